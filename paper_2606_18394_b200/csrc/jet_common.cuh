// Shared host/device helpers of the jet library (status mapping, ordered keys).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "jet.h"

namespace jet {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline jet_status launch_status() {
  return cudaGetLastError() == cudaSuccess ? JET_OK : JET_ERR_CUDA;
}

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Launch with programmatic stream serialization: the grid may be scheduled while the preceding kernel of the
// stream drains, so its launch latency is hidden.  Every kernel launched this way executes grid_dependency_wait()
// before its first access to global memory.
template <typename... KArgs, typename... Args>
inline void launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Waits until the preceding kernels of the stream have completed and their writes are visible, then lets
// the next kernel of the stream be scheduled early in turn.
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Monotone map float -> uint32 (larger float <=> larger code); -0.0 and +0.0 share a code.
__device__ __forceinline__ uint32_t f32_order(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Key whose maximum is "largest value, then lowest index".  A valid key is never 0.
__device__ __forceinline__ unsigned long long make_key(float x, uint32_t idx) {
  return (static_cast<unsigned long long>(f32_order(x)) << 32) | (0xFFFFFFFFu - idx);
}
__device__ __forceinline__ uint32_t key_index(unsigned long long k) {
  return 0xFFFFFFFFu - static_cast<uint32_t>(k);
}
// The float a key was made from (-0.0 comes back as +0.0, which adds to any partial sum identically).
__device__ __forceinline__ float key_value(unsigned long long k) {
  const uint32_t c = static_cast<uint32_t>(k >> 32);
  return __uint_as_float((c & 0x80000000u) ? (c & 0x7FFFFFFFu) : ~c);
}

// Maximum of the warp's 64-bit keys with two 32-bit warp reductions (redux.sync): the largest high word, then
// the largest low word among the lanes that hold it.  Needs no key with a zero low word other than the empty
// key 0 (the keys made here never have one: the low word holds an inverted index).
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long k) {
  const uint32_t hi = static_cast<uint32_t>(k >> 32), lo = static_cast<uint32_t>(k);
  const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
  const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
  return (static_cast<unsigned long long>(mh) << 32) | ml;
}

}  // namespace jet
