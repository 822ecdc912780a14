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

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long k) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long other = __shfl_xor_sync(0xffffffffu, k, o);
    k = other > k ? other : k;
  }
  return k;
}

}  // namespace jet
