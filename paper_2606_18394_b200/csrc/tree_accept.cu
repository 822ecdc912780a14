// jet_tree_accept: greedy acceptance of the deepest matching root-to-node path.
//
// Two launches:
//   argmax_partial_kernel  grid (chunks, batch*B rows): the one HBM pass over the target
//                          logits; each block reduces a slice of one row to a
//                          (value, lowest index) key in the workspace.  Padding rows are
//                          not read.
//   accept_path_kernel     grid (batch), one thread per node: finishes the arg-max,
//                          builds the match bit-set, tests every node's ancestor mask
//                          against it, picks the deepest accepted node and writes the
//                          path and the output tokens.
#include <atomic>
#include "jet_common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace jet {
namespace {

constexpr int kArgThreads = 256;
constexpr int kArgElems = 32;
constexpr int kArgChunk = kArgThreads * kArgElems;

__global__ void __launch_bounds__(kArgThreads)
argmax_partial_kernel(const float* __restrict__ logits, int64_t row_stride, int V, int B,
                      const int32_t* __restrict__ n_nodes, int nchunks, bool vec_ok,
                      unsigned long long* __restrict__ partial) {
  grid_dependency_wait();
  const int chunk = blockIdx.x;
  const int row = blockIdx.y;
  const int b = row / B, v = row - b * B;
  if (v >= n_nodes[b]) return;
  const int tid = threadIdx.x;
  const float* p = logits + static_cast<int64_t>(row) * row_stride;
  const int base = chunk * kArgChunk;

  float best = 0.0f;
  uint32_t best_idx = 0xFFFFFFFFu;     // none yet
  if (vec_ok && base + kArgChunk <= V) {
    const float4* p4 = reinterpret_cast<const float4*>(p + base);
    float4 x[kArgElems / 4];
#pragma unroll
    for (int i = 0; i < kArgElems / 4; ++i) x[i] = __ldcs(p4 + i * kArgThreads + tid);
#pragma unroll
    for (int i = 0; i < kArgElems / 4; ++i) {
      const uint32_t idx = base + (i * kArgThreads + tid) * 4;     // ascending in i
      if (best_idx == 0xFFFFFFFFu || x[i].x > best) { best = x[i].x; best_idx = idx; }
      if (x[i].y > best) { best = x[i].y; best_idx = idx + 1; }
      if (x[i].z > best) { best = x[i].z; best_idx = idx + 2; }
      if (x[i].w > best) { best = x[i].w; best_idx = idx + 3; }
    }
  } else if (vec_ok) {
    // the row's last, partial slice: still 16-byte loads wherever four elements are in range
    const float4* p4 = reinterpret_cast<const float4*>(p + base);
    float4 x[kArgElems / 4];
#pragma unroll
    for (int i = 0; i < kArgElems / 4; ++i) {
      const int idx = base + (i * kArgThreads + tid) * 4;
      if (idx + 3 < V) {
        x[i] = __ldcs(p4 + i * kArgThreads + tid);
      } else {
        x[i].x = idx < V ? __ldcs(p + idx) : -INFINITY;
        x[i].y = idx + 1 < V ? __ldcs(p + idx + 1) : -INFINITY;
        x[i].z = idx + 2 < V ? __ldcs(p + idx + 2) : -INFINITY;
        x[i].w = -INFINITY;
      }
    }
#pragma unroll
    for (int i = 0; i < kArgElems / 4; ++i) {
      const int idx = base + (i * kArgThreads + tid) * 4;     // ascending in i
      if (idx < V && (best_idx == 0xFFFFFFFFu || x[i].x > best)) { best = x[i].x; best_idx = idx; }
      if (idx + 1 < V && x[i].y > best) { best = x[i].y; best_idx = idx + 1; }
      if (idx + 2 < V && x[i].z > best) { best = x[i].z; best_idx = idx + 2; }
      if (idx + 3 < V && x[i].w > best) { best = x[i].w; best_idx = idx + 3; }
    }
  } else {
#pragma unroll 4
    for (int i = 0; i < kArgElems; ++i) {
      const int idx = base + i * kArgThreads + tid;
      if (idx < V) {
        const float x = __ldcs(p + idx);
        if (best_idx == 0xFFFFFFFFu || x > best) { best = x; best_idx = idx; }
      }
    }
  }
  unsigned long long key = best_idx == 0xFFFFFFFFu ? 0ull : make_key(best, best_idx);
  key = warp_max_u64(key);
  __shared__ unsigned long long warp_best[kArgThreads / 32];
  if ((tid & 31) == 0) warp_best[tid >> 5] = key;
  __syncthreads();
  if (tid < 32) {
    unsigned long long w = tid < kArgThreads / 32 ? warp_best[tid] : 0ull;
    w = warp_max_u64(w);
    if (tid == 0) partial[static_cast<size_t>(row) * nchunks + chunk] = w;
  }
}

__global__ void __launch_bounds__(JET_MAX_NODES)
accept_path_kernel(const unsigned long long* __restrict__ partial, int nchunks,
                   const int32_t* __restrict__ token, const int32_t* __restrict__ parent,
                   const int32_t* __restrict__ depth, const uint32_t* __restrict__ anc_mask,
                   const int32_t* __restrict__ n_nodes, int B, int N,
                   int32_t* __restrict__ tgt_out, int32_t* __restrict__ accept_len,
                   int32_t* __restrict__ path, int32_t* __restrict__ out_tokens) {
  grid_dependency_wait();
  __shared__ int32_t s_tgt[JET_MAX_NODES];
  __shared__ uint32_t s_match[JET_MAX_NODES / 32];
  __shared__ uint32_t s_best[JET_MAX_NODES / 32];
  __shared__ uint32_t s_end_row[JET_MAX_NODES / 32];
  __shared__ int s_end;

  const int b = blockIdx.x, v = threadIdx.x, lane = v & 31, warp = v >> 5;
  const int n = min(n_nodes[b], B);
  const int words = (B + 31) / 32;
  const size_t o = static_cast<size_t>(b) * B;
  const bool live = v < n;              // blockDim.x >= B, n <= B

  int32_t tgt = -1;
  if (live) {
    unsigned long long k = 0ull;
    const unsigned long long* pr = partial + (o + v) * nchunks;
    for (int c = 0; c < nchunks; ++c) { const unsigned long long x = pr[c]; k = x > k ? x : k; }
    tgt = static_cast<int32_t>(key_index(k));
  }
  s_tgt[v] = tgt;
  if (v < B) tgt_out[o + v] = tgt;
  __syncthreads();

  // match[v]: the root always matches; other nodes iff token == target prediction at the parent
  int my_parent = -1, my_depth = -1, my_token = -1;
  if (live) { my_parent = parent[o + v]; my_depth = depth[o + v]; my_token = token[o + v]; }
  const bool match = live && (v == 0 || (my_parent >= 0 && my_parent < n && my_token == s_tgt[my_parent]));
  const uint32_t mbits = __ballot_sync(0xffffffffu, match);
  if (lane == 0) s_match[warp] = mbits;
  __syncthreads();

  // accepted iff every node of Anc(v)+{v} matches
  bool acc = live;
  if (live) {
    const uint32_t* row = anc_mask + (o + v) * words;
    for (int w = 0; w < words; ++w) acc = acc && ((row[w] & ~s_match[w]) == 0u);
  }
  // deepest accepted node, ties -> lowest index
  uint32_t key = acc ? ((static_cast<uint32_t>(my_depth) << 16) | (0xFFFFu - v)) : 0u;
  key = __reduce_max_sync(0xffffffffu, key);
  if (lane == 0) s_best[warp] = key;
  __syncthreads();
  if (warp == 0) {
    uint32_t k = lane < blockDim.x / 32 ? s_best[lane] : 0u;
    k = __reduce_max_sync(0xffffffffu, k);
    if (lane == 0) s_end = k ? static_cast<int>(0xFFFFu - (k & 0xFFFFu)) : 0;
  }
  __syncthreads();
  const int end = s_end;
  if (v < words) s_end_row[v] = anc_mask[(o + end) * words + v];
  __syncthreads();

  // (clamped: the arrays of a tree are the caller's and are not validated; a depth outside 0 .. N must not turn
  //  into a store outside the N + 1 entries of this sequence's outputs)
  const int a = s_tgt[end] >= 0 ? min(max(depth[o + end], 0), N) : 0;
  int32_t* my_path = path + static_cast<size_t>(b) * (N + 1);
  int32_t* my_tok = out_tokens + static_cast<size_t>(b) * (N + 1);
  for (int i = v; i <= N; i += blockDim.x)
    if (i > a) { my_path[i] = -1; my_tok[i] = -1; }
  if (live && ((s_end_row[v >> 5] >> (v & 31)) & 1u) && my_depth >= 0 && my_depth <= N) {
    my_path[my_depth] = v;
    if (my_depth >= 1) my_tok[my_depth - 1] = my_token;
  }
  if (v == 0) { accept_len[b] = a; my_tok[a] = s_tgt[end]; }
}

// ------------------------------------------------------------------------------------------------
// lm_head_argmax_kernel: the target's greedy prediction straight from the final hidden states -- the logits
// never exist in memory.  One CTA computes a tile of 128 vocabulary entries for MT * 128 rows:
//   D[row, token] = sum_k X[row, k] * W[token, k]      (bf16 operands, fp32 accumulation in TMEM)
// with the LM-head weights streamed once through a ring of shared-memory stages by TMA (the hidden states come
// along per 64-wide K chunk, out of L2), tcgen05.mma issued by one thread, and an epilogue in which the thread
// that owns a row scans the tile's 128 values for (largest value, lowest token id) and folds the pair into
// the row's 64-bit key in global memory with one atomicMax.  The kernel is a weight stream: V * d * 2 bytes
// from HBM per call.  Warp roles: 0 = TMA producer, 1 = TMEM allocation + MMA issue, 2..5 = epilogue.
constexpr int kLmBM = 128, kLmBN = 128, kLmBK = 64;
constexpr int kLmBlockBytes = 128 * 128;            // one [128 rows x 64 bf16] swizzled block
constexpr int kLmThreads = 192;
constexpr uint32_t kLmWaitRounds = 1u << 17;        // bounded waits: about a second in total
constexpr uint32_t kLmWaitHintNs = 8192;

template <int MT>
struct LmCfg {
  // (two stages with two row groups: 98 KB, so that two CTAs share an SM -- with 256 TMEM columns each -- and one
  //  CTA's epilogue runs under the other's weight stream: 335 -> 319 us at 256 rows against four stages and one CTA)
  static constexpr int kStages = MT == 1 ? 3 : 2;
  static constexpr int kStageBytes = (1 + MT) * kLmBlockBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 2048;
  static constexpr int kTmemCols = 128 * MT;
};

__device__ __forceinline__ bool lm_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t i = 0; i < kLmWaitRounds; ++i) {
    if (ptx::mbar_try_wait(bar, parity, kLmWaitHintNs)) return true;
    if (*abort_flag) return false;
  }
  *abort_flag = 1u;
  return false;
}

template <int MT>
__global__ void __launch_bounds__(kLmThreads)
lm_head_argmax_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, int rows, int V,
                      int d, unsigned long long* __restrict__ keys, int32_t* __restrict__ status) {
  using C = LmCfg<MT>;
  constexpr int S = C::kStages;
  extern __shared__ uint8_t lm_smem_raw[];
  const uint32_t base = (ptx::smem_u32(lm_smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = lm_smem_raw + (base - ptx::smem_u32(lm_smem_raw));
  const uint32_t sBar = base + S * C::kStageBytes;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + S * C::kStageBytes + 256);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  auto full = [&](int s) { return sBar + 8u * s; };
  auto empty = [&](int s) { return sBar + 8u * (S + s); };
  const uint32_t tmem_full = sBar + 8u * (2 * S);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (warp == 0 && lane == 0) {
    for (int s = 0; s < S; ++s) {
      ptx::mbar_init(full(s), 1);
      ptx::mbar_init(empty(s), 1);
    }
    ptx::mbar_init(tmem_full, 1);
    ptx::fence_mbar_init();
    *abort_flag = 0u;
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_w);
  } else if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), C::kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  ptx::cta_sync();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dependency_wait();

  const int n0 = blockIdx.x * kLmBN;                  // first vocabulary entry of this tile
  const int row0 = blockIdx.y * (kLmBM * MT);         // first row of this CTA's row group
  const int KC = d / kLmBK;

  if (warp == 0) {
    if (lane == 0) {
      for (int kc = 0; kc < KC; ++kc) {
        const int s = kc % S;
        if (kc >= S && !lm_wait(empty(s), ((kc / S) - 1) & 1, abort_flag)) break;
        const uint32_t dst = base + s * C::kStageBytes;
        ptx::mbar_arrive_expect_tx(full(s), C::kStageBytes);
        ptx::tma_load_2d(dst, &tm_w, full(s), kc * kLmBK, n0);
        for (int mt = 0; mt < MT; ++mt)
          ptx::tma_load_2d(dst + (1 + mt) * kLmBlockBytes, &tm_x, full(s), kc * kLmBK, row0 + mt * kLmBM);
      }
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = ptx::umma_idesc_bf16(kLmBM, kLmBN, false);
    bool ok = true;
    for (int kc = 0; kc < KC && ok; ++kc) {
      const int s = kc % S;
      ok = lm_wait(full(s), (kc / S) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint64_t desc_w = ptx::smem_desc_sw128(base + s * C::kStageBytes, 0);
      if (ptx::elect_one()) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const uint64_t desc_x = ptx::smem_desc_sw128(base + s * C::kStageBytes + (1 + mt) * kLmBlockBytes, 0);
#pragma unroll
          for (int k4 = 0; k4 < kLmBK / 16; ++k4)
            ptx::umma_ss(tmem_base + mt * kLmBN, desc_x + static_cast<uint64_t>((k4 * 32) >> 4),
                         desc_w + static_cast<uint64_t>((k4 * 32) >> 4), idesc, (kc > 0 || k4 > 0) ? 1u : 0u);
        }
        ptx::umma_commit(empty(s));
        if (kc == KC - 1) ptx::umma_commit(tmem_full);
      }
      __syncwarp();
    }
  } else {
    const bool ok = lm_wait(tmem_full, 0, abort_flag);
    if (__all_sync(0xffffffffu, ok)) {
      ptx::tc_fence_after();
      const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
        const int row = row0 + mt * kLmBM + (warp & 3) * 32 + lane;
        float best = 0.0f;
        uint32_t best_idx = 0xFFFFFFFFu;
#pragma unroll 1
        for (int c = 0; c < kLmBN / 32; ++c) {
          uint32_t x[32];
          ptx::tmem_ld32(t_lane + mt * kLmBN + c * 32, x);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const uint32_t col = static_cast<uint32_t>(n0 + c * 32 + j);       // ascending: ties keep the lowest id
            const float vj = __uint_as_float(x[j]);
            if (col < static_cast<uint32_t>(V) && (best_idx == 0xFFFFFFFFu || vj > best)) { best = vj; best_idx = col; }
          }
        }
        if (row < rows && best_idx != 0xFFFFFFFFu) atomicMax(keys + row, make_key(best, best_idx));
      }
    }
  }
  ptx::tc_fence_before();
  ptx::cta_sync();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::kTmemCols);
  }
  if (tid == 0 && *abort_flag && status) *status = JET_ERR_TIMEOUT;
}

template <int MT>
jet_status launch_lm_head(const CUtensorMap& tx, const CUtensorMap& tw, int rows, int V, int d, unsigned long long* keys,
                          int32_t* status, cudaStream_t st) {
  using C = LmCfg<MT>;
  static std::atomic<int> configured[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return JET_ERR_CUDA;
  if (configured[dev].load(std::memory_order_acquire) == 0) {
    if (cudaFuncSetAttribute(lm_head_argmax_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess) {
      cudaGetLastError();
      return JET_ERR_CUDA;
    }
    configured[dev].store(1, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((V + kLmBN - 1) / kLmBN, (rows + kLmBM * MT - 1) / (kLmBM * MT));
  cfg.blockDim = dim3(kLmThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, lm_head_argmax_kernel<MT>, tx, tw, rows, V, d, keys, status) != cudaSuccess) {
    cudaGetLastError();
    return JET_ERR_CUDA;
  }
  return JET_OK;
}

int chunks_for(int V) { return (V + kArgChunk - 1) / kArgChunk; }

// Built-in scratch of jet_tree_accept_static: one 64-bit arg-max key per (logits row, 8192-entry
// slice).  It lives in every device context that loads the library (1 MiB) until the process exits.
constexpr size_t kStaticKeys = JET_STATIC_ACCEPT_SCRATCH_BYTES / sizeof(unsigned long long);
static __device__ __align__(256) unsigned long long g_accept_scratch[kStaticKeys];
constexpr int kMaxDevices = 64;

}  // namespace
}  // namespace jet

extern "C" size_t jet_tree_accept_workspace_bytes(int batch, int B, int V) {
  if (batch < 1 || B < 1 || V < 1) return 0;
  return jet::round_up(static_cast<size_t>(batch) * B * jet::chunks_for(V) * sizeof(unsigned long long), 256);
}

extern "C" jet_status jet_tree_accept(const float* logits, int64_t logits_row_stride,
                                      const int32_t* token, const int32_t* parent,
                                      const int32_t* depth, const uint32_t* anc_mask,
                                      const int32_t* n_nodes, int batch, int B, int V, int N,
                                      int32_t* tgt_argmax, int32_t* accept_len, int32_t* path,
                                      int32_t* out_tokens, void* workspace, size_t workspace_bytes,
                                      void* stream) {
  using namespace jet;
  if (!logits || !token || !parent || !depth || !anc_mask || !n_nodes || !tgt_argmax || !accept_len ||
      !path || !out_tokens)
    return JET_ERR_INVALID_ARG;
  if (batch < 1 || B < 1 || B > JET_MAX_NODES || V < 1 || N < 1 || N > JET_MAX_DEPTH ||
      logits_row_stride < V || static_cast<int64_t>(batch) * B > 65535)
    return JET_ERR_INVALID_ARG;
  if (!aligned(logits, 4)) return JET_ERR_INVALID_ARG;
  const size_t need = jet_tree_accept_workspace_bytes(batch, B, V);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < need) return JET_ERR_WORKSPACE;

  const int nchunks = chunks_for(V);
  const bool vec_ok = aligned(logits, 16) && logits_row_stride % 4 == 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto* partial = static_cast<unsigned long long*>(workspace);
  launch_dependent(argmax_partial_kernel, dim3(nchunks, batch * B), dim3(kArgThreads), st,
      logits, logits_row_stride, V, B, n_nodes, nchunks, vec_ok, partial);
  const int threads = (B + 31) / 32 * 32;
  launch_dependent(accept_path_kernel, dim3(batch), dim3(threads), st, partial, nchunks, token, parent, depth, anc_mask,
                                                 n_nodes, B, N, tgt_argmax, accept_len, path,
                                                 out_tokens);
  return launch_status();
}

extern "C" jet_status jet_tree_accept_static(const float* logits, int64_t logits_row_stride,
                                             const int32_t* token, const int32_t* parent,
                                             const int32_t* depth, const uint32_t* anc_mask,
                                             const int32_t* n_nodes, int batch, int B, int V, int N,
                                             int32_t* tgt_argmax, int32_t* accept_len, int32_t* path,
                                             int32_t* out_tokens, void* stream) {
  using namespace jet;
  if (batch < 1 || B < 1 || V < 1) return JET_ERR_INVALID_ARG;
  const size_t need = static_cast<size_t>(batch) * B * chunks_for(V) * sizeof(unsigned long long);
  if (need > JET_STATIC_ACCEPT_SCRATCH_BYTES) return JET_ERR_WORKSPACE;   // beyond the built-in scratch

  // Device address of the built-in array, looked up once per device with that device current.
  // (In host code the array's name is only a handle; kernels must be given this address.)  The cache is
  // one atomic pointer per device: host threads that make their first call together each look the address
  // up and store the same value.
  static std::atomic<unsigned long long*> scratch_of_device[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return JET_ERR_CUDA;
  unsigned long long* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!scratch) {
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_accept_scratch) != cudaSuccess || !addr) {
      cudaGetLastError();
      return JET_ERR_CUDA;
    }
    scratch = static_cast<unsigned long long*>(addr);
    scratch_of_device[dev].store(scratch, std::memory_order_release);
  }
  // Nothing in the scratch has to start at zero: every entry that accept_path_kernel reads was
  // written by argmax_partial_kernel of the same call.
  return jet_tree_accept(logits, logits_row_stride, token, parent, depth, anc_mask, n_nodes, batch, B, V,
                         N, tgt_argmax, accept_len, path, out_tokens, scratch,
                         JET_STATIC_ACCEPT_SCRATCH_BYTES, stream);
}

extern "C" size_t jet_tree_accept_hidden_workspace_bytes(int batch, int B) {
  if (batch < 1 || B < 1) return 0;
  return jet::round_up(static_cast<size_t>(batch) * B * sizeof(unsigned long long), 256);
}

extern "C" jet_status jet_tree_accept_hidden(const void* hidden, const void* lm_head_weight, int d,
                                             const int32_t* token, const int32_t* parent, const int32_t* depth,
                                             const uint32_t* anc_mask, const int32_t* n_nodes, int batch, int B,
                                             int V, int N, int32_t* tgt_argmax, int32_t* accept_len, int32_t* path,
                                             int32_t* out_tokens, int32_t* device_status, void* workspace,
                                             size_t workspace_bytes, void* stream) {
  using namespace jet;
  if (!hidden || !lm_head_weight || !token || !parent || !depth || !anc_mask || !n_nodes || !tgt_argmax || !accept_len ||
      !path || !out_tokens)
    return JET_ERR_INVALID_ARG;
  if (batch < 1 || B < 1 || B > JET_MAX_NODES || V < 1 || N < 1 || N > JET_MAX_DEPTH || d < 64 ||
      static_cast<int64_t>(batch) * B > 65535)
    return JET_ERR_INVALID_ARG;
  if (d % 64 != 0) return JET_ERR_UNSUPPORTED;
  if (!aligned(hidden, 16) || !aligned(lm_head_weight, 16)) return JET_ERR_INVALID_ARG;
  const size_t need = jet_tree_accept_hidden_workspace_bytes(batch, B);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < need) return JET_ERR_WORKSPACE;
  const int rows = batch * B;
  CUtensorMap tx, tw;
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(d), static_cast<uint64_t>(rows)};
    const uint64_t str[1] = {static_cast<uint64_t>(d) * 2};
    const uint32_t box[2] = {64, 128};
    if (!tma_make_map_bf16(&tx, hidden, 2, dims, str, box)) return JET_ERR_CUDA;
  }
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(d), static_cast<uint64_t>(V)};
    const uint64_t str[1] = {static_cast<uint64_t>(d) * 2};
    const uint32_t box[2] = {64, 128};
    if (!tma_make_map_bf16(&tw, lm_head_weight, 2, dims, str, box)) return JET_ERR_CUDA;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto* keys = static_cast<unsigned long long*>(workspace);
  // every row's key starts as "no entry" (0 is below any valid key)
  if (cudaMemsetAsync(keys, 0, static_cast<size_t>(rows) * sizeof(unsigned long long), st) != cudaSuccess) {
    cudaGetLastError();
    return JET_ERR_CUDA;
  }
  // rows per CTA: every row group of a CTA shares the weight tile it streams, so more rows per CTA means the
  // weights cross HBM fewer times (once for up to 512 rows)
  jet_status r;
  if (rows <= 128) r = launch_lm_head<1>(tx, tw, rows, V, d, keys, device_status, st);
  else if (rows <= 256) r = launch_lm_head<2>(tx, tw, rows, V, d, keys, device_status, st);
  else r = launch_lm_head<4>(tx, tw, rows, V, d, keys, device_status, st);
  if (r != JET_OK) return r;
  const int threads = (B + 31) / 32 * 32;
  launch_dependent(accept_path_kernel, dim3(batch), dim3(threads), st, keys, 1, token, parent, depth, anc_mask, n_nodes, B, N,
                   tgt_argmax, accept_len, path, out_tokens);
  return launch_status();
}
