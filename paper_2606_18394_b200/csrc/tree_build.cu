// jet_tree_build: per-depth top-W extraction followed by Algorithm 1 (best-first
// budgeted tree construction with the accumulated log-probability score).
// jet_tree_build_scored: the same with the expansion scores of Appendix C (per-depth
// entropy alone; accumulated log-probability + alpha * per-depth entropy): the scan
// also leaves per-slice sums of p * log p (fp64), the expansion kernel adds them up
// per depth and uses the entropy in the queue's priority.
// jet_tree_build_logits: the same fed with raw draft logits.  One more launch in front
// (lse_partial_kernel: per-slice maximum and sum of exponentials in fp64); the scan then
// forms every log-probability on the fly as float(double(z) - lse), so the [N,V]
// log-probabilities never exist in memory and the second pass over the logits comes
// out of L2.
//
// Two launches:
//   topw_partial_kernel  grid (chunks, N, batch): every block scans one slice of one
//                        vocabulary row and leaves its W best (value, token) keys in
//                        the workspace -- the only pass over the [N,V] log-probs.
//   tree_expand_kernel   grid (batch): merges the per-slice candidates, runs the
//                        sequential pop/expand loop in one warp with the pending
//                        queue held in shared memory, then emits parent / depth /
//                        token / score / ancestor bitmask.
#include "jet_common.cuh"

namespace jet {
namespace {

constexpr int kTopThreads = 256;
constexpr int kTopElems = 16;                        // elements per thread
constexpr int kTopChunk = kTopThreads * kTopElems;   // vocabulary slice per block

// One block scans a 4096-element slice of one vocabulary row and leaves its W best keys.  Almost every
// element is dismissed with one compare: an element among a warp's W best is at least as large as the W-th
// largest of the 32 per-lane maxima (tau), so only elements >= tau become candidates (as ordered 64-bit keys
// in shared memory); the block then selects its W best among the few candidates.  Exact for any input: with
// many equal values all of them become candidates and the key order (value, then lowest index) decides.
// kEntropy: the block also leaves sum(exp(l) * l) over its slice (fp64; entries of -inf contribute 0) for the
// per-depth entropy; the reduction order is fixed, so the value does not change from run to run.
// Loads the 16 elements of a thread: element e has vocabulary index
//   vec ? base + ((e >> 2) * kTopThreads + tid) * 4 + (e & 3) : base + e * kTopThreads + tid;
// elements beyond V read as -inf.
__device__ __forceinline__ void load_slice(const float* __restrict__ row, int base, int V, bool vec, int tid,
                                           float (&v)[kTopElems]) {
  if (vec) {
    const float4* row4 = reinterpret_cast<const float4*>(row + base);
#pragma unroll
    for (int i = 0; i < kTopElems / 4; ++i) {
      const float4 x = __ldg(row4 + i * kTopThreads + tid);
      v[i * 4 + 0] = x.x; v[i * 4 + 1] = x.y; v[i * 4 + 2] = x.z; v[i * 4 + 3] = x.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < kTopElems; ++i) {
      const int idx = base + i * kTopThreads + tid;
      v[i] = idx < V ? __ldg(row + idx) : -INFINITY;
    }
  }
}

// Raw logits: every block leaves (m, z) of its slice, m = the slice's maximum and z = sum(exp(double(x) - m))
// in fp64 with a fixed reduction order (a slice of -inf only: m = -inf, z = 0).
__global__ void __launch_bounds__(kTopThreads)
lse_partial_kernel(const float* __restrict__ logits, int64_t batch_stride, int64_t depth_stride, int V, int nchunks,
                   bool vec_ok, double* __restrict__ lse_partial) {
  grid_dependency_wait();
  const int chunk = blockIdx.x, d = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31;
  const float* row = logits + b * batch_stride + d * depth_stride;
  const int base = chunk * kTopChunk;
  float v[kTopElems];
  load_slice(row, base, V, vec_ok && base + kTopChunk <= V, tid, v);
  float m = -INFINITY;
#pragma unroll
  for (int i = 0; i < kTopElems; ++i) m = fmaxf(m, v[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float s_m[kTopThreads / 32];
  __shared__ double s_z[kTopThreads / 32];
  if (lane == 0) s_m[tid >> 5] = m;
  __syncthreads();
#pragma unroll
  for (int w = 0; w < kTopThreads / 32; ++w) m = fmaxf(m, s_m[w]);
  double z = 0.0;
  if (m > -INFINITY) {
    const double md = static_cast<double>(m);
#pragma unroll
    for (int i = 0; i < kTopElems; ++i)
      if (v[i] > -INFINITY) z += exp(static_cast<double>(v[i]) - md);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  if (lane == 0) s_z[tid >> 5] = z;
  __syncthreads();
  if (tid == 0) {
    double total = 0.0;
    for (int w = 0; w < kTopThreads / 32; ++w) total += s_z[w];
    double* out = lse_partial + ((static_cast<size_t>(b) * gridDim.y + d) * nchunks + chunk) * 2;
    out[0] = static_cast<double>(m);
    out[1] = total;
  }
}

// The row's log-sum-exp from the slices' (m, z): M = max m, lse = M + log(sum z * exp(m - M)), fp64, one warp,
// fixed order (every block of a row gets the same bits).
__device__ __forceinline__ double row_lse(const double* __restrict__ part, int nchunks, int lane) {
  double M = -INFINITY;
  for (int i = lane; i < nchunks; i += 32) M = fmax(M, part[2 * i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmax(M, __shfl_xor_sync(0xffffffffu, M, o));
  double Z = 0.0;
  for (int i = lane; i < nchunks; i += 32) {
    const double m = part[2 * i], z = part[2 * i + 1];
    if (z > 0.0) Z += z * exp(m - M);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
  return M + log(Z);
}

// kLogits: the row holds raw logits; lse_partial holds its slices' (m, z) and every element becomes the
// log-probability float(double(x) - lse) before anything else looks at it (block 0 of the row also leaves
// float(lse) in depth_lse_out if that is given).
template <bool kEntropy, bool kLogits>
__global__ void __launch_bounds__(kTopThreads)
topw_partial_kernel(const float* __restrict__ logp, int64_t batch_stride, int64_t depth_stride,
                    int V, int Wc, int nchunks, bool vec_ok,
                    unsigned long long* __restrict__ cand, double* __restrict__ plogp_partial,
                    const double* __restrict__ lse_partial, float* __restrict__ depth_lse_out) {
  grid_dependency_wait();
  const int chunk = blockIdx.x, d = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31;
  const float* row = logp + b * batch_stride + d * depth_stride;
  const int base = chunk * kTopChunk;

  // element e of this thread has vocabulary index idx_of(e); out-of-range elements are -inf and never candidates
  float v[kTopElems];
  const bool vec = vec_ok && base + kTopChunk <= V;
  auto idx_of = [&](int e) -> int {
    return vec ? base + ((e >> 2) * kTopThreads + tid) * 4 + (e & 3) : base + e * kTopThreads + tid;
  };
  load_slice(row, base, V, vec, tid, v);
  if constexpr (kLogits) {
    __shared__ double s_lse;
    if (tid < 32) {
      const double lse = row_lse(lse_partial + (static_cast<size_t>(b) * gridDim.y + d) * nchunks * 2, nchunks, lane);
      if (lane == 0) {
        s_lse = lse;
        if (chunk == 0 && depth_lse_out) depth_lse_out[static_cast<size_t>(b) * gridDim.y + d] = static_cast<float>(lse);
      }
    }
    __syncthreads();
    const double lse = s_lse;
#pragma unroll
    for (int i = 0; i < kTopElems; ++i) v[i] = static_cast<float>(static_cast<double>(v[i]) - lse);
  }

  if constexpr (kEntropy) {
    double acc = 0.0;
#pragma unroll
    for (int i = 0; i < kTopElems; ++i)
      if (v[i] > -INFINITY) acc += exp(static_cast<double>(v[i])) * static_cast<double>(v[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    __shared__ double s_acc[kTopThreads / 32];
    if (lane == 0) s_acc[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
      double total = 0.0;
      for (int w = 0; w < kTopThreads / 32; ++w) total += s_acc[w];
      plogp_partial[(static_cast<size_t>(b) * gridDim.y + d) * nchunks + chunk] = total;
    }
  }

  // tau = Wc-th largest of the warp's 32 lane maxima: every lane ranks its maximum (ties by lane) against
  // the others' with 32 independent shuffles; the lane of rank Wc-1 holds tau
  float lane_max = -INFINITY;
#pragma unroll
  for (int i = 0; i < kTopElems; ++i) lane_max = fmaxf(lane_max, v[i]);
  int rank = 0;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const float other = __shfl_sync(0xffffffffu, lane_max, j);
    rank += (other > lane_max || (other == lane_max && j < lane)) ? 1 : 0;
  }
  const unsigned holder = __ballot_sync(0xffffffffu, rank == Wc - 1);
  const float tau = __shfl_sync(0xffffffffu, lane_max, __ffs(holder) - 1);

  __shared__ unsigned long long s_cand[kTopChunk];      // worst case: every element of the slice
  __shared__ int s_count;
  if (tid == 0) s_count = 0;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < kTopElems; ++i) {
    const int idx = idx_of(i);
    if (v[i] >= tau && idx < V) s_cand[atomicAdd(&s_count, 1)] = make_key(v[i], static_cast<uint32_t>(idx));
  }
  __syncthreads();
  const int count = s_count;

  // the block's Wc best candidates, in rank order (keys are unique)
  unsigned long long* out = cand + ((static_cast<size_t>(b) * gridDim.y + d) * nchunks + chunk) * Wc;
  if (count <= kTopThreads) {
    // usual case: one candidate per thread, ranked against all others (broadcast reads, no serial rounds)
    if (tid < count) {
      const unsigned long long mine = s_cand[tid];
      int rank = 0;
      for (int j = 0; j < count; ++j) rank += s_cand[j] > mine ? 1 : 0;
      if (rank < Wc) out[rank] = mine;
    }
    if (tid >= count && tid < Wc) out[tid] = 0ull;          // fewer candidates than Wc: no key
    return;
  }
  // many equal values: warp 0 alone walks the candidates in rank order
  if (tid >= 32) return;
  // (more than kTopThreads candidates here, too many for registers: every round scans shared memory)
  unsigned long long prev = ~0ull;
  for (int r = 0; r < Wc; ++r) {
    unsigned long long best = 0ull;
    for (int i = lane; i < count; i += 32) {
      const unsigned long long k = s_cand[i];
      if (k < prev && k > best) best = k;
    }
    best = warp_max_u64(best);
    if (lane == 0) out[r] = best;
    prev = best;
  }
}

// Algorithm 1 in one warp.  The pending queue lives in registers: node u is kept by lane u % 32 in register
// u / 32 as a key (score, lowest index first, depth in the low byte), so a pop is a register maximum plus one
// warp reduction, and the popped node's score and depth come out of the key itself.  kSlots = registers per
// lane (32 * kSlots >= B); the instruction count of a pop grows with it, hence the template.
// kMode: 0 = priority is the accumulated log-probability (the key's value is the node's score); 1 = priority
// is the entropy of the node's depth; 2 = score + alpha * that entropy, formed as two rounded float operations.
// depth_h[d] = entropy of the distribution the tokens of depth d + 1 were drawn from.  In modes 1 and 2 the
// popped node's score is read back from shared memory.
template <int kSlots, int kMode>
__device__ __forceinline__ int expand_tree(int lane, int N, int Wc, int B, int root, const float (*top_lp)[JET_MAX_WIDTH],
                                           const int32_t (*top_tok)[JET_MAX_WIDTH], int32_t* s_parent,
                                           int32_t* s_depth, int32_t* s_token, float* s_score,
                                           const float* depth_h, float alpha) {
  unsigned long long q[kSlots];
#pragma unroll
  for (int i = 0; i < kSlots; ++i) q[i] = 0ull;
  auto queue_key = [](float score, int node, int dep) -> unsigned long long {
    return (static_cast<unsigned long long>(f32_order(score)) << 32) |
           (static_cast<unsigned long long>(0xFFFFFFu - static_cast<uint32_t>(node)) << 8) |
           static_cast<unsigned long long>(dep);
  };
  if (lane == 0) {
    s_parent[0] = -1; s_depth[0] = 0; s_token[0] = root; s_score[0] = 0.0f;
    q[0] = queue_key(0.0f, 0, 0);
  }
  int n = 1;
  while (n < B) {
    unsigned long long best = 0ull;
#pragma unroll
    for (int i = 0; i < kSlots; ++i) best = q[i] > best ? q[i] : best;
    best = warp_max_u64(best);
    if (best == 0ull) break;                        // nothing pending
    const int v = static_cast<int>(0xFFFFFFu - (static_cast<uint32_t>(best >> 8) & 0xFFFFFFu));
    const int d = static_cast<int>(best & 0xFFull);
    float sv;
    if constexpr (kMode == 0) sv = key_value(best);
    else sv = s_score[v];
#pragma unroll
    for (int i = 0; i < kSlots; ++i) if (q[i] == best) q[i] = 0ull;      // popped (only its keeper matches)
    if (d < N) {
      const int cnt = min(Wc, B - n);
      const int j = (lane - n) & 31;                // child rank whose node n + j this lane keeps
      if (j < cnt) {
        const int u = n + j;
        const float s = __fadd_rn(sv, top_lp[d][j]);
        s_parent[u] = v; s_depth[u] = d + 1; s_token[u] = top_tok[d][j]; s_score[u] = s;
        float prio = s;
        if constexpr (kMode == 1) prio = depth_h[d];
        if constexpr (kMode == 2) prio = __fadd_rn(s, __fmul_rn(alpha, depth_h[d]));
        const unsigned long long key = queue_key(prio, u, d + 1);
#pragma unroll
        for (int i = 0; i < kSlots; ++i) if (i == (u >> 5)) q[i] = key;
      }
      n += cnt;
      if constexpr (kMode != 0) __syncwarp();          // the children's scores are read back when they are popped
    }
  }
  return n;
}

constexpr int kExpThreads = 256;

template <int kMode>
__global__ void __launch_bounds__(kExpThreads)
tree_expand_kernel(const float* __restrict__ logp, int64_t batch_stride, int64_t depth_stride,
                   const int32_t* __restrict__ root_token, int N, int Wc, int B, int nchunks,
                   const unsigned long long* __restrict__ cand,
                   int32_t* __restrict__ parent_out, int32_t* __restrict__ depth_out,
                   int32_t* __restrict__ token_out, float* __restrict__ score_out,
                   uint32_t* __restrict__ anc_out, int32_t* __restrict__ n_nodes_out,
                   const double* __restrict__ plogp_partial, float alpha, float* __restrict__ depth_entropy_out,
                   const int32_t* __restrict__ node_budget) {
  grid_dependency_wait();
  __shared__ int32_t s_top_tok[JET_MAX_DEPTH][JET_MAX_WIDTH];
  __shared__ float s_top_lp[JET_MAX_DEPTH][JET_MAX_WIDTH];
  __shared__ int32_t s_parent[JET_MAX_NODES], s_depth[JET_MAX_NODES], s_token[JET_MAX_NODES];
  __shared__ float s_score[JET_MAX_NODES];
  __shared__ float s_depth_h[JET_MAX_DEPTH];
  __shared__ int s_n;

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- merge the per-slice candidates: depth d's W best of nchunks*Wc keys (keys are unique,
  //      so "largest key below the previous winner" walks them in rank order)
  for (int d = warp; d < N; d += kExpThreads / 32) {
    if constexpr (kMode != 0) {
      // entropy of row d: minus the sum of the slices' partial sums (fp64, fixed order), rounded once
      const double* part = plogp_partial + (static_cast<size_t>(b) * N + d) * nchunks;
      double acc = 0.0;
      for (int i = lane; i < nchunks; i += 32) acc += part[i];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (lane == 0) {
        const float h = static_cast<float>(-acc);
        s_depth_h[d] = h;
        if (depth_entropy_out) depth_entropy_out[static_cast<size_t>(b) * N + d] = h;
      }
    }
    const unsigned long long* c = cand + (static_cast<size_t>(b) * N + d) * nchunks * Wc;
    const int total = nchunks * Wc;
    constexpr int kHeld = 16;                 // candidates a lane can keep in registers
    unsigned long long held[kHeld];
    const bool in_regs = total <= 32 * kHeld; // usual case: one pass over global memory, rounds on registers
    if (in_regs) {
#pragma unroll
      for (int i = 0; i < kHeld; ++i) held[i] = lane + 32 * i < total ? c[lane + 32 * i] : 0ull;
    }
    unsigned long long prev = ~0ull;
    for (int r = 0; r < Wc; ++r) {
      unsigned long long best = 0ull;
      if (in_regs) {
#pragma unroll
        for (int i = 0; i < kHeld; ++i) if (held[i] < prev && held[i] > best) best = held[i];
      } else {
        for (int i = lane; i < total; i += 32) {
          const unsigned long long k = c[i];
          if (k < prev && k > best) best = k;
        }
      }
      best = warp_max_u64(best);
      if (lane == 0) {
        const uint32_t t = key_index(best);
        s_top_tok[d][r] = static_cast<int32_t>(t);
        s_top_lp[d][r] = key_value(best);            // the key holds the value itself: no second look-up
      }
      prev = best;
    }
  }
  __syncthreads();

  // ---- Algorithm 1: one warp, queue in registers (as many per lane as the budget needs)
  // this sequence's budget: B, or its own smaller one (the arrays are padded to B either way)
  const int Bmax = B;
  if (node_budget) B = max(1, min(B, node_budget[b]));
  if (warp == 0) {
    const int root = root_token[b];
    int n;
    if (B <= 32) n = expand_tree<1, kMode>(lane, N, Wc, B, root, s_top_lp, s_top_tok, s_parent, s_depth, s_token, s_score, s_depth_h, alpha);
    else if (B <= 64) n = expand_tree<2, kMode>(lane, N, Wc, B, root, s_top_lp, s_top_tok, s_parent, s_depth, s_token, s_score, s_depth_h, alpha);
    else if (B <= 128) n = expand_tree<4, kMode>(lane, N, Wc, B, root, s_top_lp, s_top_tok, s_parent, s_depth, s_token, s_score, s_depth_h, alpha);
    else if (B <= 256) n = expand_tree<8, kMode>(lane, N, Wc, B, root, s_top_lp, s_top_tok, s_parent, s_depth, s_token, s_score, s_depth_h, alpha);
    else n = expand_tree<JET_MAX_NODES / 32, kMode>(lane, N, Wc, B, root, s_top_lp, s_top_tok, s_parent, s_depth, s_token, s_score, s_depth_h, alpha);
    if (lane == 0) s_n = n;
  }
  __syncthreads();

  // ---- emit
  const int n = s_n;
  B = Bmax;
  const size_t o = static_cast<size_t>(b) * B;
  for (int v = tid; v < B; v += kExpThreads) {
    const bool live = v < n;
    parent_out[o + v] = live ? s_parent[v] : -1;
    depth_out[o + v] = live ? s_depth[v] : -1;
    token_out[o + v] = live ? s_token[v] : -1;
    if (score_out) score_out[o + v] = live ? s_score[v] : 0.0f;
  }
  if (tid == 0) n_nodes_out[b] = n;
  const int words = (B + 31) / 32;
  for (int i = tid; i < B * words; i += kExpThreads) {
    const int v = i / words, w = i - v * words;
    uint32_t bits = 0u;
    if (v < n) {
      for (int u = v; u >= 0; u = s_parent[u])
        if ((u >> 5) == w) bits |= 1u << (u & 31);
    }
    anc_out[o * words + i] = bits;
  }
}

int chunks_for(int V) { return (V + kTopChunk - 1) / kTopChunk; }

size_t cand_bytes(int batch, int N, int V, int W) {
  const size_t Wc = static_cast<size_t>(W < V ? W : V);
  return round_up(static_cast<size_t>(batch) * N * chunks_for(V) * Wc * sizeof(unsigned long long), 256);
}

// Checks and launches shared by the two entry points (score_mode: JET_SCORE_*).
jet_status tree_build_launch(const float* logp, int64_t logp_batch_stride, int64_t logp_depth_stride,
                             const int32_t* root_token, int batch, int N, int V, int W, int B, int score_mode,
                             float alpha, int32_t* parent, int32_t* depth, int32_t* token, float* score,
                             uint32_t* anc_mask, int32_t* n_nodes, float* depth_entropy,
                             const int32_t* node_budget, void* workspace, size_t workspace_bytes, size_t need,
                             void* stream, bool from_logits = false, float* depth_lse = nullptr) {
  if (!logp || !root_token || !parent || !depth || !token || !anc_mask || !n_nodes)
    return JET_ERR_INVALID_ARG;
  if (batch < 1 || batch > 65535 || N < 1 || N > JET_MAX_DEPTH || W < 1 || W > JET_MAX_WIDTH || V < 1 ||
      B < 1 || B > JET_MAX_NODES || logp_depth_stride < V || logp_batch_stride < 0)
    return JET_ERR_INVALID_ARG;
  if (score_mode < JET_SCORE_ACCUM_LOGP || score_mode > JET_SCORE_HYBRID) return JET_ERR_INVALID_ARG;
  if (score_mode == JET_SCORE_HYBRID && !(alpha == alpha && alpha > -INFINITY && alpha < INFINITY)) return JET_ERR_INVALID_ARG;
  if (!aligned(logp, 4)) return JET_ERR_INVALID_ARG;
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < need) return JET_ERR_WORKSPACE;

  const int Wc = W < V ? W : V;
  const int nchunks = chunks_for(V);
  const bool vec_ok = aligned(logp, 16) && logp_batch_stride % 4 == 0 && logp_depth_stride % 4 == 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto* cand = static_cast<unsigned long long*>(workspace);
  auto* plogp = reinterpret_cast<double*>(static_cast<uint8_t*>(workspace) + cand_bytes(batch, N, V, W));
  const double* no_lse = nullptr;
  float* no_out = nullptr;
  if (from_logits) {
    double* lse_part = plogp + round_up(static_cast<size_t>(batch) * N * nchunks * sizeof(double), 256) / sizeof(double);
    launch_dependent(lse_partial_kernel, dim3(nchunks, N, batch), dim3(kTopThreads), st,
        logp, logp_batch_stride, logp_depth_stride, V, nchunks, vec_ok, lse_part);
    const double* lse_in = lse_part;
    if (score_mode == JET_SCORE_ACCUM_LOGP)
      launch_dependent(topw_partial_kernel<false, true>, dim3(nchunks, N, batch), dim3(kTopThreads), st,
          logp, logp_batch_stride, logp_depth_stride, V, Wc, nchunks, vec_ok, cand, static_cast<double*>(nullptr),
          lse_in, depth_lse);
    else
      launch_dependent(topw_partial_kernel<true, true>, dim3(nchunks, N, batch), dim3(kTopThreads), st,
          logp, logp_batch_stride, logp_depth_stride, V, Wc, nchunks, vec_ok, cand, plogp, lse_in, depth_lse);
  } else if (score_mode == JET_SCORE_ACCUM_LOGP) {
    launch_dependent(topw_partial_kernel<false, false>, dim3(nchunks, N, batch), dim3(kTopThreads), st,
        logp, logp_batch_stride, logp_depth_stride, V, Wc, nchunks, vec_ok, cand, static_cast<double*>(nullptr),
        no_lse, no_out);
  } else {
    launch_dependent(topw_partial_kernel<true, false>, dim3(nchunks, N, batch), dim3(kTopThreads), st,
        logp, logp_batch_stride, logp_depth_stride, V, Wc, nchunks, vec_ok, cand, plogp, no_lse, no_out);
  }
  if (score_mode == JET_SCORE_ACCUM_LOGP) {
    launch_dependent(tree_expand_kernel<0>, dim3(batch), dim3(kExpThreads), st, logp, logp_batch_stride, logp_depth_stride,
        root_token, N, Wc, B, nchunks, cand, parent, depth, token, score, anc_mask, n_nodes,
        static_cast<const double*>(nullptr), 0.0f, static_cast<float*>(nullptr), node_budget);
    return launch_status();
  }
  if (score_mode == JET_SCORE_ENTROPY)
    launch_dependent(tree_expand_kernel<1>, dim3(batch), dim3(kExpThreads), st, logp, logp_batch_stride, logp_depth_stride,
        root_token, N, Wc, B, nchunks, cand, parent, depth, token, score, anc_mask, n_nodes,
        static_cast<const double*>(plogp), 0.0f, depth_entropy, node_budget);
  else
    launch_dependent(tree_expand_kernel<2>, dim3(batch), dim3(kExpThreads), st, logp, logp_batch_stride, logp_depth_stride,
        root_token, N, Wc, B, nchunks, cand, parent, depth, token, score, anc_mask, n_nodes,
        static_cast<const double*>(plogp), alpha, depth_entropy, node_budget);
  return launch_status();
}

}  // namespace
}  // namespace jet

extern "C" size_t jet_tree_build_workspace_bytes(int batch, int N, int V, int W) {
  if (batch < 1 || N < 1 || V < 1 || W < 1) return 0;
  return jet::cand_bytes(batch, N, V, W);
}

extern "C" jet_status jet_tree_build(const float* logp, int64_t logp_batch_stride,
                                     int64_t logp_depth_stride, const int32_t* root_token,
                                     int batch, int N, int V, int W, int B, int32_t* parent,
                                     int32_t* depth, int32_t* token, float* score,
                                     uint32_t* anc_mask, int32_t* n_nodes, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  const size_t need = (batch >= 1 && N >= 1 && V >= 1 && W >= 1) ? jet::cand_bytes(batch, N, V, W) : 0;
  return jet::tree_build_launch(logp, logp_batch_stride, logp_depth_stride, root_token, batch, N, V, W, B,
                                JET_SCORE_ACCUM_LOGP, 0.0f, parent, depth, token, score, anc_mask, n_nodes, nullptr,
                                nullptr, workspace, workspace_bytes, need, stream);
}

extern "C" size_t jet_tree_build_scored_workspace_bytes(int batch, int N, int V, int W) {
  if (batch < 1 || N < 1 || V < 1 || W < 1) return 0;
  return jet::cand_bytes(batch, N, V, W) +
         jet::round_up(static_cast<size_t>(batch) * N * jet::chunks_for(V) * sizeof(double), 256);
}

extern "C" jet_status jet_tree_build_scored(const float* logp, int64_t logp_batch_stride,
                                            int64_t logp_depth_stride, const int32_t* root_token,
                                            int batch, int N, int V, int W, int B, const int32_t* node_budget,
                                            int score_mode, float alpha, int32_t* parent, int32_t* depth,
                                            int32_t* token, float* score, uint32_t* anc_mask, int32_t* n_nodes,
                                            float* depth_entropy, void* workspace, size_t workspace_bytes,
                                            void* stream) {
  const size_t need = jet_tree_build_scored_workspace_bytes(batch, N, V, W);
  return jet::tree_build_launch(logp, logp_batch_stride, logp_depth_stride, root_token, batch, N, V, W, B, score_mode,
                                alpha, parent, depth, token, score, anc_mask, n_nodes, depth_entropy, node_budget,
                                workspace, workspace_bytes, need, stream);
}

extern "C" size_t jet_tree_build_logits_workspace_bytes(int batch, int N, int V, int W) {
  if (batch < 1 || N < 1 || V < 1 || W < 1) return 0;
  return jet_tree_build_scored_workspace_bytes(batch, N, V, W) +
         jet::round_up(static_cast<size_t>(batch) * N * jet::chunks_for(V) * 2 * sizeof(double), 256);
}

extern "C" jet_status jet_tree_build_logits(const float* logits, int64_t logits_batch_stride,
                                            int64_t logits_depth_stride, const int32_t* root_token,
                                            int batch, int N, int V, int W, int B, const int32_t* node_budget,
                                            int score_mode, float alpha, int32_t* parent, int32_t* depth,
                                            int32_t* token, float* score, uint32_t* anc_mask, int32_t* n_nodes,
                                            float* depth_entropy, float* depth_lse, void* workspace,
                                            size_t workspace_bytes, void* stream) {
  const size_t need = jet_tree_build_logits_workspace_bytes(batch, N, V, W);
  return jet::tree_build_launch(logits, logits_batch_stride, logits_depth_stride, root_token, batch, N, V, W, B,
                                score_mode, alpha, parent, depth, token, score, anc_mask, n_nodes, depth_entropy,
                                node_budget, workspace, workspace_bytes, need, stream, true, depth_lse);
}
