// jet_tree_accept_sample: non-greedy tree acceptance (Section 3.3, Eq. nongreedy_specdec).
//
// Two launches:
//   row_lse_partial_kernel  grid (slices, batch*B): one pass over the target logits; every block
//                           leaves the maximum and the sum of exp((x - max) / T) of one 8192-entry
//                           slice of one row in the workspace.  Padding rows are not read.
//   accept_sample_kernel    grid (batch), 512 threads: finishes the rows' log-sum-exp, computes
//                           alpha_v = min(1, p_parent(token_v) / q_depth(token_v)) and the accept
//                           bit u_v < alpha_v for every node, picks the deepest node whose whole
//                           branch is accepted, then draws the correction token at that node by
//                           inverse CDF in vocabulary order (residual max(0, p - q) if the node has
//                           rejected children, p itself if it is a leaf).
#include "jet_common.cuh"

namespace jet {
namespace {

constexpr int kLseThreads = 256;
constexpr int kLseElems = 32;
constexpr int kLseChunk = kLseThreads * kLseElems;
constexpr int kSampleThreads = 512;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float warp_max_f(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum_f(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ double warp_sum_d(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

__global__ void __launch_bounds__(kLseThreads)
row_lse_partial_kernel(const float* __restrict__ logits, int64_t row_stride, int V, int B,
                       const int32_t* __restrict__ n_nodes, int nchunks, bool vec_ok, float inv_t_log2,
                       float2* __restrict__ partial) {
  grid_dependency_wait();
  const int chunk = blockIdx.x;
  const int row = blockIdx.y;
  const int b = row / B, v = row - b * B;
  if (v >= n_nodes[b]) return;
  const int tid = threadIdx.x;
  const float* p = logits + static_cast<int64_t>(row) * row_stride;
  const int base = chunk * kLseChunk;

  float x[kLseElems];
  if (vec_ok && base + kLseChunk <= V) {
    const float4* p4 = reinterpret_cast<const float4*>(p + base);
#pragma unroll
    for (int i = 0; i < kLseElems / 4; ++i) {
      const float4 q = __ldcs(p4 + i * kLseThreads + tid);
      x[i * 4 + 0] = q.x; x[i * 4 + 1] = q.y; x[i * 4 + 2] = q.z; x[i * 4 + 3] = q.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < kLseElems; ++i) {
      const int idx = base + i * kLseThreads + tid;
      x[i] = idx < V ? __ldcs(p + idx) : -INFINITY;
    }
  }
  __shared__ float s_red[kLseThreads / 32];
  float m = -INFINITY;
#pragma unroll
  for (int i = 0; i < kLseElems; ++i) m = fmaxf(m, x[i]);
  m = warp_max_f(m);
  if ((tid & 31) == 0) s_red[tid >> 5] = m;
  __syncthreads();
  m = s_red[0];
#pragma unroll
  for (int i = 1; i < kLseThreads / 32; ++i) m = fmaxf(m, s_red[i]);
  __syncthreads();
  float s = 0.0f;
  if (m > -INFINITY) {
#pragma unroll
    for (int i = 0; i < kLseElems; ++i) s += exp2f((x[i] - m) * inv_t_log2);
  }
  s = warp_sum_f(s);
  if ((tid & 31) == 0) s_red[tid >> 5] = s;
  __syncthreads();
  if (tid == 0) {
    float tot = 0.0f;
#pragma unroll
    for (int i = 0; i < kLseThreads / 32; ++i) tot += s_red[i];
    partial[static_cast<size_t>(row) * nchunks + chunk] = make_float2(m, tot);
  }
}

__global__ void __launch_bounds__(kSampleThreads)
accept_sample_kernel(const float2* __restrict__ partial, int nchunks, const float* __restrict__ logits,
                     int64_t row_stride, float inv_t, const float* __restrict__ draft_logp,
                     int64_t logp_batch_stride, int64_t logp_depth_stride,
                     const int32_t* __restrict__ token, const int32_t* __restrict__ parent,
                     const int32_t* __restrict__ depth, const uint32_t* __restrict__ anc_mask,
                     const int32_t* __restrict__ n_nodes, const float* __restrict__ u_accept,
                     const float* __restrict__ u_sample, int B, int V, int N, float* __restrict__ alpha_out,
                     int32_t* __restrict__ accept_len, int32_t* __restrict__ path,
                     int32_t* __restrict__ out_tokens) {
  grid_dependency_wait();
  __shared__ float s_max[JET_MAX_NODES], s_lnsum[JET_MAX_NODES];      // per row: max, ln sum exp((x - max) / T)
  __shared__ uint32_t s_ok[JET_MAX_NODES / 32], s_best[kSampleThreads / 32], s_end_row[JET_MAX_NODES / 32];
  __shared__ int s_end, s_has_child, s_pick_warp, s_token;
  __shared__ double s_wsum[kSampleThreads / 32], s_before;

  const int b = blockIdx.x, v = threadIdx.x, lane = v & 31, warp = v >> 5;
  const int n = min(n_nodes[b], B);
  const int words = (B + 31) / 32;
  const size_t o = static_cast<size_t>(b) * B;
  const bool live = v < n;
  const float* lp = draft_logp + b * logp_batch_stride;

  // ---- row statistics
  if (live) {
    const float2* pr = partial + (o + v) * nchunks;
    float m = -INFINITY;
    for (int c = 0; c < nchunks; ++c) m = fmaxf(m, pr[c].x);
    float s = 0.0f;
    for (int c = 0; c < nchunks; ++c) {
      const float2 q = pr[c];
      if (q.x > -INFINITY) s += q.y * exp2f((q.x - m) * inv_t * kLog2e);
    }
    s_max[v] = m;
    s_lnsum[v] = logf(s);
  }
  if (v == 0) s_has_child = 0;
  __syncthreads();

  // ---- alpha_v = min(1, p_parent(token) / q_depth(parent)(token)); accepted iff u_v < alpha_v
  int my_parent = -1, my_depth = -1, my_token = -1;
  float alpha = 1.0f;
  bool ok = live && v == 0;
  if (live) { my_parent = parent[o + v]; my_depth = depth[o + v]; my_token = token[o + v]; }
  if (live && v > 0 && my_parent >= 0 && my_parent < n && my_token >= 0 && my_token < V) {
    const float lq = lp[static_cast<int64_t>(my_depth - 1) * logp_depth_stride + my_token];
    if (lq > -INFINITY) {
      const float x = logits[static_cast<int64_t>(o + my_parent) * row_stride + my_token];
      const float lr = (x - s_max[my_parent]) * inv_t - s_lnsum[my_parent] - lq;      // ln(p / q)
      alpha = lr >= 0.0f ? 1.0f : expf(lr);
    }
    ok = u_accept[o + v] < alpha;
  }
  if (alpha_out && v < B) alpha_out[o + v] = live ? alpha : 0.0f;
  const uint32_t okbits = __ballot_sync(0xffffffffu, ok);
  if (lane == 0 && warp < JET_MAX_NODES / 32) s_ok[warp] = okbits;
  __syncthreads();

  // ---- deepest node whose branch is accepted throughout (ties -> lowest index)
  bool acc = live;
  if (live) {
    const uint32_t* row = anc_mask + (o + v) * words;
    for (int w = 0; w < words; ++w) acc = acc && ((row[w] & ~s_ok[w]) == 0u);
  }
  uint32_t key = acc ? ((static_cast<uint32_t>(my_depth) << 16) | (0xFFFFu - v)) : 0u;
  key = __reduce_max_sync(0xffffffffu, key);
  if (lane == 0) s_best[warp] = key;
  __syncthreads();
  if (warp == 0) {
    uint32_t k = lane < kSampleThreads / 32 ? s_best[lane] : 0u;
    k = __reduce_max_sync(0xffffffffu, k);
    if (lane == 0) s_end = k ? static_cast<int>(0xFFFFu - (k & 0xFFFFu)) : 0;
  }
  __syncthreads();
  const int end = s_end;
  if (v < words) s_end_row[v] = anc_mask[(o + end) * words + v];
  if (live && my_parent == end) s_has_child = 1;          // benign race: every writer stores 1
  __syncthreads();
  const int a = n > 0 ? depth[o + end] : 0;
  const bool residual = s_has_child != 0;

  // ---- correction token: inverse CDF over the vocabulary of r(x) = max(0, p(x) - q(x)) (or p(x)).
  //      Every warp owns a contiguous range of the vocabulary; pass 1 sums the ranges, pass 2 walks the range
  //      that contains the target mass.  If the residual has no mass the draw falls back to p.
  const float* xrow = logits + static_cast<int64_t>(o + end) * row_stride;
  const float* qrow = lp + static_cast<int64_t>(a) * logp_depth_stride;      // only read when the node has children (a < N)
  const float m_e = s_max[end], ln_e = s_lnsum[end];
  constexpr int kWarps = kSampleThreads / 32;
  const int per_warp = ((V + kWarps - 1) / kWarps + 31) / 32 * 32;
  const int lo = warp * per_warp, hi = min(V, lo + per_warp);
  auto mass = [&](int idx, bool use_residual) -> float {
    const float pe = expf((xrow[idx] - m_e) * inv_t - ln_e);
    if (!use_residual) return pe;
    return fmaxf(0.0f, pe - expf(qrow[idx]));
  };
  bool use_residual = residual;
  int picked = -1;
  for (int attempt = 0; attempt < 2 && picked < 0; ++attempt) {
    double part = 0.0;
    for (int idx = lo + lane; idx < hi; idx += 32) part += static_cast<double>(mass(idx, use_residual));
    part = warp_sum_d(part);
    if (lane == 0) s_wsum[warp] = part;
    __syncthreads();
    if (v == 0) {
      double total = 0.0;
      for (int w = 0; w < kWarps; ++w) total += s_wsum[w];
      s_pick_warp = -1;
      s_token = -1;
      if (total > 0.0) {
        const double target = static_cast<double>(u_sample[b]) * total;
        double cum = 0.0;
        int pick = -1;
        for (int w = 0; w < kWarps; ++w) {
          if (s_wsum[w] > 0.0) {
            pick = w;                                  // last range with mass, unless an earlier one exceeds the target
            if (cum + s_wsum[w] > target) break;
          }
          cum += s_wsum[w];
        }
        // cum = mass before range `pick` (ranges after the break are not added)
        double before = 0.0;
        for (int w = 0; w < pick; ++w) before += s_wsum[w];
        s_before = before;
        s_pick_warp = pick;
        s_wsum[0] = target;                            // reuse: the target mass for pass 2
      }
    }
    __syncthreads();
    if (s_pick_warp < 0) {                             // no mass: fall back to the target distribution itself
      use_residual = false;
      __syncthreads();
      continue;
    }
    if (warp == s_pick_warp) {
      const double target = s_wsum[0];
      double run = s_before;
      int found = -1, last_pos = -1;
      for (int start = lo; start < hi && found < 0; start += 32) {
        const int idx = start + lane;
        const float mval = idx < hi ? mass(idx, use_residual) : 0.0f;
        // inclusive prefix sum over the warp
        double pre = static_cast<double>(mval);
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, pre, off);
          if (lane >= off) pre += up;
        }
        const bool hit = mval > 0.0f && run + pre > target;
        const unsigned hits = __ballot_sync(0xffffffffu, hit);
        const unsigned pos = __ballot_sync(0xffffffffu, mval > 0.0f);
        if (pos) last_pos = start + 31 - __clz(pos);
        if (hits) found = start + __ffs(hits) - 1;
        run += __shfl_sync(0xffffffffu, pre, 31);
      }
      if (found < 0) found = last_pos;                 // rounding left the target just above the range's mass
      if (lane == 0) s_token = found;
    }
    __syncthreads();
    picked = s_token;
    __syncthreads();
  }

  // ---- outputs
  int32_t* my_path = path + static_cast<size_t>(b) * (N + 1);
  int32_t* my_tok = out_tokens + static_cast<size_t>(b) * (N + 1);
  for (int i = v; i <= N; i += kSampleThreads)
    if (i > a) { my_path[i] = -1; my_tok[i] = -1; }
  if (live && ((s_end_row[v >> 5] >> (v & 31)) & 1u) && my_depth <= N) {
    my_path[my_depth] = v;
    if (my_depth >= 1) my_tok[my_depth - 1] = my_token;
  }
  if (v == 0) { accept_len[b] = a; my_tok[a] = picked; }
}

int lse_chunks_for(int V) { return (V + kLseChunk - 1) / kLseChunk; }

}  // namespace
}  // namespace jet

extern "C" size_t jet_tree_accept_sample_workspace_bytes(int batch, int B, int V) {
  if (batch < 1 || B < 1 || V < 1) return 0;
  return jet::round_up(static_cast<size_t>(batch) * B * jet::lse_chunks_for(V) * sizeof(float2), 256);
}

extern "C" jet_status jet_tree_accept_sample(const float* logits, int64_t logits_row_stride, float temperature,
                                             const float* draft_logp, int64_t logp_batch_stride,
                                             int64_t logp_depth_stride, const int32_t* token,
                                             const int32_t* parent, const int32_t* depth,
                                             const uint32_t* anc_mask, const int32_t* n_nodes,
                                             const float* u_accept, const float* u_sample, int batch, int B,
                                             int V, int N, float* alpha, int32_t* accept_len, int32_t* path,
                                             int32_t* out_tokens, void* workspace, size_t workspace_bytes,
                                             void* stream) {
  using namespace jet;
  if (!logits || !draft_logp || !token || !parent || !depth || !anc_mask || !n_nodes || !u_accept || !u_sample ||
      !accept_len || !path || !out_tokens)
    return JET_ERR_INVALID_ARG;
  if (batch < 1 || B < 1 || B > JET_MAX_NODES || V < 1 || N < 1 || N > JET_MAX_DEPTH || logits_row_stride < V ||
      logp_depth_stride < V || logp_batch_stride < 0 || static_cast<int64_t>(batch) * B > 65535)
    return JET_ERR_INVALID_ARG;
  if (!(temperature > 0.0f) || !(temperature < INFINITY)) return JET_ERR_INVALID_ARG;
  if (!aligned(logits, 4) || !aligned(draft_logp, 4)) return JET_ERR_INVALID_ARG;
  const size_t need = jet_tree_accept_sample_workspace_bytes(batch, B, V);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < need) return JET_ERR_WORKSPACE;

  const int nchunks = lse_chunks_for(V);
  const bool vec_ok = aligned(logits, 16) && logits_row_stride % 4 == 0;
  const float inv_t = 1.0f / temperature;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto* partial = static_cast<float2*>(workspace);
  launch_dependent(row_lse_partial_kernel, dim3(nchunks, batch * B), dim3(kLseThreads), st, logits,
                   logits_row_stride, V, B, n_nodes, nchunks, vec_ok, inv_t * kLog2e, partial);
  launch_dependent(accept_sample_kernel, dim3(batch), dim3(kSampleThreads), st,
                   static_cast<const float2*>(partial), nchunks, logits, logits_row_stride, inv_t, draft_logp,
                   logp_batch_stride, logp_depth_stride, token, parent, depth, anc_mask, n_nodes, u_accept,
                   u_sample, B, V, N, alpha, accept_len, path, out_tokens);
  return launch_status();
}
