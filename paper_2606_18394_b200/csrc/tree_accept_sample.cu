// jet_tree_accept_sample: non-greedy tree acceptance (Section 3.3, Eq. nongreedy_specdec).
//
// Two launches:
//   row_lse_partial_kernel  grid (slices, batch*B): one pass over the target logits; every block
//                           leaves the maximum and the sum of exp((x - max) / T) of one 8192-entry
//                           slice of one row in the workspace.  Padding rows are not read.
//   accept_sample_kernel    one cluster of 8 CTAs per sequence, 1024 threads each: finishes the rows' log-sum-exp, computes
//                           alpha_v = min(1, p_parent(token_v) / q_depth(token_v)) and the accept
//                           bit u_v < alpha_v for every node, picks the deepest node whose whole
//                           branch is accepted, then draws the correction token at that node by
//                           inverse CDF in vocabulary order (residual max(0, p - q) if the node has
//                           rejected children, p itself if it is a leaf).  Every CTA of the cluster
//                           repeats the (small) per-node part; the pass over the vocabulary that sums
//                           the masses is split between the CTAs, which leave their sums in the shared
//                           memory of CTA 0; CTA 0 locates the token.
#include <cooperative_groups.h>

#include "jet_common.cuh"

namespace jet {
namespace {

constexpr int kLseThreads = 256;
constexpr int kLseElems = 32;
constexpr int kLseChunk = kLseThreads * kLseElems;
constexpr int kSampleThreads = 1024;
constexpr int kSampleStep = 128;          // vocabulary entries a warp handles per step (4 per lane)
constexpr int kSampleCluster = 8;         // CTAs per sequence
constexpr int kMaxStepsTotal = 4096;      // 128-entry steps per row: vocabularies up to 524288 entries
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
                     const float* __restrict__ u_sample, int B, int V, int N, bool vec_rows, float* __restrict__ alpha_out,
                     int32_t* __restrict__ accept_len, int32_t* __restrict__ path,
                     int32_t* __restrict__ out_tokens) {
  grid_dependency_wait();
  __shared__ float s_max[JET_MAX_NODES], s_lnsum[JET_MAX_NODES];      // per row: max, ln sum exp((x - max) / T)
  __shared__ uint32_t s_ok[JET_MAX_NODES / 32], s_best[kSampleThreads / 32], s_end_row[JET_MAX_NODES / 32];
  __shared__ int s_end, s_has_child, s_pick_warp, s_pick_step, s_token;
  __shared__ double s_step[kMaxStepsTotal], s_before, s_target;      // CTA 0: mass of every 128-entry step, vocabulary order

  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / kSampleCluster, v = threadIdx.x, lane = v & 31, warp = v >> 5;
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
  if (live && v > 0 && my_parent >= 0 && my_parent < n && my_token >= 0 && my_token < V && my_depth >= 1 && my_depth <= N) {
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
  if (lane == 0 && warp < JET_MAX_NODES / 32) s_ok[warp] = okbits;      // threads beyond the budget hold no node
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
  // (clamped: the arrays of a tree are the caller's and are not validated; a depth outside 0 .. N must not turn
  //  into a store outside the N + 1 entries of this sequence's outputs)
  const int a = n > 0 ? min(max(depth[o + end], 0), N) : 0;
  const bool residual = s_has_child != 0;

  // ---- correction token: inverse CDF over the vocabulary of r(x) = max(0, p(x) - q(x)) (or p(x)).
  //      Every warp owns a contiguous range of the vocabulary and walks it in steps of 128 entries (4 per
  //      lane), keeping the mass of every step (fp64) in shared memory; one thread then finds the warp and
  //      the step that contain the target mass, and that warp recomputes the one step to locate the token.
  //      If the residual has no mass the draw falls back to p.
  const float* xrow = logits + static_cast<int64_t>(o + end) * row_stride;
  const float* qrow = lp + static_cast<int64_t>(a) * logp_depth_stride;      // only read when the node has children (a < N)
  const float m_e = s_max[end], ln_e = s_lnsum[end];
  constexpr int kWarps = kSampleThreads / 32;
  const int total_steps = (V + kSampleStep - 1) / kSampleStep;              // host checks <= kMaxStepsTotal
  const int steps = (total_steps + kWarps * kSampleCluster - 1) / (kWarps * kSampleCluster);      // per warp
  const int first_step = (rank * kWarps + warp) * steps;                    // this warp's steps, vocabulary order
  const bool vec = vec_rows;
  // masses of the 4 entries of this lane in step `g` (global step index)
  auto masses = [&](int g, bool use_residual, float (&mval)[4]) {
    const int idx = g * kSampleStep + lane * 4;
    float x4[4], q4[4] = {0.f, 0.f, 0.f, 0.f};
    if (vec && idx + 3 < V) {
      const float4 t = *reinterpret_cast<const float4*>(xrow + idx);
      x4[0] = t.x; x4[1] = t.y; x4[2] = t.z; x4[3] = t.w;
      if (use_residual) {
        const float4 u4 = *reinterpret_cast<const float4*>(qrow + idx);
        q4[0] = u4.x; q4[1] = u4.y; q4[2] = u4.z; q4[3] = u4.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        x4[j] = idx + j < V ? xrow[idx + j] : -INFINITY;
        if (use_residual) q4[j] = idx + j < V ? qrow[idx + j] : -INFINITY;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float pe = expf((x4[j] - m_e) * inv_t - ln_e);
      mval[j] = use_residual ? fmaxf(0.0f, pe - expf(q4[j])) : pe;
    }
  };
  double* step0 = cluster.map_shared_rank(&s_step[0], 0);      // the step table lives in CTA 0
  cluster.sync();                                              // every CTA of the cluster is running
  bool use_residual = residual;
  int picked = -1;
  for (int attempt = 0; attempt < 2; ++attempt) {
    for (int st = 0; st < steps; ++st) {
      const int g = first_step + st;
      if (g < total_steps) {
        float mval[4];
        masses(g, use_residual, mval);
        const double part = warp_sum_d(static_cast<double>(mval[0]) + mval[1] + mval[2] + mval[3]);
        if (lane == 0) step0[g] = part;
      }
    }
    cluster.sync();                                            // the table is complete
    bool retry = false;
    if (rank == 0) {
      if (warp == 0) {
        // lane i: mass of a contiguous run of steps; inclusive scan over the lanes = cumulative mass
        const int per_lane = (total_steps + 31) / 32;
        const int s_lo = lane * per_lane, s_hi = min(total_steps, s_lo + per_lane);
        double tot_l = 0.0;
        for (int g = s_lo; g < s_hi; ++g) tot_l += s_step[g];
        double cum_l = tot_l;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, cum_l, off);
          if (lane >= off) cum_l += up;
        }
        const double total = __shfl_sync(0xffffffffu, cum_l, 31);
        const double target = static_cast<double>(u_sample[b]) * total;
        // the run that holds the target: first with mass whose cumulative mass exceeds it, else the last with mass
        const unsigned has = __ballot_sync(0xffffffffu, tot_l > 0.0);
        const unsigned over = __ballot_sync(0xffffffffu, tot_l > 0.0 && cum_l > target);
        const int pl = over ? __ffs(over) - 1 : (has ? 31 - __clz(has) : -1);
        int ps = -1;
        double before = 0.0;
        if (lane == pl) {                                      // walk that run step by step
          double run = cum_l - tot_l;
          int last_step = -1;
          double last_before = 0.0;
          for (int g = s_lo; g < s_hi; ++g) {
            const double m = s_step[g];
            if (m > 0.0) {
              last_step = g; last_before = run;
              if (run + m > target) { ps = g; before = run; break; }
            }
            run += m;
          }
          if (ps < 0) { ps = last_step; before = last_before; }
          s_pick_step = ps;
          s_before = before;
          s_target = target;
        }
        if (lane == 0) { s_token = -1; if (pl < 0) s_pick_step = -1; }
      }
      __syncthreads();
      if (s_pick_step < 0) {
        retry = true;                                          // no mass: fall back to the target distribution itself
      } else if (warp == 0) {
        float mval[4];
        masses(s_pick_step, use_residual, mval);
        const double mine = static_cast<double>(mval[0]) + mval[1] + mval[2] + mval[3];
        double pre = mine;                                     // inclusive prefix sum over the lanes
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, pre, off);
          if (lane >= off) pre += up;
        }
        double run = s_before + pre - mine;                    // mass before this lane's entries
        int found = -1, last_pos = -1;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          run += static_cast<double>(mval[j]);
          if (mval[j] > 0.0f) {
            last_pos = j;
            if (found < 0 && run > s_target) found = j;
          }
        }
        const unsigned hits = __ballot_sync(0xffffffffu, found >= 0);
        const unsigned pos = __ballot_sync(0xffffffffu, last_pos >= 0);
        const int base_idx = s_pick_step * kSampleStep;
        if (hits) {
          const int src = __ffs(hits) - 1;
          const int j = __shfl_sync(0xffffffffu, found, src);
          if (lane == 0) s_token = base_idx + src * 4 + j;
        } else if (pos) {                                      // rounding left the target just above the step's mass
          const int src = 31 - __clz(pos);
          const int j = __shfl_sync(0xffffffffu, last_pos, src);
          if (lane == 0) s_token = base_idx + src * 4 + j;
        }
      }
      __syncthreads();
      picked = s_token;
    }
    // the whole cluster learns whether the pass has to be repeated with p itself (only when the residual is empty)
    int* retry_flag = cluster.map_shared_rank(&s_pick_warp, 0);
    if (rank == 0 && v == 0) s_pick_warp = retry ? 1 : 0;
    cluster.sync();
    const bool again = *retry_flag != 0 && use_residual;
    cluster.sync();                                            // everybody has read the flag before it changes again
    if (!again) break;
    use_residual = false;
  }
  if (rank != 0) return;                                       // CTA 0 alone writes the results

  // ---- outputs
  int32_t* my_path = path + static_cast<size_t>(b) * (N + 1);
  int32_t* my_tok = out_tokens + static_cast<size_t>(b) * (N + 1);
  for (int i = v; i <= N; i += kSampleThreads)
    if (i > a) { my_path[i] = -1; my_tok[i] = -1; }
  if (live && ((s_end_row[v >> 5] >> (v & 31)) & 1u) && my_depth >= 0 && my_depth <= N) {
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

  if (V > kMaxStepsTotal * kSampleStep) return JET_ERR_UNSUPPORTED;
  const int nchunks = lse_chunks_for(V);
  const bool vec_rows = aligned(logits, 16) && aligned(draft_logp, 16) && logits_row_stride % 4 == 0 &&
                        logp_depth_stride % 4 == 0 && logp_batch_stride % 4 == 0;
  const bool vec_ok = aligned(logits, 16) && logits_row_stride % 4 == 0;
  const float inv_t = 1.0f / temperature;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto* partial = static_cast<float2*>(workspace);
  launch_dependent(row_lse_partial_kernel, dim3(nchunks, batch * B), dim3(kLseThreads), st, logits,
                   logits_row_stride, V, B, n_nodes, nchunks, vec_ok, inv_t * kLog2e, partial);
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(batch * kSampleCluster);
    cfg.blockDim = dim3(kSampleThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kSampleCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, accept_sample_kernel, static_cast<const float2*>(partial), nchunks, logits,
                           logits_row_stride, inv_t, draft_logp, logp_batch_stride, logp_depth_stride, token, parent,
                           depth, anc_mask, n_nodes, u_accept, u_sample, B, V, N, vec_rows, alpha, accept_len, path,
                           out_tokens) != cudaSuccess) {
      cudaGetLastError();
      return JET_ERR_CUDA;
    }
  }
  return launch_status();
}
