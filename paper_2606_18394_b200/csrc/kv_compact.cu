// jet_kv_compact: commit of the accepted path.  One launch copies the K and V rows of
// every accepted node of every layer and sequence behind the prefix (contiguous or paged
// cache); a second one-block launch then advances seq_len, so that no copy block can see
// an already advanced length.
#include "jet_common.cuh"

namespace jet {
namespace {

__global__ void __launch_bounds__(256)
kv_compact_kernel(const uint4* __restrict__ tree_k, const uint4* __restrict__ tree_v,
                  uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                  int64_t layer_stride16, int64_t batch_stride16,
                  const int32_t* __restrict__ page_table, int max_pages, int page_size,
                  const int32_t* __restrict__ path, const int32_t* __restrict__ accept_len,
                  const int32_t* __restrict__ seq_len, int batch, int B, int row16, int N) {
  grid_dependency_wait();
  const int i = blockIdx.x, b = blockIdx.y, layer = blockIdx.z;
  if (i > accept_len[b]) return;
  const int node = path[static_cast<size_t>(b) * (N + 1) + i];
  if (node < 0 || node >= B) return;
  const int64_t pos = static_cast<int64_t>(seq_len[b]) + i;
  int64_t dst_row;
  if (pos < 0) return;
  if (page_table) {
    if (pos / page_size >= max_pages) return;        // (a length beyond the table is the caller's error: no access outside it)
    const int page = page_table[static_cast<size_t>(b) * max_pages + pos / page_size];
    dst_row = static_cast<int64_t>(page) * page_size + pos % page_size;
    dst_row = layer * layer_stride16 + dst_row * row16;
  } else {
    dst_row = layer * layer_stride16 + b * batch_stride16 + pos * row16;
  }
  const int64_t src = ((static_cast<int64_t>(layer) * batch + b) * B + node) * row16;
  for (int t = threadIdx.x; t < 2 * row16; t += blockDim.x) {
    if (t < row16) k_cache[dst_row + t] = tree_k[src + t];
    else v_cache[dst_row + t - row16] = tree_v[src + t - row16];
  }
}

// In-place variant: the tree's K/V rows sit in the cache at positions seq_len + node.  Row seq_len + path[i]
// moves to seq_len + i for i = 1 .. accept_len (path[i] >= i; the root stays where it is).  One block per
// (sequence, layer, K or V): all source rows are read into registers before any is written, with a block-wide
// barrier in between, so overlapping source and destination ranges are safe.
constexpr int kTailThreads = 256;
constexpr int kTailHeld = 8;           // 16-byte pieces a thread can hold: 256 * 8 * 16 bytes = 32 KiB per block pass

__global__ void __launch_bounds__(kTailThreads)
kv_compact_tail_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache, int64_t layer_stride16,
                       int64_t batch_stride16, const int32_t* __restrict__ page_table, int max_pages,
                       int page_size, const int32_t* __restrict__ path, const int32_t* __restrict__ accept_len,
                       const int32_t* __restrict__ seq_len, int B, int row16, int N) {
  grid_dependency_wait();
  const int b = blockIdx.x, layer = blockIdx.y;
  uint4* cache = blockIdx.z == 0 ? k_cache : v_cache;
  const int a = min(accept_len[b], N);
  const int64_t L = seq_len[b];
  auto row_of = [&](int64_t pos) -> int64_t {
    if (page_table) {
      // (the index is kept inside the table: a length beyond it is the caller's error and must not become an access
      //  outside the table)
      const int64_t slot = min(max(pos / page_size, static_cast<int64_t>(0)), static_cast<int64_t>(max_pages - 1));
      const int page = page_table[static_cast<size_t>(b) * max_pages + slot];
      return layer * layer_stride16 + (static_cast<int64_t>(page) * page_size + pos % page_size) * row16;
    }
    return layer * layer_stride16 + b * batch_stride16 + pos * row16;
  };
  // pieces of the rows i = 1 .. a, in passes of what the block can hold; a pass never writes a row that a later
  // pass still has to read, because rows are taken in increasing i and path[i] >= i, path increasing
  const int total = a * row16;
  for (int base = 0; base < total; base += kTailThreads * kTailHeld) {
    uint4 held[kTailHeld];
#pragma unroll
    for (int k = 0; k < kTailHeld; ++k) {
      const int e = base + k * kTailThreads + threadIdx.x;
      if (e < total) {
        const int i = 1 + e / row16, piece = e % row16;
        const int node = path[static_cast<size_t>(b) * (N + 1) + i];
        held[k] = (node >= 0 && node < B) ? cache[row_of(L + node) + piece] : make_uint4(0u, 0u, 0u, 0u);
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTailHeld; ++k) {
      const int e = base + k * kTailThreads + threadIdx.x;
      if (e < total) {
        const int i = 1 + e / row16, piece = e % row16;
        const int node = path[static_cast<size_t>(b) * (N + 1) + i];
        if (node >= 0 && node < B && node != i) cache[row_of(L + i) + piece] = held[k];
      }
    }
    __syncthreads();
  }
}

__global__ void advance_seq_len_kernel(const int32_t* __restrict__ accept_len,
                                       int32_t* __restrict__ seq_len, int batch) {
  grid_dependency_wait();
  for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < batch; b += gridDim.x * blockDim.x)
    seq_len[b] += accept_len[b] + 1;
}

}  // namespace
}  // namespace jet

extern "C" jet_status jet_kv_compact(const void* tree_k, const void* tree_v, void* k_cache,
                                     void* v_cache, int64_t cache_layer_stride,
                                     int64_t kv_batch_stride, const int32_t* page_table,
                                     int max_pages_per_seq, int page_size, const int32_t* path,
                                     const int32_t* accept_len, int32_t* seq_len, int layers,
                                     int batch, int B, int Hkv, int D, int N, void* stream) {
  using namespace jet;
  if (!tree_k || !tree_v || !k_cache || !v_cache || !path || !accept_len || !seq_len)
    return JET_ERR_INVALID_ARG;
  if (layers < 1 || layers > 65535 || batch < 1 || batch > 65535 || B < 1 || B > JET_MAX_NODES ||
      Hkv < 1 || D < 1 || N < 1 || N > JET_MAX_DEPTH)
    return JET_ERR_INVALID_ARG;
  const int64_t row_elems = static_cast<int64_t>(Hkv) * D;
  if (row_elems % 8 != 0 || cache_layer_stride % 8 != 0) return JET_ERR_INVALID_ARG;   // 16-byte rows
  if (!aligned(tree_k, 16) || !aligned(tree_v, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16))
    return JET_ERR_INVALID_ARG;
  if (page_table) {
    if (page_size < 1 || max_pages_per_seq < 1) return JET_ERR_INVALID_ARG;
  } else if (kv_batch_stride % 8 != 0 || kv_batch_stride < 0) {
    return JET_ERR_INVALID_ARG;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int row16 = static_cast<int>(row_elems / 8);
  launch_dependent(kv_compact_kernel, dim3(N + 1, batch, layers), dim3(256), st,
      static_cast<const uint4*>(tree_k), static_cast<const uint4*>(tree_v),
      static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), cache_layer_stride / 8,
      kv_batch_stride / 8, page_table, max_pages_per_seq, page_size, path, accept_len, seq_len,
      batch, B, row16, N);
  launch_dependent(advance_seq_len_kernel, dim3(1), dim3(256), st, accept_len, seq_len, batch);
  return launch_status();
}

extern "C" jet_status jet_kv_compact_tail(void* k_cache, void* v_cache, int64_t cache_layer_stride,
                                          int64_t kv_batch_stride, const int32_t* page_table,
                                          int max_pages_per_seq, int page_size, const int32_t* path,
                                          const int32_t* accept_len, int32_t* seq_len, int layers, int batch,
                                          int B, int Hkv, int D, int N, void* stream) {
  using namespace jet;
  if (!k_cache || !v_cache || !path || !accept_len || !seq_len) return JET_ERR_INVALID_ARG;
  if (layers < 1 || layers > 65535 || batch < 1 || B < 1 || B > JET_MAX_NODES || Hkv < 1 || D < 1 || N < 1 ||
      N > JET_MAX_DEPTH)
    return JET_ERR_INVALID_ARG;
  const int64_t row_elems = static_cast<int64_t>(Hkv) * D;
  if (row_elems % 8 != 0 || cache_layer_stride % 8 != 0) return JET_ERR_INVALID_ARG;   // 16-byte rows
  if (!aligned(k_cache, 16) || !aligned(v_cache, 16)) return JET_ERR_INVALID_ARG;
  if (page_table) {
    if (page_size < 1 || max_pages_per_seq < 1) return JET_ERR_INVALID_ARG;
  } else if (kv_batch_stride % 8 != 0 || kv_batch_stride < 0) {
    return JET_ERR_INVALID_ARG;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int row16 = static_cast<int>(row_elems / 8);
  launch_dependent(kv_compact_tail_kernel, dim3(batch, layers, 2), dim3(kTailThreads), st,
      static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), cache_layer_stride / 8, kv_batch_stride / 8,
      page_table, max_pages_per_seq, page_size, path, accept_len, seq_len, B, row16, N);
  launch_dependent(advance_seq_len_kernel, dim3(1), dim3(256), st, accept_len, seq_len, batch);
  return launch_status();
}
