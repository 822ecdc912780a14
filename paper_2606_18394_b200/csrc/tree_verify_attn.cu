// jet_tree_verify_attn: tree attention over prefix KV + tree KV under the ancestor mask.
//
// Kernel structure (one CTA per SM, warp-specialised):
//   work item   = (sequence b, KV head g, group of MT 128-row query tiles, key slice s).
//                 Row r of a query tile is (node v, query head g*G + j) with r = v_local*G + j,
//                 so all G heads of a KV group share every K/V tile that is loaded.
//   warp 0      = TMA producer: Q tiles once, then K and V tiles (128 keys) through a ring of
//                 shared-memory stages; paged caches are fetched one 16-row page per TMA box.
//   warp 1      = tcgen05 issuer: S = Q K^T into TMEM, O += P V into TMEM (outside the classic
//                 form of the key loop warp 1 issues the Q K^T and warp 3 the P V products; warp 2 is
//                 a second TMA producer where a paged cache or two query tiles call for one).
//   warp 2      = TMEM allocation / release.
//   warps 4..11 = two softmax warpgroups, one thread per row: the thread reads its 128 scores of a key
//                 tile from TMEM, replaces the scores of keys the row must not see (key validity,
//                 ancestor bits) by -inf, exponentiates against the row's reference maximum, adds
//                 to the row sum and writes P (bf16) back to TMEM, where the P V product reads it.
//   key loop    = with one query tile per CTA: both warpgroups (alternate key tiles) add into one
//                 accumulator against a reference fixed after the first tile; if a row overflows that
//                 reference the CTA repeats the key range in the classic form (own accumulator and
//                 running maximum per stream, accumulator rescaled when the maximum rises).  With two
//                 query tiles per CTA each warpgroup owns a tile with the classic bookkeeping, and the
//                 tiles take turns on one score buffer.  See "the key loop" below.
//   key slices  = when there are fewer work items than SMs the key range is cut into `nsplit`
//                 slices.  After the key loop every CTA stages its normalised rows (bf16) and their
//                 log-sum-exp; the rows' owner CTAs collect them -- by loads from their peers' shared
//                 memory when the slices form a thread-block cluster, else through the workspace -- combine
//                 the slices and write the output.  With few rows and many slices the combination is left
//                 to a second, small launch (tree_attn_merge_kernel) instead.
//   CTA pairs   = an optional form (JET_FORCE_PAIR=1; measured slower, never the planner's choice): two CTAs with
//                 consecutive query tiles of a work item form a cluster, each loads half of every K/V tile and
//                 the products run as tcgen05 cta_group::2 instructions.  See "CTA pairs" in the kernel.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their
// loops (still taking part in the CTA-wide and cluster barriers), outstanding TMA loads are drained,
// TMEM is released and JET_ERR_TIMEOUT is reported.
#include <cuda.h>
#include <cuda_bf16.h>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <type_traits>

#include "jet_common.cuh"
#include "sm100_ptx.cuh"

namespace jet {

#ifdef JET_TRACE
long long* g_trace_ptr = nullptr;    // debug builds only
#endif

namespace {

constexpr int kBM = 128;               // query rows per tile
constexpr int kBN = 128;               // keys per tile
constexpr int kHalfBytes = 128 * 128;  // one [128 rows x 64 bf16] swizzled block
constexpr int kMaxSplit = 20;          // most key slices (a cluster holds at most 16; more only through the workspace)
constexpr int kMaxCluster = 16;        // largest thread-block cluster the hardware launches (non-portable size)
constexpr int kMaxSorted = 128;          // batches up to this size are launched longest prefix first
constexpr float kSharedSumFloor = 8.6736174e-19f;  // 2^-60: a row that saw keys but summed to less has lost them to underflow
constexpr float kSharedSumLimit = 1.2089258e24f;   // 2^80: tile sums a fixed reference may reach before the CTA falls back
constexpr float kFastSumLimit = 256.0f;    // a row keeps its reference maximum while its tile sums stay below (so P <= 2^8)

struct AttnParams {
  const int32_t* page_table;
  const int32_t* seq_len;
  const int32_t* n_nodes;
  const uint32_t* anc_mask;
  __nv_bfloat16* out;
  float* lse;
  int32_t* status;
  int max_pages, paged;
  int tail;           // the tree's K/V rows sit in the cache behind the prefix (rows seq_len .. seq_len + n - 1)
  int batch, B, Hq, Hkv, G, words;
  int nsplit, n_mgroups, n_units;
  // The code around the key loop runs once per launch, from a cold instruction cache: its cost is its
  // instruction count.  What the host can work out arrives ready-made, and divisions by the two run-time
  // divisors are multiplications by these reciprocals (udiv below).
  int rows_per;       // ceil(128 / nsplit): rows of a query tile that one slice combines
  int npt;            // 128 / G: nodes per query tile
  uint32_t magic_S, magic_G;
  int len_hint;       // the caller's bound on the cached keys (max_seq_len); 0 = none
  uint32_t poll_limit;  // workspace merge: polls of the arrival count before the CTA gives up (about a second)
  int stable;         // JET_ATTN_STABLE_PREFIX: lengths, page table and prefix rows may be read before the dependency wait
  int via_global;     // key slices exchange their rows through the workspace instead of a cluster: 1 = inside this
                      // launch (arrival counters, bounded spin), 2 = a second launch combines them
  int* counters;      // via_global: [2][units * MT] arrival / departure counts, zero between calls
  uint8_t* partials;  // via_global: [units * nsplit * MT][128 rows][D bf16 + log2-sum-exp (fp32) + pad]
  float scale_log2;   // softmax_scale * log2(e)
#ifdef JET_TRACE
  long long* trace;   // 64 clock64() samples per CTA
#endif
};

// floor(x / d) for d <= 128 and x < 2^25, with magic = ceil(2^32 / d) (0 stands for d == 1).
__host__ __device__ inline uint32_t udiv_magic(uint32_t d) { return d == 1 ? 0u : static_cast<uint32_t>(((1ull << 32) + d - 1) / d); }
__device__ __forceinline__ uint32_t udiv(uint32_t x, uint32_t magic) { return magic ? __umulhi(x, magic) : x; }

#ifdef JET_TRACE
#define JET_TR(slot) do { if (p.trace) p.trace[(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 64 + (slot)] = clock64(); } while (0)
#else
#define JET_TR(slot) do { } while (0)
#endif

// kPair: two CTAs (a cluster of two, consecutive query tiles of one work item) share every K/V tile -- each
// loads half of it, and the products run as tcgen05 pair instructions (see "CTA pairs" in the kernel).
template <int D, int MT, bool kPair = false>
struct Cfg {
  static_assert(!kPair || (D == 128 && MT == 1), "the CTA-pair form exists for one 128-wide query tile per CTA");
  static constexpr int kHalves = D / 64;
  static constexpr int kQBytes = MT * kHalves * kHalfBytes;
  // P (probabilities, bf16) never touches shared memory: it is written to TMEM (two bf16 per 32-bit column)
  // and read from there by the P V product.
  static constexpr int kPBytes = 0;
  // (a pair's stage holds half a tile: 64 keys x D of K, or 128 keys x 64 columns of V)
  static constexpr int kStageBytes = kPair ? kHalfBytes : kHalves * kHalfBytes;
  static constexpr int kStages = kPair ? 10 : (D == 128) ? (MT == 1 ? 6 : 5) : 6;
  static constexpr int kTileBytes = kQBytes + kPBytes + kStages * kStageBytes;
  // Two softmax warpgroups in every form: with one query tile per CTA they share the tile's key tiles (even /
  // odd), with two each takes one query tile.
  static constexpr int kStreams = MT == 1 ? 2 : 1;
  static constexpr int kBarBytes = kPair ? 2048 : 1024;
  static constexpr int kSmemBytes = kTileBytes + kBarBytes + 1024;
  static constexpr int kThreads = 128 + 128 * MT * kStreams;
  // TMEM (512 columns), three layouts (the key loop's forms are described in the kernel):
  //   MT == 1, shared-accumulator pass: O [0, +D), warpgroup w: scores [128 + 128 w, +128), P [384 + 64 w, +64)
  //   MT == 1, classic pass (fallback): stream i: scores / P [i*128, +128), O [256 + i*128, +D); key tile t
  //            belongs to stream t & 1
  //   MT == 2: O of query tile mt [mt*128, +D), ONE score buffer [256, +128) that the two query tiles use in
  //            turn, P of query tile mt [384 + 64 mt, +64)
  static constexpr int kTmemCols = 512;
  __device__ static constexpr uint32_t s_col(int mt, int t) { return (t & 1) * 128; }
  __device__ static constexpr uint32_t o_col(int mt, int t) { return 256 + (t & 1) * 128; }
  // Each score buffer (and the P that replaces it) has its own barriers, so that neither side can run two
  // phases ahead of the other on one barrier: buffer index and use count of key tile t (classic pass).
  __device__ static constexpr int s_buf(int mt, int t) { return t & 1; }
  __device__ static constexpr int s_use(int t) { return t >> 1; }
  static constexpr bool kTurns = MT == 2;
  __device__ static constexpr uint32_t turn_o(int mt) { return mt * 128; }
  __device__ static constexpr uint32_t turn_s() { return 256; }
  __device__ static constexpr uint32_t turn_p(int mt) { return 384 + mt * 64; }
  __device__ static constexpr uint32_t shared_o() { return 0; }
  __device__ static constexpr uint32_t shared_s(int w) { return 128 + 128 * w; }
  __device__ static constexpr uint32_t shared_p(int w) { return 384 + 64 * w; }
  // Epilogue buffers (overlay the tile memory once the key loop is over): this CTA's 128 normalised
  // rows of one query tile -- D bf16 values followed by the row's log2-sum-exp in fp32, padded so that
  // the row-per-thread stores of a warp spread over all banks -- and the blocks received from every
  // slice.  The partial rows travel as bf16 (every one is a normalised average of V rows, so it has the
  // scale of the final output): the exchange is bandwidth-bound and this halves it.
  static constexpr int kRecvPitch = D * 2 + 16;
  static constexpr int kBlockBytes = kBM * kRecvPitch;                   // the 128 staged rows of one stream
  static constexpr int kStageOff = 0;
  static constexpr int kRecvOff = (kBlockBytes + 1023) / 1024 * 1024;
  static_assert(kRecvOff + (kBM + kMaxSplit) * kRecvPitch + 4096 <= kTileBytes, "merge buffers must fit in the tile memory");
};

struct Bars {       // offsets (in 8-byte units) inside the barrier block
  enum { kQFull = 0, kKvFull = 1, kKvEmpty = 7, kSFull = 13, kSFree = 15, kPFull = 17, kODone = 19,
         kClusterA = 21, kClusterC = 22, kRecv = 23, kOFinal = 25, kCount = 26,
         kLoopFirst = kKvFull, kLoopEnd = kClusterA };    // the key loop's barriers exist twice (one set per pass)
};

// Barriers of the CTA-pair form.  Fixed ones first, then one set of key-loop barriers per pass (a pair
// runs up to three passes over its keys, each on a fresh set: an arrival of the pass before that is still in
// flight can then never land in a later phase).  kKvFull: this CTA's half of a stage has landed; kKvReady (used
// in the even CTA): both halves are in place; kKvEmpty: the products that read the stage are complete.
struct PBars {
  enum { kQFull = 0, kQReady = 1, kRecv = 2, kFixed = 4,
         kSFull = 0, kSFree = 2, kPFull = 4, kODone = 6, kOFinal = 8, kKvFull = 9, kKvReady = 19, kKvEmpty = 29,
         kSet = 39, kPasses = 3, kCount = kFixed + kPasses * kSet };
};
static_assert(PBars::kKvReady - PBars::kKvFull == Cfg<128, 1, true>::kStages && PBars::kCount * 8 <= 1024, "pair barrier layout");

// Every wait is bounded: at most kWaitRounds suspensions of at most kWaitHintNs each -- a second at the longest; the
// hardware may end a suspension early, and waits that did run out were seen to do so after some tens of
// milliseconds, still far beyond anything a launch of well under a millisecond waits for.
// Register split (setmaxnreg): warps 0-3 (producer, MMA issuer, helpers) keep kRegsControl registers per
// thread, the softmax warpgroups get kRegsSoftmax; 128 * kRegsControl + 256 * kRegsSoftmax must not exceed
// the 384 * 168 registers the CTA is launched with.
constexpr int kRegsControl = 104;
constexpr int kRegsSoftmax = 200;
static_assert(128 * kRegsControl + 256 * kRegsSoftmax <= 384 * 168, "register split exceeds the CTA's allocation");

constexpr uint32_t kWaitRounds = 1u << 16;
constexpr uint32_t kWaitHintNs = 16384;

// Called by all 32 lanes of a warp; the result is warp-uniform.
// `site` identifies the wait in the abort flag (1 + site of the first wait that gave up).
__device__ __forceinline__ bool bounded_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                              uint32_t site) {
  bool ok = false;
  for (uint32_t i = 0; i < kWaitRounds; ++i) {
    if (ptx::mbar_try_wait(bar, parity, kWaitHintNs)) { ok = true; break; }
    if (*abort_flag) break;
  }
  if (!ok && *abort_flag == 0u) *abort_flag = 1u + site;
  return __all_sync(0xffffffffu, ok);
}

// Fast path: the phase has usually completed already, which one non-blocking test shows.
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                             uint32_t site) {
  if (__all_sync(0xffffffffu, ptx::mbar_test(bar, parity))) return true;
  return bounded_wait_slow(bar, parity, abort_flag, site);
}

// Warp-level wait on a barrier that threads of another CTA of the cluster arrive on (acquire at cluster scope).
__device__ __forceinline__ bool bounded_wait_cl(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                uint32_t site) {
  bool ok = false;
  for (uint32_t i = 0; i < kWaitRounds; ++i) {
    if (ptx::mbar_try_wait_cluster(bar, parity, kWaitHintNs)) { ok = true; break; }
    if (*abort_flag) break;
  }
  if (!ok && *abort_flag == 0u) *abort_flag = 1u + site;
  return __all_sync(0xffffffffu, ok);
}

// The same for a barrier that other CTAs of the cluster arrive on / copy into (acquire at cluster
// scope); called by every thread of the CTA, the result is CTA-uniform.
__device__ __forceinline__ bool bounded_wait_cluster(uint32_t bar, volatile uint32_t* abort_flag, uint32_t site) {
  bool ok = false;
  for (uint32_t i = 0; i < kWaitRounds; ++i) {
    if (ptx::mbar_try_wait_cluster(bar, 0, kWaitHintNs)) { ok = true; break; }
    if (*abort_flag) break;
  }
  if (!ok && *abort_flag == 0u) *abort_flag = 1u + site;
  return ptx::cta_sync_and((ok ? 1 : 0) != 0);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 pk = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&pk);
}

__device__ __forceinline__ void max_chunk(const uint32_t (&x)[32], float (&mx)[4]) {
#pragma unroll
  for (int j = 0; j < 32; ++j) mx[j & 3] = fmaxf(mx[j & 3], __uint_as_float(x[j]));
}
// Scores of keys the row must not see become -inf (bit j of `bits` = key j of the chunk is visible).
__device__ __forceinline__ void mask_chunk(uint32_t (&x)[32], uint32_t bits) {
#pragma unroll
  for (int j = 0; j < 32; ++j) x[j] = ((bits >> j) & 1u) ? x[j] : 0xFF800000u;
}

// 32 scores of one row -> probabilities (exp2 of the scaled, shifted score; a score of -inf gives exactly
// 0), added to the row sum and written as packed bf16 pairs to 16 TMEM columns of the row's lane (the A
// operand of the P V product).  The stages are kept apart so that the 32 independent exp2 are in flight
// together.  The scale-and-shift and the row sum take two values per instruction (fma.rn.f32x2 /
// add.rn.f32x2: the same roundings as the scalar forms, half the issue slots); sum[j & 3] collects column j.
__device__ __forceinline__ void exp_chunk(const uint32_t (&x)[32], float sl2, float m_ref, float (&sum)[4],
                                          uint32_t p_tmem) {
  using u64 = unsigned long long;
  auto pk2 = [](uint32_t lo, uint32_t hi) { u64 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi)); return r; };
  const u64 s2 = pk2(__float_as_uint(sl2), __float_as_uint(sl2));
  const u64 m2 = pk2(__float_as_uint(-m_ref), __float_as_uint(-m_ref));
  float e[32];
#pragma unroll
  for (int j = 0; j < 32; j += 2) {
    u64 t;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(t) : "l"(pk2(x[j], x[j + 1])), "l"(s2), "l"(m2));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(e[j]), "=f"(e[j + 1]) : "l"(t));
  }
#pragma unroll
  for (int j = 0; j < 32; ++j) e[j] = exp2f(e[j]);
  u64 acc0 = pk2(__float_as_uint(sum[0]), __float_as_uint(sum[1]));
  u64 acc1 = pk2(__float_as_uint(sum[2]), __float_as_uint(sum[3]));
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc0) : "l"(pk2(__float_as_uint(e[j]), __float_as_uint(e[j + 1]))));
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc1) : "l"(pk2(__float_as_uint(e[j + 2]), __float_as_uint(e[j + 3]))));
  }
  asm("mov.b64 {%0, %1}, %2;" : "=f"(sum[0]), "=f"(sum[1]) : "l"(acc0));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(sum[2]), "=f"(sum[3]) : "l"(acc1));
  uint32_t packed[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) packed[j] = pack_bf16(e[2 * j], e[2 * j + 1]);
  ptx::tmem_st16(p_tmem, packed);
}

// kSorted: the sequences of a batch are launched longest prefix first (see the set-up of warp 3).
// tm_k64 / tm_tk64: the K maps with boxes of 64 rows (a pair CTA's half of a key tile); unused otherwise.
template <int D, int MT, bool kSorted = false, bool kPair = false>
__global__ void __launch_bounds__(Cfg<D, MT, kPair>::kThreads, 1)
tree_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_tk,
                 const __grid_constant__ CUtensorMap tm_tv, const __grid_constant__ CUtensorMap tm_k64,
                 const __grid_constant__ CUtensorMap tm_tk64, const AttnParams p) {
  using C = Cfg<D, MT, kPair>;
  constexpr int kHalves = C::kHalves;
  constexpr int kStages = C::kStages;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) JET_TR(0);
#ifdef JET_TRACE
  if (tid == 0 && p.trace) {
    unsigned long long gt;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt));
    p.trace[(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 64 + 62] = static_cast<long long>(gt);
  }
#endif

  // ---------------- shared memory carve-up (1024-byte aligned for the 128-byte swizzle)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t sQ = smem_base;
  const uint32_t sKV = sQ + C::kQBytes;
  const uint32_t sBar = sKV + kStages * C::kStageBytes;
  uint8_t* gen_kv = smem_gen + C::kQBytes;
  uint8_t* gen_bar = gen_kv + kStages * C::kStageBytes;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_bar + (kPair ? 1024 : 2 * Bars::kCount * 8));
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile int* seq_slot = reinterpret_cast<volatile int*>(tmem_slot + 2);     // sequence of this CTA when launch order is sorted
  volatile uint32_t* redo_flag = tmem_slot + 3;          // the shared-accumulator pass met a row it cannot hold
  // pair form: redo flag of pass i at redo_flag[i]; pair_slot[pass][rank] = what each CTA of the pair reported
  volatile uint32_t* pair_slot = tmem_slot + 8;
  float* ref_s = reinterpret_cast<float*>(gen_bar + (kPair ? 1536 : 512));  // [128] the rows' common reference (shared-accumulator pass)
  static_assert(2 * Bars::kCount * 8 + 16 <= 512 && 512 + 128 * 4 <= 1024, "barrier block layout");
  constexpr int kRecvBar = kPair ? static_cast<int>(PBars::kRecv) : static_cast<int>(Bars::kRecv);
  auto bar = [&](int idx) { return sBar + 8u * idx; };
  uint32_t sBarLoop = sBar;        // base of the key loop's barrier set in use
  auto lbar = [&](int idx) { return sBarLoop + 8u * idx; };
  const int S = p.nsplit;                            // key slices = cluster size
  // ---------------- work item: what the launch parameters alone decide.  Grid = (query-tile groups x slices,
  // KV heads, sequences); CTAs are dispatched x first, so a unit's slices are neighbours.
  // CTA pairs: blockIdx.x = (pair of query tiles x slices) x 2 + rank; the two CTAs of a pair (a cluster of
  // two) take the query tiles 2k and 2k + 1 of the work item and the same key slice.
  const uint32_t prank = kPair ? (blockIdx.x & 1u) : 0u;
  const uint32_t bx_item = kPair ? (blockIdx.x >> 1) : blockIdx.x;
  const int mgroup_item = static_cast<int>(udiv(bx_item, p.magic_S));
  const int split = static_cast<int>(bx_item) - mgroup_item * S;    // = rank in the cluster of slices
  const int mgroup = kPair ? 2 * mgroup_item + static_cast<int>(prank) : mgroup_item;
  const int g = blockIdx.y;
  const int b_rank = blockIdx.z;                 // position of the sequence in launch order
  constexpr bool sorted_launch = kSorted;
  const int G = p.G;
  const int npt = p.npt;                         // nodes per query tile
  const int node_lo = mgroup * MT * npt;
  const int node_hi = min(p.B, node_lo + MT * npt);
  const int n_mt = (MT == 2 && node_hi - node_lo > npt) ? 2 : 1;     // query tiles of this CTA that hold nodes
  // last node (exclusive) of the pair's two query tiles: both CTAs of a pair walk the same key tiles
  const int node_hi_item = kPair ? min(p.B, (mgroup_item * 2 + 2) * npt) : node_hi;

  // ---------------- set-up that touches no global memory (may overlap the previous kernel's tail)
  if (kPair && warp == 0) {
    for (int i = lane; i < PBars::kCount; i += 32) {
      uint32_t count = 1;
      if (i == PBars::kQReady) count = 2;                       // one arrival per CTA of the pair
      if (i >= PBars::kFixed) {
        const int k = (i - PBars::kFixed) % PBars::kSet;
        if (k >= PBars::kSFree && k < PBars::kODone) count = 8;       // kSFree, kPFull: the four warps of a warpgroup, both CTAs
        else if (k >= PBars::kKvReady && k < PBars::kKvEmpty) count = 2;
      }
      ptx::mbar_init(bar(i), count);
      if (S > 1 && i == PBars::kRecv)
        ptx::mbar_arrive_expect_tx(bar(i), S * max(0, min(p.rows_per, kBM - split * p.rows_per)) * C::kRecvPitch);
    }
    ptx::fence_mbar_init();
    if (lane == 31) {
      redo_flag[0] = 0u;
      redo_flag[1] = 0u;
      redo_flag[2] = 0u;
      *abort_flag = 0u;
    }
  } else if (warp == 0) {
    // one lane per barrier of the block
    if (lane < Bars::kCount) {
      uint32_t count = 1;
      if (lane >= Bars::kKvEmpty && lane < Bars::kSFull) count = (MT == 1 || C::kTurns) ? 1 : n_mt;   // arrivals per stage
      else if (lane >= Bars::kSFree && lane < Bars::kODone) count = 128;                // kSFree, kPFull: a softmax warpgroup
      ptx::mbar_init(bar(lane), count);
      // slice merge: every slice sends this CTA its block of rows of query tile (lane - kRecv)
      if (S > 1 && lane >= Bars::kRecv && lane < Bars::kRecv + MT)
        ptx::mbar_arrive_expect_tx(bar(lane), S * max(0, min(p.rows_per, kBM - split * p.rows_per)) * C::kRecvPitch);
      ptx::fence_mbar_init();
    }
    if (lane == 31) {
      *redo_flag = 0u;
      *abort_flag = 0u;
    }
  } else if (warp == 2) {
    if constexpr (kPair) {
      ptx::tmem_alloc2(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), C::kTmemCols);
      ptx::tmem_relinquish2();
    } else {
      ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), C::kTmemCols);
      ptx::tmem_relinquish();
    }
    if (lane == 0) JET_TR(44);
  } else if (warp == 3) {
    if (lane == 0) {
      ptx::prefetch_tmap(&tm_q);
      ptx::prefetch_tmap(&tm_k);
      ptx::prefetch_tmap(&tm_v);
      ptx::prefetch_tmap(&tm_tk);
      ptx::prefetch_tmap(&tm_tv);
      if constexpr (kPair) {
        ptx::prefetch_tmap(&tm_k64);
        ptx::prefetch_tmap(&tm_tk64);
      }
    }
    // A single sequence's length is very often exactly the caller's bound.  On that guess this slice's first
    // key tiles are asked into L2 now -- before the grid dependency wait, under the previous kernel's tail: L2
    // is where that kernel's writes arrive, so a line prefetched early cannot go stale -- and the copies
    // proper (issued once the real lengths are known) find them there.  A wrong guess costs a few tiles of
    // traffic and nothing else.
    if (!kPair && !sorted_launch && lane == 0 && p.len_hint > 0) {
      // (the CTA index is read afresh so that nothing here lengthens a live range of the main path)
      uint32_t bx, by, bz;
      asm volatile("mov.u32 %0, %%ctaid.x;" : "=r"(bx));
      asm volatile("mov.u32 %0, %%ctaid.y;" : "=r"(by));
      asm volatile("mov.u32 %0, %%ctaid.z;" : "=r"(bz));
      const int mg = static_cast<int>(udiv(bx, p.magic_S)), sp = static_cast<int>(bx) - mg * p.nsplit;
      const int tp_g = (p.len_hint + kBN - 1) / kBN;
      const int t_all_g = tp_g + (min(p.B, (mg + 1) * MT * p.npt) + kBN - 1) / kBN;
      const int lo_g = static_cast<int>(udiv(static_cast<uint32_t>(t_all_g) * sp + p.nsplit - 1, p.magic_S));
      const int hi_g = min(tp_g, static_cast<int>(udiv(static_cast<uint32_t>(t_all_g) * (sp + 1) + p.nsplit - 1, p.magic_S)));
      // (two tiles, written out: a loop here made the register allocator spill in the key loop)
      if (lo_g < hi_g) {
        for (int h = 0; h < kHalves; ++h) ptx::tma_prefetch_4d(&tm_k, h * 64, by, lo_g * kBN, bz);
        for (int h = 0; h < kHalves; ++h) ptx::tma_prefetch_4d(&tm_v, h * 64, by, lo_g * kBN, bz);
      }
      if (lo_g + 1 < hi_g) {
        for (int h = 0; h < kHalves; ++h) ptx::tma_prefetch_4d(&tm_k, h * 64, by, (lo_g + 1) * kBN, bz);
        for (int h = 0; h < kHalves; ++h) ptx::tma_prefetch_4d(&tm_v, h * 64, by, (lo_g + 1) * kBN, bz);
      }
    }
    __syncwarp();
    if (sorted_launch) {
      // Launch order = longest prefix first (CTAs are dispatched in index order, so with more work items than
      // SMs the long sequences start early and the short ones fill the tail): this warp finds the sequence of
      // rank b_rank by counting and leaves it in shared memory.  Beyond kMaxSorted sequences the order stays
      // as given (many small items balance by themselves, and the count is quadratic).
      if (!p.stable) ptx::grid_dep_wait();
      int len[kMaxSorted / 32];
#pragma unroll
      for (int c = 0; c < kMaxSorted / 32; ++c) len[c] = c * 32 + lane < p.batch ? __ldg(p.seq_len + c * 32 + lane) : -1;
      int found = -1;
#pragma unroll
      for (int c = 0; c < kMaxSorted / 32; ++c) {
        if (c * 32 < p.batch) {
          const int mine = len[c], me = c * 32 + lane;
          int before = 0;                                // sequences that come before `me` in launch order
#pragma unroll
          for (int c2 = 0; c2 < kMaxSorted / 32; ++c2) {
            if (c2 * 32 < p.batch) {
#pragma unroll 1
              for (int j = 0; j < 32; ++j) {       // (rolled: this runs once per launch, from cold code)
                const int other = __shfl_sync(0xffffffffu, len[c2], j), ob = c2 * 32 + j;
                before += (ob < p.batch && (other > mine || (other == mine && ob < me))) ? 1 : 0;
              }
            }
          }
          if (me < p.batch && before == b_rank) found = me;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) found = max(found, __shfl_xor_sync(0xffffffffu, found, o));
      if (lane == 0) *seq_slot = found;
    }
  }
  if (tid == 0) JET_TR(40);
  ptx::tc_fence_before();
  ptx::cta_sync();
  // (a pair's barriers take arrivals from the other CTA: both sets exist before either CTA goes on)
  if constexpr (kPair) ptx::cluster_sync_all();
  ptx::tc_fence_after();
  if (tid == 0) JET_TR(41);
  // The barriers of every CTA of the cluster must exist before any CTA arrives on them remotely:
  // arrive on the hardware cluster barrier now, wait for it only when the slices are merged.
  const bool via_cluster = S > 1 && !p.via_global;
  const uint32_t tmem_base = *tmem_slot;
  if (tid == 0) JET_TR(42);
  // Inputs may be written by the preceding kernel of the stream: nothing in global memory is touched before
  // the dependency wait.  Exception (p.stable, the caller's promise): the lengths, the page table and the
  // prefix rows of the caches are older than that kernel, so the K/V producers read them at once -- under the
  // preceding kernel's tail -- and only the warps that need the query rows, the tree's own K/V rows, the
  // ancestor masks or the outputs wait, each where it first needs them.  The next kernel of the stream may be
  // scheduled once this CTA has passed its own wait (so a chain of such kernels never runs more than one ahead).
  const bool early = p.stable != 0;
  if (!early || warp == 3) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
  }
  if (tid == 96) JET_TR(43);

  // ---------------- work item, continued: what depends on device data
  const int b = sorted_launch ? *seq_slot : b_rank;
  // The query rows depend on nothing but the work item: warp 3 (idle until the first P V product) requests
  // them now, under the look-up of the sequence's lengths.
  if (warp == 3 && lane == 0) {
    JET_TR(46);
    ptx::mbar_arrive_expect_tx(bar(Bars::kQFull), n_mt * kHalves * kHalfBytes);
    for (int mt = 0; mt < n_mt; ++mt)
      for (int h = 0; h < kHalves; ++h)
        ptx::tma_load_4d(sQ + (mt * kHalves + h) * kHalfBytes, &tm_q, bar(Bars::kQFull), h * 64, 0, g,
                         b * p.B + node_lo + mt * npt);
    JET_TR(45);
  }
  const int L = p.seq_len[b];
  const int n = min(p.n_nodes[b], p.B);
  const int ntree = min(n, node_hi_item);                    // tree keys any row here can see
  // Keys that come out of the cache: the prefix, and with p.tail also the tree's own rows behind it (then
  // there are no separate tree tiles: key j >= L is tree node j - L).
  const int Lc = p.tail ? L + ntree : L;
  const int TP = (Lc + kBN - 1) / kBN;
  const int TT = p.tail ? 0 : (ntree + kBN - 1) / kBN;
  const int T_all = TP + TT;
  // key tiles of this slice; when they do not divide evenly the first slices take the extra tile, so that
  // the last slice, whose tree tile (masked) is the slowest kind, has the fewest
  int t_lo, t_hi;
  if (T_all < (1 << 20)) {
    t_lo = static_cast<int>(udiv(static_cast<uint32_t>(T_all) * split + S - 1, p.magic_S));
    t_hi = static_cast<int>(udiv(static_cast<uint32_t>(T_all) * (split + 1) + S - 1, p.magic_S));
  } else {
    t_lo = static_cast<int>((static_cast<uint32_t>(T_all) * split + S - 1) / static_cast<uint32_t>(S));
    t_hi = static_cast<int>((static_cast<uint32_t>(T_all) * (split + 1) + S - 1) / static_cast<uint32_t>(S));
  }
  const int T = t_hi - t_lo;
  // otherwise: no live node here (pair: in neither of its query tiles), or an empty key slice
  const bool has_work = (kPair ? mgroup_item * 2 * npt : node_lo) < n && T > 0;
  // A CTA without work never looks at its query rows, but they must have landed before the epilogue reuses
  // their memory (and before the CTA exits).
  if (!has_work && warp == 3) bounded_wait(bar(Bars::kQFull), 0, abort_flag, 3);
  // The first K tiles are requested here, straight after the lengths are known: the producer's own loop
  // lies some two thousand cycles of cold code further on (register re-split, set-up of the ring), and
  // the first Q K^T waits for exactly these tiles.  They are the first items of the ring in every form of
  // the key loop (ring order starts K_0 .. K_ahead); the producers start behind them.  A paged tile needs
  // its page ids first and is left to the producers.
  int n_early = (has_work && !p.paged && !kPair) ? (MT == 1 ? min(2, T) : 1) : 0;
  if (early) {         // before the dependency wait only tiles that lie wholly inside the prefix may be read
    int k = 0;
    while (k < n_early && (t_lo + k + 1) * kBN <= L) ++k;
    n_early = k;
  }
  if (warp == 0 && lane == 0) {
    for (int i = 0; i < n_early; ++i) {
      const int t = t_lo + i;
      const bool prefix = t < TP;
      const CUtensorMap* map = prefix ? &tm_k : &tm_tk;
      const int row0 = prefix ? t * kBN : (t - TP) * kBN;
      const uint32_t full = bar(Bars::kKvFull + i);
      ptx::mbar_arrive_expect_tx(full, C::kStageBytes);
      for (int h = 0; h < kHalves; ++h) ptx::tma_load_4d(sKV + i * C::kStageBytes + h * kHalfBytes, map, full, h * 64, g, row0, b);
    }
  }
  if (tid == 0) JET_TR(1);

  // per-row state of the softmax threads, live until the epilogue
  float m_used = -INFINITY;     // running reference maximum (raw score units)
  float l = 0.0f;               // running sum of exp2((s - m_used) * sl2)
  bool row_ok = has_work;       // false once a bounded wait of this warp expired
  bool classic = true;                      // the classic key loop has to run
  bool shared_result = false;               // the rows come out of the shared-accumulator pass
  float m_ref_common = 0.0f;                // softmax threads: the row's fixed reference (log2 units)
  constexpr int kAhead = 3;     // shared-accumulator form of the key loop: Q K^T runs this many key tiles ahead of P V

  // The epilogue is written once and instantiated for both register classes: `sm_side` is true for the
  // softmax warpgroups (which hold the rows, stage and combine them) and false for warps 0-3 (which take
  // part in every CTA-wide barrier and issue the bulk copies and the counter updates).
  auto epilogue = [&](auto sm_side) {
    constexpr bool kSm = decltype(sm_side)::value;
    if (!kSm && early) ptx::grid_dep_wait();      // (the softmax warps passed theirs before their first tile)
    // The slice bookkeeping is worked out again here, from the CTA index read afresh, so that none of it
    // occupies a register through the key loop (the softmax threads have none to spare).
    uint32_t e_bx;
    asm volatile("mov.u32 %0, %%ctaid.x;" : "=r"(e_bx));
    const uint32_t e_item = kPair ? (e_bx >> 1) : e_bx;
    const int e_mgroup_item = static_cast<int>(udiv(e_item, p.magic_S));
    const int split = static_cast<int>(e_item) - e_mgroup_item * S;
    const int e_mgroup = kPair ? 2 * e_mgroup_item + static_cast<int>(e_bx & 1u) : e_mgroup_item;
    const int rows_per = p.rows_per;                   // rows of a query tile that one slice combines
    const int own_lo = split * rows_per;
    const int own_n = max(0, min(rows_per, kBM - own_lo));
    // (indexed by the sequence itself, not by its rank in launch order: the merge kernel of the two-launch form
    //  addresses the slots by sequence)
    const int unit = (b * p.Hkv + static_cast<int>(blockIdx.y)) * p.n_mgroups + e_mgroup;
    // =============================================================== epilogue
    // One round per query tile: its softmax threads stage their normalised rows (D bf16 + log2-sum-exp)
    // in shared memory.  With key slices every CTA then sends each owner slice its block of rows with
    // one bulk copy credited to the owner's kRecv barrier; the owner combines the S blocks.  Without
    // slices the CTA "combines" its own staged rows.  Either way the output rows leave as coalesced
    // 16-byte stores, rows of padding nodes as zeros.
    const int e_wg = warp >= 4 ? (warp - 4) >> 2 : 0;            // softmax warpgroup of this thread
    const int e_r = (tid - 128) & 127;                           // its row within the query tile
    uint8_t* stage = smem_gen + C::kStageOff;
    bool merge_ok = true;
    ptx::cta_sync();
    // Staging of a row: normalised, D bf16 values followed by the row's log2-sum-exp (fp32).  Rows this CTA
    // computed nothing for (empty key slice, tile without nodes) get log2-sum-exp = -inf ("absent").
    const uint32_t e_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const bool active = has_work && row_ok;                      // warp-uniform: TMEM loads need whole warps
    const float own_inv = (active && l > 0.0f) ? 1.0f / l : 0.0f;
    const float own_lse2 = (active && l > 0.0f) ? m_used * p.scale_log2 + log2f(l) : -INFINITY;
    // MT == 1: the two streams of a row exchange (log2-sum-exp, 1/sum) through a scratch corner of the
    // idle tile memory; afterwards both threads of a row know both weights.
    float2* xchg = reinterpret_cast<float2*>(smem_gen + C::kTileBytes - 2048);     // [stream][row]
    // (after a shared-accumulator pass: the warpgroup's part of the row sum and the row's reference)
    if constexpr (kSm && MT == 1)
      xchg[e_wg * 128 + e_r] = shared_result ? make_float2(active ? l : 0.0f, m_ref_common) : make_float2(own_lse2, own_inv);
#pragma unroll 1
    for (int mt = 0; mt < n_mt; ++mt) {      // n_mt is the same in every CTA of the cluster
      if (mt > 0) {
        // C: everybody has combined the previous tile's rows, so both buffers are free again
        if (via_cluster) {
          __syncwarp();
          ptx::cluster_sync_all();
        } else {
          ptx::cta_sync();
        }
      }
      if constexpr (MT == 1) {
        // Both warpgroups stage half of every row (64 columns each), folding the two streams' accumulators
        // together on the way: out = wa * O_0 / l_0 + wb * O_1 / l_1 with softmax weights of the two sums.
        ptx::cta_sync();
        if constexpr (kSm) {
         if (shared_result) {
          // one accumulator, one reference: the row sum is the sum of the warpgroups' parts
          const float2 s0 = xchg[e_r], s1 = xchg[128 + e_r];
          const float lt = s0.x + s1.x;
          const bool any = lt > 0.0f && lt < INFINITY;
          const float inv = any ? 1.0f / lt : 0.0f;
          constexpr int kCols = D / 2;
          uint8_t* dst = stage + e_r * C::kRecvPitch + e_wg * kCols * 2;
#pragma unroll 1
          for (int c = 0; c < kCols / 32; ++c) {
            uint32_t o[32];
            if (active) {
              ptx::tmem_ld32(e_lane + C::shared_o() + e_wg * kCols + c * 32, o);
              ptx::tmem_wait_ld();
            }
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              uint32_t w[4] = {0u, 0u, 0u, 0u};
              if (active && any) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  w[k] = pack_bf16(__uint_as_float(o[q8 * 8 + 2 * k]) * inv, __uint_as_float(o[q8 * 8 + 2 * k + 1]) * inv);
              }
              *reinterpret_cast<uint4*>(dst + (c * 32 + q8 * 8) * 2) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
          if (e_wg == 0) *reinterpret_cast<float*>(stage + e_r * C::kRecvPitch + D * 2) = any ? s0.y + log2f(lt) : -INFINITY;
         } else {
          const float2 s0 = xchg[e_r], s1 = xchg[128 + e_r];
          const float mxl = fmaxf(s0.x, s1.x);
          float a0 = 0.0f, a1 = 0.0f, lse2 = -INFINITY;
          if (mxl > -INFINITY) {
            const float w0 = s0.x > -INFINITY ? exp2f(s0.x - mxl) : 0.0f;
            const float w1 = s1.x > -INFINITY ? exp2f(s1.x - mxl) : 0.0f;
            const float inv = 1.0f / (w0 + w1);
            a0 = w0 * inv * s0.y;
            a1 = w1 * inv * s1.y;
            lse2 = mxl + log2f(w0 + w1);
          }
          constexpr int kCols = D / 2;
          uint8_t* dst = stage + e_r * C::kRecvPitch + e_wg * kCols * 2;
#pragma unroll 1
          for (int c = 0; c < kCols / 32; ++c) {
            uint32_t o0[32], o1[32];
            if (active) {
              ptx::tmem_ld32(e_lane + C::o_col(0, 0) + e_wg * kCols + c * 32, o0);
              ptx::tmem_ld32(e_lane + C::o_col(0, 1) + e_wg * kCols + c * 32, o1);
              ptx::tmem_wait_ld();
            }
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              uint32_t w[4] = {0u, 0u, 0u, 0u};
              if (active) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const int j = q8 * 8 + 2 * k;
                  const float lo = (a0 != 0.0f ? a0 * __uint_as_float(o0[j]) : 0.0f) + (a1 != 0.0f ? a1 * __uint_as_float(o1[j]) : 0.0f);
                  const float hi = (a0 != 0.0f ? a0 * __uint_as_float(o0[j + 1]) : 0.0f) + (a1 != 0.0f ? a1 * __uint_as_float(o1[j + 1]) : 0.0f);
                  w[k] = pack_bf16(lo, hi);
                }
              }
              *reinterpret_cast<uint4*>(dst + (c * 32 + q8 * 8) * 2) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
          if (e_wg == 0) *reinterpret_cast<float*>(stage + e_r * C::kRecvPitch + D * 2) = lse2;
         }
        }
      } else if (kSm && e_wg == mt) {
        uint8_t* dst = stage + e_r * C::kRecvPitch;
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          if (active) {
            ptx::tmem_ld32(e_lane + (C::kTurns ? C::turn_o(mt) : C::o_col(mt, 0)) + c * 32, o);
            ptx::tmem_wait_ld();
          }
#pragma unroll
          for (int q8 = 0; q8 < 4; ++q8) {
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            if (active) {
#pragma unroll
              for (int k = 0; k < 4; ++k)
                w[k] = pack_bf16(__uint_as_float(o[q8 * 8 + 2 * k]) * own_inv, __uint_as_float(o[q8 * 8 + 2 * k + 1]) * own_inv);
            }
            *reinterpret_cast<uint4*>(dst + (c * 32 + q8 * 8) * 2) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
        *reinterpret_cast<float*>(dst + D * 2) = own_lse2;
      }
      if (via_cluster) {
        // The slices of the work item form a thread-block cluster: once every CTA has staged its rows (the
        // hardware cluster barrier, release / acquire, makes them visible cluster-wide), each CTA PULLS its own
        // block of rows out of every slice's shared memory into a buffer of its own -- all loads of a thread in
        // flight at once, one round trip over the SM-to-SM network -- and combines the copies.  No remote
        // writes, no arrival counters; a CTA must only not exit (or restage) before its peers have read it:
        // the cluster barriers behind the loop.  (The first version pushed the blocks with bulk copies credited
        // to the owners' mbarriers behind a cluster-wide rendezvous; the pull is 1 - 3 us per launch faster.)
        __syncwarp();
        ptx::cluster_sync_all();
        if (tid == 128 && mt == 0) JET_TR(8);
        if constexpr (kSm) {
          // gather: 16-byte chunk e of this CTA's row block, from slice c, for every (e, c) pair of the thread --
          // at most 16 pairs (fewer slices mean more rows per CTA and the other way round)
          constexpr int kChunksPerRow = C::kRecvPitch / 16;
          const int per_slice = own_n * kChunksPerRow;
          const int pairs = ((per_slice + 255) / 256) * S;
          const uint32_t local = smem_base + C::kStageOff + static_cast<uint32_t>(own_lo * C::kRecvPitch);
          uint8_t* recv = smem_gen + C::kRecvOff;
          uint4 got[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const int j = static_cast<int>(udiv(static_cast<uint32_t>(q), p.magic_S)), c = q - j * S;
            const int e = tid - 128 + 256 * j;
            if (q < pairs && e < per_slice) got[q] = ptx::ld_cluster_v4(ptx::map_to_rank(local + static_cast<uint32_t>(e * 16), c));
          }
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const int j = static_cast<int>(udiv(static_cast<uint32_t>(q), p.magic_S)), c = q - j * S;
            const int e = tid - 128 + 256 * j;
            if (q < pairs && e < per_slice)
              *reinterpret_cast<uint4*>(recv + static_cast<size_t>(c) * rows_per * C::kRecvPitch + e * 16) = got[q];
          }
          ptx::named_sync(2, 256);
        }
        if (tid == 128 && mt == 0) JET_TR(9);
      } else {
        ptx::cta_sync();
      }
      const uint8_t* src_rows = via_cluster ? smem_gen + C::kRecvOff : stage;         // S == 1: the staged rows themselves
      bool rows_ok = merge_ok;
      if (S > 1 && !via_cluster) {
        // Exchange through the workspace: publish this CTA's staged rows, count the slices of the unit
        // that have published (bounded spin), then fetch this CTA's block of rows from every slice.
        constexpr uint32_t kBlockBytes = kBM * C::kRecvPitch;
        int* arrive = p.counters + unit * MT + mt;
        int* depart = p.counters + p.n_units * MT + unit * MT + mt;
        uint8_t* slots = p.partials + (static_cast<size_t>(unit) * S * MT) * kBlockBytes;
        if (!kSm && tid == 0) JET_TR(63);
        {
          // every thread of the CTA copies its share of the staged block (consecutive threads, consecutive
          // 16 bytes); the release of the arrival count below, behind the CTA-wide barrier, publishes all of it
          const uint4* src4 = reinterpret_cast<const uint4*>(stage);
          uint4* dst4 = reinterpret_cast<uint4*>(slots + (static_cast<size_t>(split) * MT + mt) * kBlockBytes);
          for (int i = tid; i < static_cast<int>(kBlockBytes / 16); i += C::kThreads) __stcg(dst4 + i, src4[i]);
        }
        // Two launches: this one ends here; the merge kernel that follows it in the stream starts when every
        // CTA of this launch has exited, i.e. when every block is in place -- no counter, no spin, and no need
        // for the slices to be resident together.
        if (p.via_global == 2) continue;
        ptx::cta_sync();
        if (!kSm && tid == 0) {
          // the last slice to arrive knows from its own count that everybody has published
          JET_TR(29);
          bool seen = ptx::atom_add_acq_rel_gpu(arrive, 1) + 1 >= S;
          JET_TR(30);
          for (uint32_t i = 0; i < p.poll_limit && !seen; ++i) {
            if (ptx::ld_acquire_gpu(arrive) >= S) { seen = true; break; }
            __nanosleep(32);
            if (*abort_flag) break;
          }
          if (!seen && *abort_flag == 0u) *abort_flag = 1u + 16u;
          ptx::fence_proxy_async_all();
        }
        if (tid == 128 && mt == 0) JET_TR(8);
        const bool published = ptx::cta_sync_and((*abort_flag == 0u ? 1 : 0) != 0);
        if (!kSm && tid < S && published && own_n > 0)
          ptx::bulk_load_global(smem_base + C::kRecvOff + static_cast<uint32_t>(tid * rows_per * C::kRecvPitch),
                                slots + (static_cast<size_t>(tid) * MT + mt) * kBlockBytes + own_lo * C::kRecvPitch,
                                static_cast<uint32_t>(own_n * C::kRecvPitch), bar(kRecvBar + mt));
        rows_ok = published && (own_n == 0 || bounded_wait_cluster(bar(kRecvBar + mt), abort_flag, 14));
        if (own_n == 0) ptx::cta_sync();
        if (tid == 128 && mt == 0) JET_TR(9);
        src_rows = smem_gen + C::kRecvOff;
        // the last slice to have fetched its rows leaves the counters at zero for the next call
        if (!kSm && tid == 0 && ptx::atom_add_release_gpu(depart, 1) == S - 1) {
          *arrive = 0;
          *depart = 0;
          __threadfence();
        }
      }
      const uint32_t src_stride = rows_per * C::kRecvPitch;     // distance between the blocks of consecutive slices
      // The softmax warpgroups combine the blocks: one item = 8 output values of one row.  A thread first issues
      // every load of its item (the S log-sum-exps of the row and its 16 bytes of every slice), then forms the
      // softmax weights of the slice sums and the weighted sum -- one round trip to shared memory, no chain of
      // dependent loads, no table of weights and no barrier between two passes.
      if constexpr (kSm) {
        const int items = rows_ok ? own_n * (D / 8) : 0;
#pragma unroll 1
        for (int i = tid - 128; i < items; i += 256) {
          const int rl = i / (D / 8), c8 = i - rl * (D / 8);
          const int R = mt * kBM + own_lo + rl;                  // row within the unit
          const int vq = static_cast<int>(udiv(R, p.magic_G));
          const int v = node_lo + vq, h = g * G + (R - vq * G);
          if (v >= p.B) continue;
          const uint8_t* src = src_rows + rl * C::kRecvPitch;
          float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
          float lse2 = -INFINITY;
          if (S == 1) {
            // no slices: the staged row is the result
            const float lc = *reinterpret_cast<const float*>(src + D * 2);
            const uint4 x = *reinterpret_cast<const uint4*>(src + c8 * 16);
            if (v < n && lc > -INFINITY) {
              const uint32_t v4[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                acc[2 * q] = __uint_as_float(v4[q] << 16);
                acc[2 * q + 1] = __uint_as_float(v4[q] & 0xFFFF0000u);
              }
              lse2 = lc;
            }
          } else {
            // (four slices at a time: their loads are issued together, then used)
            float mx = -INFINITY;
#pragma unroll 1
            for (int c0 = 0; c0 < S; c0 += 4) {
              float l4[4];
#pragma unroll
              for (int k = 0; k < 4; ++k)
                l4[k] = c0 + k < S ? *reinterpret_cast<const float*>(src + (c0 + k) * src_stride + D * 2) : -INFINITY;
              mx = fmaxf(fmaxf(mx, fmaxf(l4[0], l4[1])), fmaxf(l4[2], l4[3]));
            }
            if (v < n && mx > -INFINITY) {
              float wsum = 0.0f;
#pragma unroll 1
              for (int c0 = 0; c0 < S; c0 += 4) {
                float l4[4];
                uint4 x4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const bool in = c0 + k < S;
                  l4[k] = in ? *reinterpret_cast<const float*>(src + (c0 + k) * src_stride + D * 2) : -INFINITY;
                  x4[k] = in ? *reinterpret_cast<const uint4*>(src + (c0 + k) * src_stride + c8 * 16) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  // absent slices (log-sum-exp -inf) get weight 0, and whatever their rows hold is not used
                  const float w = l4[k] > -INFINITY ? exp2f(l4[k] - mx) : 0.0f;
                  wsum += w;
                  const uint32_t v4[4] = {x4[k].x, x4[k].y, x4[k].z, x4[k].w};
#pragma unroll
                  for (int q = 0; q < 4; ++q) {      // bf16 pair -> fp32: the bits are the upper half of the float
                    const float lo = __uint_as_float(v4[q] << 16), hi = __uint_as_float(v4[q] & 0xFFFF0000u);
                    acc[2 * q] += w > 0.0f ? w * lo : 0.0f;
                    acc[2 * q + 1] += w > 0.0f ? w * hi : 0.0f;
                  }
                }
              }
              const float inv = 1.0f / wsum;
#pragma unroll
              for (int k = 0; k < 8; ++k) acc[k] *= inv;
              lse2 = mx + log2f(wsum);
            }
          }
          *reinterpret_cast<uint4*>(p.out + ((static_cast<size_t>(b) * p.B + v) * p.Hq + h) * D + c8 * 8) =
              make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                         pack_bf16(acc[6], acc[7]));
          if (p.lse && c8 == 0) p.lse[(static_cast<size_t>(b) * p.Hq + h) * p.B + v] = lse2 * 0.6931471805599453f;
        }
      }
    }

  };

  // ---------------- the key loop
  // Three forms (the third, for two query tiles per CTA, is described where it starts).  The classic form
  // gives every stream its own accumulator and reference maximum, which may rise
  // at any tile (the accumulator is rescaled); it is exact for any input.  With one query tile per CTA the
  // loop first runs in the shared-accumulator form: both warpgroups add into ONE accumulator against a per-row
  // reference that is fixed after the first key tile, which frees the TMEM columns for P buffers apart from
  // the score buffers -- so a warpgroup's next Q K^T runs while it still exponentiates the tile before, and
  // the chain  softmax -> P V -> Q K^T -> softmax  of the classic form becomes  softmax -> softmax.  A fixed
  // reference is exact as long as no probability overflows; a row whose tile sum passes kSharedSumLimit (or is
  // not finite) raises redo_flag, and the CTA then runs the whole key range again in the classic form (on a
  // second set of barriers; the first pass has drained by then).

  // Position in the ring of the V tile of key tile tl when K runs `ahead` tiles in front of V
  // (ring order: K_0 .. K_ahead, then V_t, K_{t+ahead+1} alternating, then the remaining V).
  auto v_item = [&](int tl, int ahead) {
    const int lead = min(ahead + 1, T);
    return lead + tl + min(tl, T - lead);
  };
  // Where a tile sits in shared memory: .x = stage, .y = parity of this use of the stage's barriers.
  //  * One producer warp: all tiles go through ONE ring in issue order (ring item i -> stage i % kStages).
  //  * Two producer warps (warp 0 requests the K tiles, warp 2 the V tiles): each warp has stages of its own, K tile
  //    t in stage t % kKStages, V tile t in stage kKStages + t % kVStages.  A parity wait tells "one phase further"
  //    from "two phases further" only for a thread that saw the phase before itself; with one shared ring a warp
  //    that runs past the other warp's tiles can be two uses of a stage ahead of the consumers (a slow load is
  //    enough), takes the stale parity for its turn and overwrites a tile that has not been read.  With stages
  //    of its own every wait of a warp follows its own previous wait on the same barrier.
  constexpr int kKStages = (kStages + 1) / 2, kVStages = kStages - kKStages;
  auto ring_pos = [&](int item) { return make_int2(item % kStages, (item / kStages) & 1); };
  auto k_pos_split = [&](int tl) { return make_int2(tl % kKStages, (tl / kKStages) & 1); };
  auto v_pos_split = [&](int tl) { return make_int2(kKStages + tl % kVStages, (tl / kVStages) & 1); };
  // The barriers of the classic pass when it follows a shared-accumulator pass: a fresh set.
  auto second_barrier_set = [&]() {
    sBarLoop = sBar + 8u * Bars::kCount;
    if (tid == 0) {
      for (int s = 0; s < kStages; ++s) {
        ptx::mbar_init(lbar(Bars::kKvFull + s), 1);
        ptx::mbar_init(lbar(Bars::kKvEmpty + s), 1);
      }
      for (int i = 0; i < 2; ++i) {
        ptx::mbar_init(lbar(Bars::kSFull + i), 1);
        ptx::mbar_init(lbar(Bars::kPFull + i), 128);
        ptx::mbar_init(lbar(Bars::kODone + i), 1);
      }
      ptx::fence_mbar_init();
    }
    ptx::cta_sync();
  };

  // End of a pass of the pair form (every thread of both CTAs calls it): each CTA tells the other whether a row
  // overflowed its reference (bit 0) and whether a wait gave up (bit 1); both go on with the same verdict.
  auto pair_verdict = [&](int pass) -> uint32_t {
    ptx::cta_sync();
    if (tid == 0) {
      const uint32_t mine = (redo_flag[pass] ? 1u : 0u) | (*abort_flag ? 2u : 0u);
      pair_slot[pass * 2 + prank] = mine;
      ptx::st_cluster_u32(ptx::map_to_rank(ptx::smem_u32(const_cast<uint32_t*>(pair_slot + pass * 2 + prank)), prank ^ 1u), mine);
    }
    __syncwarp();
    ptx::cluster_sync_all();
    return pair_slot[pass * 2] | pair_slot[pass * 2 + 1];
  };

  if (warp < 4) {
    // Warps 0-3 need few registers; what they give up goes to the softmax warpgroups, which hold a whole
    // score row (128 values) per thread.
    if (tid == 0) JET_TR(15);
    ptx::setmaxnreg_dec<kRegsControl>();
    if (tid == 0) JET_TR(18);

    // =========================================================== TMA producer (warp 0)
    // K runs `ahead` key tiles in front of V in the ring (0: K_t, V_t alternate).
    // only_c (a compile-time constant: a run-time role cost 4 % on long contiguous prefixes): -1 = this warp
    // requests every tile, 0 = the K tiles only, 1 = the V tiles only (two producer warps).
    // first: ring items already requested (K tiles 0 .. first - 1, see n_early).
    auto produce = [&](const int ahead, auto only_c, const int first) {
      constexpr int only = decltype(only_c)::value;
      if (tid == 0) JET_TR(27);
      bool ok = true;
      bool waited = !early;          // this warp has passed the dependency wait
      int issued = first;
      // paged cache: lane i holds the page of the tile's i-th 16-row block; the ids of the next tile are
      // fetched while the current tile's copies are issued, so the table look-up is off the critical path
      auto tile_page = [&](int t) -> int {
        // (the last test: a sequence length beyond what the table covers -- the caller's error -- must not become a
        //  read outside the table)
        if (!p.paged || t >= TP || lane >= 8 || t * kBN + lane * 16 >= Lc || t * 8 + lane >= p.max_pages) return 0;
        return __ldg(p.page_table + static_cast<size_t>(b) * p.max_pages + t * 8 + lane);
      };
      int kt = first, vt = 0;                   // next K tile, next V tile (first > 0 only without pages)
      int pk_cur = tile_page(t_lo), pk_next = tile_page(t_lo + 1);
      int pv_cur = pk_cur, pv_next = pk_next;
      if (tid == 0) JET_TR(28);
#pragma unroll 1
      for (; issued < 2 * T; ++issued) {
        const bool take_k = kt < T && kt <= vt + ahead;
        const int t = t_lo + (take_k ? kt : vt), kv = take_k ? 0 : 1;
        if (only >= 0 && kv != only) {          // the other producer warp's tile
          if (take_k) ++kt; else ++vt;
          continue;
        }
        // stage and how often it has been used before (see ring_pos / k_pos_split)
        const int nth = take_k ? kt : vt;
        const int stage = only < 0 ? issued % kStages : (take_k ? nth % kKStages : kKStages + nth % kVStages);
        const int use = only < 0 ? issued / kStages : (take_k ? nth / kKStages : nth / kVStages);
        if (!waited && (t + 1) * kBN > L) {      // not wholly inside the prefix: may hold rows the preceding kernel writes
          ptx::grid_dep_wait();
          waited = true;
        }
        if (use >= 1) {
          ok = bounded_wait(lbar(Bars::kKvEmpty + stage), (use - 1) & 1, abort_flag, 1);
          if (!ok) break;
        }
        const uint32_t dst = sKV + stage * C::kStageBytes;
        const uint32_t full = lbar(Bars::kKvFull + stage);
        if (t < TP && p.paged) {
          const int npages = min(8, (Lc - t * kBN + 15) / 16);
          const int page = take_k ? pk_cur : pv_cur;
          if (lane == 0) ptx::mbar_arrive_expect_tx(full, npages * kHalves * 2048);
          __syncwarp();
          if (lane < npages) {
            for (int h = 0; h < kHalves; ++h)
              ptx::tma_load_3d(dst + h * kHalfBytes + lane * 2048, kv ? &tm_v : &tm_k, full, h * 64, g, page * 16);
          }
        } else {
          const bool prefix = t < TP;
          const CUtensorMap* map = prefix ? (kv ? &tm_v : &tm_k) : (kv ? &tm_tv : &tm_tk);
          const int row0 = prefix ? t * kBN : (t - TP) * kBN;
          if (issued == 0 && lane == 0) JET_TR(48);
          if (lane == 0) {
            ptx::mbar_arrive_expect_tx(full, C::kStageBytes);
            for (int h = 0; h < kHalves; ++h) ptx::tma_load_4d(dst + h * kHalfBytes, map, full, h * 64, g, row0, b);
          }
          if (issued == 0 && lane == 0) JET_TR(49);
        }
        if (take_k) {
          ++kt;
          pk_cur = pk_next;
          pk_next = tile_page(t + 2);
        } else {
          ++vt;
          pv_cur = pv_next;
          pv_next = tile_page(t + 2);
        }
        __syncwarp();
        if (lane == 0 && issued == 0) JET_TR(14);
      }
      if (__any_sync(0xffffffffu, *abort_flag != 0u)) {
        // drain: every load that this warp issued must land before the CTA may exit
        for (int s = 0; s < kStages; ++s) {
          if (only < 0) {
            if (issued > s) {
              const int last = ((issued - 1 - s) / kStages) * kStages + s;     // last item issued to stage s
              bounded_wait(lbar(Bars::kKvFull + s), (last / kStages) & 1, abort_flag, 2);
            }
          } else {
            const bool k_stage = s < kKStages;
            const int n = k_stage ? kt : vt, ring = k_stage ? kKStages : kVStages, r = k_stage ? s : s - kKStages;
            if ((only == 0) == k_stage && n > r) {
              const int last = ((n - 1 - r) / ring) * ring + r;                // last tile of this kind in stage s
              bounded_wait(lbar(Bars::kKvFull + s), (last / ring) & 1, abort_flag, 2);
            }
          }
        }
        bounded_wait(bar(Bars::kQFull), 0, abort_flag, 3);
      }
    };

    // The tensor core queues only two or three instructions, so every instruction between two MMAs counts:
    // the whole warp runs the issue loops (uniform control flow and operands), one elected lane issues, and
    // descriptors are formed by adding precomputed offsets.
    constexpr uint32_t idesc_qk = ptx::umma_idesc_bf16(kBM, kBN, false);
    constexpr uint32_t idesc_pv = ptx::umma_idesc_bf16(kBM, D, true);
    const uint64_t desc_q0 = ptx::smem_desc_sw128(sQ, 0);
    const uint64_t desc_k0 = ptx::smem_desc_sw128(sKV, 0);
    const uint64_t desc_v0 = ptx::smem_desc_sw128(sKV, kHalfBytes);

    if constexpr (kPair) {
      // =========================================================== CTA pairs, warps 0-3
      // The two CTAs of a pair hold the query tiles 2k and 2k + 1 of one work item and walk the same key tiles
      // in the shared-accumulator form.  Every product is ONE pair instruction (M = 256) issued by the even CTA:
      // each CTA's 128 query rows (or its P rows in TMEM) meet all 128 keys of the tile, of which each CTA has
      // loaded only half -- for Q K^T 64 of the keys, for P V 64 of V's columns -- so a CTA writes and reads
      // half the shared-memory bytes per key tile that it would alone.  Roles per CTA:
      //   warp 0  TMA producer of this CTA's halves (kKvFull, local)
      //   warp 2  forwarder: tells the even CTA that a half has landed (one remote arrival per stage on its
      //           kKvReady; the V half of a tile that is not full is announced by the softmax warpgroup that
      //           clears its tail instead)
      //   warp 1 / warp 3 of the even CTA: issue Q K^T / P V; their commits arrive on the barriers of both CTAs
      //   softmax warpgroups: as in the shared-accumulator form; kSFree / kPFull arrivals (one per warp) go to
      //           the even CTA's barriers.
      // A fixed reference can overflow; the pair then repeats the key range: a pass that only finds every row's
      // true maximum, and the shared-accumulator pass again with that maximum as the reference (exact).
      constexpr uint32_t idesc_qk2 = ptx::umma_idesc_bf16(2 * kBM, kBN, false);
      constexpr uint32_t idesc_pv2 = ptx::umma_idesc_bf16(2 * kBM, D, true);
      constexpr int kKBlock = 64 * 128;          // one [64 keys x 64 bf16] swizzled block of a K half-tile
      int mode = 0;                              // 0: reference from the first key tile, 1: row maxima only, 2: given reference
#pragma unroll 1
      for (int pass = 0; pass < PBars::kPasses && has_work; ++pass) {
        sBarLoop = sBar + 8u * (PBars::kFixed + pass * PBars::kSet);
        const int n_items = mode == 1 ? T : 2 * T;
        if (warp == 0 || warp == 2) {
          // ---- producer (warp 0) and forwarder (warp 2) walk the ring in the same order
          const bool producer = warp == 0;
          bool ok = true;
          bool waited = !early || !producer;
          auto tile_page = [&](int t) -> int {
            if (!producer || !p.paged || t >= TP || lane >= 8 || t * kBN + lane * 16 >= Lc) return 0;
            return __ldg(p.page_table + static_cast<size_t>(b) * p.max_pages + t * 8 + lane);
          };
          if (!producer && pass == 0) {
            ok = bounded_wait(bar(PBars::kQFull), 0, abort_flag, 3);
            if (ok && lane == 0) ptx::mbar_arrive_peer(ptx::map_to_rank(bar(PBars::kQReady), 0));
          }
          int kt = 0, vt = 0, issued = 0;
          int pk_cur = tile_page(t_lo), pk_next = tile_page(t_lo + 1);
          int pv_cur = pk_cur, pv_next = pk_next;
#pragma unroll 1
          for (; issued < n_items && ok; ++issued) {
            const bool take_k = mode == 1 || (kt < T && kt <= vt + kAhead);
            const int t = t_lo + (take_k ? kt : vt), stage = issued % kStages;
            const uint32_t full = lbar(PBars::kKvFull + stage);
            if (producer) {
              if (!waited && (t + 1) * kBN > L) {
                ptx::grid_dep_wait();
                waited = true;
              }
              if (issued >= kStages) {
                ok = bounded_wait(lbar(PBars::kKvEmpty + stage), ((issued / kStages) - 1) & 1, abort_flag, 1);
                if (!ok) break;
              }
              const uint32_t dst = sKV + stage * C::kStageBytes;
              if (t < TP && p.paged) {
                const int npages = min(8, (Lc - t * kBN + 15) / 16);
                if (take_k) {           // this CTA's 64 keys = pages 4 rank .. 4 rank + 3 of the tile
                  const int mine = max(0, min(4, npages - 4 * static_cast<int>(prank)));
                  const int pg = __shfl_sync(0xffffffffu, pk_cur, (4 * static_cast<int>(prank) + lane) & 7);
                  if (lane == 0) ptx::mbar_arrive_expect_tx(full, mine * kHalves * 2048);
                  __syncwarp();
                  if (lane < mine) {
                    for (int h = 0; h < kHalves; ++h)
                      ptx::tma_load_3d(dst + h * kKBlock + lane * 2048, &tm_k, full, h * 64, g, pg * 16);
                  }
                } else {                // all keys, this CTA's 64 columns
                  if (lane == 0) ptx::mbar_arrive_expect_tx(full, npages * 2048);
                  __syncwarp();
                  if (lane < npages) ptx::tma_load_3d(dst + lane * 2048, &tm_v, full, static_cast<int>(prank) * 64, g, pv_cur * 16);
                }
              } else if (lane == 0) {
                const bool prefix = t < TP;
                const int row0 = prefix ? t * kBN : (t - TP) * kBN;
                ptx::mbar_arrive_expect_tx(full, C::kStageBytes);
                if (take_k) {
                  for (int h = 0; h < kHalves; ++h)
                    ptx::tma_load_4d(dst + h * kKBlock, prefix ? &tm_k64 : &tm_tk64, full, h * 64, g,
                                     row0 + 64 * static_cast<int>(prank), b);
                } else {
                  ptx::tma_load_4d(dst, prefix ? &tm_v : &tm_tv, full, static_cast<int>(prank) * 64, g, row0, b);
                }
              }
            } else {
              ok = bounded_wait(full, (issued / kStages) & 1, abort_flag, 22);
              if (!ok) break;
              bool left_to_softmax = false;         // a V tile that is not full: announced once its tail is cleared
              if (!take_k) {
                const int valid = t < TP ? min(kBN, Lc - t * kBN) : min(kBN, ntree - (t - TP) * kBN);
                left_to_softmax = valid < kBN;
              }
              if (!left_to_softmax && lane == 0) ptx::mbar_arrive_peer(ptx::map_to_rank(lbar(PBars::kKvReady + stage), 0));
            }
            if (take_k) {
              ++kt;
              pk_cur = pk_next;
              pk_next = tile_page(t + 2);
            } else {
              ++vt;
              pv_cur = pv_next;
              pv_next = tile_page(t + 2);
            }
            __syncwarp();
          }
          if (producer && __any_sync(0xffffffffu, *abort_flag != 0u)) {
            // drain: every load that was issued must land before the CTA may exit
            for (int st = 0; st < kStages; ++st) {
              if (issued > st) {
                const int last = ((issued - 1 - st) / kStages) * kStages + st;     // last item issued to stage st
                bounded_wait(lbar(PBars::kKvFull + st), (last / kStages) & 1, abort_flag, 2);
              }
            }
            bounded_wait(bar(PBars::kQFull), 0, abort_flag, 3);
          }
        } else if (prank == 0 && warp == 1) {
          // ---- Q K^T of both CTAs' query tiles against the whole key tile
          bool ok = pass > 0 || bounded_wait(bar(PBars::kQReady), 0, abort_flag, 4);
          const int lead = min(kAhead + 1, T);
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) {
            const int w = tl & 1, j = tl >> 1;
            const int item = mode == 1 ? tl : (tl < lead ? tl : 2 * tl - lead + 1);
            const int stage = item % kStages;
            if (j > 0) {
              ok = bounded_wait(lbar(PBars::kSFree + w), (j - 1) & 1, abort_flag, 20);
              if (!ok) break;
            }
            ok = bounded_wait_cl(lbar(PBars::kKvReady + stage), (item / kStages) & 1, abort_flag, 5);
            if (!ok) break;
            ptx::tc_fence_after();
            const uint64_t desc_k = desc_k0 + static_cast<uint64_t>(stage * (C::kStageBytes >> 4));
            const uint32_t s_tmem = tmem_base + C::shared_s(w);
            if (ptx::elect_one()) {
#pragma unroll
              for (int kd = 0; kd < D / 16; ++kd) {
                const uint64_t off_q = static_cast<uint64_t>(((kd / 4) * kHalfBytes + (kd % 4) * 32) >> 4);
                const uint64_t off_k = static_cast<uint64_t>(((kd / 4) * kKBlock + (kd % 4) * 32) >> 4);
                ptx::umma_ss2(s_tmem, desc_q0 + off_q, desc_k + off_k, idesc_qk2, kd > 0 ? 1u : 0u);
              }
              ptx::umma_commit2(lbar(PBars::kSFull + w), 3);
              ptx::umma_commit2(lbar(PBars::kKvEmpty + stage), 3);
            }
          }
        } else if (prank == 0 && warp == 3 && mode != 1) {
          // ---- O += P V of both CTAs
          bool ok = true;
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) {
            const int w = tl & 1, j = tl >> 1;
            const int item = v_item(tl, kAhead);
            const int stage = item % kStages;
            ok = bounded_wait(lbar(PBars::kPFull + w), j & 1, abort_flag, 8);        // (P first, as in the single-CTA form)
            if (!ok) break;
            ok = bounded_wait_cl(lbar(PBars::kKvReady + stage), (item / kStages) & 1, abort_flag, 7);
            if (!ok) break;
            ptx::tc_fence_after();
            const uint64_t desc_v = desc_v0 + static_cast<uint64_t>(stage * (C::kStageBytes >> 4));
            const uint32_t p_tmem = tmem_base + C::shared_p(w);
            const uint32_t o_tmem = tmem_base + C::shared_o();
            if (ptx::elect_one()) {
#pragma unroll
              for (int kk = 0; kk < kBN / 16; ++kk)
                ptx::umma_ts2(o_tmem, p_tmem + kk * 8, desc_v + static_cast<uint64_t>((kk * 2048) >> 4), idesc_pv2,
                              (tl == 0 && kk == 0) ? 0u : 1u);
              ptx::umma_commit2(lbar(PBars::kODone + w), 3);
              ptx::umma_commit2(lbar(PBars::kKvEmpty + stage), 3);
              if (tl == T - 1) ptx::umma_commit2(lbar(PBars::kOFinal), 3);
            }
          }
        }
        const uint32_t verdict = pair_verdict(pass);
        if ((verdict & 2u) || pass == 2 || (pass == 0 && !(verdict & 1u))) break;
        mode = pass + 1;
      }
      classic = false;
      shared_result = true;
    } else if constexpr (MT == 1) {
      if (has_work) {
        if (warp == 0) {
          // a paged tile is 16 small copies: two warps request them
          if (p.paged) produce(kAhead, std::integral_constant<int, 0>{}, 0);
          else produce(kAhead, std::integral_constant<int, -1>{}, n_early);
        } else if (warp == 2) {
          if (p.paged) produce(kAhead, std::integral_constant<int, 1>{}, 0);
        } else if (warp == 1) {
          // =========================================================== tcgen05 issuers, shared-accumulator form
          // Key tile tl belongs to warpgroup tl & 1 (score buffer and P buffer of that warpgroup).  Warp 1
          // issues every Q K^T, warp 3 every P V: the two chains depend on each other only through the softmax
          // warpgroups' barriers, and while one warp sits in the (blocking) issue of its eight instructions the
          // other gets through its waits.  A Q K^T may overwrite a score buffer once its warpgroup has read the
          // scores before (kSFree); a warpgroup may overwrite its P buffer once the P V that read it is
          // complete (kODone).  Ring positions: K_0 .. K_kAhead, then V_t, K_{t+kAhead+1} alternating.
          bool ok = bounded_wait(bar(Bars::kQFull), 0, abort_flag, 4);
          if (lane == 0) JET_TR(2);
          const int lead = min(kAhead + 1, T);
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) {
            const int w = tl & 1, j = tl >> 1;
            const int2 pos = p.paged ? k_pos_split(tl) : ring_pos(tl < lead ? tl : 2 * tl - lead + 1);
            const int stage = pos.x;
            const uint32_t par = pos.y;
            if (tl == 12 && lane == 0) JET_TR(61);
            if (j > 0) {
              ok = bounded_wait(bar(Bars::kSFree + w), (j - 1) & 1, abort_flag, 20);
              if (!ok) break;
            }
            if (tl == 12 && lane == 0) JET_TR(62);
            ok = bounded_wait(bar(Bars::kKvFull + stage), par, abort_flag, 5);
            if (!ok) break;
            if (tl == 12 && lane == 0) JET_TR(63);
            if (tl == 0 && lane == 0) JET_TR(3);
            ptx::tc_fence_after();
            const uint64_t desc_k = desc_k0 + static_cast<uint64_t>(stage * (C::kStageBytes >> 4));
            const uint32_t s_tmem = tmem_base + C::shared_s(w);
            if (ptx::elect_one()) {
#pragma unroll
              for (int kd = 0; kd < D / 16; ++kd) {
                const uint64_t off = static_cast<uint64_t>(((kd / 4) * kHalfBytes + (kd % 4) * 32) >> 4);
                ptx::umma_ss(s_tmem, desc_q0 + off, desc_k + off, idesc_qk, kd > 0 ? 1u : 0u);
              }
              ptx::umma_commit(bar(Bars::kSFull + w));
              ptx::umma_commit(bar(Bars::kKvEmpty + stage));
            }
          }
        } else if (warp == 3) {
          bool ok = true;
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) {
            const int w = tl & 1, j = tl >> 1;
            const int2 pos = p.paged ? v_pos_split(tl) : ring_pos(v_item(tl, kAhead));
            const int stage = pos.x;
            const uint32_t par = pos.y;
            if (tl == 8 && lane == 0) JET_TR(58);
            // P first: once P of this tile exists its Q K^T is complete, i.e. every K tile up to this one has landed.
            // In the shared ring the stages of V tiles 1 and 2 were first used by K tiles 0 and 2, whose phases this
            // warp has not seen; behind the P wait the parity of the V tile's phase cannot be mistaken for theirs.
            ok = bounded_wait(bar(Bars::kPFull + w), j & 1, abort_flag, 8);
            if (!ok) break;
            if (tl == 8 && lane == 0) JET_TR(59);
            ok = bounded_wait(bar(Bars::kKvFull + stage), par, abort_flag, 7);
            if (!ok) break;
            if (tl == 8 && lane == 0) JET_TR(60);
            ptx::tc_fence_after();
            if (w == 0 && j < 8 && lane == 0) JET_TR(50 + j);
            const uint64_t desc_v = desc_v0 + static_cast<uint64_t>(stage * (C::kStageBytes >> 4));
            const uint32_t p_tmem = tmem_base + C::shared_p(w);
            const uint32_t o_tmem = tmem_base + C::shared_o();
            if (ptx::elect_one()) {
#pragma unroll
              for (int kk = 0; kk < kBN / 16; ++kk)      // 16 keys = 8 TMEM columns of packed bf16 pairs
                ptx::umma_ts(o_tmem, p_tmem + kk * 8, desc_v + static_cast<uint64_t>((kk * 2048) >> 4), idesc_pv,
                             (tl == 0 && kk == 0) ? 0u : 1u);
              ptx::umma_commit(bar(Bars::kODone + w));
              ptx::umma_commit(bar(Bars::kKvEmpty + stage));
              if (tl == T - 1) ptx::umma_commit(bar(Bars::kOFinal));
            }
          }
        }
      }
      ptx::cta_sync();                                  // every role has left the shared-accumulator pass
      classic = *redo_flag != 0u && *abort_flag == 0u;
      shared_result = !classic;
      if (classic) second_barrier_set();
    }

    if constexpr (C::kTurns) {
      // =========================================================== two query tiles per CTA
      // Each query tile (stream) keeps the classic bookkeeping -- own accumulator, running reference, rescale
      // when it rises -- but the two tiles take turns on ONE score buffer, which leaves TMEM columns for a P
      // buffer per tile: a thread releases the score buffer as soon as it has read its row, the other tile's
      // Q K^T (warp 1) follows at once, and the P V products (warp 3) read P from buffers of their own.  The
      // chain softmax -> P V -> Q K^T -> softmax of the classic form is gone.
      classic = false;
      if (has_work) {
        if (warp == 0) {
          produce(0, std::integral_constant<int, 0>{}, n_early);            // K tiles
        } else if (warp == 2) {
          produce(0, std::integral_constant<int, 1>{}, n_early);            // V tiles (a paged tile is 16 small copies: two warps request them)
        } else if (warp == 1) {
          bool ok = bounded_wait(bar(Bars::kQFull), 0, abort_flag, 4);
          int prev_mt = -1, prev_tl = 0;
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) {
            const int2 pos = k_pos_split(tl);
            const int stage = pos.x;
            ok = bounded_wait(bar(Bars::kKvFull + stage), pos.y, abort_flag, 5);
            if (!ok) break;
            const uint64_t desc_k = desc_k0 + static_cast<uint64_t>((stage * C::kStageBytes) >> 4);
            for (int mt = 0; mt < n_mt && ok; ++mt) {
              if (prev_mt >= 0) {       // the warpgroup that used the score buffer before has read its scores
                ok = bounded_wait(bar(Bars::kSFree + prev_mt), prev_tl & 1, abort_flag, 20);
                if (!ok) break;
              }
              ptx::tc_fence_after();
              const uint64_t desc_q = desc_q0 + static_cast<uint64_t>(mt * ((kHalves * kHalfBytes) >> 4));
              const uint32_t s_tmem = tmem_base + C::turn_s();
              if (ptx::elect_one()) {
#pragma unroll
                for (int kd = 0; kd < D / 16; ++kd) {
                  const uint64_t off = static_cast<uint64_t>(((kd / 4) * kHalfBytes + (kd % 4) * 32) >> 4);
                  ptx::umma_ss(s_tmem, desc_q + off, desc_k + off, idesc_qk, kd > 0 ? 1u : 0u);
                }
                ptx::umma_commit(bar(Bars::kSFull + mt));
                if (mt == n_mt - 1) ptx::umma_commit(bar(Bars::kKvEmpty + stage));    // K tile read
              }
              prev_mt = mt;
              prev_tl = tl;
            }
          }
        } else if (warp == 3) {
          bool ok = true;
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) {
            const int2 pos = v_pos_split(tl);
            const int stage = pos.x;
            ok = bounded_wait(bar(Bars::kKvFull + stage), pos.y, abort_flag, 7);
            if (!ok) break;
            const uint64_t desc_v = desc_v0 + static_cast<uint64_t>((stage * C::kStageBytes) >> 4);
            for (int mt = 0; mt < n_mt && ok; ++mt) {
              ok = bounded_wait(bar(Bars::kPFull + mt), tl & 1, abort_flag, 8);
              if (!ok) break;
              ptx::tc_fence_after();
              const uint32_t p_tmem = tmem_base + C::turn_p(mt);
              const uint32_t o_tmem = tmem_base + C::turn_o(mt);
              if (ptx::elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk)
                  ptx::umma_ts(o_tmem, p_tmem + kk * 8, desc_v + static_cast<uint64_t>((kk * 2048) >> 4), idesc_pv,
                               (tl == 0 && kk == 0) ? 0u : 1u);
                ptx::umma_commit(bar(Bars::kODone + mt));
                if (mt == n_mt - 1) ptx::umma_commit(bar(Bars::kKvEmpty + stage));    // V tile read
              }
            }
          }
        }
      }
    }

    if (!kPair && !C::kTurns && classic && has_work) {
      if (warp == 0) {
        produce(0, std::integral_constant<int, -1>{}, 0);
      } else if (warp == 1) {
        // =========================================================== tcgen05 issuer, classic form
        // A stream is a chain  S = Q K^T -> softmax -> O += P V -> next S  on its own score buffer (which the P
        // overwrites) and accumulator: with one query tile per CTA the two streams take alternate key tiles,
        // with two each stream is one query tile and takes every key tile.  The streams take turns: a turn
        // issues one tile's P V and the stream's next Q K^T, so that one stream's softmax runs under the other
        // stream's products.  Within a stream the next Q K^T overwrites the P of the tile before; it is issued
        // after that tile's P V, and one thread's MMAs execute in issue order, so it needs no further wait.
        constexpr int kStep = MT == 1 ? 2 : 1;            // distance between a stream's tiles
        bool ok = bounded_wait(bar(Bars::kQFull), 0, abort_flag, 4);
        if (lane == 0) JET_TR(2);
        auto issue_qk = [&](int stream, int tl) {
          const int item = 2 * tl, stage = item % kStages;
          ok = bounded_wait(lbar(Bars::kKvFull + stage), (item / kStages) & 1, abort_flag, 5);
          if (!ok) return;
          if (tl == 0 && stream == 0 && lane == 0) JET_TR(3);
          ptx::tc_fence_after();
          const int mt = MT == 1 ? 0 : stream;
          const uint64_t desc_q = desc_q0 + static_cast<uint64_t>(mt * ((kHalves * kHalfBytes) >> 4));
          const uint64_t desc_k = desc_k0 + static_cast<uint64_t>(stage * (C::kStageBytes >> 4));
          const uint32_t s_tmem = tmem_base + C::s_col(mt, tl);
          if (ptx::elect_one()) {
#pragma unroll
            for (int kd = 0; kd < D / 16; ++kd) {
              const uint64_t off = static_cast<uint64_t>(((kd / 4) * kHalfBytes + (kd % 4) * 32) >> 4);
              ptx::umma_ss(s_tmem, desc_q + off, desc_k + off, idesc_qk, kd > 0 ? 1u : 0u);
            }
            ptx::umma_commit(lbar(Bars::kSFull + stream));
            ptx::umma_commit(lbar(Bars::kKvEmpty + stage));     // this stream has read the K tile
          }
        };
        auto turn = [&](int stream, int tl) {
          // ---- O += P V of tile tl (rows of masked keys of the V tile were cleared by the softmax threads)
          const int item = 2 * tl + 1, stage = item % kStages;
          ok = bounded_wait(lbar(Bars::kKvFull + stage), (item / kStages) & 1, abort_flag, 7);
          if (!ok) return;
          ok = bounded_wait(lbar(Bars::kPFull + stream), C::s_use(tl) & 1, abort_flag, 8);
          if (!ok) return;
          ptx::tc_fence_after();
          if (stream == 0 && tl / kStep < 8 && lane == 0) JET_TR(50 + tl / kStep);
          const int mt = MT == 1 ? 0 : stream;
          const uint64_t desc_v = desc_v0 + static_cast<uint64_t>(stage * (C::kStageBytes >> 4));
          const uint32_t s_tmem = tmem_base + C::s_col(mt, tl);
          const uint32_t o_tmem = tmem_base + C::o_col(mt, tl);
          const bool first = tl < kStep;                       // first product of this accumulator
          if (ptx::elect_one()) {
#pragma unroll
            for (int kk = 0; kk < kBN / 16; ++kk)      // 16 keys = 8 TMEM columns of packed bf16 pairs
              ptx::umma_ts(o_tmem, s_tmem + kk * 8, desc_v + static_cast<uint64_t>((kk * 2048) >> 4), idesc_pv,
                           (first && kk == 0) ? 0u : 1u);
            ptx::umma_commit(lbar(Bars::kODone + stream));
            ptx::umma_commit(lbar(Bars::kKvEmpty + stage));      // this stream has read the V tile
          }
          // ---- S = Q K^T of the stream's next tile
          if (tl + kStep < T) issue_qk(stream, tl + kStep);
        };
        if constexpr (MT == 1) {
          if (ok) issue_qk(0, 0);
          if (ok && T > 1) issue_qk(1, 1);
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl) turn(tl & 1, tl);
        } else {
          for (int mt = 0; mt < n_mt && ok; ++mt) issue_qk(mt, 0);
#pragma unroll 1
          for (int tl = 0; tl < T && ok; ++tl)
            for (int mt = 0; mt < n_mt && ok; ++mt) turn(mt, tl);
        }
      }
    }
    epilogue(std::false_type{});
  } else {
    ptx::setmaxnreg_inc<kRegsSoftmax>();
    if (early) ptx::grid_dep_wait();        // ancestor masks, outputs and the workspace belong behind the wait
    constexpr int kChunks = kBN / 32;                       // 32-key chunks per row and tile
    static_assert(kChunks == 4, "the register-resident row is written out for four 32-key chunks");
    constexpr int kStreams = C::kStreams;
    const int wg = (warp - 4) >> 2;
    const int mt = MT == 1 ? 0 : wg;                        // query tile of this warpgroup
    const int stream = MT == 1 ? wg : 0;                    // its share of the key tiles (tl % kStreams)
    const int r = (tid - 128) & 127;                        // row of the query tile = TMEM lane
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const int v = node_lo + mt * npt + static_cast<int>(udiv(r, p.magic_G));
    const bool row_live = v < n;
    const uint32_t* mask_row = p.anc_mask + (static_cast<size_t>(b) * p.B + (row_live ? v : 0)) * p.words;
    const float sl2 = p.scale_log2;
    // visibility bits of this row for 32-key chunk c of key tile t (a tile that is not full)
    auto chunk_bits = [&](int t, int c) -> uint32_t {
      if (t < TP) {
        const int nv = (L - t * kBN) - c * 32;              // prefix keys in this chunk (all of them visible)
        if (nv >= 32) return 0xFFFFFFFFu;
        const uint32_t prefix_bits = nv <= 0 ? 0u : ((1u << nv) - 1u);
        if (!p.tail) return prefix_bits;
        // the rest of the chunk are tree nodes s, s + 1, ... (s = -nv; negative: the chunk starts in the prefix)
        auto word = [&](int i) -> uint32_t { return (row_live && i >= 0 && i < p.words) ? __ldg(mask_row + i) : 0u; };
        if (nv > 0) return prefix_bits | (word(0) << nv);
        const int s = -nv, w = s >> 5, sh = s & 31;
        return sh ? ((word(w) >> sh) | (word(w + 1) << (32 - sh))) : word(w);
      }
      const int w = (t - TP) * 4 + c;
      return (row_live && w < p.words) ? __ldg(mask_row + w) : 0u;
    };
    // Masked keys get P = 0 exactly, but 0 * NaN is NaN: the V rows of keys beyond the valid ones (stale
    // cache rows, rows of padding nodes) are cleared before the P V product may read them.  `item` = the V
    // tile's position in the ring.  Returns false if the wait for the tile gave up.
    auto clear_v_tail = [&](int t, int2 pos) -> bool {
      const int valid = t < TP ? min(kBN, Lc - t * kBN) : min(kBN, ntree - (t - TP) * kBN);
      if (valid >= kBN) return true;
      const int stage = pos.x;
      if (!bounded_wait(lbar(Bars::kKvFull + stage), pos.y, abort_flag, 10)) return false;
      uint8_t* vt = gen_kv + stage * C::kStageBytes;
      const int chunks = (kBN - valid) * 8;                // 16-byte chunks per 64-column block
      for (int h = 0; h < kHalves; ++h)
        for (int i = r; i < chunks; i += 128)
          *reinterpret_cast<uint4*>(vt + h * kHalfBytes + valid * 128 + i * 16) = make_uint4(0u, 0u, 0u, 0u);
      ptx::fence_proxy_async_smem();
      return true;
    };

    if constexpr (kPair) {
      // =========================================================== CTA pairs, softmax warpgroups
      // The shared-accumulator form on this CTA's own query tile; arrivals that the issuing warps wait for go to
      // the even CTA's barriers, one per warp.
      auto arrive_pair = [&](uint32_t local_bar) {
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_peer(ptx::map_to_rank(local_bar, 0));
      };
      // This CTA's half of a V tile (all keys, 64 columns): rows of keys beyond the valid ones are cleared, then
      // the warpgroup announces the half to the even CTA in the forwarder's place.
      auto clear_v_half = [&](int t, int item) -> bool {
        const int valid = t < TP ? min(kBN, Lc - t * kBN) : min(kBN, ntree - (t - TP) * kBN);
        if (valid >= kBN) return true;
        const int stage = item % kStages;
        const bool landed = bounded_wait(lbar(PBars::kKvFull + stage), (item / kStages) & 1, abort_flag, 10);
        if (landed) {
          uint8_t* vt = gen_kv + stage * C::kStageBytes;
          const int chunks = (kBN - valid) * 8;
          for (int i = r; i < chunks; i += 128) *reinterpret_cast<uint4*>(vt + valid * 128 + i * 16) = make_uint4(0u, 0u, 0u, 0u);
          ptx::fence_proxy_async_all();
        }
        ptx::named_sync(3 + wg, 128);
        if (landed && r == 0) ptx::mbar_arrive_remote(ptx::map_to_rank(lbar(PBars::kKvReady + stage), 0));
        return landed;
      };
      float m_ref = 0.0f;
      int mode = 0;
      const uint32_t tS = t_lane + C::shared_s(wg);
      const uint32_t tP = t_lane + C::shared_p(wg);
#pragma unroll 1
      for (int pass = 0; pass < PBars::kPasses && has_work; ++pass) {
        sBarLoop = sBar + 8u * (PBars::kFixed + pass * PBars::kSet);
        bool ok = true;
        bool synced = false;
        bool saw_key = false;
        float m_run = -INFINITY;
        l = 0.0f;
        if (tid == 128) JET_TR(5 + pass);
#pragma unroll 1
        for (int tl = wg; tl < T && ok; tl += 2) {
          const int t = t_lo + tl, j = tl >> 1;
          const bool full_tile = t < TP && (L - t * kBN) >= kBN;
          ok = bounded_wait(lbar(PBars::kSFull + wg), j & 1, abort_flag, 9);
          if (!ok) break;
          ptx::tc_fence_after();
          if (tid == 128 && pass == 0 && j < 4) JET_TR(19 + 2 * j);
          if (tid == 128 && pass == 0 && j == 8) JET_TR(36);
          if (tid == 128 && pass == 0 && j == 16) JET_TR(37);
          uint32_t xa[32], xb[32], xc[32], xd[32];
          uint32_t b0 = 0xFFFFFFFFu, b1 = 0xFFFFFFFFu, b2 = 0xFFFFFFFFu, b3 = 0xFFFFFFFFu;
          if (!full_tile) { b0 = chunk_bits(t, 0); b1 = chunk_bits(t, 1); b2 = chunk_bits(t, 2); b3 = chunk_bits(t, 3); }
          saw_key = saw_key || (b0 | b1 | b2 | b3) != 0u;
          ptx::tmem_ld32(tS, xa);
          ptx::tmem_ld32(tS + 32, xb);
          ptx::tmem_ld32(tS + 64, xc);
          ptx::tmem_ld32(tS + 96, xd);
          ptx::tmem_wait_ld();
          ptx::tc_fence_before();
          arrive_pair(lbar(PBars::kSFree + wg));            // the scores are in registers
          if (tid == 128 && pass == 0 && j == 8) JET_TR(52);
          if (!full_tile) {
            mask_chunk(xa, b0);
            mask_chunk(xb, b1);
            mask_chunk(xc, b2);
            mask_chunk(xd, b3);
          }
          if (mode == 1 || (mode == 0 && j == 0 && wg == 0)) {
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            max_chunk(xa, mx);
            max_chunk(xb, mx);
            max_chunk(xc, mx);
            max_chunk(xd, mx);
            m_run = fmaxf(m_run, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])));
          }
          if (mode == 1) continue;
          if (mode == 0 && j == 0) {
            // the reference of a row: its maximum over the first key tile (0 if it sees no key there)
            if (wg == 0) {
              m_ref = (m_run == -INFINITY) ? -0.0f : m_run * sl2;
              if (T > 1) {
                ref_s[r] = m_ref;
                ptx::named_arrive(1, 256);
              }
            } else {
              ptx::named_sync(1, 256);
              m_ref = ref_s[r];
            }
            synced = true;
          }
          if (j > 0) {
            ok = bounded_wait(lbar(PBars::kODone + wg), (j - 1) & 1, abort_flag, 21);
            if (!ok) break;
          }
          if (tid == 128 && pass == 0 && j == 8) JET_TR(53);
          float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          exp_chunk(xa, sl2, m_ref, sum, tP);
          exp_chunk(xb, sl2, m_ref, sum, tP + 16);
          exp_chunk(xc, sl2, m_ref, sum, tP + 32);
          exp_chunk(xd, sl2, m_ref, sum, tP + 48);
          const float tile_sum = (sum[0] + sum[1]) + (sum[2] + sum[3]);
          if (row_live && !(tile_sum <= kSharedSumLimit)) redo_flag[pass] = 1u;
          l += tile_sum;
          if (tid == 128 && pass == 0 && j == 8) JET_TR(54);
          if (!full_tile) {
            ok = clear_v_half(t, v_item(tl, kAhead));
            if (!ok) break;
          }
          ptx::tmem_wait_st();                     // P is in TMEM
          ptx::tc_fence_before();
          arrive_pair(lbar(PBars::kPFull + wg));
          if (tid == 128 && pass == 0 && j < 4) JET_TR(20 + 2 * j);
          if (tid == 128 && pass == 0 && j == 8) JET_TR(55);
        }
        if (mode == 0) {
          // (see the shared-accumulator form: a row without a reference of its own may have lost its keys to underflow)
          if (row_live && saw_key && __float_as_uint(m_ref) == 0x80000000u && !(l >= kSharedSumFloor)) redo_flag[pass] = 1u;
          if (T > 1 && !synced) {
            if (wg == 0) ptx::named_arrive(1, 256);
            else ptx::named_sync(1, 256);
          }
        } else if (mode == 1) {
          // the row's true maximum over all keys of the slice, from both warpgroups
          if (wg == 1) ref_s[r] = m_run;
          ptx::named_sync(1, 256);
          if (wg == 0) {
            const float m = fmaxf(m_run, ref_s[r]);
            m_ref = (m == -INFINITY) ? 0.0f : m * sl2;
            ref_s[r] = m_ref;
          }
          ptx::named_sync(1, 256);
          if (wg == 1) m_ref = ref_s[r];
        }
        if (mode != 1) {
          if (ok) ok = bounded_wait(lbar(PBars::kOFinal), 0, abort_flag, 11);      // the last P V is complete
          if (ok) ptx::tc_fence_after();
        }
        row_ok = ok;
        const uint32_t verdict = pair_verdict(pass);
#ifdef JET_TRACE
        if (tid == 128 && p.trace) p.trace[(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 64 + 56 + pass] = 100 + verdict;
#endif
        if ((verdict & 2u) || pass == 2 || (pass == 0 && !(verdict & 1u))) break;
        mode = pass + 1;
      }
      m_ref_common = m_ref;
      classic = false;
      shared_result = true;
    } else if constexpr (MT == 1) {
      if (has_work) {
        // =========================================================== softmax, shared-accumulator form
        // Warpgroup wg takes key tiles wg, wg + 2, ...  A thread reads its whole score row from TMEM, hands
        // the score buffer back at once (the tile after next can be computed into it), exponentiates against
        // the row's fixed reference and writes P to the warpgroup's P buffer.
        bool ok = true;
        bool synced = false;                 // the two warpgroups have met at the reference hand-over
        bool saw_key = false;                // some key of this warpgroup's tiles is visible to the row
        float m_ref = 0.0f;
        const uint32_t tS = t_lane + C::shared_s(wg);
        const uint32_t tP = t_lane + C::shared_p(wg);
#pragma unroll 1
        for (int tl = wg; tl < T && ok; tl += 2) {
          const int t = t_lo + tl, j = tl >> 1;
          const bool full_tile = t < TP && (L - t * kBN) >= kBN;      // uniform: every key visible to every row
          ok = bounded_wait(bar(Bars::kSFull + wg), j & 1, abort_flag, 9);
          if (!ok) break;
          ptx::tc_fence_after();
          if (tid == 128 && j == 4) JET_TR(4);
          if (tid == 128 && j < 4) JET_TR(19 + 2 * j);
          if (tid == 256 && j < 4) JET_TR(32 + 2 * j);
          uint32_t xa[32], xb[32], xc[32], xd[32];
          uint32_t b0 = 0xFFFFFFFFu, b1 = 0xFFFFFFFFu, b2 = 0xFFFFFFFFu, b3 = 0xFFFFFFFFu;
          if (!full_tile) { b0 = chunk_bits(t, 0); b1 = chunk_bits(t, 1); b2 = chunk_bits(t, 2); b3 = chunk_bits(t, 3); }
          saw_key = saw_key || (b0 | b1 | b2 | b3) != 0u;
          ptx::tmem_ld32(tS, xa);
          ptx::tmem_ld32(tS + 32, xb);
          ptx::tmem_ld32(tS + 64, xc);
          ptx::tmem_ld32(tS + 96, xd);
          ptx::tmem_wait_ld();
          ptx::tc_fence_before();
          ptx::mbar_arrive(bar(Bars::kSFree + wg));          // the scores are in registers
          if (!full_tile) {
            mask_chunk(xa, b0);
            mask_chunk(xb, b1);
            mask_chunk(xc, b2);
            mask_chunk(xd, b3);
          }
          if (j == 0) {
            // The reference of a row: its maximum over the first key tile (0 if it sees no key there), found
            // by warpgroup 0 and handed to warpgroup 1 through shared memory.
            if (wg == 0) {
              float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
              max_chunk(xa, mx);
              max_chunk(xb, mx);
              max_chunk(xc, mx);
              max_chunk(xd, mx);
              const float m = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
              m_ref = (m == -INFINITY) ? -0.0f : m * sl2;     // -0.0 marks "no reference of its own" (same arithmetic as 0)
              if (T > 1) {
                ref_s[r] = m_ref;
                ptx::named_arrive(1, 256);          // warpgroup 1 waits for this, warpgroup 0 goes on
              }
            } else {
              ptx::named_sync(1, 256);
              m_ref = ref_s[r];
            }
            synced = true;
          }
          if (tid == 128 && j == 4) JET_TR(5);
          if (j > 0) {
            // the P V product of this warpgroup's tile before has read the P buffer
            ok = bounded_wait(bar(Bars::kODone + wg), (j - 1) & 1, abort_flag, 21);
            if (!ok) break;
          }
          if (tid == 128 && j == 4) JET_TR(16);
          float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          exp_chunk(xa, sl2, m_ref, sum, tP);
          exp_chunk(xb, sl2, m_ref, sum, tP + 16);
          exp_chunk(xc, sl2, m_ref, sum, tP + 32);
          exp_chunk(xd, sl2, m_ref, sum, tP + 48);
          const float tile_sum = (sum[0] + sum[1]) + (sum[2] + sum[3]);
          if (row_live && !(tile_sum <= kSharedSumLimit)) *redo_flag = 1u;
          l += tile_sum;
          if (tid == 128 && j == 4) JET_TR(17);
          if (!full_tile) {
            ok = clear_v_tail(t, p.paged ? v_pos_split(tl) : ring_pos(v_item(tl, kAhead)));
            if (!ok) break;
          }
          ptx::tmem_wait_st();                     // P is in TMEM
          ptx::tc_fence_before();
          ptx::mbar_arrive(bar(Bars::kPFull + wg));
          if (tid == 128 && j == 4) JET_TR(6);
          if (tid == 128 && j < 4) JET_TR(20 + 2 * j);
          if (tid == 256 && j < 4) JET_TR(33 + 2 * j);
        }
        // A row whose reference was not taken from scores of its own (no key of the first tile was visible to it:
        // reference 0) may have lost its keys to underflow; such a row sums to (almost) nothing although it saw
        // keys, and the CTA repeats the key range in the classic form.  (A row with a reference of its own sums
        // to at least 1 in warpgroup 0.  The test is per warpgroup and errs on the safe side.)
        if (row_live && saw_key && __float_as_uint(m_ref) == 0x80000000u && !(l >= kSharedSumFloor)) *redo_flag = 1u;
        if (T > 1 && !synced) {                   // a warpgroup that gave up early still takes part in the hand-over
          if (wg == 0) ptx::named_arrive(1, 256);
          else ptx::named_sync(1, 256);
        }
        if (tid == 128) JET_TR(10);
        if (ok) ok = bounded_wait(bar(Bars::kOFinal), 0, abort_flag, 11);      // the last P V is complete
        if (ok) ptx::tc_fence_after();
        row_ok = ok;
        m_ref_common = m_ref;
      }
      ptx::cta_sync();                                  // every role has left the shared-accumulator pass
      classic = *redo_flag != 0u && *abort_flag == 0u;
      shared_result = !classic;
      if (classic) {
        second_barrier_set();
        m_used = -INFINITY;
        l = 0.0f;
        row_ok = has_work;
      }
    }

    if constexpr (C::kTurns) {
      classic = false;
      if (has_work && wg < n_mt) {
        // =========================================================== softmax, one query tile of two
        bool ok = true;
        const uint32_t tS = t_lane + C::turn_s();
        const uint32_t tO = t_lane + C::turn_o(mt);
        const uint32_t tP = t_lane + C::turn_p(mt);
        int last_tl = -1;
#pragma unroll 1
        for (int tl = 0; tl < T && ok; ++tl) {
          const int t = t_lo + tl;
          const bool full_tile = t < TP && (L - t * kBN) >= kBN;      // uniform: every key visible to every row
          ok = bounded_wait(bar(Bars::kSFull + mt), tl & 1, abort_flag, 9);
          if (!ok) break;
          ptx::tc_fence_after();
          uint32_t xa[32], xb[32], xc[32], xd[32];
          uint32_t b0 = 0xFFFFFFFFu, b1 = 0xFFFFFFFFu, b2 = 0xFFFFFFFFu, b3 = 0xFFFFFFFFu;
          if (!full_tile) { b0 = chunk_bits(t, 0); b1 = chunk_bits(t, 1); b2 = chunk_bits(t, 2); b3 = chunk_bits(t, 3); }
          ptx::tmem_ld32(tS, xa);
          ptx::tmem_ld32(tS + 32, xb);
          ptx::tmem_ld32(tS + 64, xc);
          ptx::tmem_ld32(tS + 96, xd);
          ptx::tmem_wait_ld();
          ptx::tc_fence_before();
          ptx::mbar_arrive(bar(Bars::kSFree + mt));            // the scores are in registers: the other tile's turn
          if (!full_tile) {
            mask_chunk(xa, b0);
            mask_chunk(xb, b1);
            mask_chunk(xc, b2);
            mask_chunk(xd, b3);
          }
          if (__any_sync(0xffffffffu, m_used == -INFINITY)) {
            // nothing accumulated yet for some row: its reference is this tile's own row maximum
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            max_chunk(xa, mx);
            max_chunk(xb, mx);
            max_chunk(xc, mx);
            max_chunk(xd, mx);
            if (m_used == -INFINITY) m_used = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          }
          float m_ref = (m_used == -INFINITY) ? 0.0f : m_used * sl2;
          float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          if (tl >= 1) {
            // the P V product of the tile before is complete: the P buffer is free and O may be rescaled
            ok = bounded_wait(bar(Bars::kODone + mt), (tl - 1) & 1, abort_flag, 21);
            if (!ok) break;
            ptx::tc_fence_after();
          }
          exp_chunk(xa, sl2, m_ref, sum, tP);
          exp_chunk(xb, sl2, m_ref, sum, tP + 16);
          exp_chunk(xc, sl2, m_ref, sum, tP + 32);
          exp_chunk(xd, sl2, m_ref, sum, tP + 48);
          float tile_sum = (sum[0] + sum[1]) + (sum[2] + sum[3]);
          float factor = 1.0f;
          if (__any_sync(0xffffffffu, !(tile_sum <= kFastSumLimit))) {
            // The reference was too low for some row of this warp (or a value is not finite): take the tile's
            // true row maximum as the new reference and compute the tile again (the scores are in registers).
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            max_chunk(xa, mx);
            max_chunk(xb, mx);
            max_chunk(xc, mx);
            max_chunk(xd, mx);
            const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            if (m_tile > m_used) {
              if (m_used > -INFINITY) factor = exp2f((m_used - m_tile) * sl2);
              m_used = m_tile;
            }
            m_ref = (m_used == -INFINITY) ? 0.0f : m_used * sl2;
            sum[0] = sum[1] = sum[2] = sum[3] = 0.0f;
            ptx::tmem_wait_st();
            exp_chunk(xa, sl2, m_ref, sum, tP);
            exp_chunk(xb, sl2, m_ref, sum, tP + 16);
            exp_chunk(xc, sl2, m_ref, sum, tP + 32);
            exp_chunk(xd, sl2, m_ref, sum, tP + 48);
            tile_sum = (sum[0] + sum[1]) + (sum[2] + sum[3]);
            if (__any_sync(0xffffffffu, factor != 1.0f) && tl > 0) {
#pragma unroll 1
              for (int c = 0; c < D / 32; ++c) {
                ptx::tmem_ld32(tO + c * 32, xa);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) xa[j] = __float_as_uint(__uint_as_float(xa[j]) * factor);
                ptx::tmem_st32(tO + c * 32, xa);
              }
            }
          }
          l = l * factor + tile_sum;
          if (!full_tile) {
            ok = clear_v_tail(t, v_pos_split(tl));
            if (!ok) break;
          }
          ptx::tmem_wait_st();                     // P (and a rescaled O) are in TMEM
          ptx::tc_fence_before();
          ptx::mbar_arrive(bar(Bars::kPFull + mt));
          last_tl = tl;
        }
        // O is complete once the last P V of this accumulator has been committed
        if (ok && last_tl >= 0) ok = bounded_wait(bar(Bars::kODone + mt), last_tl & 1, abort_flag, 11);
        if (ok) ptx::tc_fence_after();
        row_ok = ok;
      }
    }

    if (!kPair && !C::kTurns && classic && has_work && (MT == 1 || wg < n_mt)) {
      // =========================================================== softmax, classic form
      bool ok = true;
      int last_tl = -1;

#pragma unroll 1
      for (int tl = stream; tl < T && ok; tl += kStreams) {
        const int t = t_lo + tl;
        const uint32_t tS = t_lane + C::s_col(mt, tl);
        const uint32_t tO = t_lane + C::o_col(mt, tl);
        const bool full_tile = t < TP && (L - t * kBN) >= kBN;      // uniform: every key visible to every row

        ok = bounded_wait(lbar(Bars::kSFull + C::s_buf(mt, tl)), C::s_use(tl) & 1, abort_flag, 9);
        if (!ok) break;
        ptx::tc_fence_after();
        if (tid == 128 && tl < 1) JET_TR(4);
        if (tid == 128 && tl / kStreams < 4) JET_TR(19 + 2 * (tl / kStreams));
        if (tid == 128 && tl / kStreams == 3) JET_TR(58);
        if (tid == 256 && tl / kStreams < 4) JET_TR(32 + 2 * (tl / kStreams));

        // (The P V product of this accumulator's previous tile is complete: the Q K^T that produced these
        //  scores was only issued after it.  So O may be rescaled and the score buffer overwritten with P.)
        // ---- The thread reads its whole score row (128 values) from TMEM once.  Keys the row must not see
        //      (ragged end of the prefix, tree keys outside the ancestor set) are replaced by -inf right away,
        //      so they get probability exactly 0 whatever the cache rows behind them hold.  The row is then
        //      exponentiated against the reference maximum it already has -- no pass for the row maximum, except
        //      in the first tile of a stream.  Any reference is exact as long as nothing overflows; the row sum
        //      of the tile shows whether the reference was too low (then, or if a value is not finite, the tile
        //      is redone with its true maximum).
        uint32_t xa[32], xb[32], xc[32], xd[32];
        uint32_t b0 = 0xFFFFFFFFu, b1 = 0xFFFFFFFFu, b2 = 0xFFFFFFFFu, b3 = 0xFFFFFFFFu;
        if (!full_tile) { b0 = chunk_bits(t, 0); b1 = chunk_bits(t, 1); b2 = chunk_bits(t, 2); b3 = chunk_bits(t, 3); }
        ptx::tmem_ld32(tS, xa);
        ptx::tmem_ld32(tS + 32, xb);
        ptx::tmem_ld32(tS + 64, xc);
        ptx::tmem_ld32(tS + 96, xd);
        ptx::tmem_wait_ld();
        if (!full_tile) {
          mask_chunk(xa, b0);
          mask_chunk(xb, b1);
          mask_chunk(xc, b2);
          mask_chunk(xd, b3);
        }
        if (__any_sync(0xffffffffu, m_used == -INFINITY)) {
          // nothing accumulated yet for some row: its reference is the tile's own row maximum (which stays
          // -inf if the row sees no key of this tile)
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          max_chunk(xa, mx);
          max_chunk(xb, mx);
          max_chunk(xc, mx);
          max_chunk(xd, mx);
          if (m_used == -INFINITY) m_used = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        }
        if (tid == 128 && tl < 1) JET_TR(5);
        if (tid == 128 && tl / kStreams == 3) JET_TR(59);
        float m_ref = (m_used == -INFINITY) ? 0.0f : m_used * sl2;
        float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        // P is stored chunk by chunk, under the arithmetic of the next chunk.  It overwrites the score columns
        // of the first two chunks, so those two stay in registers (xa, xb) in case the tile has to be redone;
        // the last two chunks go first, their score columns stay intact in TMEM.
        exp_chunk(xc, sl2, m_ref, sum, tS + 32);
        exp_chunk(xd, sl2, m_ref, sum, tS + 48);
        exp_chunk(xa, sl2, m_ref, sum, tS);
        exp_chunk(xb, sl2, m_ref, sum, tS + 16);
        float tile_sum = (sum[0] + sum[1]) + (sum[2] + sum[3]);
        if (tid == 128 && tl < 1) JET_TR(17);
        if (tid == 128 && tl / kStreams == 3) JET_TR(60);
        float factor = 1.0f;
        if (__any_sync(0xffffffffu, !(tile_sum <= kFastSumLimit))) {
          // The reference was too low for some row of this warp (or a value is not finite): take the tile's
          // true row maximum as the new reference and compute the tile again.
          ptx::tmem_ld32(tS + 64, xc);
          ptx::tmem_ld32(tS + 96, xd);
          ptx::tmem_wait_ld();
          if (!full_tile) {
            mask_chunk(xc, b2);
            mask_chunk(xd, b3);
          }
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          max_chunk(xa, mx);
          max_chunk(xb, mx);
          max_chunk(xc, mx);
          max_chunk(xd, mx);
          const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          if (m_tile > m_used) {
            if (m_used > -INFINITY) factor = exp2f((m_used - m_tile) * sl2);
            m_used = m_tile;
          }
          m_ref = (m_used == -INFINITY) ? 0.0f : m_used * sl2;
          sum[0] = sum[1] = sum[2] = sum[3] = 0.0f;
          ptx::tmem_wait_st();
          exp_chunk(xc, sl2, m_ref, sum, tS + 32);
          exp_chunk(xd, sl2, m_ref, sum, tS + 48);
          exp_chunk(xa, sl2, m_ref, sum, tS);
          exp_chunk(xb, sl2, m_ref, sum, tS + 16);
          tile_sum = (sum[0] + sum[1]) + (sum[2] + sum[3]);
          if (__any_sync(0xffffffffu, factor != 1.0f) && last_tl >= 0) {
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              ptx::tmem_ld32(tO + c * 32, xa);
              ptx::tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) xa[j] = __float_as_uint(__uint_as_float(xa[j]) * factor);
              ptx::tmem_st32(tO + c * 32, xa);
            }
          }
        }
        l = l * factor + tile_sum;
        if (!full_tile) {
          ok = clear_v_tail(t, ring_pos(2 * tl + 1));
          if (!ok) break;
        }
        ptx::tmem_wait_st();                     // P (and a rescaled O) are in TMEM
        ptx::tc_fence_before();
        ptx::mbar_arrive(lbar(Bars::kPFull + C::s_buf(mt, tl)));
        if (tid == 128 && tl < 1) JET_TR(6);
        if (tid == 128 && tl / kStreams < 4) JET_TR(20 + 2 * (tl / kStreams));
        if (tid == 256 && tl / kStreams < 4) JET_TR(33 + 2 * (tl / kStreams));
        last_tl = tl;
      }
      if (tid == 128) JET_TR(10);
      // O is complete once the last P V of this accumulator has been committed
      if (ok && last_tl >= 0)
        ok = bounded_wait(lbar(Bars::kODone + C::s_buf(mt, last_tl)), C::s_use(last_tl) & 1, abort_flag, 11);
      if (ok) ptx::tc_fence_after();
      row_ok = ok;
    }
    epilogue(std::true_type{});
  }

  // ---------------- teardown
  if (tid == 128) JET_TR(12);
  if (via_cluster) {
    __syncwarp();
    ptx::cluster_sync_all();     // every CTA of the cluster has read this CTA's staged rows
  }
  ptx::tc_fence_before();
  ptx::cta_sync();
  if constexpr (kPair) {
    ptx::cluster_sync_all();       // the pair's TMEM is released together, once both CTAs are done with theirs
    if (warp == 2) {
      ptx::tc_fence_after();
      ptx::tmem_dealloc2(tmem_base, C::kTmemCols);
    }
  } else if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::kTmemCols);
  }
  if (tid == 0) {
    JET_TR(13);
#ifdef JET_TRACE
    if (p.trace) {
      unsigned long long gt;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt));
      p.trace[(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 64 + 61] = static_cast<long long>(gt);
    }
#endif
    if (*abort_flag && p.status) *p.status = JET_ERR_TIMEOUT;
#ifdef JET_TRACE
    if (*abort_flag && p.trace) p.trace[(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 64 + 31] = *abort_flag;
#endif
  }
}

// ------------------------------------------------------------------------------------------ merge kernel
// Second launch of the two-launch slice merge: every key slice of a work item has left its 128 normalised rows
// (D bf16 values + log2-sum-exp, fp32) in the workspace; one thread combines 8 output values of one row over the
// S slices with softmax weights of the slice sums and writes them (bf16), the first thread of a row also its
// log-sum-exp.  All loads of a thread are independent of each other: one round trip to L2.
struct MergeParams {
  const uint8_t* partials;
  const int32_t* n_nodes;
  __nv_bfloat16* out;
  float* lse;
  int B, Hq, Hkv, G, S, MT, n_mgroups, npt;
  uint32_t magic_G;
};

template <int D>
__global__ void __launch_bounds__(256) tree_attn_merge_kernel(const MergeParams p) {
  constexpr int kPitch = D * 2 + 16;
  constexpr int kItemsPerRow = D / 8;
  constexpr int kRowsPerCta = 256 / kItemsPerRow;
  constexpr int kBlocksPerTile = kBM / kRowsPerCta;
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  int bx = static_cast<int>(blockIdx.x);
  const int rb = bx % kBlocksPerTile;
  bx /= kBlocksPerTile;
  const int mt = bx % p.MT, mgroup = bx / p.MT;
  const int g = blockIdx.y, b = blockIdx.z;
  const int row = rb * kRowsPerCta + static_cast<int>(threadIdx.x) / kItemsPerRow;
  const int c8 = static_cast<int>(threadIdx.x) % kItemsPerRow;
  const int R = mt * kBM + row;                              // row within the work item
  const int vq = static_cast<int>(udiv(R, p.magic_G));
  const int v = mgroup * p.MT * p.npt + vq, h = g * p.G + (R - vq * p.G);
  if (v >= p.B) return;
  const int n = min(p.n_nodes[b], p.B);
  const int unit = (b * p.Hkv + g) * p.n_mgroups + mgroup;
  const int S = p.S;
  const size_t stride = static_cast<size_t>(p.MT) * kBM * kPitch;       // distance between consecutive slices
  const uint8_t* row0 = p.partials + (static_cast<size_t>(unit) * S * p.MT + mt) * (static_cast<size_t>(kBM) * kPitch) +
                        static_cast<size_t>(row) * kPitch;
  // every load of the thread is issued before any is used (the slots are valid memory for any row)
  float lc[kMaxSplit];
  uint4 x[kMaxSplit];
#pragma unroll
  for (int c = 0; c < kMaxSplit; ++c) {
    if (c < S) {
      lc[c] = __ldcg(reinterpret_cast<const float*>(row0 + c * stride + D * 2));
      x[c] = __ldcg(reinterpret_cast<const uint4*>(row0 + c * stride + c8 * 16));
    } else {
      lc[c] = -INFINITY;
      x[c] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  float lse2 = -INFINITY;
  float mx = -INFINITY;
#pragma unroll
  for (int c = 0; c < kMaxSplit; ++c) mx = fmaxf(mx, lc[c]);
  if (v < n && mx > -INFINITY) {
    float wsum = 0.0f;
#pragma unroll
    for (int c = 0; c < kMaxSplit; ++c) {
      const float w = lc[c] > -INFINITY ? exp2f(lc[c] - mx) : 0.0f;       // absent slices get weight 0 ...
      wsum += w;
      const uint32_t v4[4] = {x[c].x, x[c].y, x[c].z, x[c].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {      // bf16 pair -> fp32: the bits are the upper half of the float
        const float lo = __uint_as_float(v4[q] << 16), hi = __uint_as_float(v4[q] & 0xFFFF0000u);
        acc[2 * q] += w > 0.0f ? w * lo : 0.0f;                          // ... and whatever they hold is not used
        acc[2 * q + 1] += w > 0.0f ? w * hi : 0.0f;
      }
    }
    const float inv = 1.0f / wsum;
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] *= inv;
    lse2 = mx + log2f(wsum);
  }
  *reinterpret_cast<uint4*>(p.out + ((static_cast<size_t>(b) * p.B + v) * p.Hq + h) * D + c8 * 8) =
      make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                 pack_bf16(acc[6], acc[7]));
  if (p.lse && c8 == 0) p.lse[(static_cast<size_t>(b) * p.Hq + h) * p.B + v] = lse2 * 0.6931471805599453f;
}

// ------------------------------------------------------------------------------------------ host
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return static_cast<EncodeFn>(nullptr);
    return reinterpret_cast<EncodeFn>(sym);
  }();
  return fn;
}

// bf16 tensor map, 128-byte swizzle, innermost box of 64 elements.
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[5], gstr[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), gdim, gstr, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Everything the host side caches about the GPU is kept per device (a process may drive several).
constexpr int kMaxDevices = 64;
int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return 0;
  }
  return dev;
}

int sm_count() {
  static std::atomic<int> cache[kMaxDevices];
  const int dev = current_device();
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
      cudaGetLastError();
      v = 148;
    }
    n = v;
    cache[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

struct Plan {
  int mt;          // query tiles per CTA (1 or 2)
  int n_mgroups;   // groups of mt query tiles per (sequence, KV head)
  int units;       // work items before key slicing
  int nsplit;      // key slices
  int via_global;  // 1: slices exchange rows through the workspace (no cluster), 0: through a cluster
  int pair;        // 1: CTA pairs (clusters of two CTAs with consecutive query tiles share the K/V tiles)
};

constexpr size_t kCounterBytes = 4096;     // head of the workspace: arrival / departure counters

template <int D, int MT, bool kPair = false>
bool configure_kernel() {
  static std::atomic<int> states[kMaxDevices];      // per device: 0 = not yet, 1 = ok, -1 = failed
  std::atomic<int>& state_ref = states[current_device()];
  int state = state_ref.load(std::memory_order_acquire);
  if (state == 0) {
    auto set = [](auto kernel) {
      return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D, MT, kPair>::kSmemBytes) ==
                 cudaSuccess &&
             cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    };
    state = (set(tree_attn_kernel<D, MT, false, kPair>) && set(tree_attn_kernel<D, MT, true, kPair>))
                ? 1
                : -1;
    if (state < 0) cudaGetLastError();
    state_ref.store(state, std::memory_order_release);
  }
  return state > 0;
}

// How many clusters of `cluster` CTAs of this kernel the device can hold at once (one CTA per SM, and a
// cluster must fit inside one GPC).  Asked of the driver once per cluster size and cached.
template <int D, int MT>
int max_active_clusters(int cluster) {
  static std::atomic<int> caches[kMaxDevices][kMaxSplit + 1];      // per device: 0 = unknown, -1 = none
  if (cluster < 1 || cluster > kMaxCluster) return 0;       // (the occupancy query does not refuse larger ones)
  std::atomic<int>* cache = caches[current_device()];
  if (cache[cluster].load(std::memory_order_relaxed) == 0) {
    int n = 0;
    if (configure_kernel<D, MT>()) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(cluster * 64);
      cfg.blockDim = dim3(Cfg<D, MT>::kThreads);
      cfg.dynamicSmemBytes = Cfg<D, MT>::kSmemBytes;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = cluster;
      at[0].val.clusterDim.y = 1;
      at[0].val.clusterDim.z = 1;
      cfg.attrs = at;
      cfg.numAttrs = 1;
      if (cudaOccupancyMaxActiveClusters(&n, tree_attn_kernel<D, MT>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        n = 0;
      }
    }
    cache[cluster].store(n > 0 ? n : -1, std::memory_order_relaxed);
  }
  const int have = cache[cluster].load(std::memory_order_relaxed);
  return have > 0 ? have : 0;
}

int max_active_clusters_for(int D, int mt, int cluster) {
  if (D == 128) return mt == 1 ? max_active_clusters<128, 1>(cluster) : max_active_clusters<128, 2>(cluster);
  return mt == 1 ? max_active_clusters<64, 1>(cluster) : max_active_clusters<64, 2>(cluster);
}

// Picks the query-tile grouping and the number of key slices with a cost model fitted to measurements, in
// units of one key tile of a one-query-tile CTA whose K/V comes out of L2 (about 1900 cycles):
//   key tile, one query tile per CTA   1 + 0.75 / g    g = CTAs that read the same K/V tile side by side
//                                                      (the first one fetches it from HBM, the others hit L2)
//   key tile, two query tiles per CTA  max(2.2, 1 + 0.75 / g)   two softmax chains share the tensor core,
//                                                      but the K/V tile is loaded once for both
//   fixed cost of a CTA                6 (no slices), 8 (slices merged inside a cluster), 10 (through the
//                                      workspace); 1.6 times that with two query tiles (two merge rounds)
// and the CTAs run in waves of what the device holds at once.
// Measured: a key tile costs a pair CTA 1800 cycles against 1475 for a CTA on its own (the hand-overs cross two SMs),
// so the planner never prefers the pair form; JET_FORCE_PAIR=1 selects it.
constexpr double kPairTile = 1.22;    // a pair CTA's key tile against a single CTA's
constexpr double kPairFixed = 1.0;    // what a pair adds per CTA (cluster barriers at set-up, end of pass, teardown)

Plan make_plan(int batch, int B, int Hq, int Hkv, int D, int max_seq_len) {
  const int G = Hq / Hkv;
  const int rows = B * G;
  const int tiles = (max_seq_len + kBN - 1) / kBN + (B + kBN - 1) / kBN;
  Plan best{};
  double best_cost = -1.0;
  // Test hooks (read once per process): JET_FORCE_MT = query tiles per CTA, JET_FORCE_SPLIT = "slices" or
  // "slices,g" (g = merge through the workspace); a forced choice the device cannot hold is ignored.
  static const int force_mt = [] { const char* e = getenv("JET_FORCE_MT"); return e ? atoi(e) : 0; }();
  static const int force_ns = [] { const char* e = getenv("JET_FORCE_SPLIT"); return e ? atoi(e) : 0; }();
  // ",g": exchange inside the launch (counters and a bounded spin); ",h": exchange finished by a second launch
  // JET_FORCE_PAIR: 1 = CTA pairs wherever the shape allows them, -1 = never
  static const int force_pair = [] { const char* e = getenv("JET_FORCE_PAIR"); return e ? atoi(e) : 0; }();
  static const int force_via = [] {
    const char* e = getenv("JET_FORCE_SPLIT");
    return (e && strstr(e, ",g")) ? 1 : ((e && strstr(e, ",h")) ? 2 : 0);
  }();
  for (int mt = 1; mt <= (rows > kBM ? 2 : 1); ++mt) {
    if (force_mt && mt != force_mt && !(force_mt == 2 && rows <= kBM)) continue;
    Plan pl;
    pl.mt = mt;
    pl.n_mgroups = (rows + mt * kBM - 1) / (mt * kBM);
    pl.units = batch * Hkv * pl.n_mgroups;
    const double shared = 1.0 + 0.75 / pl.n_mgroups;
    const double tile_cost = mt == 1 ? shared : (shared > 2.2 ? shared : 2.2);
    const double fixed_scale = mt == 1 ? 1.0 : 1.6;
    // CTA pairs: one 128-wide query tile per CTA, an even number of them per work item
    const bool pair_ok = D == 128 && mt == 1 && pl.n_mgroups % 2 == 0;
    auto consider = [&](int ns, int via_global, double waves, double fixed, double given_cost = -1.0, int pair = 0) {
      if (force_ns && (ns != force_ns || (ns > 1 && via_global != force_via))) return;
      if (force_pair && (force_pair > 0) != (pair != 0) && (pair || pair_ok)) return;
      const double cost = given_cost >= 0.0 ? given_cost
                                            : waves * (((tiles + ns - 1) / ns) * tile_cost * (pair ? kPairTile : 1.0) +
                                                       (fixed + (pair ? kPairFixed : 0.0)) * fixed_scale);
      if (best_cost < 0.0 || cost < best_cost) {
        best = pl;
        best.nsplit = ns;
        best.via_global = via_global;
        best.pair = pair;
        best_cost = cost;
      }
    };

    for (int ns = 1; ns <= kMaxSplit && ns <= tiles; ++ns) {
      // (a) the slices of a unit form a thread-block cluster and merge through distributed shared memory
      const int resident = max_active_clusters_for(D, mt, ns);
      if (resident > 0) consider(ns, 0, static_cast<double>((pl.units + resident - 1) / resident), ns == 1 ? 6.0 : 8.0);
      if (pair_ok && ns == 1) consider(1, 0, static_cast<double>((pl.units + sm_count() - 1) / sm_count()), 6.0, -1.0, 1);
      // (b) independent CTAs that merge through the workspace: all of them must be resident at once
      //     (a cluster has to fit into one GPC, which can leave a third of the SMs idle)
      //     -- either inside the launch (arrival counters, bounded spin), or with a second small launch that
      //     combines the blocks once the first has ended (nothing waits inside a kernel)
      if (ns > 1 && static_cast<long>(pl.units) * ns <= sm_count() &&
          static_cast<size_t>(pl.units) * mt * 2 * sizeof(int) <= kCounterBytes) {
        // measured (Qwen3-8B layer shape, prefix 4096 / 16384): with one query tile per KV head (few rows, many
        // slices) the two-launch form is 1-3 % faster, with more query tiles the single launch is (2.6 % at 64 nodes)
        const int via = force_via ? force_via : (pl.n_mgroups == 1 ? 2 : 1);
        if (via == 2 && mt == 1 && pl.n_mgroups == 1) {
          // One query tile per KV head: few work items, so the launch is a handful of tiles per CTA plus the
          // merge.  Fitted to a sweep of 6 .. 18 slices at prefixes 2048 .. 16384 (budgets 16 and 32): 0.6 us per
          // key tile of a CTA, 0.1 us per slice for the second launch, 0.25 us more per slice beyond 12 (in the
          // planner's unit of 0.8 us: 0.75, 0.125, 0.31).  9 - 11 slices win up to prefix 8192, 13 - 18 beyond.
          consider(ns, via, 1.0, 0.0, ((tiles + ns - 1) / ns) * 0.75 + 0.125 * ns + 0.31 * (ns > 12 ? ns - 12 : 0) + 9.7);
        } else {
          consider(ns, via, 1.0, 10.0);
          if (pair_ok) consider(ns, via, 1.0, 10.0, -1.0, 1);
        }
      }
    }
  }
  if (best_cost < 0.0) {        // the occupancy query failed: plain launch without slices
    best.mt = rows > kBM ? 2 : 1;
    best.n_mgroups = (rows + best.mt * kBM - 1) / (best.mt * kBM);
    best.units = batch * Hkv * best.n_mgroups;
    best.nsplit = 1;
    best.via_global = 0;
    best.pair = 0;
  }
  return best;
}

size_t workspace_need(const Plan& pl, int D) {
  if (!pl.via_global) return 256;
  return kCounterBytes + static_cast<size_t>(pl.units) * pl.nsplit * pl.mt * kBM * (D * 2 + 16);
}

template <int D, int MT, bool kPair = false>
jet_status launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& ttk,
                  const CUtensorMap& ttv, const CUtensorMap& tk64, const CUtensorMap& ttk64, const AttnParams& p,
                  const Plan& pl, cudaStream_t st) {
  using C = Cfg<D, MT, kPair>;
  if (!configure_kernel<D, MT, kPair>()) return JET_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(pl.n_mgroups * pl.nsplit, p.Hkv, p.batch);
  cfg.blockDim = dim3(C::kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attrs[2];
  int na = 0;
  attrs[na].id = cudaLaunchAttributeClusterDimension;
  attrs[na].val.clusterDim.x = kPair ? 2 : (pl.via_global ? 1 : pl.nsplit);
  attrs[na].val.clusterDim.y = 1;
  attrs[na].val.clusterDim.z = 1;
  ++na;
  // Programmatic dependent launch: this grid may be scheduled while the previous kernel of the stream
  // drains; the kernel touches no global memory before its griddepcontrol.wait.
  attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[na].val.programmaticStreamSerializationAllowed = 1;
  ++na;
  cfg.attrs = attrs;
  cfg.numAttrs = na;
  const bool sorted = p.batch > 1 && p.batch <= kMaxSorted;
  const cudaError_t err =
      sorted ? cudaLaunchKernelEx(&cfg, tree_attn_kernel<D, MT, true, kPair>, tq, tk, tv, ttk, ttv, tk64, ttk64, p)
             : cudaLaunchKernelEx(&cfg, tree_attn_kernel<D, MT, false, kPair>, tq, tk, tv, ttk, ttv, tk64, ttk64, p);
  if (err != cudaSuccess) {
#ifdef JET_TRACE
    fprintf(stderr, "attention launch failed: %s (grid %d x %d x %d, cluster %d, %d slices, merge form %d, D %d, MT %d)\n",
            cudaGetErrorString(err), pl.n_mgroups * pl.nsplit, p.Hkv, p.batch, pl.via_global ? 1 : pl.nsplit, pl.nsplit,
            pl.via_global, D, MT);
#endif
    cudaGetLastError();
    return JET_ERR_CUDA;
  }
  if (pl.via_global == 2) {
    MergeParams m;
    m.partials = p.partials;
    m.n_nodes = p.n_nodes;
    m.out = p.out;
    m.lse = p.lse;
    m.B = p.B; m.Hq = p.Hq; m.Hkv = p.Hkv; m.G = p.G; m.S = pl.nsplit; m.MT = MT; m.n_mgroups = pl.n_mgroups; m.npt = p.npt;
    m.magic_G = p.magic_G;
    constexpr int kRowsPerCta = 256 / (D / 8);
    launch_dependent(tree_attn_merge_kernel<D>, dim3((kBM / kRowsPerCta) * MT * pl.n_mgroups, p.Hkv, p.batch), dim3(256), st, m);
  }
  return launch_status();
}

}  // namespace
}  // namespace jet

#ifdef JET_TRACE
extern "C" JET_API void jet_debug_set_attn_trace(void* ptr) { jet::g_trace_ptr = static_cast<long long*>(ptr); }
extern "C" JET_API int jet_debug_max_clusters(int cluster) {
  using namespace jet;
  using C = Cfg<128, 1>;
  cudaFuncSetAttribute(tree_attn_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  cudaFuncSetAttribute(tree_attn_kernel<128, 1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cluster * 32);
  cfg.blockDim = dim3(C::kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = -1;
  if (cudaOccupancyMaxActiveClusters(&n, tree_attn_kernel<128, 1>, &cfg) != cudaSuccess) { cudaGetLastError(); return -1; }
  return n;
}
#endif

extern "C" size_t jet_tree_verify_attn_workspace_bytes(int batch, int B, int Hq, int Hkv, int D,
                                                       int max_seq_len) {
  if (batch < 1 || batch > 65535 || B < 1 || Hq < 1 || Hkv < 1 || Hkv > 65535 || Hq % Hkv != 0 || max_seq_len < 0 ||
      (D != 64 && D != 128))
    return 0;
  return jet::workspace_need(jet::make_plan(batch, B, Hq, Hkv, D, max_seq_len), D);
}

extern "C" int jet_tree_verify_attn_plan(int batch, int B, int Hq, int Hkv, int D, int max_seq_len, int32_t* plan) {
  if (!plan || batch < 1 || batch > 65535 || B < 1 || Hq < 1 || Hkv < 1 || Hkv > 65535 || Hq % Hkv != 0 || max_seq_len < 0 ||
      (D != 64 && D != 128))
    return 0;
  const jet::Plan pl = jet::make_plan(batch, B, Hq, Hkv, D, max_seq_len);
  plan[0] = pl.mt;
  plan[1] = pl.n_mgroups;
  plan[2] = pl.nsplit;
  plan[3] = pl.nsplit > 1 ? (pl.via_global == 0 ? 1 : pl.via_global + 1) : 0;     // 0 none, 1 cluster, 2 workspace in one launch, 3 second launch
  plan[4] = pl.pair;
  return 1;
}

extern "C" int jet_tree_verify_attn_launches(int batch, int B, int Hq, int Hkv, int D, int max_seq_len) {
  if (batch < 1 || batch > 65535 || B < 1 || Hq < 1 || Hkv < 1 || Hkv > 65535 || Hq % Hkv != 0 || max_seq_len < 0 ||
      (D != 64 && D != 128))
    return 0;
  return jet::make_plan(batch, B, Hq, Hkv, D, max_seq_len).via_global == 2 ? 2 : 1;
}

namespace jet {
namespace {

// Checks, tensor maps and launch shared by the two entry points.  tail: the tree's K/V rows are in the cache
// behind the prefix (tree_k / tree_v unused), and max_seq_len bounds seq_len + n_nodes.
jet_status attn_call(const void* q, const void* k_cache, const void* v_cache, const int32_t* page_table,
                     int max_pages_per_seq, int page_size, int64_t num_pages, const int32_t* seq_len,
                     int max_seq_len, const void* tree_k, const void* tree_v, bool tail, const uint32_t* anc_mask,
                     const int32_t* n_nodes, int batch, int B, int Hq, int Hkv, int D, int64_t kv_batch_stride,
                     float softmax_scale, void* out, float* lse, int32_t* device_status, void* workspace,
                     size_t workspace_bytes, void* stream, uint32_t flags) {
  if (!q || !seq_len || !anc_mask || !n_nodes || !out) return JET_ERR_INVALID_ARG;
  if (flags & ~static_cast<uint32_t>(JET_ATTN_STABLE_PREFIX)) return JET_ERR_INVALID_ARG;
  if (tail ? (!k_cache || !v_cache || max_seq_len < 1) : (!tree_k || !tree_v)) return JET_ERR_INVALID_ARG;
  if (batch < 1 || batch > 65535 || B < 1 || B > JET_MAX_NODES || Hq < 1 || Hkv < 1 || Hkv > 65535 || Hq % Hkv != 0 ||
      max_seq_len < 0)        // (sequences and KV heads are grid dimensions)
    return JET_ERR_INVALID_ARG;
  if (max_seq_len > 0 && (!k_cache || !v_cache)) return JET_ERR_INVALID_ARG;
  const int G = Hq / Hkv;
  // the running reference maximum is kept in raw score units, which needs a positive, finite scale
  if (!(softmax_scale > 0.0f) || !(softmax_scale < INFINITY)) return JET_ERR_INVALID_ARG;
  if (D != 64 && D != 128) return JET_ERR_UNSUPPORTED;
  if (G > 16 || (G & (G - 1)) != 0) return JET_ERR_UNSUPPORTED;
  const bool paged = page_table != nullptr;
  if (paged && (page_size != 16 || max_pages_per_seq < 1 || num_pages < 1)) return JET_ERR_UNSUPPORTED;
  if (paged && static_cast<int64_t>(max_pages_per_seq) * 16 < max_seq_len) return JET_ERR_INVALID_ARG;
  if (!paged && batch > 1 && (kv_batch_stride < static_cast<int64_t>(max_seq_len) * Hkv * D || kv_batch_stride % 8 != 0))
    return JET_ERR_INVALID_ARG;
  if (!aligned(q, 16) || (!tail && (!aligned(tree_k, 16) || !aligned(tree_v, 16))) || !aligned(out, 16) ||
      (k_cache && !aligned(k_cache, 16)) || (v_cache && !aligned(v_cache, 16)))
    return JET_ERR_INVALID_ARG;
  if (static_cast<int64_t>(batch) * B >= (1ll << 31)) return JET_ERR_INVALID_ARG;
  const Plan pl = make_plan(batch, B, Hq, Hkv, D, max_seq_len);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < workspace_need(pl, D)) return JET_ERR_WORKSPACE;

  // ---- tensor maps (bf16, 128-byte swizzle, 64-element inner box)
  CUtensorMap tq = {}, tk = {}, tv = {}, ttk = {}, ttv = {}, tk64 = {}, ttk64 = {};     // (maps a call does not use stay zeroed; the last two: K with boxes of 64 rows, for CTA pairs)
  const uint64_t eb = 2;
  {
    const uint64_t dims[4] = {static_cast<uint64_t>(D), static_cast<uint64_t>(G), static_cast<uint64_t>(Hkv),
                              static_cast<uint64_t>(batch) * B};
    const uint64_t str[3] = {D * eb, static_cast<uint64_t>(G) * D * eb, static_cast<uint64_t>(Hq) * D * eb};
    const uint32_t box[4] = {64, static_cast<uint32_t>(G), 1, static_cast<uint32_t>(kBM / G)};
    if (!make_map(&tq, q, 4, dims, str, box)) return JET_ERR_CUDA;
  }
  if (!tail) {
    const uint64_t dims[4] = {static_cast<uint64_t>(D), static_cast<uint64_t>(Hkv), static_cast<uint64_t>(B),
                              static_cast<uint64_t>(batch)};
    const uint64_t str[3] = {D * eb, static_cast<uint64_t>(Hkv) * D * eb, static_cast<uint64_t>(B) * Hkv * D * eb};
    const uint32_t box[4] = {64, 1, kBN, 1};
    const uint32_t box64[4] = {64, 1, 64, 1};
    if (!make_map(&ttk, tree_k, 4, dims, str, box) || !make_map(&ttv, tree_v, 4, dims, str, box))
      return JET_ERR_CUDA;
    if (pl.pair && !make_map(&ttk64, tree_k, 4, dims, str, box64)) return JET_ERR_CUDA;
  }
  if (max_seq_len == 0) {
    tk = ttk;   // never dereferenced: there are no prefix tiles
    tv = ttv;
    tk64 = ttk64;
  } else if (paged) {
    const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(Hkv),
                              static_cast<uint64_t>(num_pages) * 16};
    const uint64_t str[2] = {D * eb, static_cast<uint64_t>(Hkv) * D * eb};
    const uint32_t box[3] = {64, 1, 16};
    if (!make_map(&tk, k_cache, 3, dims, str, box) || !make_map(&tv, v_cache, 3, dims, str, box))
      return JET_ERR_CUDA;
  } else {
    const uint64_t bstride = batch > 1 ? static_cast<uint64_t>(kv_batch_stride)
                                       : static_cast<uint64_t>(max_seq_len) * Hkv * D;
    const uint64_t dims[4] = {static_cast<uint64_t>(D), static_cast<uint64_t>(Hkv),
                              static_cast<uint64_t>(max_seq_len), static_cast<uint64_t>(batch)};
    const uint64_t str[3] = {D * eb, static_cast<uint64_t>(Hkv) * D * eb, bstride * eb};
    const uint32_t box[4] = {64, 1, kBN, 1};
    const uint32_t box64[4] = {64, 1, 64, 1};
    if (!make_map(&tk, k_cache, 4, dims, str, box) || !make_map(&tv, v_cache, 4, dims, str, box))
      return JET_ERR_CUDA;
    if (pl.pair && !make_map(&tk64, k_cache, 4, dims, str, box64)) return JET_ERR_CUDA;
  }
  if (!pl.pair || paged) tk64 = tk;        // (unused: a paged tile is fetched page by page)
  if (!pl.pair || tail) ttk64 = tail ? tk64 : ttk;

  AttnParams p;
  p.page_table = page_table;
  p.seq_len = seq_len;
  p.n_nodes = n_nodes;
  p.anc_mask = anc_mask;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  p.status = device_status;
  p.max_pages = max_pages_per_seq;
  p.paged = paged ? 1 : 0;
  p.tail = tail ? 1 : 0;
  p.batch = batch; p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.words = (B + 31) / 32;
  p.nsplit = pl.nsplit;
  p.n_mgroups = pl.n_mgroups;
  p.n_units = pl.units;
  p.rows_per = (kBM + pl.nsplit - 1) / pl.nsplit;
  p.npt = kBM / G;
  p.magic_S = udiv_magic(static_cast<uint32_t>(pl.nsplit));
  p.magic_G = udiv_magic(static_cast<uint32_t>(G));
  // (measured: a gain of 3-9 % with one query tile per KV head, none to a small loss with two or more)
  p.len_hint = (!pl.pair && !paged && !tail && batch == 1 && pl.n_mgroups == 1 && max_seq_len > 0 && max_seq_len < (1 << 26)) ? max_seq_len : 0;
  p.stable = (flags & JET_ATTN_STABLE_PREFIX) ? 1 : 0;
  // Test hook (read once per process): JET_TEST_POLL_LIMIT shortens the bounded spin of the workspace merge so
  // that a test can make it run out within milliseconds.
  static const uint32_t poll_limit = [] {
    const char* e = getenv("JET_TEST_POLL_LIMIT");
    const long v = e ? atol(e) : 0;
    return v > 0 ? static_cast<uint32_t>(v) : (1u << 22);
  }();
  p.poll_limit = poll_limit;
  p.via_global = pl.via_global;
  p.counters = static_cast<int*>(workspace);
  p.partials = static_cast<uint8_t*>(workspace) + kCounterBytes;
  p.scale_log2 = softmax_scale * 1.4426950408889634f;
#ifdef JET_TRACE
  p.trace = g_trace_ptr;
#endif

  if (tail) {       // no separate tree tiles: the maps are never used
    ttk = tk;
    ttv = tv;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (pl.pair) return launch<128, 1, true>(tq, tk, tv, ttk, ttv, tk64, ttk64, p, pl, st);
  if (D == 128) return pl.mt == 1 ? launch<128, 1>(tq, tk, tv, ttk, ttv, tk64, ttk64, p, pl, st)
                                  : launch<128, 2>(tq, tk, tv, ttk, ttv, tk64, ttk64, p, pl, st);
  return pl.mt == 1 ? launch<64, 1>(tq, tk, tv, ttk, ttv, tk64, ttk64, p, pl, st)
                    : launch<64, 2>(tq, tk, tv, ttk, ttv, tk64, ttk64, p, pl, st);
}

}  // namespace
}  // namespace jet

extern "C" jet_status jet_tree_verify_attn(const void* q, const void* k_cache, const void* v_cache,
                                           const int32_t* page_table, int max_pages_per_seq, int page_size,
                                           int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                           const void* tree_k, const void* tree_v, const uint32_t* anc_mask,
                                           const int32_t* n_nodes, int batch, int B, int Hq, int Hkv, int D,
                                           int64_t kv_batch_stride, float softmax_scale, void* out, float* lse,
                                           int32_t* device_status, void* workspace, size_t workspace_bytes,
                                           void* stream) {
  return jet::attn_call(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len, max_seq_len,
                        tree_k, tree_v, false, anc_mask, n_nodes, batch, B, Hq, Hkv, D, kv_batch_stride, softmax_scale,
                        out, lse, device_status, workspace, workspace_bytes, stream, 0u);
}

extern "C" jet_status jet_tree_verify_attn_ex(const void* q, const void* k_cache, const void* v_cache,
                                              const int32_t* page_table, int max_pages_per_seq, int page_size,
                                              int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                              const void* tree_k, const void* tree_v, const uint32_t* anc_mask,
                                              const int32_t* n_nodes, int batch, int B, int Hq, int Hkv, int D,
                                              int64_t kv_batch_stride, float softmax_scale, void* out, float* lse,
                                              int32_t* device_status, void* workspace, size_t workspace_bytes,
                                              void* stream, uint32_t flags) {
  return jet::attn_call(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len, max_seq_len,
                        tree_k, tree_v, false, anc_mask, n_nodes, batch, B, Hq, Hkv, D, kv_batch_stride, softmax_scale,
                        out, lse, device_status, workspace, workspace_bytes, stream, flags);
}

extern "C" jet_status jet_tree_verify_attn_tail(const void* q, const void* k_cache, const void* v_cache,
                                                const int32_t* page_table, int max_pages_per_seq, int page_size,
                                                int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                                const uint32_t* anc_mask, const int32_t* n_nodes, int batch, int B,
                                                int Hq, int Hkv, int D, int64_t kv_batch_stride,
                                                float softmax_scale, void* out, float* lse, int32_t* device_status,
                                                void* workspace, size_t workspace_bytes, void* stream) {
  return jet::attn_call(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len, max_seq_len,
                        nullptr, nullptr, true, anc_mask, n_nodes, batch, B, Hq, Hkv, D, kv_batch_stride, softmax_scale,
                        out, lse, device_status, workspace, workspace_bytes, stream, 0u);
}

extern "C" jet_status jet_tree_verify_attn_tail_ex(const void* q, const void* k_cache, const void* v_cache,
                                                   const int32_t* page_table, int max_pages_per_seq, int page_size,
                                                   int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                                   const uint32_t* anc_mask, const int32_t* n_nodes, int batch,
                                                   int B, int Hq, int Hkv, int D, int64_t kv_batch_stride,
                                                   float softmax_scale, void* out, float* lse,
                                                   int32_t* device_status, void* workspace, size_t workspace_bytes,
                                                   void* stream, uint32_t flags) {
  return jet::attn_call(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len, max_seq_len,
                        nullptr, nullptr, true, anc_mask, n_nodes, batch, B, Hq, Hkv, D, kv_batch_stride, softmax_scale,
                        out, lse, device_status, workspace, workspace_bytes, stream, flags);
}
