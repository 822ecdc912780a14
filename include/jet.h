/*
 * jet.h -- C ABI of the tree-verification hot path of parallel-tree-drafting
 * speculative decoding (sm_100a).
 *
 * Four operations, in the order one verification step runs them:
 *
 *   jet_tree_build        per-depth draft log-probs -> budgeted candidate tree
 *   jet_tree_verify_attn  attention of all tree nodes over prefix KV + tree KV
 *                         under the ancestor mask (once per layer)
 *   jet_tree_accept       greedy acceptance of the deepest matching path
 *   jet_kv_compact        commit of the accepted path's K/V into the cache
 *
 * and their variants:
 *
 *   jet_tree_build_scored      entropy / hybrid expansion scores, per-sequence budgets
 *   jet_tree_build_logits      the same fed with raw draft logits (log-softmax on the fly)
 *   jet_tree_verify_attn_tail  the tree's K/V rows live in the cache behind the prefix
 *   jet_tree_verify_attn_ex, jet_tree_verify_attn_tail_ex   the same with a flags word
 *   jet_kv_compact_tail        in-place commit for that layout
 *   jet_tree_accept_static     greedy acceptance on scratch built into the library
 *   jet_tree_accept_hidden     greedy acceptance from the final hidden states (LM head inside, arg-max only)
 *   jet_tree_accept_sample     non-greedy (min(1, p/q)) acceptance with a correction draw
 *
 * Conventions shared by every call
 *   - Every pointer is a DEVICE pointer owned by the caller unless a comment
 *     says "host".  The library allocates nothing and frees nothing.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *     return; no call synchronises the host with the device.
 *   - `workspace` is caller-provided device scratch of at least the size the
 *     matching *_workspace_bytes() query returns, 256-byte aligned.  Its
 *     contents need not be initialised and are undefined afterwards.  Two calls
 *     that may overlap on the device must not share a workspace.
 *   - Argument errors are detected on the host before anything is launched and
 *     reported as a negative jet_status; outputs are then untouched.
 *   - B is the node budget INCLUDING the root (1 <= B <= JET_MAX_NODES).
 *     Node rows v >= n_nodes[b] are padding: parent = depth = token = -1, mask
 *     row zero, attention output row zero; acceptance ignores them.
 *   - Ancestor mask: row v has mask_words = ceil(B/32) uint32 words; bit
 *     (u mod 32) of word (u div 32) is set iff u is v or an ancestor of v.
 *   - All element offsets are 64-bit.
 */
#ifndef JET_H_
#define JET_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define JET_API __attribute__((visibility("default")))
#else
#define JET_API
#endif

typedef int32_t jet_status;

enum {
  JET_OK = 0,
  JET_ERR_INVALID_ARG = -1, /* null pointer, size out of range, bad alignment */
  JET_ERR_UNSUPPORTED = -2, /* shape outside the compiled instantiations       */
  JET_ERR_WORKSPACE = -3,   /* workspace null, misaligned or too small         */
  JET_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed             */
  JET_ERR_TIMEOUT = -5      /* a bounded device-side wait gave up              */
};

#define JET_MAX_NODES 512 /* largest node budget B                      */
#define JET_MAX_WIDTH 32  /* largest branching width W                  */
#define JET_MAX_DEPTH 64  /* largest draft depth N                      */

/* Human-readable name of a status code (host pointer to a static string). */
JET_API const char* jet_status_string(jet_status s);

/* ---------------------------------------------------------------------------
 * jet_tree_build -- Algorithm 1 (Parallel Tree Drafting) with the accumulated
 * draft log-probability score of Section 3.3, preceded by the per-depth top-W
 * extraction that Section 3.3 / Appendix E describe.
 *
 * For each sequence b: candidates of depth d are the W largest entries of
 * logp[b,d,:] (ties -> lowest token id, -0.0 == +0.0).  Node 0 is the root
 * (token root_token[b], score 0, depth 0).  Repeatedly the pending node with
 * the largest score (ties -> lowest node index) is taken; if its depth is N it
 * is dropped, otherwise its min(W,V) children are appended in rank order with
 * score = fl32(score[parent] + logp[b, depth[parent], token]) until the tree
 * holds B nodes or no node is pending.  Nodes are numbered in creation order,
 * so parent[v] < v.
 *
 *   logp         fp32 [batch, N, V]; element (b,d,t) at
 *                b*logp_batch_stride + d*logp_depth_stride + t.  No NaN.
 *   root_token   i32 [batch]
 *   parent, depth, token   i32 [batch, B] out
 *   score        fp32 [batch, B] out, may be NULL
 *   anc_mask     u32 [batch, B, ceil(B/32)] out
 *   n_nodes      i32 [batch] out
 * Limits: 1 <= N <= JET_MAX_DEPTH, 1 <= W <= JET_MAX_WIDTH, V >= 1.
 */
JET_API size_t jet_tree_build_workspace_bytes(int batch, int N, int V, int W);

JET_API jet_status jet_tree_build(const float* logp, int64_t logp_batch_stride, int64_t logp_depth_stride,
                          const int32_t* root_token, int batch, int N, int V, int W, int B,
                          int32_t* parent, int32_t* depth, int32_t* token, float* score,
                          uint32_t* anc_mask, int32_t* n_nodes, void* workspace,
                          size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * jet_tree_build_scored -- jet_tree_build with the alternative expansion scores
 * of Appendix C (tree-drafting ablation).  Everything is as for jet_tree_build,
 * except the priority by which the pending node is taken:
 *   JET_SCORE_ACCUM_LOGP  the accumulated log-probability (= jet_tree_build);
 *   JET_SCORE_ENTROPY     H of the node's depth alone;
 *   JET_SCORE_HYBRID      fl32(score + fl32(alpha * H of the node's depth)).
 * H of depth d >= 1 is the entropy of the distribution the depth-d tokens were
 * drawn from, H = -sum_t exp(l_t) * l_t over logp[b, d-1, :], summed in fp64
 * (entries of -inf contribute 0) and rounded once to fp32; the root's H is 0.
 * (The appendix gives the formula "sum log r + alpha * H" only; taken here: the
 * entropy of the node's own depth, so that a large alpha gives the entropy-only
 * rule as the appendix states.)  Ties -> lowest node index; `score` is the
 * accumulated log-probability in every mode.
 *
 *   node_budget   i32 [batch] or NULL: sequence b's own budget min(B, max(1,
 *                 node_budget[b])) (load-dependent budgets, which Section 5 leaves
 *                 to future work); every array keeps its [batch, B] shape, rows
 *                 past n_nodes[b] are padding as usual
 *   score_mode    one of JET_SCORE_*
 *   alpha         finite; used by JET_SCORE_HYBRID only
 *   depth_entropy fp32 [batch, N] out, may be NULL: H of logp[b, d, :]
 *                 (not written with JET_SCORE_ACCUM_LOGP)
 * Workspace: jet_tree_build_scored_workspace_bytes (larger than jet_tree_build's).
 */
#define JET_SCORE_ACCUM_LOGP 0
#define JET_SCORE_ENTROPY 1
#define JET_SCORE_HYBRID 2

JET_API size_t jet_tree_build_scored_workspace_bytes(int batch, int N, int V, int W);

JET_API jet_status jet_tree_build_scored(const float* logp, int64_t logp_batch_stride, int64_t logp_depth_stride,
                                 const int32_t* root_token, int batch, int N, int V, int W, int B,
                                 const int32_t* node_budget, int score_mode, float alpha, int32_t* parent,
                                 int32_t* depth,
                                 int32_t* token, float* score, uint32_t* anc_mask, int32_t* n_nodes,
                                 float* depth_entropy, void* workspace, size_t workspace_bytes,
                                 void* stream);

/* ---------------------------------------------------------------------------
 * jet_tree_build_logits -- jet_tree_build_scored fed with RAW draft logits z
 * (Section 3.3: the draft head's one forward gives logits for N depths; the
 * tree is scored with their log-probabilities).  Computes exactly what a
 * log-softmax followed by jet_tree_build_scored computes, without the [N,V]
 * log-probabilities ever existing in memory:
 *   lse[b,d]  = log sum_t exp(z[b,d,t]), formed in fp64 as max + log(sum exp(z - max));
 *   logp[b,d,t] = fl32(double(z[b,d,t]) - lse[b,d])   (one rounding);
 * candidates are ranked by these fp32 log-probabilities (two logits that round
 * to the same log-probability tie -> lowest token id), entropies are taken of
 * them, scores add them.  The fp64 sums are formed in a fixed order (per 4096-
 * entry slice, then over the slices), so results do not change from run to run;
 * against another summation order lse can differ in its last bits, which moves
 * a log-probability only if it sits within ~1e-15 (relative) of a rounding
 * boundary.
 *
 *   logits       fp32 [batch, N, V], strides as for logp.  No NaN, no +inf; a
 *                row must hold at least one finite entry (-inf = probability 0)
 *   depth_lse    fp32 [batch, N] out, may be NULL: fl32(lse[b,d])
 *   every other argument as for jet_tree_build_scored
 * Workspace: jet_tree_build_logits_workspace_bytes.
 */
JET_API size_t jet_tree_build_logits_workspace_bytes(int batch, int N, int V, int W);

JET_API jet_status jet_tree_build_logits(const float* logits, int64_t logits_batch_stride,
                                 int64_t logits_depth_stride, const int32_t* root_token, int batch, int N,
                                 int V, int W, int B, const int32_t* node_budget, int score_mode, float alpha,
                                 int32_t* parent, int32_t* depth, int32_t* token, float* score,
                                 uint32_t* anc_mask, int32_t* n_nodes, float* depth_entropy, float* depth_lse,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * jet_tree_verify_attn -- the masked tree attention of Section 3.2 (tree-causal
 * mask: a node sees the whole prefix, its ancestors and itself), as used by the
 * one-pass tree verification of Section 3.3 / Appendix E.  One call = one layer.
 *
 * For sequence b, node v < n_nodes[b], query head h (KV head g = h / (Hq/Hkv)):
 *   out[b,v,h,:] = softmax_j( softmax_scale * <q[b,v,h,:], K_j> ) . V_j
 * over the seq_len[b] prefix keys (all visible) and the tree keys u whose bit
 * is set in anc_mask[b,v].  bf16 operands, fp32 accumulation, bf16 output.
 *
 *   q            bf16 [batch, B, Hq, D]
 *   k_cache, v_cache
 *                bf16.  page_table == NULL: contiguous, position j of sequence
 *                b at element ((b*kv_batch_stride) + j*Hkv*D + g*D).
 *                page_table != NULL: paged [num_pages, page_size, Hkv, D];
 *                position j of sequence b is row (j mod page_size) of page
 *                page_table[b*max_pages_per_seq + j / page_size].
 *   num_pages    pages in the pool (paged) -- bounds the tensor map; ignored
 *                when contiguous.
 *   max_seq_len  host value, >= every seq_len[b]; sizes the grid and, when
 *                contiguous, bounds the rows per sequence.
 *   softmax_scale  positive and finite (1/sqrt(D) in the paper), else JET_ERR_INVALID_ARG
 *   seq_len      i32 [batch] prefix lengths (0 allowed)
 *   tree_k, tree_v  bf16 [batch, B, Hkv, D]
 *   out          bf16 [batch, B, Hq, D]
 *   lse          fp32 [batch, Hq, B] natural-log sum of exp of the visible
 *                scaled scores; may be NULL.  Padding rows get -inf.
 *   device_status  i32[1], may be NULL: set to JET_ERR_TIMEOUT if a bounded
 *                wait inside the kernel expired (outputs are then undefined).
 * Limits: D in {64,128}; Hq % Hkv == 0 and Hq/Hkv a power of two <= 16;
 * page_size == 16 when paged; all base pointers 16-byte aligned; batch and Hkv
 * at most 65535 (they are grid dimensions).  max_seq_len is a bound, but a call
 * with one sequence whose seq_len equals it exactly starts a little faster (the
 * first key tiles are prefetched on that guess).
 * Workspace: unlike the other calls, the first 4096 bytes of this workspace hold
 * counters that must be ZERO when the call starts.  Zero them once after
 * allocating the workspace; every call that completes leaves them zero again.
 * (A call that reported JET_ERR_TIMEOUT may leave them dirty: zero them again.
 * Counters that are not zero on entry are the caller's error: the key slices of
 * a work item then never see each other arrive, every CTA gives up after its
 * bounded wait, device_status reads JET_ERR_TIMEOUT and the outputs are
 * undefined; nothing faults and the next call on a zeroed workspace is correct.)
 * When a sequence has fewer work items than the GPU has SMs, its key range is cut
 * into slices that run as separate CTAs and hand each other their partial rows
 * through this workspace inside the one launch.  That exchange assumes that all
 * CTAs of the launch are resident at once: the plan is sized from the device's SM
 * count, so give the call the whole GPU (no other kernel holding SMs at the same
 * time through another stream, MPS or a green context).  If some CTAs cannot
 * start until others finish, the waiting ones give up after about a second with
 * JET_ERR_TIMEOUT instead of hanging.
 * (For shapes with few query rows per KV head -- one 128-row query tile, e.g.
 * up to 32 nodes at 4 query heads per KV head -- the slices only WRITE their rows
 * in the first launch and a second, small launch combines them: then nothing
 * waits inside a kernel, the counters are unused and the residency assumption
 * falls away; jet_tree_verify_attn_launches tells which form a shape gets.
 * JET_FORCE_SPLIT="<slices>,g" / ",h" selects the one- / two-launch form.)
 * Stream capture: the first call for a shape family on a device configures the
 * kernel (shared-memory size, cluster attribute) and asks the driver how many
 * clusters fit; make it outside any stream capture (one warm-up call per head
 * size and query-tile grouping is enough), later calls can be captured.
 * Test hooks, read from the environment once per process and meant for the
 * test-suite only: JET_FORCE_MT / JET_FORCE_SPLIT force a launch plan (query
 * tiles per CTA; key slices, with ",g" / ",h" through the workspace in one / two launches),
 * JET_TEST_POLL_LIMIT shortens the bounded wait of the workspace exchange,
 * JET_FORCE_PAIR=1 runs pairs of consecutive query tiles of a work item as CTA
 * pairs that share every K/V tile (D = 128, one query tile per CTA, an even
 * number of query tiles per KV head; built and kept for measurement: slower than
 * the default form, which the planner therefore always prefers).
 */
JET_API size_t jet_tree_verify_attn_workspace_bytes(int batch, int B, int Hq, int Hkv, int D,
                                            int max_seq_len);

/* Kernel launches one attention call of this shape enqueues: 1, or 2 when the key range of a work item is cut
 * into slices whose partial rows a second, small kernel combines (0 for an invalid shape).  For callers that
 * count launches (CUDA-graph sizing, launch statistics); same arguments as the workspace query.
 */
JET_API int jet_tree_verify_attn_launches(int batch, int B, int Hq, int Hkv, int D, int max_seq_len);

/* The launch plan of one attention call of this shape on the calling thread's current device, for tests and for
 * reading timings: plan (HOST pointer, 5 entries) receives
 *   [0] query tiles of 128 rows per CTA (1 or 2)         [1] groups of such tiles per (sequence, KV head)
 *   [2] key slices per work item                         [3] how the slices are combined: 0 = no slices, 1 = inside
 *       a thread-block cluster, 2 = through the workspace in the one launch, 3 = by a second launch
 *   [4] 1 if consecutive query tiles run as CTA pairs (tcgen05 cta_group::2; only with JET_FORCE_PAIR=1).
 * Returns 1, or 0 for an invalid shape.  Same arguments as the workspace query.
 */
JET_API int jet_tree_verify_attn_plan(int batch, int B, int Hq, int Hkv, int D, int max_seq_len, int32_t* plan);

JET_API jet_status jet_tree_verify_attn(const void* q, const void* k_cache, const void* v_cache,
                                const int32_t* page_table, int max_pages_per_seq, int page_size,
                                int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                const void* tree_k, const void* tree_v, const uint32_t* anc_mask,
                                const int32_t* n_nodes, int batch, int B, int Hq, int Hkv, int D,
                                int64_t kv_batch_stride, float softmax_scale, void* out, float* lse,
                                int32_t* device_status, void* workspace, size_t workspace_bytes,
                                void* stream);

/* jet_tree_verify_attn_tail -- the same attention for a cache that already holds
 * the tree's K/V rows behind the prefix (the serving layout of Appendix E: the
 * tree lives in the tail of the paged cache): node v of sequence b is the cache
 * row at position seq_len[b] + v (contiguous or through the page table), there are
 * no tree_k / tree_v buffers.  The key tiles then run over positions
 * 0 .. seq_len[b] + n_nodes[b] - 1 without a break between prefix and tree.
 * max_seq_len bounds seq_len[b] + n_nodes[b] (and is the row extent of a
 * contiguous cache); rows of padding nodes may hold anything.  Everything else as
 * for jet_tree_verify_attn; same workspace query.
 */
JET_API jet_status jet_tree_verify_attn_tail(const void* q, const void* k_cache, const void* v_cache,
                                     const int32_t* page_table, int max_pages_per_seq, int page_size,
                                     int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                     const uint32_t* anc_mask, const int32_t* n_nodes, int batch, int B,
                                     int Hq, int Hkv, int D, int64_t kv_batch_stride, float softmax_scale,
                                     void* out, float* lse, int32_t* device_status, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* jet_tree_verify_attn_ex / jet_tree_verify_attn_tail_ex -- the two attention calls
 * with a `flags` word (0 = exactly the plain calls).  The operation is that of
 * Section 3.2 / Appendix E as above; the flag only tells the kernel what it may
 * read EARLY.
 *
 * The kernel is launched so that it may begin while the kernel before it in the
 * stream is still finishing (programmatic dependent launch); normally it touches
 * no global memory until that kernel has completed.  Within a decoding step most
 * of its inputs are much older than that: the cached prefix was committed by
 * earlier steps, lengths and page table were set when the step began.
 *
 *   JET_ATTN_STABLE_PREFIX   the caller promises that seq_len, n_nodes, page_table
 *       and every cache row at a position below seq_len[b] were written by work
 *       that had finished before the kernel DIRECTLY PRECEDING this call in the
 *       stream could let its successor start (for the kernels of this library,
 *       which signal only after their own dependency wait, and for ordinary
 *       launches: "not written by the directly preceding launch, nor by
 *       anything running concurrently on another stream").  The kernel then
 *       reads the lengths and streams the prefix K/V tiles into shared memory
 *       before its dependency wait, i.e. under the preceding kernel's tail.
 *       q, tree_k / tree_v (tail layout: the rows at and behind seq_len[b]),
 *       anc_mask and every output are still read / written only behind the wait.
 *       A broken promise gives undefined attention outputs (stale reads), no
 *       fault.  In a layer stack: set it for every layer but the first when the
 *       tree (n_nodes) was built by the launch right before the first layer.
 * Any other bit: JET_ERR_INVALID_ARG.
 */
#define JET_ATTN_STABLE_PREFIX 1u

JET_API jet_status jet_tree_verify_attn_ex(const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* page_table, int max_pages_per_seq, int page_size,
                                   int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                   const void* tree_k, const void* tree_v, const uint32_t* anc_mask,
                                   const int32_t* n_nodes, int batch, int B, int Hq, int Hkv, int D,
                                   int64_t kv_batch_stride, float softmax_scale, void* out, float* lse,
                                   int32_t* device_status, void* workspace, size_t workspace_bytes,
                                   void* stream, uint32_t flags);

JET_API jet_status jet_tree_verify_attn_tail_ex(const void* q, const void* k_cache, const void* v_cache,
                                        const int32_t* page_table, int max_pages_per_seq, int page_size,
                                        int64_t num_pages, const int32_t* seq_len, int max_seq_len,
                                        const uint32_t* anc_mask, const int32_t* n_nodes, int batch, int B,
                                        int Hq, int Hkv, int D, int64_t kv_batch_stride, float softmax_scale,
                                        void* out, float* lse, int32_t* device_status, void* workspace,
                                        size_t workspace_bytes, void* stream, uint32_t flags);

/* ---------------------------------------------------------------------------
 * jet_tree_accept -- greedy acceptance (Section 3.3, Appendix E): a node is
 * accepted iff its token equals the target's arg-max prediction at its parent;
 * the deepest fully accepted root-to-node path is selected and the target's
 * prediction at its last node is the correction token.
 *
 *   logits       fp32, row (b*B + v) at logits + (b*B+v)*logits_row_stride,
 *                V entries.  Arg-max ties -> lowest index.  No NaN.
 *   token, parent, depth   i32 [batch, B]  (from jet_tree_build)
 *   anc_mask, n_nodes      as produced by jet_tree_build
 *                The tree arrays are not validated (they live in device memory).
 *                Arrays that do not describe a tree give a meaningless result,
 *                but never a store outside the outputs: n_nodes is clipped to B,
 *                a depth outside 0 .. N is clamped / its node left out of path
 *                and out_tokens, a parent outside the tree never matches.  The
 *                same holds for the _static, _hidden and _sample forms.
 *   tgt_argmax   i32 [batch, B] out (-1 on padding rows)
 *   accept_len   i32 [batch] out: a = number of accepted draft nodes (root not
 *                counted); end node v* = deepest accepted node, ties -> lowest
 *                index
 *   path         i32 [batch, N+1] out: node ids root .. v*, then -1
 *   out_tokens   i32 [batch, N+1] out: the a accepted tokens, then the
 *                correction token tgt_argmax[v*], then -1
 */
JET_API size_t jet_tree_accept_workspace_bytes(int batch, int B, int V);

JET_API jet_status jet_tree_accept(const float* logits, int64_t logits_row_stride, const int32_t* token,
                           const int32_t* parent, const int32_t* depth, const uint32_t* anc_mask,
                           const int32_t* n_nodes, int batch, int B, int V, int N,
                           int32_t* tgt_argmax, int32_t* accept_len, int32_t* path,
                           int32_t* out_tokens, void* workspace, size_t workspace_bytes,
                           void* stream);

/* ---------------------------------------------------------------------------
 * jet_tree_accept_hidden -- greedy acceptance (Section 3.3, Appendix E: "the target
 * model's greedy prediction" at every node) straight from the target's FINAL HIDDEN
 * STATES: the LM head is applied inside the call and only the arg-max of every row
 * is kept, so the [batch*B, V] logits are neither written nor read.
 *
 *   logit[r, t] = sum_k hidden[r, k] * lm_head_weight[t, k]   bf16 operands, fp32
 *                 accumulation (tensor cores, accumulation order unspecified);
 *   tgt_argmax[r] = arg max_t logit[r, t], ties -> lowest t, -0.0 == +0.0;
 * then exactly jet_tree_accept's path selection.  Because the sums are formed in
 * fp32 in an unspecified order, two tokens whose exact logits differ by less than
 * the rounding of a K-term fp32 sum (about K * 2^-24 * sum_k |hidden * weight|) may
 * come out in either order; everything else matches an exact evaluation.
 *
 *   hidden          bf16 [batch*B, d], rows contiguous (row r = sequence r / B, node r % B);
 *                   rows of padding nodes may hold anything
 *   lm_head_weight  bf16 [V, d], rows contiguous (the usual [vocab, hidden] layout)
 *   d               hidden size, a multiple of 64
 *   every other argument as for jet_tree_accept; device_status as for the attention call
 * Cost: one pass over the weights (V * d * 2 bytes from HBM) for up to 512 rows; more
 * rows stream them once per group of 512.
 * Workspace: jet_tree_accept_hidden_workspace_bytes (one 64-bit key per row; need not
 * be initialised).
 */
JET_API size_t jet_tree_accept_hidden_workspace_bytes(int batch, int B);

JET_API jet_status jet_tree_accept_hidden(const void* hidden, const void* lm_head_weight, int d,
                                  const int32_t* token, const int32_t* parent, const int32_t* depth,
                                  const uint32_t* anc_mask, const int32_t* n_nodes, int batch, int B,
                                  int V, int N, int32_t* tgt_argmax, int32_t* accept_len, int32_t* path,
                                  int32_t* out_tokens, int32_t* device_status, void* workspace,
                                  size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * jet_tree_accept_static -- the same operation as jet_tree_accept for callers that cannot
 * provide scratch memory.  (The paper has no counterpart; this is a library convenience.)
 *
 * Who needs it: code that runs after all device memory has been handed out (a serving engine
 * that reserved the rest of the GPU for its KV cache at start-up, so a late cudaMalloc fails or
 * fragments the pool), and code on a latency-critical decode loop where an allocator call is
 * forbidden because cudaMalloc / cudaFree may synchronise the whole device.
 *
 * Instead of a caller workspace the arg-max partials go to an array built into the library:
 * JET_STATIC_ACCEPT_SCRATCH_BYTES of device memory that every GPU which loads the library
 * holds until the process exits.  The call makes no cudaMalloc / cudaFree and uses no
 * allocating library routine.  Inputs and outputs are exactly those of jet_tree_accept.
 *
 * Limit: batch * B * ceil(V / 8192) * 8 bytes must fit in JET_STATIC_ACCEPT_SCRATCH_BYTES
 * (e.g. 4096 logits rows of a 151936-entry vocabulary); larger problems are rejected on the
 * host with JET_ERR_WORKSPACE and nothing is launched.
 * First call on a device: looks up the array's device address (cudaGetSymbolAddress, with the
 * calling thread's current device); make that first call outside any stream capture.
 * Sharing: all calls on one GPU use the same array, which keeps the previous call's contents.
 * Nothing in it has to be cleared between calls, but two calls that can overlap on the GPU
 * (different streams) race on it -- serialise them, or use jet_tree_accept with separate
 * workspaces.
 */
#define JET_STATIC_ACCEPT_SCRATCH_BYTES (1u << 20)

JET_API jet_status jet_tree_accept_static(const float* logits, int64_t logits_row_stride, const int32_t* token,
                                  const int32_t* parent, const int32_t* depth, const uint32_t* anc_mask,
                                  const int32_t* n_nodes, int batch, int B, int V, int N,
                                  int32_t* tgt_argmax, int32_t* accept_len, int32_t* path,
                                  int32_t* out_tokens, void* stream);

/* ---------------------------------------------------------------------------
 * jet_tree_accept_sample -- non-greedy tree acceptance (Section 3.3, the
 * rejection-sampling rule of Eq. nongreedy_specdec applied along every branch).
 *
 * Target distribution of row v: p_v = softmax(logits[v,:] / temperature).
 * Draft distribution for the children of a depth-d node: q_d = exp(draft_logp[b,d,:]).
 * For every node v >= 1 with parent w and token y:
 *     alpha_v = min(1, p_w(y) / q_depth(w)(y))   (1 where q is 0),
 *     the node passes iff u_accept[b,v] < alpha_v.
 * The accepted prefix ends at the deepest node all of whose branch passes (several
 * at that depth: lowest index); accept_len = its depth, path / out_tokens as in
 * jet_tree_accept.  The correction token (out_tokens[accept_len]) is drawn by
 * inverse CDF in vocabulary order with u_sample[b] -- the first token whose
 * cumulative mass exceeds u_sample * total -- from max(0, p - q) at the end node if
 * that node has children in the tree (all rejected; a residual without mass falls
 * back to p), and from p itself if it is a leaf.  The random numbers are inputs:
 * uniform in [0,1), one per node and one per sequence.
 *
 *   logits       fp32 [batch*B rows, V], row stride in elements
 *   draft_logp   fp32 [batch, N, V] log-probabilities (strides in elements)
 *   u_accept     fp32 [batch, B]; u_sample fp32 [batch]
 *   alpha        optional out fp32 [batch, B] (0 for padding rows, 1 for the root)
 *   accept_len   i32 [batch]; path, out_tokens i32 [batch, N+1], -1 padded
 * What distribution comes out: on a CHAIN whose tokens were drawn from q the
 * emitted tokens follow the target distribution exactly (the guarantee of
 * speculative sampling).  On a BRANCHED tree the rule above is applied to every
 * sibling on its own and the deepest passing branch wins, which is the per-branch
 * rule the paper states but does not preserve the target distribution (two
 * siblings with p == q both pass, and the one with the lower node index is always
 * the one emitted; the residual after several rejected siblings is the single-draft
 * one).  A caller that needs exact target sampling at temperature > 0 verifies
 * chains (W = 1) with this call, or uses greedy acceptance on trees.
 * Precision: fp32 throughout, cumulative masses in fp64; a draw or a test that
 * falls within rounding of its threshold may differ from an fp64 evaluation.
 * temperature must be positive and finite.
 */
JET_API size_t jet_tree_accept_sample_workspace_bytes(int batch, int B, int V);

JET_API jet_status jet_tree_accept_sample(const float* logits, int64_t logits_row_stride, float temperature,
                                  const float* draft_logp, int64_t logp_batch_stride,
                                  int64_t logp_depth_stride, const int32_t* token, const int32_t* parent,
                                  const int32_t* depth, const uint32_t* anc_mask, const int32_t* n_nodes,
                                  const float* u_accept, const float* u_sample, int batch, int B, int V,
                                  int N, float* alpha, int32_t* accept_len, int32_t* path,
                                  int32_t* out_tokens, void* workspace, size_t workspace_bytes,
                                  void* stream);

/* ---------------------------------------------------------------------------
 * jet_kv_compact -- commit of the accepted path (Appendix E: "the accepted path
 * is committed"): for every layer l, sequence b and i in [0, accept_len[b]] the
 * K and V rows of tree node path[b,i] are copied to cache position
 * seq_len[b] + i (the root's K/V is committed too); afterwards
 * seq_len[b] += accept_len[b] + 1.  All layers in one call.
 *
 *   tree_k, tree_v  bf16 [layers, batch, B, Hkv, D]
 *   k_cache, v_cache  bf16; layer l starts cache_layer_stride elements after
 *                layer l-1.  Within a layer the layout is that of
 *                jet_tree_verify_attn (contiguous with kv_batch_stride, or
 *                paged when page_table != NULL).
 *   page_table   i32 [batch, max_pages_per_seq] or NULL.  The pages covering
 *                positions seq_len[b] .. seq_len[b]+N must already be assigned.
 *   path         i32 [batch, N+1], accept_len i32 [batch] (from jet_tree_accept)
 *   seq_len      i32 [batch], read and then updated in place
 * Every cache byte outside the written rows is left untouched.
 */
JET_API jet_status jet_kv_compact(const void* tree_k, const void* tree_v, void* k_cache, void* v_cache,
                          int64_t cache_layer_stride, int64_t kv_batch_stride,
                          const int32_t* page_table, int max_pages_per_seq, int page_size,
                          const int32_t* path, const int32_t* accept_len, int32_t* seq_len,
                          int layers, int batch, int B, int Hkv, int D, int N, void* stream);

/* jet_kv_compact_tail -- the commit for the layout of jet_tree_verify_attn_tail:
 * for every layer, sequence b and i in [1, accept_len[b]] the K and V rows at
 * position seq_len[b] + path[b,i] move to position seq_len[b] + i (the root's row
 * is already in place; all rows are read before any is written); afterwards
 * seq_len[b] += accept_len[b] + 1.  Rows behind the new length keep what they held.
 */
JET_API jet_status jet_kv_compact_tail(void* k_cache, void* v_cache, int64_t cache_layer_stride,
                               int64_t kv_batch_stride, const int32_t* page_table, int max_pages_per_seq,
                               int page_size, const int32_t* path, const int32_t* accept_len,
                               int32_t* seq_len, int layers, int batch, int B, int Hkv, int D, int N,
                               void* stream);

#ifdef __cplusplus
}
#endif
#endif /* JET_H_ */
