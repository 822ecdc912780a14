"""Plain CPU statement of the tree-verification path (NumPy, fp64 arithmetic).

TEST INFRASTRUCTURE ONLY -- never imported by the product package.

Each function follows one passage of the paper:

* ``tree_build_ref``   -- Algorithm 1 (Parallel Tree Drafting) with the
  accumulated draft log-probability score of Eq. (accum_logp) in Section 3.3,
  fed by the per-depth top-W extraction described in Section 3.3 / Appendix E;
  its ``score_mode`` argument selects the alternative expansion scores of
  Appendix C (per-depth entropy alone, accumulated log-probability plus alpha
  times the per-depth entropy), with ``depth_entropy_ref`` as the entropy.
  ``tree_build_logits_ref`` is the same fed with raw draft logits
  (``log_softmax_ref`` first).
* ``tree_attn_ref``    -- the tree-causal mask and masked attention equations
  of Section 3.2 (prefix visible to every node, a node sees Anc(v) + {v}).
* ``tree_accept_ref``  -- the greedy acceptance rule of Section 3.3 and
  Appendix E: a node is accepted iff its token equals the target's greedy
  prediction at its parent; the deepest fully accepted root-to-node path wins
  and the target prediction at its last node is the correction token.
* ``kv_compact_ref``   -- "the accepted path is committed" (Appendix E): the
  K/V rows of the accepted path are copied behind the prefix;
  ``kv_compact_tail_ref`` is the same commit for a cache that already holds the
  tree's rows behind the prefix (the serving layout of Appendix E).
* ``lm_head_argmax_ref`` -- that greedy prediction taken from the target's final hidden
  states (logit = hidden . LM-head row, arg-max per row, ties to the lowest id).
* ``tree_accept_sample_ref`` -- the non-greedy acceptance rule of Section 3.3
  (Eq. nongreedy_specdec): along every branch a draft token is accepted with
  probability min(1, p/q); a correction token is sampled from the target where
  the accepted prefix ends.

Nothing here is blocked, fused or reordered; loops are literal so the code can
be checked against the paper by eye.  Readings taken where the paper is silent
(root counted in the budget B, root score 0, ties to the lowest index, fp32
score adds, contiguous GQA groups, root K/V committed) are listed in the
design notes of the repository and repeated in the docstrings below.

Pins (tests marked "not gpu"): brute-force full-tree enumeration, closed forms
(W=1 chain, N=1 star, B=1, B >= full tree) and hand-worked fixtures for
``tree_build_ref``; causal-attention / decode-attention special cases against
torch's CPU scaled_dot_product_attention, zero influence of masked nodes and
uniform-V for ``tree_attn_ref``; the expected-token closed form of Eq. (1) on
chains, the ancestor-bitmask formulation and planted paths for
``tree_accept_ref``; attention-after-commit round trip for ``kv_compact_ref``,
and agreement of ``kv_compact_tail_ref`` with it on a cache whose tail holds the tree.
The tie-break conventions themselves have no counterpart to be checked
against (the authors' code is not available): parity unpinned for tie-breaks
only.  ``tree_accept_sample_ref`` is pinned by the defining property of
speculative sampling (on a chain whose tokens are drawn from the draft
distribution the emitted token is distributed exactly as the target's), the
closed-form expected accepted length, and the q == p / disjoint-support
special cases; its reading of the rule for several rejected siblings (the
single-draft residual max(0, p - q)) has no counterpart to be checked against:
parity unpinned for that reading only.  The expansion scores of Appendix C are
pinned by the limits the appendix states (alpha = 0 gives the default tree, a
large alpha the entropy-only tree), closed-form entropies (uniform, two-point),
closed-form trees for monotone entropies (level order / comb) and by replaying
the pop order against priorities recomputed from the paths; whether the entropy
term is that of the node's own depth or a sum along the branch is a reading
with no counterpart to check against: parity unpinned for that reading only.  ``log_softmax_ref`` is pinned against
scipy's log_softmax, closed forms (uniform, two-point), rows summing to one and
shift invariance; the two helpers ``bf16_bits_to_f64`` (fixed bit patterns whose values the bfloat16
format itself gives) and ``gather_paged_prefix`` (a cache whose rows hold their own page and offset)
have pins of their own; ``lm_head_argmax_ref`` is pinned by brute-force integer sums on small
integer-valued inputs (every product and sum exact), one-hot hidden states that select a weight column,
ties to the lowest id and the sign flip that turns the arg-max into the arg-min; ``tree_build_logits_ref`` by the invariance of the tree under
a per-row shift of the logits and by agreement with ``tree_build_ref`` on
log-probabilities that scipy computed.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# helpers (no method arithmetic)
# --------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    bits = np.asarray(bits)
    if bits.dtype != np.uint16:
        return np.asarray(bits, dtype=np.float64)
    as_f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return as_f32.astype(np.float64)


def gather_paged_prefix(cache: np.ndarray, page_table_row: np.ndarray, L: int) -> np.ndarray:
    """Rows 0..L-1 of one sequence out of a paged cache [num_pages, page_size, Hkv, D].

    Position j lives in page ``page_table_row[j // page_size]`` at offset
    ``j % page_size``.
    """
    page_size = cache.shape[1]
    rows = [cache[int(page_table_row[j // page_size]), j % page_size] for j in range(L)]
    if not rows:
        return np.zeros((0,) + cache.shape[2:], dtype=cache.dtype)
    return np.stack(rows, axis=0)


# --------------------------------------------------------------------------
# O0  target prediction from hidden states (Section 3.3 / Appendix E: "the target model's greedy prediction")
# --------------------------------------------------------------------------
def lm_head_argmax_ref(hidden, weight):
    """The target's greedy prediction of every row from its final hidden state.

    ``hidden`` [R, d] and ``weight`` [V, d] are bfloat16 bit patterns (uint16) or numbers; they are widened
    exactly to float64 and logit[r, t] = sum_k hidden[r, k] * weight[t, k] is formed in float64 (a library
    matrix product).  Returns a dict: ``logits`` [R, V] float64; ``tgt`` [R] = arg-max per row, ties to the
    lowest token id; ``abs_dot`` [R, V] = sum_k |hidden[r, k] * weight[t, k]|, the scale of the rounding error
    that a K-term fp32 evaluation of the same sum may make (about K * 2**-24 of it), which the GPU parity test
    uses to tell a genuine disagreement from two tokens whose exact logits are closer than that."""
    h = bf16_bits_to_f64(hidden)
    w = bf16_bits_to_f64(weight)
    logits = h @ w.T
    return dict(logits=logits, tgt=np.argmax(logits, axis=1).astype(np.int32), abs_dot=np.abs(h) @ np.abs(w).T)


# --------------------------------------------------------------------------
# O1  tree_build  -- Algorithm 1 + Eq. (accum_logp)
# --------------------------------------------------------------------------
def depth_entropy_ref(logp: np.ndarray, N: int) -> np.ndarray:
    """Per-depth entropy of the draft distributions (Appendix C): H[d] = -sum_v exp(l_v) * l_v over row d of
    the log-probabilities, summed in float64 (entries of -inf contribute 0) and rounded once to float32."""
    H = np.zeros(N, dtype=np.float32)
    for d in range(N):
        l = np.asarray(logp[d], dtype=np.float64)
        fin = np.isfinite(l)
        H[d] = np.float32(-np.sum(np.exp(l[fin]) * l[fin]))
    return H


def log_softmax_ref(logits: np.ndarray):
    """Draft log-probabilities from raw draft logits (Section 3.3: the tree is scored with log q): per row
    lse = log sum_v exp(z_v), formed in float64 as max + log(sum(exp(z - max))), and
    logp_v = float32(float64(z_v) - lse), rounded once.  Returns (logp [N,V] float32, lse [N] float64).
    Entries of -inf stay -inf (probability 0)."""
    z = np.asarray(logits, dtype=np.float64)
    m = z.max(axis=1)
    lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
    return (z - lse[:, None]).astype(np.float32), lse


def tree_build_logits_ref(logits: np.ndarray, root_token: int, N: int, W: int, B: int,
                          score_mode: str = "accum_logp", alpha: float = 0.0) -> dict:
    """Algorithm 1 fed with raw draft logits: exactly log_softmax_ref followed by tree_build_ref (the
    candidates are ranked by their rounded float32 log-probabilities, so two logits that round to the same
    log-probability tie and the lower token id comes first, as in tree_build_ref).  Adds ``depth_lse``
    (float32 rounding of each row's lse) to the result."""
    logp, lse = log_softmax_ref(np.asarray(logits)[:N])
    out = tree_build_ref(logp, root_token, N, W, B, score_mode=score_mode, alpha=alpha)
    out["depth_lse"] = lse.astype(np.float32)
    return out


def tree_build_ref(logp: np.ndarray, root_token: int, N: int, W: int, B: int,
                   score_mode: str = "accum_logp", alpha: float = 0.0) -> dict:
    """Algorithm 1 for one sequence.

    ``logp`` is [N, V] float32: row d is the draft log-distribution that the
    children of every depth-d node draw their candidates from.  B counts the
    root.  Returns arrays padded to B with -1 (mask rows zero) and ``n_nodes``.

    Readings: root token is given, root score is 0 (empty sum); candidates per
    depth are the W largest log-probs, ties to the lowest token id; the queue
    pops the largest score, ties to the smallest node index; a child's score is
    one float32 add ``score[parent] + logp[depth[parent], token]``; a popped
    node at depth N is discarded (stays in the tree as a leaf); all of a
    node's children are appended at once, cut short only by the budget.

    Expansion scores (Appendix C).  ``score_mode`` selects the queue's priority; the
    ``score`` output is the accumulated log-probability in every mode:
      "accum_logp"  priority = score (Eq. accum_logp, the default);
      "entropy"     priority = H of the node's depth alone;
      "hybrid"      priority = score + alpha * H of the node's depth.
    H of depth d >= 1 is the entropy of the distribution the depth-d tokens were
    drawn from (row d-1 of ``logp``), see depth_entropy_ref; the root's H is 0.
    Readings: the entropy term is the one of the node's own depth, not a sum along
    the branch (so that alpha -> infinity is the entropy-only rule, as the appendix
    states); it enters with a plus sign; the priority is formed in float32 as
    fl(score + fl(alpha * H)), two roundings, no fused multiply-add.
    """
    assert score_mode in ("accum_logp", "entropy", "hybrid")
    logp = np.asarray(logp)
    assert logp.dtype == np.float32 and logp.ndim == 2 and logp.shape[0] >= N
    V = logp.shape[1]
    Wc = min(W, V)
    words = (B + 31) // 32

    # per-depth top-W: sort by (value descending, token id ascending)
    ids = np.arange(V)
    top = []
    for d in range(N):
        order = np.lexsort((ids, -logp[d].astype(np.float64)))
        top.append(order[:Wc])

    parent = np.full(B, -1, dtype=np.int32)
    depth = np.full(B, -1, dtype=np.int32)
    token = np.full(B, -1, dtype=np.int32)
    score = np.zeros(B, dtype=np.float32)
    score64 = np.zeros(B, dtype=np.float64)

    H = depth_entropy_ref(logp, N)                     # H[d-1] belongs to the nodes of depth d
    prio = np.zeros(B, dtype=np.float32)
    alpha32 = np.float32(alpha)

    def priority(u):
        h = np.float32(0.0) if depth[u] == 0 else H[depth[u] - 1]
        if score_mode == "accum_logp":
            return score[u]
        if score_mode == "entropy":
            return h
        return np.float32(score[u] + np.float32(alpha32 * h))

    parent[0], depth[0], token[0] = -1, 0, int(root_token)
    score[0] = np.float32(0.0)
    prio[0] = priority(0)
    n = 1
    queue = [0]
    pops = []
    while n < B and queue:
        best = queue[0]
        for v in queue[1:]:
            if prio[v] > prio[best] or (prio[v] == prio[best] and v < best):
                best = v
        queue.remove(best)
        v = best
        pops.append(v)
        if depth[v] == N:
            continue
        d = int(depth[v])
        for r in range(Wc):
            if n == B:
                break
            u = n
            n += 1
            y = int(top[d][r])
            parent[u], depth[u], token[u] = v, d + 1, y
            score[u] = np.float32(score[v]) + np.float32(logp[d, y])
            score64[u] = score64[v] + float(logp[d, y])
            prio[u] = priority(u)
            queue.append(u)

    anc = np.zeros((B, words), dtype=np.uint32)
    for u in range(n):
        if u > 0:
            anc[u] = anc[parent[u]]
        anc[u, u // 32] |= np.uint32(1) << np.uint32(u % 32)

    return dict(parent=parent, depth=depth, token=token, score=score, score64=score64,
                anc_mask=anc, n_nodes=n, pops=pops, priority=prio, depth_entropy=H,
                top_tok=np.stack(top).astype(np.int32) if N > 0 else np.zeros((0, Wc), np.int32))


def anc_from_parent(parent, n_nodes: int, B: int) -> np.ndarray:
    """Ancestor bitmask rows of the mask equation in Section 3.2: bit u of row v
    is set iff u is v or an ancestor of v (found by walking parent pointers)."""
    words = (B + 31) // 32
    anc = np.zeros((B, words), dtype=np.uint32)
    for v in range(n_nodes):
        u = v
        while u != -1:
            anc[v, u // 32] |= np.uint32(1) << np.uint32(u % 32)
            u = int(parent[u])
    return anc


# --------------------------------------------------------------------------
# O2  tree_verify_attn  -- mask + attention equations of Section 3.2
# --------------------------------------------------------------------------
def _visible_nodes(anc_row: np.ndarray, B: int) -> list:
    return [u for u in range(B) if (int(anc_row[u // 32]) >> (u % 32)) & 1]


def tree_attn_rows_ref(q, k_prefix, v_prefix, tree_k, tree_v, anc_mask, n_nodes,
                       scale, rows):
    """Attention outputs for selected (node v, query head h) pairs of one sequence.

    q [B,Hq,D]; k_prefix/v_prefix [L,Hkv,D]; tree_k/tree_v [B,Hkv,D]; any of
    them may be bfloat16 bit patterns (uint16), widened exactly to fp64.
    Query head h reads KV head h // (Hq // Hkv).  Every prefix key is visible;
    tree key u is visible to node v iff bit u of ``anc_mask[v]`` is set.
    Masked keys get exactly zero weight.  Returns (o [len(rows), D] fp64,
    lse [len(rows)] fp64, natural log).  A padding node (v >= n_nodes) gives a
    zero row and lse = -inf.
    """
    q = bf16_bits_to_f64(q)
    k_prefix = bf16_bits_to_f64(k_prefix)
    v_prefix = bf16_bits_to_f64(v_prefix)
    tree_k = bf16_bits_to_f64(tree_k)
    tree_v = bf16_bits_to_f64(tree_v)
    B, Hq, D = q.shape
    Hkv = tree_k.shape[1]
    G = Hq // Hkv
    L = k_prefix.shape[0]
    out = np.zeros((len(rows), D), dtype=np.float64)
    lse = np.full(len(rows), -np.inf, dtype=np.float64)
    for i, (v, h) in enumerate(rows):
        if v >= n_nodes:
            continue
        g = h // G
        vis = _visible_nodes(anc_mask[v], B)
        s = np.empty(L + len(vis), dtype=np.float64)
        for j in range(L):
            s[j] = scale * np.dot(q[v, h], k_prefix[j, g])
        for c, u in enumerate(vis):
            s[L + c] = scale * np.dot(q[v, h], tree_k[u, g])
        m = s.max()
        p = np.exp(s - m)
        denom = p.sum()
        acc = np.zeros(D, dtype=np.float64)
        for j in range(L):
            acc += p[j] * v_prefix[j, g]
        for c, u in enumerate(vis):
            acc += p[L + c] * tree_v[u, g]
        out[i] = acc / denom
        lse[i] = m + np.log(denom)
    return out, lse


def tree_attn_ref(q, k_prefix, v_prefix, tree_k, tree_v, anc_mask, n_nodes, scale):
    """All rows of one sequence: out [B,Hq,D] fp64, lse [Hq,B] fp64.

    Same definition as ``tree_attn_rows_ref`` but with the two key loops
    written as matrix-vector products per (node, head) so that the full
    Qwen3-8B-shaped layer finishes in seconds.
    """
    q = bf16_bits_to_f64(q)
    k_prefix = bf16_bits_to_f64(k_prefix)
    v_prefix = bf16_bits_to_f64(v_prefix)
    tree_k = bf16_bits_to_f64(tree_k)
    tree_v = bf16_bits_to_f64(tree_v)
    B, Hq, D = q.shape
    Hkv = tree_k.shape[1]
    G = Hq // Hkv
    L = k_prefix.shape[0]
    out = np.zeros((B, Hq, D), dtype=np.float64)
    lse = np.full((Hq, B), -np.inf, dtype=np.float64)
    kp = [np.ascontiguousarray(k_prefix[:, g, :]) for g in range(Hkv)]
    vp = [np.ascontiguousarray(v_prefix[:, g, :]) for g in range(Hkv)]
    for v in range(min(n_nodes, B)):
        vis = _visible_nodes(anc_mask[v], B)
        for h in range(Hq):
            g = h // G
            s_prefix = scale * (kp[g] @ q[v, h])                 # [L]
            s_tree = scale * (tree_k[vis, g, :] @ q[v, h])       # [len(vis)]
            s = np.concatenate([s_prefix, s_tree])
            m = s.max()
            p = np.exp(s - m)
            denom = p.sum()
            acc = p[:L] @ vp[g] + p[L:] @ tree_v[vis, g, :]
            out[v, h] = acc / denom
            lse[h, v] = m + np.log(denom)
    return out, lse


# --------------------------------------------------------------------------
# O3  tree_accept  -- greedy acceptance, brute force over root-to-leaf paths
# --------------------------------------------------------------------------
def tree_accept_ref(logits, token, parent, depth, n_nodes, N) -> dict:
    """Greedy acceptance for one sequence.

    ``logits`` [B,V] fp32: row v is the target's next-token logits after node
    v.  tgt[v] = first index of the row maximum.  Every root-to-leaf path is
    enumerated; along it draft tokens are accepted while
    ``token[v_t] == tgt[v_{t-1}]``.  The result is the longest accepted prefix
    over all leaves (if several end nodes tie, the smallest node index).
    The root is always on the path and is not counted in ``accept_len``.
    ``out_tokens`` = accepted draft tokens followed by the correction token
    ``tgt[v*]``; ``path`` and ``out_tokens`` are padded to N+1 with -1.
    """
    logits = np.asarray(logits)
    B = len(token)
    tgt = np.full(B, -1, dtype=np.int32)
    for v in range(n_nodes):
        tgt[v] = int(np.argmax(logits[v]))          # first occurrence of the max

    has_child = np.zeros(B, dtype=bool)
    for v in range(1, n_nodes):
        has_child[parent[v]] = True
    best_len, best_end = 0, 0
    for leaf in range(n_nodes):
        if has_child[leaf]:
            continue
        chain = []
        v = leaf
        while v != -1:
            chain.append(v)
            v = int(parent[v])
        chain.reverse()                              # root .. leaf
        r = 0
        for t in range(1, len(chain)):
            if token[chain[t]] == tgt[chain[t - 1]]:
                r = t
            else:
                break
        end = chain[r]
        if r > best_len or (r == best_len and end < best_end):
            best_len, best_end = r, end

    chain = []
    v = best_end
    while v != -1:
        chain.append(v)
        v = int(parent[v])
    chain.reverse()
    path = np.full(N + 1, -1, dtype=np.int32)
    out_tokens = np.full(N + 1, -1, dtype=np.int32)
    path[: len(chain)] = chain
    for t in range(1, len(chain)):
        out_tokens[t - 1] = token[chain[t]]
    out_tokens[best_len] = tgt[best_end]
    return dict(tgt=tgt, accept_len=best_len, end_node=best_end, path=path, out_tokens=out_tokens)


# --------------------------------------------------------------------------
# O3b  non-greedy acceptance (Section 3.3, Eq. nongreedy_specdec)
# --------------------------------------------------------------------------
def target_probs_ref(logits_row, temperature: float) -> np.ndarray:
    """softmax(logits / temperature) of one row in fp64."""
    z = np.asarray(logits_row, dtype=np.float64) / float(temperature)
    z = z - z.max()
    e = np.exp(z)
    return e / e.sum()


def tree_accept_sample_ref(logits, temperature, draft_logp, token, parent, depth, n_nodes, N,
                           u_accept, u_sample) -> dict:
    """Non-greedy tree acceptance for one sequence.

    ``logits`` [B,V] fp32: row v is the target's next-token logits after node
    v; p_v = softmax(row / temperature).  ``draft_logp`` [N,V]: row d is the
    draft's log-distribution for the children of depth-d nodes; q_d = exp(row).
    ``u_accept`` [B] and ``u_sample`` (scalar) are uniform numbers in [0,1)
    supplied by the caller (the method's randomness is an input).

    For every node v >= 1 with parent w and token y:
        alpha_v = min(1, p_w(y) / q_{depth(w)}(y)),   A_v = [u_accept[v] < alpha_v]
    (alpha_v = 1 where q is 0).  A node is accepted iff A holds for it and all
    its ancestors below the root; the deepest accepted node v* ends the prefix
    (several at that depth: smallest index), accept_len = depth[v*].

    Correction token at v* (depth d): if v* has children in the tree (all of
    them were rejected) it is drawn from the residual max(0, p_{v*} - q_d)
    normalised -- the single-draft rule; a residual without mass falls back to
    p_{v*} -- and from p_{v*} itself if v* is a leaf.  Drawing = inverse CDF in
    vocabulary order: the first token whose cumulative mass exceeds
    u_sample * total.
    """
    logits = np.asarray(logits)
    draft_logp = np.asarray(draft_logp, dtype=np.float64)
    B = len(token)
    alpha = np.ones(B, dtype=np.float64)
    ok = np.zeros(B, dtype=bool)
    ok[0] = True
    probs = {}

    def p_of(v):
        if v not in probs:
            probs[v] = target_probs_ref(logits[v], temperature)
        return probs[v]

    for v in range(1, n_nodes):
        w = int(parent[v])
        y = int(token[v])
        q = float(np.exp(draft_logp[int(depth[w]), y]))
        pw = float(p_of(w)[y])
        alpha[v] = 1.0 if q == 0.0 else min(1.0, pw / q)
        ok[v] = bool(u_accept[v] < alpha[v])

    accepted = np.zeros(B, dtype=bool)
    accepted[0] = True
    for v in range(1, n_nodes):                      # parent[v] < v: parents come first
        accepted[v] = ok[v] and accepted[int(parent[v])]
    best_end, best_len = 0, 0
    for v in range(n_nodes):
        if accepted[v] and int(depth[v]) > best_len:
            best_end, best_len = v, int(depth[v])

    has_child = any(int(parent[v]) == best_end for v in range(1, n_nodes))
    p_end = p_of(best_end)
    dist = p_end
    if has_child:
        resid = np.maximum(0.0, p_end - np.exp(draft_logp[int(depth[best_end])]))
        if resid.sum() > 0.0:
            dist = resid
    cdf = np.cumsum(dist)
    target = float(u_sample) * float(cdf[-1])
    corr = int(np.searchsorted(cdf, target, side="right"))       # first index with cdf > target
    corr = min(corr, len(dist) - 1)

    chain = []
    v = best_end
    while v != -1:
        chain.append(v)
        v = int(parent[v])
    chain.reverse()
    path = np.full(N + 1, -1, dtype=np.int32)
    out_tokens = np.full(N + 1, -1, dtype=np.int32)
    path[: len(chain)] = chain
    for t in range(1, len(chain)):
        out_tokens[t - 1] = token[chain[t]]
    out_tokens[best_len] = corr
    return dict(alpha=alpha, ok=ok, accept_len=best_len, end_node=best_end, path=path, out_tokens=out_tokens,
                correction=corr, dist=dist, cdf=cdf, residual_used=bool(has_child and dist is not p_end))


# --------------------------------------------------------------------------
# O4  kv_compact  -- commit of the accepted path
# --------------------------------------------------------------------------
def kv_compact_ref(tree_k, tree_v, k_cache, v_cache, page_table, path, accept_len, seq_len):
    """Copy the accepted path's K/V rows behind each sequence's prefix.

    tree_k/tree_v [layers,batch,B,Hkv,D].  Contiguous cache (``page_table`` is
    None): [layers,batch,Lmax,Hkv,D]; paged: [layers,num_pages,page_size,Hkv,D]
    with position j of sequence b in page ``page_table[b, j // page_size]`` at
    offset ``j % page_size``.  For i = 0..accept_len[b] (root included) the row
    of node ``path[b,i]`` goes to position ``seq_len[b] + i``; the new length
    is ``seq_len[b] + accept_len[b] + 1``.  Returns new (k_cache, v_cache,
    seq_len); inputs are not modified.
    """
    k_out = np.array(k_cache, copy=True)
    v_out = np.array(v_cache, copy=True)
    new_len = np.array(seq_len, copy=True)
    layers, batch = tree_k.shape[0], tree_k.shape[1]
    for layer in range(layers):
        for b in range(batch):
            for i in range(int(accept_len[b]) + 1):
                node = int(path[b, i])
                pos = int(seq_len[b]) + i
                if page_table is None:
                    k_out[layer, b, pos] = tree_k[layer, b, node]
                    v_out[layer, b, pos] = tree_v[layer, b, node]
                else:
                    page_size = k_cache.shape[2]
                    page = int(page_table[b, pos // page_size])
                    k_out[layer, page, pos % page_size] = tree_k[layer, b, node]
                    v_out[layer, page, pos % page_size] = tree_v[layer, b, node]
    for b in range(batch):
        new_len[b] = seq_len[b] + accept_len[b] + 1
    return k_out, v_out, new_len


def kv_compact_tail_ref(k_cache, v_cache, page_table, path, accept_len, seq_len):
    """The commit when the tree's K/V rows already sit in the cache behind the prefix (node v of
    sequence b at position ``seq_len[b] + v``; layouts as in kv_compact_ref): for i = 1..accept_len[b]
    the row at position ``seq_len[b] + path[b,i]`` moves to position ``seq_len[b] + i`` (the root's row
    stays), every row is read before any is written, and the new length is ``seq_len[b] +
    accept_len[b] + 1``.  Rows beyond the new length keep whatever they held.  Returns new
    (k_cache, v_cache, seq_len)."""
    k_out = np.array(k_cache, copy=True)
    v_out = np.array(v_cache, copy=True)
    new_len = np.array(seq_len, copy=True)
    layers = k_cache.shape[0]
    batch = len(seq_len)

    def slot(b, pos):
        if page_table is None:
            return (b, pos)
        page_size = k_cache.shape[2]
        return (int(page_table[b, pos // page_size]), pos % page_size)

    for layer in range(layers):
        for b in range(batch):
            L = int(seq_len[b])
            for i in range(1, int(accept_len[b]) + 1):
                src = slot(b, L + int(path[b, i]))
                dst = slot(b, L + i)
                k_out[(layer,) + dst] = k_cache[(layer,) + src]        # sources are read from the old cache
                v_out[(layer,) + dst] = v_cache[(layer,) + src]
    for b in range(batch):
        new_len[b] = seq_len[b] + accept_len[b] + 1
    return k_out, v_out, new_len
