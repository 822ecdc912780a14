"""Seeded input generators (NumPy PCG64).  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np

# Workload shapes.  "sigma" values are standard deviations.  W is the branching
# width (4 for the tiny case, 7 -- the paper's production width -- elsewhere).
CONFIGS = {
    "tiny": dict(batch=1, layers=1, Hq=8, Hkv=2, D=64, L=512, N=4, V=1024, W=4, B=16,
                 sigma_draft=2.0, sigma_target=2.0, plant=3, paged=False),
    "qwen3_8b": dict(batch=1, layers=36, Hq=32, Hkv=8, D=128, L=4096, N=8, V=151936, W=7, B=64,
                     sigma_draft=3.0, sigma_target=2.0, plant=5, paged=False),
    "sweep_16k": dict(batch=1, layers=36, Hq=32, Hkv=8, D=128, L=16384, V=151936, W=7,
                      budgets=(16, 32, 64, 128, 256), sigma_draft=3.0, sigma_target=2.0, paged=False),
    "batched_paged": dict(batch=32, layers=36, Hq=32, Hkv=8, D=128, L_range=(1024, 8192), N=8,
                          V=151936, W=7, B=64, page_size=16, sigma_draft=3.0, sigma_target=2.0,
                          paged=True),
    "moe_30b": dict(batch=(1, 8), layers=48, Hq=32, Hkv=4, D=128, L=32768, N=12, V=151936, W=7,
                    budgets=(128, 512), sigma_draft=3.0, sigma_target=2.0, paged=False),
}


# ---------------------------------------------------------------- storage types
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _randn_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


# ---------------------------------------------------------------- draft log-probs
def make_logp(rng: np.random.Generator, N: int, V: int, sigma: float, peaked_p: float | None = None):
    """[N,V] float32 log_softmax of N(0, sigma) logits, evaluated in fp64 then rounded.

    With ``peaked_p`` one random token per depth is raised so that its
    probability is ``peaked_p`` (draft heads of real workloads are confident;
    flat random rows give trees too shallow to plant long paths).
    """
    logits = (rng.standard_normal((N, V), dtype=np.float32) * np.float32(sigma)).astype(np.float64)
    if peaked_p is not None:
        for d in range(N):
            t = int(rng.integers(0, V))
            rest = np.delete(logits[d], t)
            m = rest.max()
            log_rest = m + np.log(np.exp(rest - m).sum())
            logits[d, t] = np.log(peaked_p / (1.0 - peaked_p)) + log_rest
    m = logits.max(axis=1, keepdims=True)
    lse = m + np.log(np.exp(logits - m).sum(axis=1, keepdims=True))
    return (logits - lse).astype(np.float32)


def make_draft_logits(rng: np.random.Generator, N: int, V: int, sigma: float, peaked_p: float | None = None,
                      offset: float = 0.0):
    """[N,V] float32 raw draft logits: N(0, sigma) + offset, not normalised; with ``peaked_p`` one random token
    per depth is raised to about that probability (as in make_logp)."""
    logits = (rng.standard_normal((N, V), dtype=np.float32) * np.float32(sigma)).astype(np.float64)
    if peaked_p is not None:
        for d in range(N):
            t = int(rng.integers(0, V))
            rest = np.delete(logits[d], t)
            m = rest.max()
            logits[d, t] = np.log(peaked_p / (1.0 - peaked_p)) + m + np.log(np.exp(rest - m).sum())
    return (logits + offset).astype(np.float32)


# ---------------------------------------------------------------- attention operands
def make_attn_inputs(rng: np.random.Generator, B: int, Hq: int, Hkv: int, D: int, L: int):
    """q [B,Hq,D], k/v prefix [L,Hkv,D], tree_k/tree_v [B,Hkv,D]; N(0,1) rounded to bf16 bits."""
    return dict(
        q=_randn_bf16(rng, (B, Hq, D)),
        k_prefix=_randn_bf16(rng, (L, Hkv, D)),
        v_prefix=_randn_bf16(rng, (L, Hkv, D)),
        tree_k=_randn_bf16(rng, (B, Hkv, D)),
        tree_v=_randn_bf16(rng, (B, Hkv, D)),
    )


def make_paged_cache(rng: np.random.Generator, seq_lens, page_size: int, Hkv: int, D: int,
                     reserve: int, spare_pages: int = 3):
    """Paged K and V pools with a shuffled page table.

    Every sequence gets pages for ``seq_len + reserve`` positions.  Returns
    (k_pages, v_pages [num_pages,page_size,Hkv,D] bf16 bits, page_table
    [batch,max_pages] int32, -1 where unallocated).  All pool rows are random,
    so rows beyond a sequence's length hold junk that must not be read.
    """
    need = [(int(L) + reserve + page_size - 1) // page_size for L in seq_lens]
    num_pages = sum(need) + spare_pages
    perm = rng.permutation(num_pages)
    max_pages = max(need)
    table = np.full((len(seq_lens), max_pages), -1, dtype=np.int32)
    pos = 0
    for b, cnt in enumerate(need):
        table[b, :cnt] = perm[pos:pos + cnt]
        pos += cnt
    k_pages = _randn_bf16(rng, (num_pages, page_size, Hkv, D))
    v_pages = _randn_bf16(rng, (num_pages, page_size, Hkv, D))
    return k_pages, v_pages, table


# ---------------------------------------------------------------- target logits
def make_target_logits(rng: np.random.Generator, B: int, V: int, sigma: float) -> np.ndarray:
    return rng.standard_normal((B, V), dtype=np.float32) * np.float32(sigma)


def plant_path(logits: np.ndarray, token, parent, depth, n_nodes: int, length: int,
               rng: np.random.Generator):
    """Make the target's arg-max follow one random tree path of ``length`` draft nodes.

    Picks a node at depth min(length, deepest level) uniformly; on every edge
    (p -> u) of its root path sets ``logits[p, token[u]]`` above the row maximum,
    and at the end node raises a token that none of its children carries.
    Modifies ``logits`` in place; returns (end_node, effective_length).
    """
    depth = np.asarray(depth)
    max_depth = int(depth[:n_nodes].max())
    eff = min(length, max_depth)
    cands = [v for v in range(n_nodes) if depth[v] == eff]
    end = int(cands[int(rng.integers(0, len(cands)))])
    u = end
    while parent[u] != -1:
        p = int(parent[u])
        logits[p, token[u]] = logits[p].max() + np.float32(1.0)
        u = p
    child_tokens = {int(token[c]) for c in range(n_nodes) if parent[c] == end}
    V = logits.shape[1]
    t = int(rng.integers(0, V))
    while t in child_tokens:
        t = (t + 1) % V
    logits[end, t] = logits[end].max() + np.float32(1.0)
    return end, eff


# ---------------------------------------------------------------- hand-made tree shapes
def _finish(parent, rng, V):
    B = len(parent)
    depth = np.zeros(B, dtype=np.int32)
    for v in range(1, B):
        depth[v] = depth[parent[v]] + 1
    if rng is None:
        token = np.arange(B, dtype=np.int32)
    else:
        token = rng.integers(0, V, size=B).astype(np.int32)
    return np.asarray(parent, dtype=np.int32), depth, token


def chain_tree(B: int, rng=None, V: int = 1 << 30):
    return _finish([-1] + list(range(B - 1)), rng, V)


def star_tree(B: int, rng=None, V: int = 1 << 30):
    return _finish([-1] + [0] * (B - 1), rng, V)


def binary_tree(B: int, rng=None, V: int = 1 << 30):
    return _finish([-1] + [(v - 1) // 2 for v in range(1, B)], rng, V)


def random_tree(B: int, rng: np.random.Generator, V: int = 1 << 30, max_depth: int | None = None):
    """Random tree with parent[v] < v (each node hangs under a uniformly chosen earlier node)."""
    parent = [-1]
    depth = [0]
    for v in range(1, B):
        while True:
            p = int(rng.integers(0, v))
            if max_depth is None or depth[p] < max_depth:
                break
        parent.append(p)
        depth.append(depth[p] + 1)
    return _finish(parent, rng, V)
