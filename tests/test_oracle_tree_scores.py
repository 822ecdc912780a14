"""Pins for the alternative expansion scores of the tree-construction oracle (Appendix C:
per-depth entropy alone, accumulated log-probability plus alpha times the per-depth entropy).

None of these re-run the oracle's loop: they use the limits the appendix states, closed forms
of the entropy, closed-form trees for monotone entropies, and a replay of the pop order against
priorities recomputed from the paths.
"""
import math

import numpy as np
import pytest

from jet_inputs import make_logp
from oracle import depth_entropy_ref, tree_build_ref


def _same_tree(a, b):
    return (a["n_nodes"] == b["n_nodes"] and np.array_equal(a["parent"], b["parent"]) and
            np.array_equal(a["depth"], b["depth"]) and np.array_equal(a["token"], b["token"]) and
            np.array_equal(a["anc_mask"], b["anc_mask"]))


# ---------------------------------------------------------------- the entropy itself
def test_entropy_closed_forms():
    V = 1000
    uniform = np.full(V, -math.log(V), np.float32)
    two = np.full(V, -np.inf, np.float32)
    two[3], two[77] = math.log(0.25), math.log(0.75)
    one = np.full(V, -np.inf, np.float32)
    one[5] = 0.0
    H = depth_entropy_ref(np.stack([uniform, two, one]), 3)
    assert H.dtype == np.float32
    assert abs(H[0] - math.log(V)) < 1e-5 * math.log(V)
    assert abs(H[1] - (-(0.25 * math.log(0.25) + 0.75 * math.log(0.75)))) < 1e-6
    assert H[2] == 0.0


def test_entropy_against_scipy_on_random_rows():
    from scipy.stats import entropy
    rng = np.random.default_rng(11)
    logp = make_logp(rng, 4, 5000, 2.0)
    H = depth_entropy_ref(logp, 4)
    for d in range(4):
        ref = entropy(np.exp(logp[d].astype(np.float64)))          # normalises: the rows sum to 1 within fp32 rounding
        assert abs(H[d] - ref) < 2e-5 * max(1.0, ref)


# ---------------------------------------------------------------- limits stated by the appendix
@pytest.mark.parametrize("seed", range(4))
def test_hybrid_with_alpha_zero_is_the_default_tree(seed):
    rng = np.random.default_rng(seed)
    N, W, B, V = 6, 5, 48, 3000
    logp = make_logp(rng, N, V, 2.5)
    a = tree_build_ref(logp, 1, N, W, B)
    b = tree_build_ref(logp, 1, N, W, B, score_mode="hybrid", alpha=0.0)
    assert _same_tree(a, b) and a["pops"] == b["pops"]
    assert np.array_equal(a["score"], b["score"])


@pytest.mark.parametrize("seed", range(4))
def test_hybrid_with_huge_alpha_is_the_entropy_only_tree(seed):
    """With alpha * (smallest entropy gap) far above any accumulated log-probability the entropy term decides
    every comparison between depths.  Within one depth hybrid falls back to the accumulated score and
    entropy-only to the node index, so the trees are compared where a depth holds one node (W = 1), and the
    sequence of popped DEPTHS where it holds several."""
    rng = np.random.default_rng(100 + seed)
    N, W, B, V = 4, 1, 5, 50            # W = 1: one node per depth, no ties inside a depth
    logp = make_logp(rng, N, V, 1.0 + seed)
    H = depth_entropy_ref(logp, N)
    gap = np.min(np.abs(np.diff(np.sort(H))))
    assert gap > 1e-4
    a = tree_build_ref(logp, 0, N, W, B, score_mode="entropy")
    b = tree_build_ref(logp, 0, N, W, B, score_mode="hybrid", alpha=1e6)
    assert _same_tree(a, b)
    # and with several nodes per depth the depth ORDER of the pops agrees
    N, W, B = 3, 3, 13
    logp = make_logp(rng, N, V, 2.0)
    a = tree_build_ref(logp, 0, N, W, B, score_mode="entropy")
    b = tree_build_ref(logp, 0, N, W, B, score_mode="hybrid", alpha=1e6)
    assert [int(a["depth"][v]) for v in a["pops"]] == [int(b["depth"][v]) for v in b["pops"]]


# ---------------------------------------------------------------- closed-form trees
def _rows_with_entropies(rng, V, targets):
    """Rows whose entropies are ordered like `targets` (temperature-scaled random logits)."""
    rows = []
    for t in targets:
        x = rng.standard_normal(V) * t
        x = x - np.log(np.sum(np.exp(x)))
        rows.append(x.astype(np.float32))
    return np.stack(rows)


def test_entropy_only_decreasing_entropies_give_level_order():
    """H_1 > H_2 > H_3: every node of depth d is popped before any node of depth d + 1 (among equal
    priorities the lowest index first), so the tree is the complete W-ary tree in level order, cut by B."""
    rng = np.random.default_rng(5)
    N, W, V, B = 3, 3, 400, 30
    logp = _rows_with_entropies(rng, V, [0.5, 1.5, 3.0])          # sharper rows have less entropy
    H = depth_entropy_ref(logp, N)
    assert H[0] > H[1] > H[2]
    t = tree_build_ref(logp, 9, N, W, B, score_mode="entropy")
    assert t["n_nodes"] == B
    # level order: node u >= 1 has parent (u - 1) // W
    assert t["parent"][1:B].tolist() == [(u - 1) // W for u in range(1, B)]
    assert t["depth"][:B].tolist() == [0] + [1] * 3 + [2] * 9 + [3] * 17


def test_entropy_only_increasing_entropies_give_a_comb():
    """H_1 < H_2 < H_3: the newest (deepest) children always have the highest priority, so the walk goes
    down the first child until depth N; nodes of depth N are discarded when popped, then the remaining
    nodes of depth N - 1 are expanded in index order, and so on."""
    rng = np.random.default_rng(6)
    N, W, V = 3, 2, 400
    logp = _rows_with_entropies(rng, V, [3.0, 1.5, 0.5])
    H = depth_entropy_ref(logp, N)
    assert H[0] < H[1] < H[2]
    t = tree_build_ref(logp, 9, N, W, 15, score_mode="entropy")
    # root -> 1,2 ; pop 1 -> 3,4 ; pop 3 -> 5,6 (depth 3) ; 5,6 discarded ; pop 4 -> 7,8 ; 7,8 discarded ;
    # pop 2 -> 9,10 ; pop 9 -> 11,12 ; discarded ; pop 10 -> 13,14
    assert t["n_nodes"] == 15
    assert t["parent"].tolist() == [-1, 0, 0, 1, 1, 3, 3, 4, 4, 2, 2, 9, 9, 10, 10]
    assert t["pops"][:4] == [0, 1, 3, 5]


# ---------------------------------------------------------------- replay
@pytest.mark.parametrize("mode,alpha", [("entropy", 0.0), ("hybrid", 0.5), ("hybrid", 4.0)])
@pytest.mark.parametrize("seed", range(3))
def test_pop_order_replays_against_recomputed_priorities(mode, alpha, seed):
    """Priorities recomputed from the finished tree (path log-probabilities summed from the root in fp32,
    entropy from the closed-form helper) must make every pop the maximum of the frontier at that moment."""
    rng = np.random.default_rng(40 + seed)
    N, W, B, V = 5, 4, 40, 2000
    logp = make_logp(rng, N, V, 2.0)
    t = tree_build_ref(logp, 3, N, W, B, score_mode=mode, alpha=alpha)
    n = t["n_nodes"]
    H = depth_entropy_ref(logp, N)
    prio = np.zeros(n, np.float32)
    for u in range(n):
        path = []
        v = u
        while v > 0:
            path.append(v)
            v = int(t["parent"][v])
        s = np.float32(0.0)
        for v in reversed(path):
            s = np.float32(s + logp[t["depth"][v] - 1, t["token"][v]])
        h = np.float32(0.0) if u == 0 else H[t["depth"][u] - 1]
        prio[u] = h if mode == "entropy" else np.float32(s + np.float32(np.float32(alpha) * h))
    assert np.array_equal(prio, t["priority"][:n])
    # replay: children of a popped node join the frontier; the next pop is the frontier's best
    children = {v: [u for u in range(n) if t["parent"][u] == v] for v in range(n)}
    frontier = {0}
    for v in t["pops"]:
        best = max(frontier, key=lambda u: (prio[u], -u))
        assert v == best
        frontier.remove(v)
        frontier.update(children[v])
