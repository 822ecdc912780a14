"""Pins for the tree-construction oracle (Algorithm 1, accumulated log-prob score).

None of these re-run the oracle's own loop: they check it against a hand-worked
example, closed forms for degenerate parameters, a brute-force construction that
never uses a queue, and structural invariants.
"""
import itertools
import json
import os

import numpy as np
import pytest

from jet_inputs import make_logp
from oracle import tree_build_ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_handworked_example():
    g = json.load(open(os.path.join(GOLDEN, "tree_build_handworked.json")))
    logp = np.log(np.array(g["probs"], dtype=np.float64)).astype(np.float32)
    t = tree_build_ref(logp, g["root_token"], g["N"], g["W"], g["B"])
    assert t["n_nodes"] == g["B"]
    assert t["parent"].tolist() == g["parent"]
    assert t["depth"].tolist() == g["depth"]
    assert t["token"].tolist() == g["token"]
    assert t["pops"] == g["pops"]
    assert t["anc_mask"][:, 0].tolist() == g["anc_mask"]
    np.testing.assert_allclose(np.exp(t["score"].astype(np.float64)), g["score_probs"], rtol=1e-6)


def _brute_force_tree(logp, root_token, N, W, B):
    """Queue-free construction: enumerate the complete W-ary depth-N tree, sort all
    of its nodes by path score, and hand out children in that order.

    Valid only without score ties.  Best-first search with non-positive
    increments pops nodes in globally sorted score order, so the node created
    k-th is the k-th child slot when walking the sorted list.
    """
    V = logp.shape[1]
    Wc = min(W, V)
    top = [sorted(range(V), key=lambda t: (-float(logp[d, t]), t))[:Wc] for d in range(N)]
    # every node of the complete tree = tuple of ranks; score summed in float32 left to right
    nodes = {(): np.float32(0.0)}
    for d in range(1, N + 1):
        for ranks in itertools.product(range(Wc), repeat=d):
            nodes[ranks] = np.float32(nodes[ranks[:-1]] + logp[d - 1, top[d - 1][ranks[-1]]])
    scores = sorted(nodes.values())
    assert all(a != b for a, b in zip(scores, scores[1:])), "score tie: brute force not applicable"
    order = sorted(nodes, key=lambda r: -float(nodes[r]))
    index = {(): 0}
    parent, depth, token = [-1], [0], [root_token]
    for ranks in order:
        if len(parent) >= B:
            break
        if ranks not in index:
            # a node is reached in sorted order only after its parent created it,
            # unless the budget ran out first
            continue
        if len(ranks) == N:
            continue
        for r in range(Wc):
            if len(parent) == B:
                break
            child = ranks + (r,)
            index[child] = len(parent)
            parent.append(index[ranks])
            depth.append(len(child))
            token.append(top[len(ranks)][r])
    return parent, depth, token


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("N,W,B,V", [(4, 4, 16, 1024), (3, 3, 11, 50), (4, 2, 31, 17), (2, 5, 40, 9)])
def test_matches_queue_free_brute_force(seed, N, W, B, V):
    rng = np.random.default_rng(100 + seed)
    logp = make_logp(rng, N, V, 2.0)
    t = tree_build_ref(logp, 7, N, W, B)
    parent, depth, token = _brute_force_tree(logp, 7, N, W, B)
    n = len(parent)
    full = sum(min(W, V) ** d for d in range(N + 1))
    assert t["n_nodes"] == n == min(B, full)
    assert t["parent"][:n].tolist() == parent
    assert t["depth"][:n].tolist() == depth
    assert t["token"][:n].tolist() == token
    assert (t["parent"][n:] == -1).all() and (t["token"][n:] == -1).all()
    assert (t["anc_mask"][n:] == 0).all()


def test_width_one_is_argmax_chain():
    rng = np.random.default_rng(1)
    N, V = 6, 300
    logp = make_logp(rng, N, V, 2.0)
    for B in (1, 2, 4, 7, 12):
        t = tree_build_ref(logp, 3, N, 1, B)
        n = min(B, N + 1)
        assert t["n_nodes"] == n
        assert t["parent"][:n].tolist() == [-1] + list(range(n - 1))
        assert t["token"][1:n].tolist() == [int(np.argmax(logp[d])) for d in range(n - 1)]
        cum = np.float32(0)
        for v in range(1, n):
            cum = np.float32(cum + logp[v - 1].max())
            assert t["score"][v] == cum


def test_depth_one_is_star_in_rank_order():
    rng = np.random.default_rng(2)
    V, W = 200, 7
    logp = make_logp(rng, 1, V, 2.0)
    ranked = np.argsort(-logp[0], kind="stable")
    for B in (2, 5, 8, 20):
        t = tree_build_ref(logp, 0, 1, W, B)
        n = min(B, W + 1)
        assert t["n_nodes"] == n
        assert t["parent"][1:n].tolist() == [0] * (n - 1)
        assert t["token"][1:n].tolist() == ranked[: n - 1].tolist()
        assert t["score"][1:n].tolist() == logp[0, ranked[: n - 1]].tolist()


def test_budget_beyond_full_tree_gives_complete_tree():
    rng = np.random.default_rng(3)
    N, W, V = 3, 3, 40
    logp = make_logp(rng, N, V, 2.0)
    full = (W ** (N + 1) - 1) // (W - 1)
    t = tree_build_ref(logp, 0, N, W, full + 9)
    assert t["n_nodes"] == full
    counts = np.bincount(t["depth"][:full])
    assert counts.tolist() == [W ** d for d in range(N + 1)]
    # queue-empty termination popped every node exactly once
    assert sorted(t["pops"]) == list(range(full))


def test_root_only():
    logp = make_logp(np.random.default_rng(4), 3, 10, 1.0)
    t = tree_build_ref(logp, 42, 3, 2, 1)
    assert t["n_nodes"] == 1 and t["token"][0] == 42 and t["parent"][0] == -1
    assert t["anc_mask"][0, 0] == 1


@pytest.mark.parametrize("seed", range(4))
def test_invariants(seed):
    rng = np.random.default_rng(50 + seed)
    N, W, B, V = 8, 7, 64, 5000
    logp = make_logp(rng, N, V, 3.0, peaked_p=0.7 if seed % 2 else None)
    t = tree_build_ref(logp, 1, N, W, B)
    n = t["n_nodes"]
    p, d, tok, s, anc = t["parent"], t["depth"], t["token"], t["score"], t["anc_mask"]
    assert n == B
    for v in range(1, n):
        assert 0 <= p[v] < v
        assert d[v] == d[p[v]] + 1 <= N
        assert s[v] <= s[p[v]]
        assert tok[v] in np.argsort(-logp[d[v] - 1], kind="stable")[:W]
    # sibling tokens distinct and in rank order, siblings contiguous
    for v in range(n):
        kids = [u for u in range(n) if p[u] == v]
        assert kids == list(range(kids[0], kids[0] + len(kids))) if kids else True
        assert len({int(tok[u]) for u in kids}) == len(kids)
        lps = [logp[d[v], tok[u]] for u in kids]
        assert lps == sorted(lps, reverse=True)
    # successive pops have non-increasing scores
    ps = [s[v] for v in t["pops"]]
    assert all(a >= b for a, b in zip(ps, ps[1:]))
    # mask rows: popcount = depth + 1; row v = row parent | bit v; intersection = common chain
    for v in range(n):
        bits = [u for u in range(B) if (int(anc[v, u // 32]) >> (u % 32)) & 1]
        assert len(bits) == d[v] + 1 and bits[-1] == v
        assert [int(d[u]) for u in bits] == list(range(d[v] + 1))
        if v:
            assert bits[:-1] == [u for u in range(B) if (int(anc[p[v], u // 32]) >> (u % 32)) & 1]
    # fp32 vs fp64 accumulation agree to rounding
    np.testing.assert_allclose(s[:n], t["score64"][:n], rtol=1e-5, atol=1e-5)


def test_token_relabelling_permutes_tokens_only():
    rng = np.random.default_rng(9)
    N, W, B, V = 4, 4, 16, 256
    logp = make_logp(rng, N, V, 2.0)
    perm = rng.permutation(V)                      # new id of old token t is perm[t]
    logp2 = np.empty_like(logp)
    logp2[:, perm] = logp
    a = tree_build_ref(logp, 5, N, W, B)
    b = tree_build_ref(logp2, 5, N, W, B)
    assert a["parent"].tolist() == b["parent"].tolist()
    assert a["score"].tolist() == b["score"].tolist()
    assert b["token"][1:].tolist() == perm[a["token"][1:]].tolist()


def test_tie_breaks_are_lowest_index():
    # two equal maxima per row: rank order must put the lower token id first;
    # equal node scores: the earlier node pops first.
    logp = np.full((2, 6), -5.0, dtype=np.float32)
    logp[0, [4, 2]] = -1.0
    logp[1, [5, 1]] = -1.0
    t = tree_build_ref(logp, 0, 2, 2, 7)
    assert t["token"].tolist() == [0, 2, 4, 1, 5, 1, 5]
    assert t["parent"].tolist() == [-1, 0, 0, 1, 1, 2, 2]
    # signed zeros compare equal: lower index wins
    z = np.array([[-0.0, 0.0, -1.0]], dtype=np.float32)
    assert tree_build_ref(z, 0, 1, 2, 3)["token"].tolist() == [0, 0, 1]
    z = np.array([[-1.0, 0.0, -0.0]], dtype=np.float32)
    assert tree_build_ref(z, 0, 1, 2, 3)["token"].tolist() == [0, 1, 2]
