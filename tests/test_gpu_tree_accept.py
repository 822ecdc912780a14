"""GPU parity: jet_tree_accept against the oracle, bit-exact."""
import numpy as np
import pytest

from jet_inputs import (CONFIGS, chain_tree, make_logp, make_target_logits, plant_path, random_tree,
                        star_tree)
from oracle import anc_from_parent, tree_accept_ref, tree_build_ref

pytestmark = pytest.mark.gpu


def _compare(logits, token, parent, depth, anc, n_nodes, N):
    import jet_harness as H
    got = H.run_tree_accept(logits, token, parent, depth, anc, n_nodes, N)
    for b in range(logits.shape[0]):
        ref = tree_accept_ref(logits[b], token[b], parent[b], depth[b], int(n_nodes[b]), N)
        assert np.array_equal(got["tgt"][b], ref["tgt"]), b
        assert got["accept_len"][b] == ref["accept_len"], (b, got["accept_len"][b], ref["accept_len"])
        assert np.array_equal(got["path"][b], ref["path"]), (b, got["path"][b], ref["path"])
        assert np.array_equal(got["out_tokens"][b], ref["out_tokens"]), b
    return got


def _built(rng, batch, N, W, B, V, sigma, peaked=0.7):
    trees = [tree_build_ref(make_logp(rng, N, V, sigma, peaked_p=peaked), 1, N, W, B) for _ in range(batch)]
    stack = lambda k: np.stack([t[k] for t in trees])
    return stack("token"), stack("parent"), stack("depth"), stack("anc_mask"), np.array([t["n_nodes"] for t in trees])


@pytest.mark.parametrize("seed", range(3))
def test_tiny_config_planted(seed):
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(1000 + seed)
    token, parent, depth, anc, n = _built(rng, 1, c["N"], c["W"], c["B"], c["V"], c["sigma_draft"])
    logits = make_target_logits(rng, c["B"], c["V"], c["sigma_target"])[None]
    end, eff = plant_path(logits[0], token[0], parent[0], depth[0], int(n[0]), c["plant"], rng)
    got = _compare(logits, token, parent, depth, anc, n, c["N"])
    assert got["accept_len"][0] == eff


@pytest.mark.parametrize("plant", [0, 5, 8])
def test_qwen3_8b_config_planted(plant):
    c = CONFIGS["qwen3_8b"]
    rng = np.random.default_rng(2000 + plant)
    token, parent, depth, anc, n = _built(rng, 1, c["N"], c["W"], c["B"], c["V"], c["sigma_draft"])
    logits = make_target_logits(rng, c["B"], c["V"], c["sigma_target"])[None]
    end, eff = plant_path(logits[0], token[0], parent[0], depth[0], int(n[0]), plant, rng)
    got = _compare(logits, token, parent, depth, anc, n, c["N"])
    assert got["accept_len"][0] == eff == min(plant, depth[0].max())


def test_batched_ragged_plants_and_padding():
    rng = np.random.default_rng(4000)
    batch, N, W, B, V = 6, 8, 7, 64, 20011
    token, parent, depth, anc, n = _built(rng, batch, N, W, B, V, 3.0)
    # shrink two trees so that they carry padding rows
    for b, keep in ((1, 40), (4, 1)):
        n[b] = keep
        token[b, keep:] = parent[b, keep:] = depth[b, keep:] = -1
        anc[b, keep:] = 0
    logits = np.stack([make_target_logits(rng, B, V, 2.0) for _ in range(batch)])
    for b in range(batch):
        plant_path(logits[b], token[b], parent[b], depth[b], int(n[b]), int(rng.integers(1, 9)), rng)
    _compare(logits, token, parent, depth, anc, n, N)


@pytest.mark.parametrize("B,V", [(1, 1), (2, 5), (33, 8191), (512, 300), (100, 8193), (31, 16385)])
def test_random_trees_small_vocab_many_matches(B, V):
    rng = np.random.default_rng(B * 7 + V)
    N = 12
    parent, depth, token = random_tree(B, rng, V=min(V, 4), max_depth=N)
    anc = anc_from_parent(parent, B, B)
    logits = make_target_logits(rng, B, V, 1.0)
    logits[:, : min(V, 4)] += 6.0                    # predictions fall in the small token range
    _compare(logits[None], token[None], parent[None], depth[None], anc[None], np.array([B]), N)


def test_argmax_ties_take_lowest_index_across_slices():
    B, V, N = 4, 40000, 3
    parent, depth, token = chain_tree(B)
    logits = np.zeros((1, B, V), dtype=np.float32)             # all equal -> index 0
    logits[0, 1, [39999, 123, 20000]] = 2.0                    # equal maxima in three slices -> 123
    logits[0, 2, [8192, 8191]] = [1.0, 1.0]
    logits[0, 3, :] = -np.inf
    token = np.array([9, 0, 123, 8191], dtype=np.int32)
    anc = anc_from_parent(parent, B, B)
    got = _compare(logits, token[None], parent[None], depth[None], anc[None], np.array([B]), N)
    assert got["tgt"][0].tolist() == [0, 123, 8191, 0]
    assert got["accept_len"][0] == 3


def test_subnormal_logits_are_compared_by_value():
    """The arg-max is an IEEE fp32 compare without flush-to-zero: a subnormal beats +-0 and a more negative
    subnormal loses to -0.0; -0.0 == +0.0 still tie to the lowest index."""
    tiny = np.float32(1e-40)
    assert 0 < tiny < np.finfo(np.float32).tiny
    B, V, N = 6, 20000, 5
    parent, depth, token = chain_tree(B)
    logits = np.zeros((1, B, V), dtype=np.float32)
    logits[0, 0, 15000] = tiny                                  # subnormal > 0: wins over index 0
    logits[0, 1, :] = -tiny
    logits[0, 1, 9000] = -0.0                                   # -0.0 > -1e-40
    logits[0, 2, :] = -0.0
    logits[0, 2, 8200] = 0.0                                    # +0.0 == -0.0: index 0 wins
    logits[0, 3, :] = -2 * tiny
    logits[0, 3, [17000, 300]] = -tiny                          # equal subnormal maxima in two slices -> 300
    logits[0, 4, :] = -np.inf
    logits[0, 4, 19999] = -np.finfo(np.float32).max
    logits[0, 5, [1, 2]] = [tiny, 2 * tiny]
    token = np.array([1, 15000, 9000, 0, 300, 19999], dtype=np.int32)
    anc = anc_from_parent(parent, B, B)
    got = _compare(logits, token[None], parent[None], depth[None], anc[None], np.array([B]), N)
    assert got["tgt"][0].tolist() == [15000, 9000, 0, 300, 19999, 2]
    assert got["accept_len"][0] == 5


def test_star_and_duplicate_sibling_tokens():
    B, V, N = 9, 50, 2
    parent, depth, token = star_tree(B)
    token = np.array([0, 7, 7, 7, 3, 3, 1, 2, 4], dtype=np.int32)
    logits = make_target_logits(np.random.default_rng(1), B, V, 1.0)
    logits[0, 7] = 50.0
    anc = anc_from_parent(parent, B, B)
    got = _compare(logits[None], token[None], parent[None], depth[None], anc[None], np.array([B]), N)
    assert got["path"][0].tolist() == [0, 1, -1]


def test_tree_arrays_that_are_not_a_tree_stay_inside_the_outputs():
    """The tree arrays are the caller's and are not validated.  Whatever they hold -- depths outside 0 .. N, parents
    outside the tree, node counts beyond the budget, arbitrary mask bits -- every store of the call must stay inside
    its output tensors (sentinel margins around them are checked) and the call must end without an error."""
    import jet_harness as H
    rng = np.random.default_rng(77)
    batch, B, V, N = 3, 70, 1000, 6
    logits = rng.standard_normal((batch, B, V)).astype(np.float32)
    token = rng.integers(-5, V + 5, size=(batch, B)).astype(np.int32)
    parent = rng.integers(-5, 2 * B, size=(batch, B)).astype(np.int32)
    depth = rng.integers(-1000, 1000, size=(batch, B)).astype(np.int32)
    anc = rng.integers(0, 2 ** 32, size=(batch, B, (B + 31) // 32), dtype=np.uint64).astype(np.uint32)
    n_nodes = np.array([B + 100, B, 1], np.int32)
    got = H.run_tree_accept(logits, token, parent, depth, anc, n_nodes, N)       # checks the margins
    assert ((got["accept_len"] >= 0) & (got["accept_len"] <= N)).all()
    u = rng.random((batch, B)).astype(np.float32)
    logp = np.log(np.full((batch, N, V), 1.0 / V, np.float32))
    got = H.run_tree_accept_sample(logits, 1.0, logp, token, parent, depth, anc, np.minimum(n_nodes, B), N, u,
                                   rng.random(batch).astype(np.float32))
    assert ((got["accept_len"] >= 0) & (got["accept_len"] <= N)).all()
