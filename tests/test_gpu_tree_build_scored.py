"""GPU parity: jet_tree_build_scored (expansion scores of Appendix C) against the oracle.

The entropy is a float32 value that decides integers (which node is taken next), so both sides must use
the same one: the library's per-depth entropy must equal the oracle's fp64 sum rounded to float32 -- bit for
bit, except that a different order of the fp64 additions may move a sum that lies within 1e-13 (relative)
of a float32 rounding boundary by one ulp; such a case would be reported by the first assertion, and every
array is then compared bit-exactly.
"""
import numpy as np
import pytest

from jet_inputs import CONFIGS, make_logp
from oracle import depth_entropy_ref, tree_build_ref

pytestmark = pytest.mark.gpu

MODES = {"accum_logp": 0, "entropy": 1, "hybrid": 2}


def _compare(logp, roots, N, W, B, mode, alpha):
    import jet_harness as H
    got = H.run_tree_build_scored(logp, roots, N, W, B, MODES[mode], alpha)
    for b in range(logp.shape[0]):
        if mode != "accum_logp":
            Href = depth_entropy_ref(logp[b], N)
            assert np.array_equal(got["depth_entropy"][b].view(np.uint32), Href.view(np.uint32)), \
                (b, got["depth_entropy"][b], Href)
        ref = tree_build_ref(logp[b], int(roots[b]), N, W, B, score_mode=mode, alpha=alpha)
        assert got["n_nodes"][b] == ref["n_nodes"], (b, got["n_nodes"][b], ref["n_nodes"])
        for k in ("parent", "depth", "token"):
            assert np.array_equal(got[k][b], ref[k]), (b, k)
        assert np.array_equal(got["score"][b].view(np.uint32), ref["score"].view(np.uint32)), b
        assert np.array_equal(got["anc_mask"][b], ref["anc_mask"]), b
    return got


@pytest.mark.parametrize("mode,alpha", [("accum_logp", 0.0), ("entropy", 0.0), ("hybrid", 0.25), ("hybrid", 1.0),
                                        ("hybrid", 8.0)])
@pytest.mark.parametrize("seed", range(2))
def test_tiny_config(mode, alpha, seed):
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(1000 + seed)
    logp = make_logp(rng, c["N"], c["V"], c["sigma_draft"])[None]
    _compare(logp, [5], c["N"], c["W"], c["B"], mode, alpha)


@pytest.mark.parametrize("mode,alpha", [("entropy", 0.0), ("hybrid", 0.5), ("hybrid", 4.0)])
@pytest.mark.parametrize("peaked", [None, 0.7])
def test_qwen3_8b_config(mode, alpha, peaked):
    c = CONFIGS["qwen3_8b"]
    rng = np.random.default_rng(2000)
    logp = make_logp(rng, c["N"], c["V"], c["sigma_draft"], peaked_p=peaked)[None]
    _compare(logp, [11], c["N"], c["W"], c["B"], mode, alpha)


@pytest.mark.parametrize("B,N", [(16, 8), (128, 12), (512, 12)])
@pytest.mark.parametrize("mode,alpha", [("entropy", 0.0), ("hybrid", 2.0)])
def test_budget_sweep_full_vocab(B, N, mode, alpha):
    rng = np.random.default_rng(3000 + B)
    # rows of different sharpness, so that the depths' entropies differ and the entropy term matters
    logp = np.stack([make_logp(rng, 1, 151936, 1.0 + 0.5 * d, peaked_p=0.7 if d % 3 == 0 else None)[0]
                     for d in range(N)])[None]
    _compare(logp, [1], N, 7, B, mode, alpha)


def test_batched_sequences_each_own_tree():
    rng = np.random.default_rng(4000)
    batch, N, V = 4, 8, 151936
    logp = np.stack([make_logp(rng, N, V, 2.0 + b, peaked_p=0.7 if b % 2 else None) for b in range(batch)])
    _compare(logp, np.arange(batch) + 100, N, 7, 64, "hybrid", 1.0)
    _compare(logp, np.arange(batch) + 100, N, 7, 64, "entropy", 0.0)


@pytest.mark.parametrize("N,W,B,V", [(1, 1, 1, 1), (3, 5, 40, 3), (4, 32, 512, 50), (2, 7, 9, 4097),
                                     (64, 1, 70, 33), (6, 4, 33, 4095), (3, 2, 31, 12289)])
def test_edge_shapes(N, W, B, V):
    rng = np.random.default_rng(N * 1000 + W * 100 + B)
    logp = make_logp(rng, N, V, 2.0)[None]
    _compare(logp, [0], N, W, B, "hybrid", 0.75)
    _compare(logp, [0], N, W, B, "entropy", 0.0)


def test_hybrid_with_alpha_zero_and_mode_zero_equal_jet_tree_build():
    import jet_harness as H
    rng = np.random.default_rng(77)
    N, W, B, V = 8, 7, 64, 151936
    logp = make_logp(rng, N, V, 3.0, peaked_p=0.7)[None]
    base = H.run_tree_build(logp, [3], N, W, B)
    for mode, alpha in ((0, 0.0), (2, 0.0)):
        got = H.run_tree_build_scored(logp, [3], N, W, B, mode, alpha)
        for k in ("parent", "depth", "token", "anc_mask", "n_nodes"):
            assert np.array_equal(got[k], base[k]), (mode, k)
        assert np.array_equal(got["score"].view(np.uint32), base["score"].view(np.uint32))


def test_rows_with_minus_infinity_entries():
    """Log-probabilities of -inf (zero-probability tokens) contribute nothing to the entropy."""
    rng = np.random.default_rng(5)
    N, V = 4, 9000
    logp = make_logp(rng, N, V, 2.0)
    logp[:, ::3] = -np.inf
    logp = logp - np.log(np.sum(np.exp(logp.astype(np.float64)), axis=1, keepdims=True)).astype(np.float32)
    _compare(logp[None].astype(np.float32), [2], N, 5, 48, "hybrid", 1.5)


def test_argument_errors():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    N, V, W, B = 2, 100, 3, 8
    logp = torch.zeros((1, N, V), dtype=torch.float32, device=H.DEV)
    root = torch.zeros(1, dtype=torch.int32, device=H.DEV)
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(jet.jet_tree_build_scored_workspace_bytes(1, N, V, W))
    args = lambda mode, alpha, w: (logp, root, 1, N, V, W, B, mode, alpha, i32(1, B), i32(1, B), i32(1, B), None,
                                   i32(1, B, 1), i32(1), None, w)
    assert jet.jet_tree_build_scored(*args(3, 0.0, ws), check=False) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_build_scored(*args(-1, 0.0, ws), check=False) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_build_scored(*args(2, float("nan"), ws), check=False) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_build_scored(*args(2, float("inf"), ws), check=False) == jet.JET_ERR_INVALID_ARG
    small = H.workspace(jet.jet_tree_build_workspace_bytes(1, N, V, W))
    if small.numel() < ws.numel():
        assert jet.jet_tree_build_scored(*args(1, 0.0, small), check=False) == jet.JET_ERR_WORKSPACE
    assert jet.jet_tree_build_scored(*args(1, 0.0, ws), check=False) == jet.JET_OK


@pytest.mark.parametrize("mode,alpha", [("accum_logp", 0.0), ("hybrid", 1.0)])
def test_per_sequence_budgets(mode, alpha):
    """Each sequence of a batch with its own budget: the tree equals the oracle's tree for that budget, padded
    to B like any shorter tree (a budget above B counts as B, below 1 as 1)."""
    import jet_harness as H
    rng = np.random.default_rng(4100)
    batch, N, V, W, B = 6, 8, 20000, 7, 128
    budgets = [128, 64, 17, 1, 500, 0]
    logp = np.stack([make_logp(rng, N, V, 3.0, peaked_p=0.7) for _ in range(batch)])
    got = H.run_tree_build_scored(logp, np.arange(batch), N, W, B, MODES[mode], alpha, node_budget=budgets)
    words = (B + 31) // 32
    for b in range(batch):
        Bb = max(1, min(B, budgets[b]))
        ref = tree_build_ref(logp[b], b, N, W, Bb, score_mode=mode, alpha=alpha)
        n = ref["n_nodes"]
        assert got["n_nodes"][b] == n
        for k in ("parent", "depth", "token"):
            assert np.array_equal(got[k][b][:Bb], ref[k]) and (got[k][b][Bb:] == -1).all(), (b, k)
        assert np.array_equal(got["score"][b][:n].view(np.uint32), ref["score"][:n].view(np.uint32))
        anc = np.zeros((B, words), np.uint32)
        anc[:Bb, :ref["anc_mask"].shape[1]] = ref["anc_mask"]
        assert np.array_equal(got["anc_mask"][b], anc), b
