"""GPU parity: jet_tree_build_logits (raw draft logits in, log-softmax on the fly) against the oracle's
log_softmax_ref + tree_build_ref.

Every log-probability is a float32 rounding of a float64 difference, and decides integers (the candidates'
ranks, the pop order), so both sides must produce the same float32 values: the library's lse must agree with
the oracle's to the last few bits of the float64 (checked first, on the float32 rounding the library
returns), and then every array is compared bit-exactly.  A different order of the fp64 additions can move a
log-probability only if it lies within ~1e-15 (relative) of a float32 rounding boundary.
"""
import numpy as np
import pytest

from jet_inputs import CONFIGS, make_draft_logits
from oracle import depth_entropy_ref, log_softmax_ref, tree_build_logits_ref

pytestmark = pytest.mark.gpu

MODES = {"accum_logp": 0, "entropy": 1, "hybrid": 2}


def _compare(logits, roots, N, W, B, mode, alpha, node_budget=None):
    import jet_harness as H
    got = H.run_tree_build_logits(logits, roots, N, W, B, MODES[mode], alpha, node_budget=node_budget)
    words = (B + 31) // 32
    for b in range(logits.shape[0]):
        Bb = B if node_budget is None else max(1, min(B, int(node_budget[b])))
        ref = tree_build_logits_ref(logits[b], int(roots[b]), N, W, Bb, score_mode=mode, alpha=alpha)
        assert np.array_equal(got["depth_lse"][b].view(np.uint32), ref["depth_lse"].view(np.uint32)), \
            (b, got["depth_lse"][b], ref["depth_lse"])
        if mode != "accum_logp":
            Href = depth_entropy_ref(log_softmax_ref(logits[b][:N])[0], N)
            assert np.array_equal(got["depth_entropy"][b].view(np.uint32), Href.view(np.uint32)), \
                (b, got["depth_entropy"][b], Href)
        n = ref["n_nodes"]
        assert got["n_nodes"][b] == n, (b, got["n_nodes"][b], n)
        for k in ("parent", "depth", "token"):
            assert np.array_equal(got[k][b][:Bb], ref[k]) and (got[k][b][Bb:] == -1).all(), (b, k)
        assert np.array_equal(got["score"][b][:n].view(np.uint32), ref["score"][:n].view(np.uint32)), b
        anc = np.zeros((B, words), np.uint32)
        anc[:Bb, :ref["anc_mask"].shape[1]] = ref["anc_mask"]
        assert np.array_equal(got["anc_mask"][b], anc), b
    return got


@pytest.mark.parametrize("mode,alpha", [("accum_logp", 0.0), ("entropy", 0.0), ("hybrid", 0.5)])
@pytest.mark.parametrize("seed", range(2))
def test_tiny_config(mode, alpha, seed):
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(1100 + seed)
    z = make_draft_logits(rng, c["N"], c["V"], c["sigma_draft"])[None]
    _compare(z, [5], c["N"], c["W"], c["B"], mode, alpha)


@pytest.mark.parametrize("mode,alpha", [("accum_logp", 0.0), ("entropy", 0.0), ("hybrid", 2.0)])
@pytest.mark.parametrize("peaked,offset", [(None, 0.0), (0.7, 0.0), (0.7, 37.5), (None, -300.0)])
def test_qwen3_8b_config(mode, alpha, peaked, offset):
    c = CONFIGS["qwen3_8b"]
    rng = np.random.default_rng(2100)
    z = make_draft_logits(rng, c["N"], c["V"], c["sigma_draft"], peaked_p=peaked, offset=offset)[None]
    _compare(z, [11], c["N"], c["W"], c["B"], mode, alpha)


@pytest.mark.parametrize("B,N", [(16, 8), (128, 12), (512, 12)])
def test_budget_sweep_full_vocab(B, N):
    rng = np.random.default_rng(3100 + B)
    z = np.stack([make_draft_logits(rng, 1, 151936, 1.0 + 0.5 * d, peaked_p=0.7 if d % 3 == 0 else None,
                                    offset=3.0 * d)[0] for d in range(N)])[None]
    _compare(z, [1], N, 7, B, "hybrid", 1.0)
    _compare(z, [1], N, 7, B, "accum_logp", 0.0)


def test_batched_sequences_with_their_own_budgets():
    rng = np.random.default_rng(4200)
    batch, N, V = 5, 8, 50000
    z = np.stack([make_draft_logits(rng, N, V, 2.0 + b, peaked_p=0.7 if b % 2 else None, offset=-5.0 * b)
                  for b in range(batch)])
    _compare(z, np.arange(batch) + 100, N, 7, 64, "accum_logp", 0.0)
    _compare(z, np.arange(batch) + 100, N, 7, 64, "hybrid", 1.0, node_budget=[64, 3, 40, 1, 100])


@pytest.mark.parametrize("N,W,B,V", [(1, 1, 1, 1), (3, 5, 40, 3), (4, 32, 512, 50), (2, 7, 9, 4097),
                                     (64, 1, 70, 33), (6, 4, 33, 4095), (3, 2, 31, 12289)])
def test_edge_shapes(N, W, B, V):
    rng = np.random.default_rng(N * 1000 + W * 100 + B + 1)
    z = make_draft_logits(rng, N, V, 2.0, offset=1.5)[None]
    _compare(z, [0], N, W, B, "accum_logp", 0.0)
    _compare(z, [0], N, W, B, "hybrid", 0.75)


def test_zero_probability_tokens_and_whole_slices_of_them():
    """-inf logits (probability 0): inside a slice, and filling whole 4096-entry slices."""
    rng = np.random.default_rng(6)
    N, V = 4, 4096 * 3 + 100
    z = make_draft_logits(rng, N, V, 2.0)
    z[:, ::3] = -np.inf
    z[:, 4096:8192] = -np.inf
    _compare(z[None], [2], N, 5, 48, "hybrid", 1.5)
    _compare(z[None], [2], N, 5, 48, "accum_logp", 0.0)


def test_logits_that_collapse_to_one_log_probability():
    """Distinct logits whose log-probabilities round to the same float32: the lower token id ranks first,
    also when the two sit in different slices of the scan and at the cut between rank W and W + 1."""
    V = 4096 * 2 + 64
    z = np.full((1, 2, V), -30.0, np.float32)
    one = np.float32(1.0)
    below = np.nextafter(one, np.float32(0.0))
    z[0, :, 5] = 20.0                          # pushes lse up: log-probabilities near -19 have coarser ulps
    z[0, 0, 5000] = one
    z[0, 0, 10] = below                        # ties with token 5000 after the rounding, lower id, other slice
    z[0, 1, 8000] = one
    z[0, 1, 7000] = below
    z[0, 1, 100] = below
    lp, _ = log_softmax_ref(z[0])
    assert lp[0, 5000] == lp[0, 10] and lp[1, 8000] == lp[1, 100]
    for W in (2, 3, 4):
        _compare(z, [0], 2, W, 12, "accum_logp", 0.0)


def test_unaligned_rows_take_the_scalar_path():
    rng = np.random.default_rng(8)
    N, V = 3, 9001                               # odd V: rows after the first are not 16-byte aligned
    z = make_draft_logits(rng, N, V, 2.5, peaked_p=0.6)[None]
    _compare(z, [3], N, 6, 32, "hybrid", 0.3)


def test_argument_errors():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    N, V, W, B = 2, 100, 3, 8
    z = torch.zeros((1, N, V), dtype=torch.float32, device=H.DEV)
    root = torch.zeros(1, dtype=torch.int32, device=H.DEV)
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(jet.jet_tree_build_logits_workspace_bytes(1, N, V, W))
    args = lambda mode, w: (z, root, 1, N, V, W, B, mode, 0.0, i32(1, B), i32(1, B), i32(1, B), None, i32(1, B, 1),
                            i32(1), None, None, w)
    assert jet.jet_tree_build_logits(*args(3, ws), check=False) == jet.JET_ERR_INVALID_ARG
    small = H.workspace(jet.jet_tree_build_scored_workspace_bytes(1, N, V, W))
    if small.numel() < ws.numel():
        assert jet.jet_tree_build_logits(*args(0, small), check=False) == jet.JET_ERR_WORKSPACE
    assert jet.jet_tree_build_logits(*args(0, ws), check=False) == jet.JET_OK
    torch.cuda.synchronize()
