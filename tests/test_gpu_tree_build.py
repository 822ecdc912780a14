"""GPU parity: jet_tree_build against the oracle, bit-exact on every output array."""
import numpy as np
import pytest

from jet_inputs import CONFIGS, make_logp
from oracle import tree_build_ref

pytestmark = pytest.mark.gpu


def _compare(logp, roots, N, W, B):
    import jet_harness as H
    got = H.run_tree_build(logp, roots, N, W, B)
    for b in range(logp.shape[0]):
        ref = tree_build_ref(logp[b], int(roots[b]), N, W, B)
        assert got["n_nodes"][b] == ref["n_nodes"], (b, got["n_nodes"][b], ref["n_nodes"])
        for k in ("parent", "depth", "token"):
            assert np.array_equal(got[k][b], ref[k]), (b, k)
        assert np.array_equal(got["score"][b].view(np.uint32), ref["score"].view(np.uint32)), b
        assert np.array_equal(got["anc_mask"][b], ref["anc_mask"]), b


@pytest.mark.parametrize("seed", range(3))
def test_tiny_config(seed):
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(1000 + seed)
    logp = make_logp(rng, c["N"], c["V"], c["sigma_draft"])[None]
    _compare(logp, [5], c["N"], c["W"], c["B"])


@pytest.mark.parametrize("peaked", [None, 0.7])
def test_qwen3_8b_config(peaked):
    c = CONFIGS["qwen3_8b"]
    rng = np.random.default_rng(2000)
    logp = make_logp(rng, c["N"], c["V"], c["sigma_draft"], peaked_p=peaked)[None]
    _compare(logp, [11], c["N"], c["W"], c["B"])


@pytest.mark.parametrize("B,N", [(16, 8), (32, 8), (128, 12), (256, 12), (512, 12)])
def test_budget_sweep_full_vocab(B, N):
    rng = np.random.default_rng(3000 + B)
    logp = make_logp(rng, N, 151936, 3.0, peaked_p=0.7)[None]
    _compare(logp, [1], N, 7, B)


def test_batched_sequences_each_own_tree():
    rng = np.random.default_rng(4000)
    batch, N, V = 5, 8, 151936
    logp = np.stack([make_logp(rng, N, V, 3.0, peaked_p=0.7 if b % 2 else None) for b in range(batch)])
    _compare(logp, np.arange(batch) + 100, N, 7, 64)


@pytest.mark.parametrize("N,W,B,V", [(1, 1, 1, 1), (3, 5, 40, 3), (4, 32, 512, 50), (2, 7, 9, 4097),
                                     (64, 1, 70, 33), (5, 3, 2, 8192), (6, 4, 33, 4095), (3, 2, 31, 12289)])
def test_edge_shapes(N, W, B, V):
    rng = np.random.default_rng(N * 1000 + W * 100 + B)
    logp = make_logp(rng, N, V, 2.0)[None]
    _compare(logp, [0], N, W, B)


def test_ties_signed_zero_and_minus_inf():
    logp = np.full((1, 3, 9000), -5.0, dtype=np.float32)
    logp[0, 0, [8000, 17, 4500]] = -1.0           # three equal maxima in different slices
    logp[0, 1, [3, 2]] = [-0.0, 0.0]
    logp[0, 2, :] = -np.inf
    logp[0, 2, 8999] = -2.0
    _compare(logp, [0], 3, 3, 30)
    flat = np.zeros((1, 2, 100), dtype=np.float32)  # every score ties: pops go by node index
    _compare(flat, [0], 2, 4, 19)


def test_subnormal_log_probabilities_are_not_flushed():
    """IEEE fp32 without flush-to-zero: a subnormal increment under a zero parent score stays subnormal in
    `score`, and subnormals rank among each other and against +-0 by value."""
    tiny = np.float32(1e-40)                                  # subnormal (smallest normal is 1.18e-38)
    assert tiny > 0 and tiny < np.finfo(np.float32).tiny
    N, V, W, B = 3, 9000, 4, 40
    logp = np.full((1, N, V), -3.0, dtype=np.float32)
    # depth 0: four candidates -1e-40 < -0.0 == +0.0 ... ranked by value, ties to the lowest id
    logp[0, 0, [8500, 40, 4100, 7]] = [-tiny, -0.0, 0.0, -2 * tiny]
    # depth 1: subnormals in different 4096-entry slices, and a value one ulp below the largest
    logp[0, 1, [5, 4097, 8999]] = [-3 * tiny, -tiny, -2 * tiny]
    logp[0, 2, [100, 200]] = [-tiny, -tiny]                   # equal subnormals: lowest id first
    ref = tree_build_ref(logp[0], 0, N, W, B)
    assert ref["token"][1:5].tolist() == [40, 4100, 8500, 7]
    assert (np.abs(ref["score"][1:ref["n_nodes"]]) < np.finfo(np.float32).tiny).any()   # the oracle keeps subnormals
    _compare(logp, [0], N, W, B)
    # a subnormal against a normal neighbour: the sum must round as IEEE does, not from a flushed operand
    logp2 = np.full((1, 2, 64), -np.inf, dtype=np.float32)
    logp2[0, 0, :3] = [-np.finfo(np.float32).tiny, -tiny, -5.0]
    logp2[0, 1, :3] = [-tiny, -np.finfo(np.float32).tiny * np.float32(0.5), -1.0]
    _compare(logp2, [1], 2, 3, 13)


def test_unaligned_rows_take_the_scalar_path():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    rng = np.random.default_rng(77)
    N, V, W, B = 4, 5001, 5, 20
    logp = make_logp(rng, N, V, 2.0)
    flat = torch.zeros(N * V + 1, dtype=torch.float32, device=H.DEV)
    flat[1:] = torch.from_numpy(logp.reshape(-1)).to(H.DEV)
    view = flat[1:]                                  # 4-byte aligned only
    words = 1
    parent = torch.zeros((1, B), dtype=torch.int32, device=H.DEV)
    depth, token = torch.zeros_like(parent), torch.zeros_like(parent)
    anc = torch.zeros((1, B, words), dtype=torch.int32, device=H.DEV)
    n_nodes = torch.zeros(1, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(jet.jet_tree_build_workspace_bytes(1, N, V, W))
    jet.jet_tree_build(view, H.dev(np.array([3], np.int32)), 1, N, V, W, B, parent, depth, token, None, anc,
                       n_nodes, ws, logp_batch_stride=N * V, logp_depth_stride=V)
    torch.cuda.synchronize()
    ref = tree_build_ref(logp, 3, N, W, B)
    assert np.array_equal(parent.cpu().numpy()[0], ref["parent"])
    assert np.array_equal(token.cpu().numpy()[0], ref["token"])


def test_argument_errors_are_reported_before_launch():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    logp = torch.zeros((1, 2, 16), device=H.DEV)
    i32 = lambda *s: torch.full(s, -9, dtype=torch.int32, device=H.DEV)
    parent, depth, token, anc, n = i32(1, 4), i32(1, 4), i32(1, 4), i32(1, 4, 1), i32(1)
    ws = H.workspace(1024)
    root = i32(1)
    bad = jet.jet_tree_build(logp, root, 1, 2, 16, 2, 0, parent, depth, token, None, anc, n, ws, check=False)
    assert bad == jet.JET_ERR_INVALID_ARG
    bad = jet.jet_tree_build(logp, root, 1, 2, 16, 33, 4, parent, depth, token, None, anc, n, ws, check=False)
    assert bad == jet.JET_ERR_INVALID_ARG
    bad = jet.jet_tree_build(logp, root, 1, 2, 16, 2, 4, parent, depth, token, None, anc, n, ws,
                             workspace_bytes=8, check=False)
    assert bad == jet.JET_ERR_WORKSPACE
    bad = jet.jet_tree_build(logp, None, 1, 2, 16, 2, 4, parent, depth, token, None, anc, n, ws, check=False)
    assert bad == jet.JET_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert (parent == -9).all() and (n == -9).all()
