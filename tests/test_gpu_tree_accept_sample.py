"""GPU parity: jet_tree_accept_sample against the oracle.

The accept decisions compare a supplied uniform number with a probability ratio computed in fp32 on the GPU and
in fp64 by the oracle.  So that both sides take every decision the same way, the test first asks the oracle for
the ratios and moves any uniform number that lies within 1e-3 of its threshold away from it; after that the
accepted prefix must match exactly.  The correction token is a draw by inverse CDF: the GPU's token must own the
target mass within the fp32 rounding of the cumulative sums (and equals the oracle's token except at such
boundaries)."""
import numpy as np
import pytest

from jet_inputs import CONFIGS, chain_tree, make_logp, star_tree
from oracle import anc_from_parent, tree_accept_sample_ref, tree_build_ref

pytestmark = pytest.mark.gpu


def _settle(u, alpha, rng):
    """Move uniform numbers away from their thresholds (the decision must not hinge on rounding)."""
    u = u.copy()
    close = np.abs(u - alpha) < 1e-3
    u[close] = np.where(alpha[close] > 0.5, alpha[close] - 0.01, alpha[close] + 0.01)
    return np.clip(u, 0.0, 0.999999).astype(np.float32)


def _check(logits, temperature, logp, token, parent, depth, anc, n_nodes, N, rng):
    import jet_harness as H
    batch, B, V = logits.shape
    u = rng.random((batch, B)).astype(np.float32)
    u_s = rng.random(batch).astype(np.float32)
    for b in range(batch):        # pre-pass: only the thresholds are taken from the oracle
        pre = tree_accept_sample_ref(logits[b], temperature, logp[b], token[b], parent[b], depth[b], int(n_nodes[b]), N,
                                     u[b], u_s[b])
        u[b] = _settle(u[b], pre["alpha"], rng)
    got = H.run_tree_accept_sample(logits, temperature, logp, token, parent, depth, anc, n_nodes, N, u, u_s)
    exact = 0
    for b in range(batch):
        n = int(n_nodes[b])
        ref = tree_accept_sample_ref(logits[b], temperature, logp[b], token[b], parent[b], depth[b], n, N, u[b], u_s[b])
        assert np.allclose(got["alpha"][b, :n], ref["alpha"][:n], rtol=2e-4, atol=1e-6), b
        assert (got["alpha"][b, n:] == 0).all()
        a = ref["accept_len"]
        assert got["accept_len"][b] == a, (b, got["accept_len"][b], a)
        assert np.array_equal(got["path"][b], ref["path"]), b
        assert np.array_equal(got["out_tokens"][b, :a], ref["out_tokens"][:a]), b
        assert (got["out_tokens"][b, a + 1:] == -1).all()
        t = int(got["out_tokens"][b, a])
        cdf, dist = ref["cdf"], ref["dist"]
        target, tol = float(u_s[b]) * cdf[-1], 3e-5 * cdf[-1]
        assert 0 <= t < V and dist[t] > 0, (b, t)
        assert (cdf[t - 1] if t else 0.0) - tol <= target <= cdf[t] + tol, (b, t, ref["correction"])
        exact += int(t == ref["correction"])
    return exact, got


def _built(rng, batch, N, W, B, V, sigma, peaked=0.7):
    logps = [make_logp(rng, N, V, sigma, peaked_p=peaked) for _ in range(batch)]
    trees = [tree_build_ref(lp, 1, N, W, B) for lp in logps]
    stack = lambda k: np.stack([t[k] for t in trees])
    return (np.stack(logps), stack("token"), stack("parent"), stack("depth"), stack("anc_mask"),
            np.array([t["n_nodes"] for t in trees]))


def _target_near_draft(rng, logp, token, parent, depth, n_nodes, B, V, noise):
    """Target logits per node = the draft's log-probs of the node's depth plus noise: ratios p/q of order one."""
    batch, N = logp.shape[0], logp.shape[1]
    out = rng.standard_normal((batch, B, V), dtype=np.float32) * np.float32(noise)
    for b in range(batch):
        for v in range(int(n_nodes[b])):
            d = min(int(depth[b, v]), N - 1)
            out[b, v] += np.maximum(logp[b, d], -30.0)
    return out


@pytest.mark.parametrize("seed", range(3))
def test_tiny_config(seed):
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(7000 + seed)
    logp, token, parent, depth, anc, n = _built(rng, 1, c["N"], c["W"], c["B"], c["V"], c["sigma_draft"])
    logits = _target_near_draft(rng, logp, token, parent, depth, n, c["B"], c["V"], 0.7)
    for temperature in (1.0, 0.6):
        _check(logits, temperature, logp, token, parent, depth, anc, n, c["N"], rng)


def test_qwen3_8b_shape_batch():
    c = CONFIGS["qwen3_8b"]
    rng = np.random.default_rng(7100)
    batch = 4
    logp, token, parent, depth, anc, n = _built(rng, batch, c["N"], c["W"], c["B"], c["V"], c["sigma_draft"])
    logits = _target_near_draft(rng, logp, token, parent, depth, n, c["B"], c["V"], 0.5)
    exact, got = _check(logits, 1.0, logp, token, parent, depth, anc, n, c["N"], rng)
    assert exact >= batch - 1
    assert got["accept_len"].max() >= 1          # the inputs do exercise accepted prefixes


def test_equal_distributions_accept_to_the_leaf_and_draw_from_the_target():
    rng = np.random.default_rng(7200)
    N, V, B = 6, 4096, 7
    logp = make_logp(rng, N, V, 2.0)[None]
    parent, depth, token = chain_tree(B)
    token = np.array([0] + [int(rng.integers(V)) for _ in range(B - 1)], np.int32)
    anc = anc_from_parent(parent, B, B)
    logits = np.zeros((1, B, V), np.float32)
    for v in range(B):
        logits[0, v] = logp[0, min(v, N - 1)]            # p == q at every depth
    exact, got = _check(logits, 1.0, logp, token[None], parent[None], depth[None], anc[None], np.array([B]), N, rng)
    assert got["accept_len"][0] == B - 1 and exact == 1


def test_star_with_every_child_rejected_draws_from_the_residual():
    rng = np.random.default_rng(7300)
    N, V, B = 4, 2048, 9
    logp = make_logp(rng, N, V, 2.0)[None]
    parent, depth, _ = star_tree(B)
    token = np.arange(B, dtype=np.int32) * 3
    anc = anc_from_parent(parent, B, B)
    logits = rng.standard_normal((1, B, V), dtype=np.float32)
    logits[0, 0, token[1:]] = -np.inf                    # the target gives the drafted tokens no mass
    import jet_harness as H
    u = rng.random((1, B)).astype(np.float32)
    u_s = np.array([0.37], np.float32)
    got = H.run_tree_accept_sample(logits, 1.0, logp, token[None], parent[None], depth[None], anc[None], np.array([B]), N,
                                   u, u_s)
    ref = tree_accept_sample_ref(logits[0], 1.0, logp[0], token, parent, depth, B, N, u[0], u_s[0])
    assert got["accept_len"][0] == 0 and ref["accept_len"] == 0 and ref["residual_used"]
    t = int(got["out_tokens"][0, 0])
    assert t not in set(token[1:].tolist()) and ref["dist"][t] > 0
    target, tol = float(u_s[0]) * ref["cdf"][-1], 3e-5 * ref["cdf"][-1]
    assert (ref["cdf"][t - 1] if t else 0.0) - tol <= target <= ref["cdf"][t] + tol


def test_two_siblings_follow_the_per_branch_reading():
    """Branched tree, the documented reading: every sibling is tested on its own, the deepest passing branch wins
    (lowest node index first).  With q == p both siblings always pass and the first one is emitted; the GPU and
    the oracle agree on every draw."""
    import jet_harness as H
    rng = np.random.default_rng(17)
    V, N, B = 4099, 2, 3
    p_logits = (rng.standard_normal(V) * 2.0).astype(np.float32)
    z = p_logits.astype(np.float64)
    logp0 = (z - (z.max() + np.log(np.exp(z - z.max()).sum()))).astype(np.float32)     # q == p at depth 0
    logp = np.stack([logp0, make_logp(rng, 1, V, 2.0)[0]])[None]
    order = np.argsort(-p_logits)
    token = np.array([[7, int(order[1]), int(order[0])]], np.int32)     # two children of the root
    parent = np.array([[-1, 0, 0]], np.int32)
    depth = np.array([[0, 1, 1]], np.int32)
    anc = anc_from_parent(parent[0], B, B)[None]
    logits = np.stack([p_logits, (rng.standard_normal(V) * 2).astype(np.float32),
                       (rng.standard_normal(V) * 2).astype(np.float32)])[None]
    for _ in range(20):
        u = rng.random((1, B)).astype(np.float32) * 0.98
        u_s = rng.random(1).astype(np.float32)
        got = H.run_tree_accept_sample(logits, 1.0, logp, token, parent, depth, anc, np.array([B]), N, u, u_s)
        ref = tree_accept_sample_ref(logits[0], 1.0, logp[0], token[0], parent[0], depth[0], B, N, u[0], u_s[0])
        assert got["accept_len"][0] == ref["accept_len"] == 1
        assert np.array_equal(got["path"][0], ref["path"]) and got["path"][0, 1] == 1
        assert got["out_tokens"][0, 0] == ref["out_tokens"][0] == token[0, 1]


def test_padding_nodes_and_argument_errors():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(7400)
    logp, token, parent, depth, anc, n = _built(rng, 2, c["N"], c["W"], c["B"], c["V"], c["sigma_draft"])
    n = np.array([5, c["B"]])
    for b in range(2):                                    # cut sequence 0 down to 5 nodes
        token[b, n[b]:] = -1; parent[b, n[b]:] = -1; depth[b, n[b]:] = -1; anc[b, n[b]:] = 0
    logits = _target_near_draft(rng, logp, token, parent, depth, n, c["B"], c["V"], 0.7)
    _check(logits, 1.0, logp, token, parent, depth, anc, n, c["N"], rng)
    t = torch.zeros(4096, dtype=torch.float32, device=H.DEV)
    i32 = torch.zeros(64, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(1 << 16)
    args = dict(logits=t, logits_row_stride=64, temperature=1.0, draft_logp=t, logp_batch_stride=256,
                logp_depth_stride=64, token=i32, parent=i32, depth=i32, anc_mask=i32, n_nodes=i32, u_accept=t,
                u_sample=t, batch=1, B=8, V=64, N=4, alpha=None, accept_len=i32, path=i32, out_tokens=i32,
                workspace=ws, check=False)
    assert jet.jet_tree_accept_sample(**{**args, "temperature": 0.0}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_accept_sample(**{**args, "u_sample": None}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_accept_sample(**{**args, "B": 513}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_accept_sample(**{**args, "workspace": None}) == jet.JET_ERR_WORKSPACE
