"""GPU parity: jet_tree_accept_hidden (LM head inside the acceptance call, arg-max only) against the oracle.

The GPU forms each logit in fp32 on the tensor cores, in an order of its own; the oracle forms it in fp64.  So
the test does not ask for the oracle's arg-max outright: the GPU's token must be the oracle's wherever the
oracle's best logit leads the runner-up by more than the worst-case rounding of a d-term fp32 sum
(d * 2^-24 * sum_k |hidden * weight| of the two candidates), and otherwise it must be one of the tokens that
are within that bound of the best (a complete validity check).  After that the path selection is exact: it is
replayed through the oracle's acceptance on the GPU's own predictions.
"""
import numpy as np
import pytest

from jet_inputs import f32_to_bf16_bits, make_logp, random_tree
from oracle import anc_from_parent, lm_head_argmax_ref, tree_build_ref

pytestmark = pytest.mark.gpu


def _run(hidden_bits, weight_bits, token, parent, depth, anc, n_nodes, N):
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    batch, B = token.shape
    V, d = weight_bits.shape
    tgt = H.guarded_full((batch, B), -7, torch.int32)
    acc = H.guarded_full((batch,), -7, torch.int32)
    path = H.guarded_full((batch, N + 1), -7, torch.int32)
    toks = H.guarded_full((batch, N + 1), -7, torch.int32)
    status = H.guarded_full((1,), 0, torch.int32)
    ws = torch.full((max(jet.jet_tree_accept_hidden_workspace_bytes(batch, B), 256),), 0xCD, dtype=torch.uint8, device=H.DEV)
    jet.jet_tree_accept_hidden(H.dev_bf16(hidden_bits), H.dev_bf16(weight_bits), d, H.dev(token.astype(np.int32)),
                               H.dev(parent.astype(np.int32)), H.dev(depth.astype(np.int32)), H.dev(anc.view(np.int32)),
                               H.dev(np.asarray(n_nodes, dtype=np.int32)), batch, B, V, N, tgt, acc, path, toks, status, ws)
    H.check_guards()
    assert int(status.item()) == 0
    return dict(tgt=tgt.cpu().numpy(), accept_len=acc.cpu().numpy(), path=path.cpu().numpy(), out_tokens=toks.cpu().numpy())


def _check_predictions(got_tgt, ref, n_live_rows, d):
    logits, abs_dot = ref["logits"], ref["abs_dot"]
    exact = 0
    for r in n_live_rows:
        t = int(got_tgt[r])
        best = int(ref["tgt"][r])
        assert 0 <= t < logits.shape[1], (r, t)
        bound = d * 2.0 ** -24 * max(abs_dot[r, t], abs_dot[r, best])
        if t == best:
            exact += 1
            continue
        # a different token is only acceptable if the exact logits are closer than an fp32 sum can resolve
        assert logits[r, best] - logits[r, t] <= 2 * bound, (r, t, best, logits[r, best] - logits[r, t], bound)
        assert t > best or logits[r, t] >= logits[r, best] - 2 * bound
    return exact


def _replay_accept(tgt, token, parent, depth, n, N):
    """The oracle's greedy path selection fed with given predictions (one-hot logits reproduce them exactly)."""
    from oracle import tree_accept_ref
    B = len(token)
    V = int(max(tgt.max(), token.max())) + 2
    logits = np.zeros((B, V), dtype=np.float32)
    for v in range(n):
        logits[v, int(tgt[v])] = 1.0
    return tree_accept_ref(logits, token, parent, depth, n, N)


@pytest.mark.parametrize("rows_case", ["qwen3_8b", "small_vocab_ragged", "two_row_groups", "three_row_groups"])
def test_predictions_and_paths(rows_case):
    rng = np.random.default_rng({"qwen3_8b": 1, "small_vocab_ragged": 2, "two_row_groups": 3, "three_row_groups": 4}[rows_case])
    if rows_case == "qwen3_8b":
        batch, B, N, d, V = 1, 64, 8, 4096, 151936        # the headline step's acceptance: 64 rows, full vocabulary
    elif rows_case == "small_vocab_ragged":
        batch, B, N, d, V = 3, 20, 5, 192, 1000           # vocabulary that ends inside a 128-entry tile; padding nodes
    elif rows_case == "two_row_groups":
        batch, B, N, d, V = 2, 100, 6, 256, 4099          # 200 rows: two 128-row groups share every weight tile
    else:
        batch, B, N, d, V = 5, 128, 6, 128, 777           # 640 rows: more than one CTA row group
    hidden = f32_to_bf16_bits(rng.standard_normal((batch * B, d), dtype=np.float32))
    weight = f32_to_bf16_bits(rng.standard_normal((V, d), dtype=np.float32) * np.float32(0.02))
    ref = lm_head_argmax_ref(hidden, weight)
    # trees whose tokens follow the oracle's predictions along one planted path per sequence
    token = np.full((batch, B), -1, np.int32); parent = np.full((batch, B), -1, np.int32); depth = np.full((batch, B), -1, np.int32)
    n_nodes = np.full(batch, B, np.int32)
    if rows_case == "small_vocab_ragged":
        n_nodes[:] = [20, 7, 1]
    ancs = []
    for b in range(batch):
        n = int(n_nodes[b])
        p, dep, tok = random_tree(n, rng, V=V, max_depth=N)
        parent[b, :n], depth[b, :n], token[b, :n] = p, dep, tok
        leaf = int(rng.integers(0, n))
        chain = []
        u = leaf
        while u > 0:
            chain.append(u)
            u = int(p[u])
        for u in chain:                                    # every node on the path carries its parent's prediction
            token[b, u] = ref["tgt"][b * B + int(p[u])]
        ancs.append(anc_from_parent(p, n, B))
    anc = np.stack(ancs)
    if rows_case == "small_vocab_ragged":                  # rows of padding nodes hold junk
        for b in range(batch):
            hidden[b * B + n_nodes[b]:(b + 1) * B] = 0x7FC0
    got = _run(hidden, weight, token, parent, depth, anc, n_nodes, N)
    live = [b * B + v for b in range(batch) for v in range(int(n_nodes[b]))]
    exact = _check_predictions(got["tgt"].reshape(-1), ref, live, d)
    assert exact >= 0.99 * len(live)                       # near-ties are rare with these inputs
    for b in range(batch):
        n = int(n_nodes[b])
        assert (got["tgt"][b, n:] == -1).all()
        want = _replay_accept(got["tgt"][b], token[b], parent[b], depth[b], n, N)
        assert got["accept_len"][b] == want["accept_len"], b
        assert np.array_equal(got["path"][b], want["path"]), b
        assert np.array_equal(got["out_tokens"][b], want["out_tokens"]), b


def test_exact_ties_and_signed_zero_take_the_lowest_token():
    """Integer-valued inputs: every product and every partial sum is exact in fp32, so ties are real ties and
    the lowest token id must win, also across 128-entry tiles and for rows that are all zero (-0.0 == +0.0)."""
    rng = np.random.default_rng(9)
    B, N, d, V = 8, 3, 64, 700
    h = rng.integers(-2, 3, size=(B, d)).astype(np.float32)
    w = rng.integers(-2, 3, size=(V, d)).astype(np.float32)
    w[650] = w[5]                                           # the same row twice, in different tiles
    w[300] = w[5]
    h[3] = 0.0                                              # every logit is +-0: token 0
    h[4] = -0.0
    ref = lm_head_argmax_ref(f32_to_bf16_bits(h), f32_to_bf16_bits(w))
    parent, depth, token = random_tree(B, rng, V=V, max_depth=N)
    anc = anc_from_parent(parent, B, B)
    got = _run(f32_to_bf16_bits(h), f32_to_bf16_bits(w), token[None], parent[None], depth[None], anc[None], [B], N)
    assert np.array_equal(got["tgt"][0], ref["tgt"])
    assert got["tgt"][0, 3] == 0 and got["tgt"][0, 4] == 0


def test_argument_errors():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    t = torch.zeros(1 << 16, dtype=torch.bfloat16, device=H.DEV)
    i32 = torch.zeros(64, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(4096)
    args = dict(hidden=t, lm_head_weight=t, d=128, token=i32, parent=i32, depth=i32, anc_mask=i32, n_nodes=i32, batch=1,
                B=8, V=100, N=4, tgt_argmax=i32, accept_len=i32, path=i32, out_tokens=i32, device_status=None,
                workspace=ws, check=False)
    assert jet.jet_tree_accept_hidden(**{**args, "d": 100}) == jet.JET_ERR_UNSUPPORTED
    assert jet.jet_tree_accept_hidden(**{**args, "hidden": None}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_accept_hidden(**{**args, "B": 513}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_accept_hidden(**{**args, "workspace": None}) == jet.JET_ERR_WORKSPACE
    assert jet.jet_tree_accept_hidden(**{**args, "workspace_bytes": 8}) == jet.JET_ERR_WORKSPACE
