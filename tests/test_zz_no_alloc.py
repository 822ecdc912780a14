"""jet_tree_accept_static: acceptance without a caller workspace, for callers that cannot allocate
device memory (all of it already handed out, or allocator calls banned on the decode loop).

Collected last on purpose.  The new entry point must give bit-identical results to
jet_tree_accept on two calls in a row; the second call is smaller than the first so that
whatever the first left in the shared built-in scratch would show if it leaked.
"""
import numpy as np
import pytest

from jet_inputs import make_logp, make_target_logits, plant_path
from oracle import tree_accept_ref, tree_build_ref

pytestmark = pytest.mark.gpu


def _case(rng, batch, N, W, B, V):
    trees = [tree_build_ref(make_logp(rng, N, V, 3.0, peaked_p=0.7), 1, N, W, B) for _ in range(batch)]
    stack = lambda k: np.stack([t[k] for t in trees])
    logits = np.stack([make_target_logits(rng, B, V, 2.0) for _ in range(batch)])
    for b, t in enumerate(trees):
        plant_path(logits[b], t["token"], t["parent"], t["depth"], t["n_nodes"], int(rng.integers(0, N + 1)), rng)
    return logits, stack("token"), stack("parent"), stack("depth"), stack("anc_mask"), \
        np.array([t["n_nodes"] for t in trees], dtype=np.int32)


def _run_static(logits, token, parent, depth, anc, n_nodes, N):
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    batch, B, V = logits.shape
    out = {k: torch.full(shape, -7, dtype=torch.int32, device=H.DEV)
           for k, shape in (("tgt", (batch, B)), ("accept_len", (batch,)), ("path", (batch, N + 1)),
                            ("out_tokens", (batch, N + 1)))}
    jet.jet_tree_accept_static(H.dev(logits), V, H.dev(token.astype(np.int32)), H.dev(parent.astype(np.int32)),
                               H.dev(depth.astype(np.int32)), H.dev(anc.view(np.int32)), H.dev(n_nodes), batch, B, V,
                               N, out["tgt"], out["accept_len"], out["path"], out["out_tokens"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    import jet_harness as H
    rng = np.random.default_rng(2024)
    shapes = ((3, 8, 7, 64, 40000), (1, 4, 4, 16, 9000))
    cases = [_case(rng, *shape) for shape in shapes]
    wants = [H.run_tree_accept(*args, shape[1]) for args, shape in zip(cases, shapes)]
    gots = [_run_static(*args, shape[1]) for args, shape in zip(cases, shapes)]     # two calls in a row
    for got, want, shape, args in zip(gots, wants, shapes, cases):
        for k in ("tgt", "accept_len", "path", "out_tokens"):
            assert np.array_equal(got[k], want[k]), (shape, k)
        # and against the CPU oracle itself, sequence by sequence
        logits, token, parent, depth, _, n_nodes = args
        for b in range(shape[0]):
            ref = tree_accept_ref(logits[b], token[b], parent[b], depth[b], int(n_nodes[b]), shape[1])
            assert np.array_equal(got["tgt"][b], ref["tgt"]), (shape, b)
            assert got["accept_len"][b] == ref["accept_len"], (shape, b)
            assert np.array_equal(got["path"][b], ref["path"]), (shape, b)
            assert np.array_equal(got["out_tokens"][b], ref["out_tokens"]), (shape, b)


def test_static_call_leaves_device_memory_as_it_was():
    """What the entry point is for: free device memory is the same before and after the call (inputs and
    outputs are allocated beforehand; the built-in scratch was set aside when the library was loaded)."""
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    rng = np.random.default_rng(5)
    logits, token, parent, depth, anc, n_nodes = _case(rng, 2, 6, 5, 48, 30000)
    batch, B, V = logits.shape
    N = 6
    d = [H.dev(logits), H.dev(token.astype(np.int32)), H.dev(parent.astype(np.int32)),
         H.dev(depth.astype(np.int32)), H.dev(anc.view(np.int32)), H.dev(n_nodes)]
    outs = [torch.full(shape, -7, dtype=torch.int32, device=H.DEV)
            for shape in ((batch, B), (batch,), (batch, N + 1), (batch, N + 1))]
    # first call on this device (address look-up) happens here at the latest
    jet.jet_tree_accept_static(d[0], V, d[1], d[2], d[3], d[4], d[5], batch, B, V, N, *outs)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    reserved_before = torch.cuda.memory_reserved()
    for _ in range(3):
        jet.jet_tree_accept_static(d[0], V, d[1], d[2], d[3], d[4], d[5], batch, B, V, N, *outs)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before and torch.cuda.memory_reserved() == reserved_before
    ref = tree_accept_ref(logits[1], token[1], parent[1], depth[1], int(n_nodes[1]), N)
    assert np.array_equal(outs[2].cpu().numpy()[1], ref["path"])


def test_static_scratch_size_boundary():
    """batch * B * ceil(V / 8192) * 8 bytes == the built-in scratch exactly is accepted (and agrees with the
    workspace call); one more slice per row, or one more sequence, is rejected before anything is launched."""
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    batch, B, N = 64, 512, 4
    V = 3 * 8192 + 1                                   # 4 slices per row: 64 * 512 * 4 * 8 B = 1 MiB
    assert batch * B * 4 * 8 == jet.JET_STATIC_ACCEPT_SCRATCH_BYTES
    logits = torch.zeros((batch * B, V), dtype=torch.float32, device=H.DEV)          # 3.2 GB of zeros
    logits[::B, 77] = 1.0                              # the root rows predict token 77
    i32 = lambda shape, fill: torch.full(shape, fill, dtype=torch.int32, device=H.DEV)
    token, parent, depth = i32((batch, B), -1), i32((batch, B), -1), i32((batch, B), -1)
    token[:, 0], depth[:, 0] = 5, 0
    anc = i32((batch, B, B // 32), 0)
    anc[:, 0, 0] = 1
    n_nodes = i32((batch,), 1)
    res = []
    for static in (True, False):
        outs = [i32((batch, B), -7), i32((batch,), -7), i32((batch, N + 1), -7), i32((batch, N + 1), -7)]
        if static:
            st = jet.jet_tree_accept_static(logits, V, token, parent, depth, anc, n_nodes, batch, B, V, N, *outs,
                                            check=False)
        else:
            ws = H.workspace(jet.jet_tree_accept_workspace_bytes(batch, B, V))
            st = jet.jet_tree_accept(logits, V, token, parent, depth, anc, n_nodes, batch, B, V, N, *outs, ws,
                                     check=False)
        assert st == jet.JET_OK
        torch.cuda.synchronize()
        res.append([o.cpu().numpy() for o in outs])
    for a, b in zip(*res):
        assert np.array_equal(a, b)
    assert (res[0][1] == 0).all() and (res[0][3][:, 0] == 77).all() and (res[0][0][:, 0] == 77).all()
    outs = [i32((batch, B), -7), i32((batch,), -7), i32((batch, N + 1), -7), i32((batch, N + 1), -7)]
    for bad_batch, bad_V in ((batch, 4 * 8192 + 1), (batch + 1, V)):
        st = jet.jet_tree_accept_static(logits, bad_V, token, parent, depth, anc, n_nodes, bad_batch, B, bad_V, N,
                                        *outs, check=False)
        assert st == jet.JET_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert all(bool((o == -7).all()) for o in outs)


def test_static_scratch_rejects_oversized_problems():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    i32 = torch.zeros(8, dtype=torch.int32, device=H.DEV)
    f32 = torch.zeros(8, dtype=torch.float32, device=H.DEV)
    # 128 sequences x 512 nodes x 19 slices x 8 bytes is far beyond the 1 MiB built-in scratch
    st = jet.jet_tree_accept_static(f32, 151936, i32, i32, i32, i32, i32, 128, 512, 151936, 8, i32, i32, i32, i32,
                                    check=False)
    assert st == jet.JET_ERR_WORKSPACE
