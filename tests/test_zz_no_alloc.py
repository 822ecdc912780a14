"""jet_tree_accept_static: acceptance without a caller workspace, for callers that cannot allocate
device memory (all of it already handed out, or allocator calls banned on the decode loop).

Collected last on purpose.  The new entry point must give bit-identical results to
jet_tree_accept on two calls in a row; the second call is smaller than the first so that
whatever the first left in the shared built-in scratch would show if it leaked.
"""
import numpy as np
import pytest

from jet_inputs import make_logp, make_target_logits, plant_path
from oracle import tree_build_ref

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
    for got, want, shape in zip(gots, wants, shapes):
        for k in ("tgt", "accept_len", "path", "out_tokens"):
            assert np.array_equal(got[k], want[k]), (shape, k)


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
