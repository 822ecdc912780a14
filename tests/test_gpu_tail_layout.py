"""GPU parity for the in-cache tree layout (jet_tree_verify_attn_tail, jet_kv_compact_tail): the tree's
K/V rows sit in the cache behind each prefix.  The attention is compared with the fp64 oracle on the same
prefix and tree (the layout does not change what is computed); the commit is compared bit for bit with
kv_compact_tail_ref.
"""
import numpy as np
import pytest

from jet_inputs import make_attn_inputs, random_tree
from oracle import anc_from_parent, kv_compact_tail_ref, tree_attn_ref

pytestmark = pytest.mark.gpu

MAX_ERR, MEAN_ERR, LSE_ERR = 2e-2, 2e-3, 1e-3
NAN_BITS = np.uint16(0x7FC0)


def _contiguous_case(rng, B, n, Hq, Hkv, D, L, extra=24):
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(n, rng)
    anc = anc_from_parent(parent, n, B)
    rows = L + B + extra
    kc = np.full((1, rows, Hkv, D), NAN_BITS, np.uint16)             # junk wherever nothing valid lives
    vc = np.full_like(kc, NAN_BITS)
    kc[0, :L], vc[0, :L] = x["k_prefix"], x["v_prefix"]
    kc[0, L:L + n], vc[0, L:L + n] = x["tree_k"][:n], x["tree_v"][:n]
    return x, anc, kc, vc, rows


@pytest.mark.parametrize("L", [0, 127, 128, 129, 1000])
@pytest.mark.parametrize("B,n", [(16, 16), (33, 20), (64, 64)])
def test_contiguous_tail_with_early_prefix_reads(L, B, n):
    """JET_ATTN_STABLE_PREFIX in the tail layout: the tiles that hold tree rows (at and behind seq_len) must
    still be read behind the dependency wait; results equal those of the plain call bit for bit."""
    import jet_harness as H
    rng = np.random.default_rng(L * 100 + B)
    Hq, Hkv, D = 8, 2, 128
    x, anc, kc, vc, rows = _contiguous_case(rng, B, n, Hq, Hkv, D, L)
    scale = 1.0 / np.sqrt(D)
    plain, lse_p, st_p = H.run_tree_attn_tail(x["q"][None], kc, vc, None, [L], anc[None], [n], scale, rows, Hkv)
    early, lse_e, st_e = H.run_tree_attn_tail(x["q"][None], kc, vc, None, [L], anc[None], [n], scale, rows, Hkv,
                                              flags=1)
    assert st_p == 0 and st_e == 0
    assert np.array_equal(plain, early) and np.array_equal(lse_p, lse_e)
    ref, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, n, scale)
    err = np.abs(early[0] - ref)
    assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR


@pytest.mark.parametrize("L", [0, 1, 100, 127, 128, 129, 300, 1000])
@pytest.mark.parametrize("B,n", [(1, 1), (16, 16), (33, 20), (64, 64)])
def test_contiguous_tail_against_oracle(L, B, n):
    import jet_harness as H
    rng = np.random.default_rng(L * 100 + B)
    Hq, Hkv, D = 8, 2, 128
    x, anc, kc, vc, rows = _contiguous_case(rng, B, n, Hq, Hkv, D, L)
    scale = 1.0 / np.sqrt(D)
    ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, n, scale)
    out, lse, st = H.run_tree_attn_tail(x["q"][None], kc, vc, None, [L], anc[None], [n], scale, rows, Hkv)
    assert st == 0 and not np.isnan(out).any()
    err = np.abs(out[0] - ref)
    assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR
    assert (out[0, n:] == 0).all()
    assert np.abs(lse[0][:, :n] - rlse[:, :n]).max() <= LSE_ERR


@pytest.mark.parametrize("B,Hq,Hkv,D,L", [(64, 32, 8, 128, 4096), (256, 32, 8, 128, 2000), (128, 32, 4, 128, 777),
                                          (40, 4, 2, 64, 700)])
def test_tail_equals_separate_buffers(B, Hq, Hkv, D, L):
    """Same inputs through both layouts: the outputs agree to the output rounding (the tiles are cut at other
    positions, so the sums are formed in another order) and both meet the oracle's tolerance."""
    import jet_harness as H
    rng = np.random.default_rng(B + L)
    x, anc, kc, vc, rows = _contiguous_case(rng, B, B, Hq, Hkv, D, L)
    scale = 1.0 / np.sqrt(D)
    a, lse_a, st_a = H.run_tree_attn_tail(x["q"][None], kc, vc, None, [L], anc[None], [B], scale, rows, Hkv)
    b, lse_b, st_b = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L],
                                     x["tree_k"][None], x["tree_v"][None], anc[None], [B], scale)
    assert st_a == 0 and st_b == 0
    assert np.abs(a - b).max() <= 2e-2 and np.abs(lse_a - lse_b).max() <= 1e-3
    if B * L <= 64 * 4096:
        ref, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
        err = np.abs(a[0] - ref)
        assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR


def test_batched_paged_ragged_tail():
    import jet_harness as H
    rng = np.random.default_rng(12)
    batch, B, Hq, Hkv, D, page = 5, 48, 8, 2, 128, 16
    seq = np.array([0, 17, 333, 1024, 2047], dtype=np.int32)
    n_nodes = np.array([48, 1, 30, 48, 9], dtype=np.int32)
    need = [(int(L) + B + page - 1) // page for L in seq]
    num_pages = sum(need) + 3
    perm = rng.permutation(num_pages)
    table = np.zeros((batch, max(need)), np.int32)
    pos = 0
    for b, cnt in enumerate(need):
        table[b, :cnt] = perm[pos:pos + cnt]
        pos += cnt
    kp = np.full((num_pages, page, Hkv, D), NAN_BITS, np.uint16)
    vp = np.full_like(kp, NAN_BITS)
    qs, ancs, refs, lses = [], [], [], []
    scale = 1.0 / np.sqrt(D)
    for b in range(batch):
        L, n = int(seq[b]), int(n_nodes[b])
        x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
        parent, _, _ = random_tree(n, rng)
        anc = anc_from_parent(parent, n, B)
        for j in range(L):
            kp[table[b, j // page], j % page] = x["k_prefix"][j]
            vp[table[b, j // page], j % page] = x["v_prefix"][j]
        for v in range(n):
            j = L + v
            kp[table[b, j // page], j % page] = x["tree_k"][v]
            vp[table[b, j // page], j % page] = x["tree_v"][v]
        ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, n, scale)
        qs.append(x["q"]); ancs.append(anc); refs.append(ref); lses.append(rlse)
    out, lse, st = H.run_tree_attn_tail(np.stack(qs), kp, vp, table, seq, np.stack(ancs), n_nodes, scale,
                                        int((seq + B).max()), Hkv)
    assert st == 0 and not np.isnan(out).any()
    for b in range(batch):
        n = int(n_nodes[b])
        err = np.abs(out[b] - refs[b])
        assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR, b
        assert (out[b, n:] == 0).all()
        assert np.abs(lse[b][:, :n] - lses[b][:, :n]).max() <= LSE_ERR


@pytest.mark.parametrize("paged", [False, True])
def test_commit_in_place(paged):
    import jet_harness as H
    rng = np.random.default_rng(31)
    layers, batch, B, Hkv, D, N, page = 3, 4, 64, 8, 128, 8, 16
    seq = np.array([5, 100, 0, 1000], dtype=np.int32)
    path = np.full((batch, N + 1), -1, np.int32)
    path[0, :4] = [0, 2, 5, 63]
    path[1, :1] = [0]
    path[2, :9] = [0, 1, 2, 3, 4, 5, 6, 7, 8]                       # nothing moves
    path[3, :9] = [0, 7, 9, 20, 21, 40, 41, 50, 62]
    acc = np.array([3, 0, 8, 8], dtype=np.int32)
    if not paged:
        Lmax = int(seq.max()) + B + 8
        k = rng.integers(0, 1 << 16, size=(layers, batch, Lmax, Hkv, D)).astype(np.uint16)
        v = rng.integers(0, 1 << 16, size=(layers, batch, Lmax, Hkv, D)).astype(np.uint16)
        table = None
    else:
        need = [(int(L) + B + page - 1) // page for L in seq]
        num_pages = sum(need) + 2
        perm = rng.permutation(num_pages)
        table = np.zeros((batch, max(need)), np.int32)
        pos = 0
        for b, cnt in enumerate(need):
            table[b, :cnt] = perm[pos:pos + cnt]
            pos += cnt
        k = rng.integers(0, 1 << 16, size=(layers, num_pages, page, Hkv, D)).astype(np.uint16)
        v = rng.integers(0, 1 << 16, size=(layers, num_pages, page, Hkv, D)).astype(np.uint16)
    k_ref, v_ref, len_ref = kv_compact_tail_ref(k, v, table, path, acc, seq)
    k_new, v_new, len_new = H.run_kv_compact_tail(k, v, table, path, acc, seq, B)
    assert len_new.tolist() == len_ref.tolist()
    assert np.array_equal(k_new.reshape(k.shape), k_ref) and np.array_equal(v_new.reshape(v.shape), v_ref)


def test_argument_errors():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    B, Hq, Hkv, D, L = 16, 8, 2, 128, 64
    bf = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device=H.DEV)
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=H.DEV)
    ws = torch.zeros(jet.jet_tree_verify_attn_workspace_bytes(1, B, Hq, Hkv, D, L + B), dtype=torch.uint8, device=H.DEV)
    q, k, v, out = bf(1, B, Hq, D), bf(1, L + B, Hkv, D), bf(1, L + B, Hkv, D), bf(1, B, Hq, D)
    call = lambda kk, msl: jet.jet_tree_verify_attn_tail(q, kk, v, None, 0, 0, 0, i32(1), msl, i32(1, B, 1), i32(1), 1, B,
                                                        Hq, Hkv, D, (L + B) * Hkv * D, 0.1, out, None, None, ws,
                                                        check=False)
    assert call(None, L + B) == jet.JET_ERR_INVALID_ARG            # the tail needs a cache
    assert call(k, 0) == jet.JET_ERR_INVALID_ARG
    assert call(k, L + B) == jet.JET_OK
    torch.cuda.synchronize()
