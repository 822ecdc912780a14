"""Pins for the commit oracle (Appendix E: the accepted path is committed)."""
import numpy as np

from jet_inputs import make_attn_inputs, make_paged_cache, random_tree
from oracle import (anc_from_parent, gather_paged_prefix, kv_compact_ref, kv_compact_tail_ref, tree_attn_ref)


def _setup(rng, layers, batch, B, Hkv, D, Lmax):
    tk = rng.integers(0, 1 << 16, size=(layers, batch, B, Hkv, D)).astype(np.uint16)
    tv = rng.integers(0, 1 << 16, size=(layers, batch, B, Hkv, D)).astype(np.uint16)
    kc = rng.integers(0, 1 << 16, size=(layers, batch, Lmax, Hkv, D)).astype(np.uint16)
    vc = rng.integers(0, 1 << 16, size=(layers, batch, Lmax, Hkv, D)).astype(np.uint16)
    return tk, tv, kc, vc


def test_contiguous_rows_land_behind_prefix_and_rest_untouched():
    rng = np.random.default_rng(0)
    layers, batch, B, Hkv, D, Lmax, N = 3, 2, 8, 2, 4, 20, 4
    tk, tv, kc, vc = _setup(rng, layers, batch, B, Hkv, D, Lmax)
    path = np.array([[0, 2, 5, -1, -1], [0, -1, -1, -1, -1]], dtype=np.int32)
    acc = np.array([2, 0], dtype=np.int32)
    seq = np.array([7, 15], dtype=np.int32)
    k2, v2, seq2 = kv_compact_ref(tk, tv, kc, vc, None, path, acc, seq)
    assert seq2.tolist() == [10, 16]
    touched = np.zeros(kc.shape, dtype=bool)
    for l in range(layers):
        for b in range(batch):
            for i in range(acc[b] + 1):
                assert np.array_equal(k2[l, b, seq[b] + i], tk[l, b, path[b, i]])
                assert np.array_equal(v2[l, b, seq[b] + i], tv[l, b, path[b, i]])
                touched[l, b, seq[b] + i] = True
    assert np.array_equal(k2[~touched], kc[~touched]) and np.array_equal(v2[~touched], vc[~touched])
    assert touched.sum() == layers * (3 + 1) * Hkv * D


def test_paged_round_trip_attention_over_new_prefix():
    """Commit, then attend with a one-node tree over the new prefix: equals attention over
    the hand-concatenated [old prefix ; accepted rows]."""
    rng = np.random.default_rng(5)
    B, Hq, Hkv, D, page = 10, 4, 2, 16, 4
    seq = np.array([9, 14], dtype=np.int32)
    N = 4
    kp, vp, table = make_paged_cache(rng, seq, page, Hkv, D, reserve=N + 1)
    trees = [make_attn_inputs(rng, B, Hq, Hkv, D, 0) for _ in range(2)]
    tk = np.stack([t["tree_k"] for t in trees])[None]
    tv = np.stack([t["tree_v"] for t in trees])[None]
    path = np.array([[0, 3, 4, 9, -1], [0, 1, -1, -1, -1]], dtype=np.int32)
    acc = np.array([3, 1], dtype=np.int32)
    k2, v2, seq2 = kv_compact_ref(tk, tv, kp[None], vp[None], table, path, acc, seq)
    assert seq2.tolist() == [13, 16]
    # pages not owned by a written position are untouched
    changed = {int(p) for p in np.nonzero((k2[0] != kp).reshape(kp.shape[0], -1).any(1))[0]}
    owned = {int(table[b, (seq[b] + i) // page]) for b in range(2) for i in range(acc[b] + 1)}
    assert changed <= owned
    one = np.array([[1]], dtype=np.uint32)
    for b in range(2):
        new_k = gather_paged_prefix(k2[0], table[b], seq2[b])
        new_v = gather_paged_prefix(v2[0], table[b], seq2[b])
        old_k = gather_paged_prefix(kp, table[b], seq[b])
        old_v = gather_paged_prefix(vp, table[b], seq[b])
        nodes = path[b, : acc[b] + 1]
        cat_k = np.concatenate([old_k, tk[0, b, nodes]], 0)
        cat_v = np.concatenate([old_v, tv[0, b, nodes]], 0)
        assert np.array_equal(new_k, cat_k) and np.array_equal(new_v, cat_v)
        probe = make_attn_inputs(rng, 1, Hq, Hkv, D, 0)
        a, _ = tree_attn_ref(probe["q"], new_k, new_v, probe["tree_k"], probe["tree_v"], one, 1, 0.25)
        c, _ = tree_attn_ref(probe["q"], cat_k, cat_v, probe["tree_k"], probe["tree_v"], one, 1, 0.25)
        assert np.array_equal(a, c)


def test_chain_commit_equals_extending_the_chain():
    """Attention of a later node over (prefix + committed chain) equals tree attention of that
    node inside the uncommitted chain tree: commit keeps exactly what the mask let it see."""
    rng = np.random.default_rng(7)
    B, Hq, Hkv, D, L = 6, 2, 1, 8, 12
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent = np.array([-1, 0, 1, 2, 2, 4])
    anc = anc_from_parent(parent, B, B)
    full, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, 0.3)
    kc = np.zeros((1, 1, L + 8, Hkv, D), np.uint16); vc = np.zeros_like(kc)
    kc[0, 0, :L] = x["k_prefix"]; vc[0, 0, :L] = x["v_prefix"]
    path = np.array([[0, 1, 2, 4, -1, -1]], dtype=np.int32)
    k2, v2, seq2 = kv_compact_ref(x["tree_k"][None, None], x["tree_v"][None, None], kc, vc, None,
                                  path, np.array([3]), np.array([L]))
    # node 5 (child of 4) as a single-node tree over the committed prefix
    one = np.array([[1]], dtype=np.uint32)
    o, _ = tree_attn_ref(x["q"][5:6], k2[0, 0, : seq2[0]], v2[0, 0, : seq2[0]],
                         x["tree_k"][5:6], x["tree_v"][5:6], one, 1, 0.3)
    np.testing.assert_allclose(o[0], full[5], rtol=1e-12, atol=1e-14)


def test_tail_commit_agrees_with_the_copying_commit():
    """A cache whose rows seq_len .. seq_len + B - 1 hold the tree: committing in place must leave the new
    prefix (positions < new length) exactly as the copying commit from separate tree buffers does; both
    contiguous and paged."""
    rng = np.random.default_rng(9)
    layers, batch, B, Hkv, D, N, page = 2, 3, 12, 2, 8, 5, 4
    seq = np.array([5, 9, 2], dtype=np.int32)
    path = np.array([[0, 2, 5, 11, -1, -1], [0, -1, -1, -1, -1, -1], [0, 1, 2, 3, 4, 5]], dtype=np.int32)
    acc = np.array([3, 0, 5], dtype=np.int32)
    tk = rng.integers(0, 1 << 16, size=(layers, batch, B, Hkv, D)).astype(np.uint16)
    tv = rng.integers(0, 1 << 16, size=(layers, batch, B, Hkv, D)).astype(np.uint16)
    # contiguous
    Lmax = 24
    kc = rng.integers(0, 1 << 16, size=(layers, batch, Lmax, Hkv, D)).astype(np.uint16)
    vc = rng.integers(0, 1 << 16, size=(layers, batch, Lmax, Hkv, D)).astype(np.uint16)
    kt, vt = kc.copy(), vc.copy()
    for b in range(batch):
        kt[:, b, seq[b]:seq[b] + B] = tk[:, b]
        vt[:, b, seq[b]:seq[b] + B] = tv[:, b]
    k_ref, v_ref, len_ref = kv_compact_ref(tk, tv, kc, vc, None, path, acc, seq)
    k_new, v_new, len_new = kv_compact_tail_ref(kt, vt, None, path, acc, seq)
    assert len_new.tolist() == len_ref.tolist()
    for b in range(batch):
        n = int(len_new[b])
        assert np.array_equal(k_new[:, b, :n], k_ref[:, b, :n]) and np.array_equal(v_new[:, b, :n], v_ref[:, b, :n])
        assert np.array_equal(k_new[:, b, seq[b] + B:], kt[:, b, seq[b] + B:])        # nothing behind the tail is touched
    # paged
    need = [(int(L) + B + page - 1) // page for L in seq]
    num_pages = sum(need) + 2
    perm = rng.permutation(num_pages)
    table = np.zeros((batch, max(need)), np.int32)
    pos = 0
    for b, cnt in enumerate(need):
        table[b, :cnt] = perm[pos:pos + cnt]
        pos += cnt
    kp = rng.integers(0, 1 << 16, size=(layers, num_pages, page, Hkv, D)).astype(np.uint16)
    vp = rng.integers(0, 1 << 16, size=(layers, num_pages, page, Hkv, D)).astype(np.uint16)
    kpt, vpt = kp.copy(), vp.copy()
    for b in range(batch):
        for v in range(B):
            j = int(seq[b]) + v
            kpt[:, table[b, j // page], j % page] = tk[:, b, v]
            vpt[:, table[b, j // page], j % page] = tv[:, b, v]
    k_ref, v_ref, _ = kv_compact_ref(tk, tv, kp, vp, table, path, acc, seq)
    k_new, v_new, len_new = kv_compact_tail_ref(kpt, vpt, table, path, acc, seq)
    for b in range(batch):
        for layer in range(layers):
            got = gather_paged_prefix(k_new[layer], table[b], int(len_new[b]))
            ref = gather_paged_prefix(k_ref[layer], table[b], int(len_new[b]))
            assert np.array_equal(got, ref)
            assert np.array_equal(gather_paged_prefix(v_new[layer], table[b], int(len_new[b])),
                                  gather_paged_prefix(v_ref[layer], table[b], int(len_new[b])))
