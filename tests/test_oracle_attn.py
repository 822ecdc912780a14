"""Pins for the tree-attention oracle (mask and attention equations of Section 3.2).

Checked against: a hand-worked example, torch's CPU scaled_dot_product_attention
in fp64 for the chain (= causal) and single-node (= decode) special cases, and
properties the definition fixes (masked nodes have no influence, convexity,
uniform values, log-sum-exp, relabelling).
"""
import json
import os

import numpy as np
import pytest
import torch

from jet_inputs import binary_tree, chain_tree, make_attn_inputs, random_tree, star_tree
from oracle import anc_from_parent, bf16_bits_to_f64, tree_attn_ref, tree_attn_rows_ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _inputs(seed, B, Hq, Hkv, D, L):
    return make_attn_inputs(np.random.default_rng(seed), B, Hq, Hkv, D, L)


def test_handworked_example():
    g = json.load(open(os.path.join(GOLDEN, "tree_attn_handworked.json")))
    B = 3
    q = np.array(g["q"]).reshape(B, 1, 1)
    kp = np.log(np.array(g["prefix_weight"])).reshape(-1, 1, 1)
    vp = np.array(g["prefix_v"]).reshape(-1, 1, 1)
    kt = np.log(np.array(g["tree_weight"])).reshape(B, 1, 1)
    vt = np.array(g["tree_v"]).reshape(B, 1, 1)
    anc = anc_from_parent(g["parent"], B, B)
    out, lse = tree_attn_ref(q, kp, vp, kt, vt, anc, B, 1.0)
    np.testing.assert_allclose(out[:, 0, 0], g["out"], rtol=1e-13)
    np.testing.assert_allclose(np.exp(lse[0]), g["sum_weights"], rtol=1e-13)
    rows = [(v, 0) for v in range(B)]
    o2, l2 = tree_attn_rows_ref(q, kp, vp, kt, vt, anc, B, 1.0, rows)
    np.testing.assert_allclose(o2[:, 0], g["out"], rtol=1e-13)


def _sdpa(q, k, v, mask, scale):
    """torch CPU fp64: q [H,Tq,D], k/v [H,Tk,D], boolean mask [Tq,Tk] (True = visible)."""
    return torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None],
        attn_mask=torch.from_numpy(mask), scale=scale)[0].numpy()


@pytest.mark.parametrize("L", [0, 1, 37])
def test_chain_tree_is_causal_attention(L):
    B, Hq, Hkv, D = 9, 4, 2, 16
    x = _inputs(11 + L, B, Hq, Hkv, D, L)
    parent, _, _ = chain_tree(B)
    anc = anc_from_parent(parent, B, B)
    scale = 1.0 / np.sqrt(D)
    out, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
    # textbook: causal attention of the last B positions of a length L+B sequence
    G = Hq // Hkv
    k_all = np.concatenate([bf16_bits_to_f64(x["k_prefix"]), bf16_bits_to_f64(x["tree_k"])], 0)
    v_all = np.concatenate([bf16_bits_to_f64(x["v_prefix"]), bf16_bits_to_f64(x["tree_v"])], 0)
    k_h = np.repeat(k_all.transpose(1, 0, 2), G, axis=0)      # [Hq, L+B, D], contiguous GQA groups
    v_h = np.repeat(v_all.transpose(1, 0, 2), G, axis=0)
    q_h = bf16_bits_to_f64(x["q"]).transpose(1, 0, 2).copy()  # [Hq, B, D]
    causal = np.tril(np.ones((L + B, L + B), dtype=bool))[L:]
    ref = _sdpa(q_h, k_h, v_h, causal, scale).transpose(1, 0, 2)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)


def test_single_node_tree_is_decode_attention():
    Hq, Hkv, D, L = 8, 2, 64, 100
    x = _inputs(5, 1, Hq, Hkv, D, L)
    anc = np.array([[1]], dtype=np.uint32)
    scale = 1.0 / np.sqrt(D)
    out, lse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, 1, scale)
    G = Hq // Hkv
    k_all = np.concatenate([bf16_bits_to_f64(x["k_prefix"]), bf16_bits_to_f64(x["tree_k"])], 0)
    v_all = np.concatenate([bf16_bits_to_f64(x["v_prefix"]), bf16_bits_to_f64(x["tree_v"])], 0)
    q = bf16_bits_to_f64(x["q"])
    for h in range(Hq):
        g = h // G
        s = (k_all[:, g] @ q[0, h]) * scale
        w = np.exp(s - s.max())
        w /= w.sum()
        np.testing.assert_allclose(out[0, h], w @ v_all[:, g], rtol=1e-12)
        np.testing.assert_allclose(lse[h, 0], np.log(np.exp(s).sum()), rtol=1e-12)


def test_general_tree_against_dense_mask_sdpa():
    B, Hq, Hkv, D, L = 21, 6, 3, 32, 50
    rng = np.random.default_rng(21)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(B, rng)
    anc = anc_from_parent(parent, B, B)
    scale = 0.3
    out, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
    # dense visibility matrix built by walking ancestors (independent of the bitmask)
    vis = np.zeros((B, L + B), dtype=bool)
    vis[:, :L] = True
    for v in range(B):
        u = v
        while u != -1:
            vis[v, L + u] = True
            u = parent[u]
    G = Hq // Hkv
    k_all = np.concatenate([bf16_bits_to_f64(x["k_prefix"]), bf16_bits_to_f64(x["tree_k"])], 0)
    v_all = np.concatenate([bf16_bits_to_f64(x["v_prefix"]), bf16_bits_to_f64(x["tree_v"])], 0)
    ref = _sdpa(bf16_bits_to_f64(x["q"]).transpose(1, 0, 2).copy(),
                np.repeat(k_all.transpose(1, 0, 2), G, axis=0),
                np.repeat(v_all.transpose(1, 0, 2), G, axis=0), vis, scale).transpose(1, 0, 2)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)


def test_masked_nodes_have_zero_influence():
    B, Hq, Hkv, D, L = 15, 4, 2, 16, 20
    x = _inputs(3, B, Hq, Hkv, D, L)
    parent, _, _ = binary_tree(B)
    anc = anc_from_parent(parent, B, B)
    base, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, 0.25)
    for v in (0, 4, 9, 14):
        k2 = bf16_bits_to_f64(x["tree_k"]).copy()
        v2 = bf16_bits_to_f64(x["tree_v"]).copy()
        for u in range(B):
            if not (int(anc[v, 0]) >> u) & 1:
                k2[u] = 1e4
                v2[u] = -7e5
        out, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], k2, v2, anc, B, 0.25)
        assert np.array_equal(out[v], base[v])


def test_star_children_see_prefix_root_self_only():
    B, Hq, Hkv, D, L = 6, 2, 1, 8, 5
    x = _inputs(8, B, Hq, Hkv, D, L)
    parent, _, _ = star_tree(B)
    anc = anc_from_parent(parent, B, B)
    out, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, 0.5)
    q = bf16_bits_to_f64(x["q"])
    kt, vt = bf16_bits_to_f64(x["tree_k"]), bf16_bits_to_f64(x["tree_v"])
    kp, vp = bf16_bits_to_f64(x["k_prefix"]), bf16_bits_to_f64(x["v_prefix"])
    for v in range(1, B):
        keys = np.concatenate([kp[:, 0], kt[[0, v], 0]])
        vals = np.concatenate([vp[:, 0], vt[[0, v], 0]])
        for h in range(Hq):
            s = 0.5 * keys @ q[v, h]
            w = np.exp(s - s.max())
            np.testing.assert_allclose(out[v, h], (w / w.sum()) @ vals, rtol=1e-12)


def test_uniform_values_and_convexity():
    B, Hq, Hkv, D, L = 10, 4, 4, 8, 30
    rng = np.random.default_rng(4)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(B, rng)
    anc = anc_from_parent(parent, B, B)
    c = np.linspace(-2, 2, D)
    vp = np.broadcast_to(c, (L, Hkv, D)).copy()
    vt = np.broadcast_to(c, (B, Hkv, D)).copy()
    out, _ = tree_attn_ref(x["q"], x["k_prefix"], vp, x["tree_k"], vt, anc, B, 0.35)
    np.testing.assert_allclose(out, np.broadcast_to(c, out.shape), rtol=0, atol=1e-14)
    out, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, 0.35)
    vals = np.concatenate([bf16_bits_to_f64(x["v_prefix"]), bf16_bits_to_f64(x["tree_v"])], 0)
    assert (out <= vals.max() + 1e-12).all() and (out >= vals.min() - 1e-12).all()


def test_padding_rows_and_row_subset():
    B, Hq, Hkv, D, L = 12, 4, 2, 16, 33
    rng = np.random.default_rng(6)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    n = 9
    parent, _, _ = random_tree(n, rng)
    anc = anc_from_parent(parent, n, B)
    out, lse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, n, 0.25)
    assert (out[n:] == 0).all() and np.isneginf(lse[:, n:]).all()
    rows = [(v, h) for v in range(B) for h in range(Hq)]
    o2, l2 = tree_attn_rows_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"],
                                anc, n, 0.25, rows)
    np.testing.assert_allclose(o2.reshape(B, Hq, D), out, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(l2.reshape(B, Hq).T[:, :n], lse[:, :n], rtol=1e-12)


def test_parent_consistent_relabelling_permutes_rows():
    B, Hq, Hkv, D, L = 7, 2, 2, 8, 11
    rng = np.random.default_rng(12)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent = np.array([-1, 0, 0, 1, 1, 2, 2])
    new_of_old = np.array([0, 2, 1, 5, 6, 3, 4])     # swap the two subtrees; parents stay before children
    parent2 = np.full(B, -1)
    for old in range(1, B):
        parent2[new_of_old[old]] = new_of_old[parent[old]]
    a, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"],
                         anc_from_parent(parent, B, B), B, 0.4)
    inv = np.argsort(new_of_old)
    b, _ = tree_attn_ref(x["q"][inv], x["k_prefix"], x["v_prefix"], x["tree_k"][inv], x["tree_v"][inv],
                         anc_from_parent(parent2, B, B), B, 0.4)
    np.testing.assert_allclose(b[new_of_old], a, rtol=1e-12, atol=1e-14)


def test_bf16_widening_of_fixed_bit_patterns():
    """bf16_bits_to_f64 against values the bfloat16 format itself fixes (1 sign, 8 exponent, 7 mantissa bits):
    a wrong shift, a dropped sign or a mantissa taken as the exponent fails one of these."""
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x8000, 0x7F80, 0xFF80, 0x3FC0, 0x4049, 0x0001, 0x0080, 0x7F7F, 0x3B80],
                    dtype=np.uint16)
    want = [1.0, -2.0, 0.0, -0.0, np.inf, -np.inf, 1.5, 3.140625, 2.0 ** -133, 2.0 ** -126,
            (2.0 - 2.0 ** -7) * 2.0 ** 127, 2.0 ** -8]
    got = bf16_bits_to_f64(bits)
    assert got.dtype == np.float64
    np.testing.assert_array_equal(got, np.array(want, dtype=np.float64))
    assert np.signbit(got[3]) and not np.signbit(got[2])
    assert np.isnan(bf16_bits_to_f64(np.array([0x7FC0], dtype=np.uint16)))[0]
    # arrays that are not bit patterns pass through as values
    np.testing.assert_array_equal(bf16_bits_to_f64(np.array([0.5, -3.0])), [0.5, -3.0])


def test_paged_gather_on_a_cache_with_known_rows():
    """gather_paged_prefix on a cache whose every row holds its own (page, offset): position j must come
    from page table[j // page_size], offset j % page_size -- a swapped division or a page taken as a row
    shows at once."""
    from oracle import gather_paged_prefix
    num_pages, page_size = 5, 4
    cache = np.zeros((num_pages, page_size, 2, 3), dtype=np.int64)
    for pg in range(num_pages):
        for off in range(page_size):
            cache[pg, off] = 100 * pg + off
    table = np.array([3, 0, 4, 1])
    got = gather_paged_prefix(cache, table, 10)
    want = [300, 301, 302, 303, 0, 1, 2, 3, 400, 401]
    assert got.shape == (10, 2, 3)
    for j in range(10):
        assert (got[j] == want[j]).all(), j
    assert gather_paged_prefix(cache, table, 0).shape == (0, 2, 3)
    # a prefix that ends inside a page stops there
    assert gather_paged_prefix(cache, table, 5)[-1, 0, 0] == 0
