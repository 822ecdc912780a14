"""GPU parity: jet_tree_verify_attn on seeded random configurations against the fp64 oracle.

Every case draws head layout (G = 1 .. 16, 1 .. 4 KV heads, D 64 / 128), batch (1 .. 5), budget (1 .. 300 nodes),
ragged prefix lengths (0 .. 2600, contiguous or paged), live node counts, tree shape, softmax scale and the
stable-prefix flag, so that the launch planner is exercised far from the benchmark shapes: every merge form of
the key slices, one and two query tiles per CTA, sorted launch order with slices, clusters up to the largest
size.  All rows of every sequence are compared.  120 further cases use the in-cache layout (tree rows behind the prefix).

Tolerance: the arithmetic bound |err| <= 2^-8 (|ref| + max |v|) + 2e-3 element-wise (probabilities rounded to
bf16 before they weigh V entries of size up to 4.5, output rounded to bf16), mean |err| <= 2.5e-3 over the live
rows, log-sum-exp within 2e-3.

Cases pinned by name because randomized runs found faults with them:
  * a paged cache with one query tile per CTA at scale: K and V tiles come from two producer warps there; with one
    shared ring of stages a warp could run two uses of a stage ahead of the consumers when a load was slow and
    overwrite a tile that had not been read (the warps now have stages of their own);
  * small trees in a ragged batch: one query tile per KV head, key slices combined by the second launch,
    sequences launched longest first -- the partial rows were addressed by launch rank instead of by sequence;
  * 17 key tiles with few work items: a plan with a cluster of 17 CTAs, which the hardware does not launch.
"""
import numpy as np
import pytest

from jet_inputs import binary_tree, chain_tree, make_attn_inputs, make_paged_cache, random_tree, star_tree
from oracle import anc_from_parent, gather_paged_prefix, tree_attn_ref, tree_attn_rows_ref

pytestmark = pytest.mark.gpu

NAN_BITS = np.uint16(0x7FC0)
V_MAX = 4.5


def _run_case(rng, D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale, wide_bound):
    import jet_harness as H
    Hq = G * Hkv
    qs, tks, tvs, ancs, kpre, vpre = [], [], [], [], [], []
    for b in range(batch):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, int(seq[b]))
        n = int(n_nodes[b])
        kind = rng.choice(["random", "chain", "star", "binary"])
        parent = {"random": lambda: random_tree(n, rng), "chain": lambda: chain_tree(n),
                  "star": lambda: star_tree(n), "binary": lambda: binary_tree(n)}[kind]()[0]
        tk, tv = x["tree_k"].copy(), x["tree_v"].copy()
        tk[n:], tv[n:] = NAN_BITS, NAN_BITS                      # padding nodes hold junk
        qs.append(x["q"]); tks.append(tk); tvs.append(tv); ancs.append(anc_from_parent(parent, n, B))
        kpre.append(x["k_prefix"]); vpre.append(x["v_prefix"])
    Lmax = int(seq.max())
    if paged:
        kp, vp, table = make_paged_cache(rng, seq, 16, Hkv, D, reserve=0)
        kp[:], vp[:] = NAN_BITS, NAN_BITS                        # every row outside a prefix is junk
        for b in range(batch):
            for pos in range(int(seq[b])):
                kp[table[b, pos // 16], pos % 16] = kpre[b][pos]
                vp[table[b, pos // 16], pos % 16] = vpre[b][pos]
        bound = table.shape[1] * 16 if wide_bound else max(Lmax, 1)
        out, lse, st = H.run_tree_attn(np.stack(qs), kp, vp, table, seq, np.stack(tks), np.stack(tvs), np.stack(ancs),
                                       n_nodes, scale, max_seq_len=bound, flags=flags)
    else:
        rows = Lmax + (37 if wide_bound else 0)
        if rows == 0:
            kc = vc = None
        else:
            kc = np.full((batch, rows, Hkv, D), NAN_BITS, np.uint16)
            vc = np.full_like(kc, NAN_BITS)
            for b in range(batch):
                kc[b, :seq[b]], vc[b, :seq[b]] = kpre[b], vpre[b]
        out, lse, st = H.run_tree_attn(np.stack(qs), kc, vc, None, seq, np.stack(tks), np.stack(tvs), np.stack(ancs),
                                       n_nodes, scale, max_seq_len=rows, flags=flags)
    assert st == 0
    assert not np.isnan(out).any()
    for b in range(batch):
        n = int(n_nodes[b])
        ref, rlse = tree_attn_ref(qs[b], kpre[b], vpre[b], tks[b], tvs[b], ancs[b], n, scale)
        err = np.abs(out[b] - ref)[:n]
        assert (err <= 2.0 ** -8 * (np.abs(ref[:n]) + V_MAX) + 2e-3).all(), (b, float(err.max()))
        assert err.mean() <= 2.5e-3, (b, float(err.mean()))
        assert (out[b, n:] == 0).all()
        assert np.abs(lse[b][:, :n] - rlse[:, :n]).max() <= 2e-3
        assert np.isneginf(lse[b][:, n:]).all()


def _draw(rng):
    D = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    Hkv = int(rng.choice([1, 2, 4]))
    batch = int(rng.choice([1, 1, 1, 2, 3, 5]))
    B = int(rng.choice([1, 7, 16, 31, 32, 33, 64, 65, 100, 128, 129, 200, 256, 300]))
    B = min(B, max(1, 2048 // G))
    Lmax = int(rng.choice([0, 5, 127, 128, 129, 300, 700, 1500, 2600]))
    work = batch * B * G * Hkv
    if work * max(Lmax, 1) > 6e7:                     # keeps the oracle at a second or so per case
        Lmax = int(6e7 / work)
    seq = rng.integers(0, Lmax + 1, size=batch).astype(np.int32)
    if rng.random() < 0.5:
        seq[rng.integers(0, batch)] = Lmax
    paged = bool(rng.random() < 0.4) and Lmax > 0
    flags = int(rng.random() < 0.5)
    scale = float(rng.choice([1.0 / np.sqrt(D), 0.3, 0.02]))
    n_nodes = rng.integers(1, B + 1, size=batch)
    if rng.random() < 0.5:
        n_nodes[0] = B
    wide = bool(rng.random() < 0.5)
    return D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale, wide


@pytest.mark.parametrize("block", range(8))
def test_random_configurations(block):
    """8 x 40 seeded cases (one oracle call per sequence, about a second per case at most)."""
    for it in range(40):
        rng = np.random.default_rng(77003 * block + it)
        D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale, wide = _draw(rng)
        try:
            _run_case(rng, D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale, wide)
        except AssertionError as e:
            raise AssertionError(f"case {block}/{it}: D={D} G={G} Hkv={Hkv} batch={batch} B={B} seq={seq.tolist()} "
                                 f"n={n_nodes.tolist()} paged={paged} flags={flags} scale={scale}: {e}") from e


def _run_case_in_cache(rng, D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale):
    """The same comparison for the in-cache layout: node v of sequence b sits at cache position seq[b] + v."""
    import jet_harness as H
    Hq = G * Hkv
    xs, qs, ancs = [], [], []
    for b in range(batch):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, int(seq[b]))
        parent = random_tree(int(n_nodes[b]), rng)[0]
        xs.append(x); qs.append(x["q"]); ancs.append(anc_from_parent(parent, int(n_nodes[b]), B))
    if paged:
        kp, vp, table = make_paged_cache(rng, seq, 16, Hkv, D, reserve=B)
        kp[:], vp[:] = NAN_BITS, NAN_BITS
        for b in range(batch):
            n, L = int(n_nodes[b]), int(seq[b])
            rows_k = np.concatenate([xs[b]["k_prefix"], xs[b]["tree_k"][:n]])
            rows_v = np.concatenate([xs[b]["v_prefix"], xs[b]["tree_v"][:n]])
            for pos in range(L + n):
                kp[table[b, pos // 16], pos % 16] = rows_k[pos]
                vp[table[b, pos // 16], pos % 16] = rows_v[pos]
        out, lse, st = H.run_tree_attn_tail(np.stack(qs), kp, vp, table, seq, np.stack(ancs), n_nodes, scale,
                                            table.shape[1] * 16, Hkv, flags=flags)
    else:
        rows = int(seq.max()) + B + 7
        kc = np.full((batch, rows, Hkv, D), NAN_BITS, np.uint16)
        vc = np.full_like(kc, NAN_BITS)
        for b in range(batch):
            n, L = int(n_nodes[b]), int(seq[b])
            kc[b, :L], vc[b, :L] = xs[b]["k_prefix"], xs[b]["v_prefix"]
            kc[b, L:L + n], vc[b, L:L + n] = xs[b]["tree_k"][:n], xs[b]["tree_v"][:n]
        out, lse, st = H.run_tree_attn_tail(np.stack(qs), kc, vc, None, seq, np.stack(ancs), n_nodes, scale, rows, Hkv,
                                            flags=flags)
    assert st == 0 and not np.isnan(out).any()
    for b in range(batch):
        n = int(n_nodes[b])
        ref, rlse = tree_attn_ref(qs[b], xs[b]["k_prefix"], xs[b]["v_prefix"], xs[b]["tree_k"], xs[b]["tree_v"], ancs[b],
                                  n, scale)
        err = np.abs(out[b] - ref)[:n]
        assert (err <= 2.0 ** -8 * (np.abs(ref[:n]) + V_MAX) + 2e-3).all(), (b, float(err.max()))
        assert (out[b, n:] == 0).all()
        assert np.abs(lse[b][:, :n] - rlse[:, :n]).max() <= 2e-3


@pytest.mark.parametrize("block", range(4))
def test_random_configurations_in_cache_layout(block):
    for it in range(30):
        rng = np.random.default_rng(99991 * (block + 1) + it)
        D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale, _ = _draw(rng)
        try:
            _run_case_in_cache(rng, D, G, Hkv, batch, B, seq, n_nodes, paged, flags, scale)
        except AssertionError as e:
            raise AssertionError(f"case {block}/{it}: D={D} G={G} Hkv={Hkv} batch={batch} B={B} seq={seq.tolist()} "
                                 f"n={n_nodes.tolist()} paged={paged} flags={flags} scale={scale}: {e}") from e


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("D,G,Hkv,B,seq,n_nodes,paged", [
    (64, 2, 2, 32, [282, 2582, 1298, 222, 646], [32, 13, 26, 14, 26], False),
    (64, 16, 4, 1, [1627, 937, 445, 1423, 1701], [1, 1, 1, 1, 1], False),
    (64, 2, 4, 16, [1566, 2600, 1069], [15, 5, 16], True),
    (128, 16, 2, 7, [1340, 1167, 1637, 1282, 1680], [7, 5, 7, 2, 4], False),
    (64, 1, 4, 128, [925, 809, 1214, 644, 1500], [110, 96, 13, 117, 41], True),
])
def test_small_trees_in_a_ragged_batch(D, G, Hkv, B, seq, n_nodes, paged, flags):
    """One query tile per KV head, several key slices per work item, sequences of different lengths: the slices
    of a sequence must be combined with that sequence's own partial rows whatever the launch order."""
    rng = np.random.default_rng(5100 + B)
    seq = np.asarray(seq, np.int32)
    _run_case(rng, D, G, Hkv, len(seq), B, seq, np.asarray(n_nodes), paged, flags, 1.0 / np.sqrt(D), False)


@pytest.mark.parametrize("paged", [False, True])
def test_seventeen_key_tiles_with_few_work_items(paged):
    """3 work items with 17 key tiles each: the cheapest plan on paper is one key tile per CTA in clusters of 17,
    which do not exist; the planner must stop at the largest launchable cluster."""
    rng = np.random.default_rng(5200)
    seq = np.asarray([1973, 1000, 1571], np.int32)
    _run_case(rng, 64, 2, 1, 3, 32, seq, np.asarray([28, 18, 23]), paged, 1, 0.125, False)


@pytest.mark.parametrize("G,Hkv,batch,B,L,ragged,flags", [
    (4, 8, 2, 384, 9000, False, 1),       # 12 query tiles per KV head, two key slices in clusters of two, three waves
    (1, 4, 16, 96, 4100, False, 0),       # one query tile per KV head, two slices combined by the second launch
    (1, 8, 32, 128, 3988, True, 0),       # 256 work items, two waves, sequences launched longest first
    (1, 8, 32, 16, 4100, False, 1),
    (4, 8, 32, 16, 4096, False, 1),
])
def test_paged_cache_one_query_tile_per_cta_at_scale(G, Hkv, batch, B, L, ragged, flags):
    """Sampled rows of the first, last, shortest and longest sequence against the oracle (D = 128)."""
    import jet_harness as H
    D, Hq = 128, G * Hkv
    rng = np.random.default_rng(5300 + batch * B)
    seq = (rng.integers(L // 5, L + 1, size=batch) if ragged else np.full(batch, L)).astype(np.int32)
    n_nodes = np.full(batch, B)
    qs, tks, tvs, ancs = [], [], [], []
    for b in range(batch):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, 0)
        parent = random_tree(B, rng)[0]
        qs.append(x["q"]); tks.append(x["tree_k"]); tvs.append(x["tree_v"]); ancs.append(anc_from_parent(parent, B, B))
    kp, vp, table = make_paged_cache(rng, seq, 16, Hkv, D, reserve=0)
    scale = 1.0 / np.sqrt(D)
    for _ in range(3):                    # (the fault depended on timing: a few launches)
        out, lse, st = H.run_tree_attn(np.stack(qs), kp, vp, table, seq, np.stack(tks), np.stack(tvs), np.stack(ancs),
                                       n_nodes, scale, flags=flags)
        assert st == 0 and not np.isnan(out).any()
    for b in sorted({0, batch - 1, int(np.argmin(seq)), int(np.argmax(seq))}):
        kpre = gather_paged_prefix(kp, table[b], int(seq[b]))
        vpre = gather_paged_prefix(vp, table[b], int(seq[b]))
        rows = [(int(rng.integers(0, B)), int(rng.integers(0, Hq))) for _ in range(10)] + [(0, 0), (B - 1, Hq - 1)]
        ref, rlse = tree_attn_rows_ref(qs[b], kpre, vpre, tks[b], tvs[b], ancs[b], B, scale, rows)
        got = np.stack([out[b, v, h] for v, h in rows])
        err = np.abs(got - ref)
        assert (err <= 2.0 ** -8 * (np.abs(ref) + V_MAX) + 2e-3).all(), (b, float(err.max()))
        assert np.abs(np.array([lse[b, h, v] for v, h in rows]) - rlse).max() <= 2e-3
