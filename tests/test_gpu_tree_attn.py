"""GPU parity: jet_tree_verify_attn against the fp64 oracle.

Tolerance (bf16 operands, fp32 accumulation, bf16 output): max |err| <= 2e-2 and
mean |err| <= 2e-3 against the fp64 oracle; log-sum-exp within 1e-3.
"""
import numpy as np
import pytest

from jet_inputs import (CONFIGS, binary_tree, chain_tree, make_attn_inputs, make_logp, make_paged_cache,
                        random_tree, star_tree)
from oracle import anc_from_parent, gather_paged_prefix, tree_attn_ref, tree_attn_rows_ref, tree_build_ref

pytestmark = pytest.mark.gpu

MAX_ERR, MEAN_ERR, LSE_ERR = 2e-2, 2e-3, 1e-3
NAN_BITS = np.uint16(0x7FC0)
# (Where the stated bound comes from: every probability is rounded to bf16, 2^-9 relative, before it multiplies
# V entries of size up to ~4.5, the row sum keeps the unrounded values, and the output is rounded to bf16 --
# 2^-8 * 4.5 = 1.8e-2 in the worst case of a row that sees one or two keys.  With thousands of keys the errors
# average out; the full-size tests hold the kernel to 4e-3 / 4e-4 there.)


def _check(out, lse, ref, rlse, n):
    assert not np.isnan(out).any()
    err = np.abs(out - ref)[:n]                 # live rows only: the zero rows of padding nodes would dilute the mean
    assert err.max() <= MAX_ERR, err.max()
    assert err.mean() <= MEAN_ERR, err.mean()
    assert (out[n:] == 0).all()
    if lse is not None:
        assert np.abs(lse[:, :n] - rlse[:, :n]).max() <= LSE_ERR
        assert np.isneginf(lse[:, n:]).all()


def _tree(kind, n, rng):
    return {"random": lambda: random_tree(n, rng), "chain": lambda: chain_tree(n),
            "star": lambda: star_tree(n), "binary": lambda: binary_tree(n)}[kind]()


def _run_contiguous(B, Hq, Hkv, D, L, seed, n=None, kind="random", junk_rows=40, scale=None, flags=0):
    import jet_harness as H
    rng = np.random.default_rng(seed)
    n = n or B
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = _tree(kind, n, rng)
    anc = anc_from_parent(parent, n, B)
    scale = scale or 1.0 / np.sqrt(D)
    ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, n, scale)
    # cache rows beyond the prefix hold NaN junk that must never influence the result
    kc = np.full((1, L + junk_rows, Hkv, D), NAN_BITS, np.uint16)
    vc = np.full_like(kc, NAN_BITS)
    kc[0, :L], vc[0, :L] = x["k_prefix"], x["v_prefix"]
    tk, tv = x["tree_k"].copy(), x["tree_v"].copy()
    tk[n:], tv[n:] = NAN_BITS, NAN_BITS                       # padding nodes hold junk too
    out, lse, st = H.run_tree_attn(x["q"][None], kc, vc, None, [L], tk[None], tv[None], anc[None], [n], scale,
                                   max_seq_len=L + junk_rows, flags=flags)
    assert st == 0
    _check(out[0], lse[0], ref, rlse, n)
    return out[0], ref


@pytest.mark.parametrize("B,Hq,Hkv,D,L", [(32, 8, 2, 128, 0), (32, 8, 2, 128, 127), (33, 8, 2, 128, 128),
                                          (64, 8, 2, 128, 1000), (64, 32, 8, 128, 4096), (16, 32, 8, 128, 4097),
                                          (256, 8, 2, 128, 700), (40, 4, 2, 64, 700)])
def test_stable_prefix_flag_reads_early_and_computes_the_same(B, Hq, Hkv, D, L):
    """JET_ATTN_STABLE_PREFIX only moves reads of the lengths and of whole prefix tiles in front of the dependency
    wait; prefixes that end inside a tile, empty prefixes and junk behind the prefix give the same results."""
    plain, _ = _run_contiguous(B, Hq, Hkv, D, L, 900 + B + L)
    early, _ = _run_contiguous(B, Hq, Hkv, D, L, 900 + B + L, flags=1)
    assert np.array_equal(plain, early)


def test_unknown_attention_flags_are_rejected():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    t = torch.zeros(1 << 16, dtype=torch.bfloat16, device=H.DEV)
    i32 = torch.ones(64, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(1 << 20)
    st = jet.jet_tree_verify_attn_ex(t, t, t, None, 0, 0, 0, i32, 16, t, t, i32, i32, 1, 8, 8, 2, 128, 0, 0.1, t, None,
                                     None, ws, 2, check=False)
    assert st == jet.JET_ERR_INVALID_ARG


@pytest.mark.parametrize("seed", range(2))
def test_tiny_config(seed):
    c = CONFIGS["tiny"]
    _run_contiguous(c["B"], c["Hq"], c["Hkv"], c["D"], c["L"], 1000 + seed)


def test_tiny_config_with_built_tree():
    import jet_harness as H
    c = CONFIGS["tiny"]
    rng = np.random.default_rng(1000)
    t = tree_build_ref(make_logp(rng, c["N"], c["V"], c["sigma_draft"]), 1, c["N"], c["W"], c["B"])
    x = make_attn_inputs(rng, c["B"], c["Hq"], c["Hkv"], c["D"], c["L"])
    scale = 1.0 / np.sqrt(c["D"])
    ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], t["anc_mask"],
                              t["n_nodes"], scale)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [c["L"]],
                                   x["tree_k"][None], x["tree_v"][None], t["anc_mask"][None], [t["n_nodes"]], scale)
    assert st == 0
    _check(out[0], lse[0], ref, rlse, t["n_nodes"])


def test_qwen3_8b_config():
    c = CONFIGS["qwen3_8b"]
    _run_contiguous(c["B"], c["Hq"], c["Hkv"], c["D"], c["L"], 2000)


@pytest.mark.parametrize("L", [0, 1, 127, 128, 129, 255, 257])
@pytest.mark.parametrize("B", [1, 2, 31, 32, 33])
def test_tile_boundaries(L, B):
    _run_contiguous(B, 8, 2, 128, L, 31 * L + B)


@pytest.mark.parametrize("kind", ["chain", "star", "binary"])
def test_tree_shapes(kind):
    _run_contiguous(48, 8, 2, 128, 200, 5, kind=kind)


@pytest.mark.parametrize("B,Hq,Hkv,D,L", [(64, 8, 8, 128, 333), (40, 4, 2, 64, 700), (128, 32, 4, 128, 520),
                                          (200, 16, 1, 64, 130), (512, 8, 2, 128, 140), (512, 8, 1, 128, 260)])
def test_head_group_and_budget_variants(B, Hq, Hkv, D, L):
    _run_contiguous(B, Hq, Hkv, D, L, B + L)


def test_padding_nodes_give_zero_rows():
    _run_contiguous(64, 8, 2, 128, 300, 9, n=37)
    _run_contiguous(300, 8, 2, 128, 100, 10, n=129)
    _run_contiguous(64, 32, 8, 128, 50, 11, n=1)


def test_masked_nodes_have_no_influence_and_output_is_deterministic():
    out_a, ref = _run_contiguous(64, 8, 2, 128, 500, 77)
    out_b, _ = _run_contiguous(64, 8, 2, 128, 500, 77)
    assert np.array_equal(out_a, out_b)


def test_large_scores_stay_finite():
    # scale 1.0 with head_dim 128 gives scores of +-30: exercises the running-max rescaling
    _run_contiguous(64, 8, 2, 128, 900, 3, scale=1.0)


@pytest.mark.parametrize("jump", [12.0, 40.0])
@pytest.mark.parametrize("where", ["prefix", "tree"])
def test_scores_far_above_the_first_tile(jump, where):
    """One query tile per CTA keeps the row reference of the first key tile for the whole key range; keys whose
    scores lie far above it (here by about 2^110 and by more than the fp32 range, in the later prefix tiles or only
    in the tree) must send the CTA through its exact two-accumulator pass.  Rows stay within tolerance."""
    import jet_harness as H
    from jet_inputs import bf16_bits_to_f32, f32_to_bf16_bits
    B, Hq, Hkv, D, L = 32, 8, 2, 128, 700
    rng = np.random.default_rng(77)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    q = np.abs(bf16_bits_to_f32(x["q"])) * 0.25                  # every score against an all-positive key is positive
    x["q"] = f32_to_bf16_bits(q)
    k = bf16_bits_to_f32(x["k_prefix"]) * 0.05
    tk = bf16_bits_to_f32(x["tree_k"]) * 0.05
    if where == "prefix":
        k[300:520] = jump * 0.25                                 # keys 300..519: scores of about 25 * jump * 0.25 * 0.8
    else:
        tk[:] = jump * 0.25                                      # the tree's own keys only
    x["k_prefix"], x["tree_k"] = f32_to_bf16_bits(k), f32_to_bf16_bits(tk)
    parent, _, _ = random_tree(B, rng)
    anc = anc_from_parent(parent, B, B)
    scale = 1.0
    s_big = (bf16_bits_to_f32(x["q"])[0, 0] * jump * 0.25).sum() * scale * 1.4427
    assert s_big > (100 if jump == 12.0 else 130)                 # log2 units above the first tile's scores
    ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L],
                                   x["tree_k"][None], x["tree_v"][None], anc[None], [B], scale)
    assert st == 0
    _check(out[0], None, ref, rlse, B)
    assert np.abs(lse[0] - rlse).max() <= 1e-3 * max(1.0, np.abs(rlse).max())


def test_scores_far_above_the_first_tile_headline_shape():
    """The same at the benchmark's shape (16 work items x 9 key slices that merge through the workspace): only
    some slices contain the overflowing keys, so CTAs that kept the fixed reference and CTAs that fell back to
    the exact pass are merged with each other."""
    import jet_harness as H
    from jet_inputs import bf16_bits_to_f32, f32_to_bf16_bits
    B, Hq, Hkv, D, L = 64, 32, 8, 128, 4096
    rng = np.random.default_rng(78)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    x["q"] = f32_to_bf16_bits(np.abs(bf16_bits_to_f32(x["q"])) * 0.25)
    k = bf16_bits_to_f32(x["k_prefix"]) * 0.05
    k[1500:1700] = 10.0                                         # inside the 4th of the 9 slices, not at its start
    x["k_prefix"] = f32_to_bf16_bits(k)
    parent, _, _ = random_tree(B, rng)
    anc = anc_from_parent(parent, B, B)
    scale = 1.0
    rows = [(int(rng.integers(0, B)), int(rng.integers(0, Hq))) for _ in range(64)] + [(0, 0), (B - 1, Hq - 1)]
    ref, rlse = tree_attn_rows_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale,
                                   rows)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L],
                                   x["tree_k"][None], x["tree_v"][None], anc[None], [B], scale)
    assert st == 0 and not np.isnan(out).any()
    got = np.stack([out[0, v, h] for v, h in rows])
    err = np.abs(got - ref)
    assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR
    got_lse = np.array([lse[0, h, v] for v, h in rows])
    assert np.abs(got_lse - rlse).max() <= 1e-3 * max(1.0, np.abs(rlse).max())


def test_rows_without_a_key_in_their_first_tile_and_very_negative_scores():
    """512-node tree, no prefix: the rows of the later query tiles see no key in the first key tiles of
    their slices (their ancestors lie elsewhere), so those rows start without a reference of their own; all
    scores are about -300 (far below what exp2 can represent against a reference of 0).  The result must still
    be the softmax over the visible keys."""
    import jet_harness as H
    from jet_inputs import bf16_bits_to_f32, f32_to_bf16_bits
    B, Hq, Hkv, D, L = 512, 4, 1, 128, 0
    rng = np.random.default_rng(91)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    x["q"] = f32_to_bf16_bits(np.abs(bf16_bits_to_f32(x["q"])) * 0.5 + 0.5)
    x["tree_k"] = f32_to_bf16_bits(-(np.abs(bf16_bits_to_f32(x["tree_k"])) * 0.5 + 2.0))
    parent = np.zeros(B, dtype=np.int32)                     # a star: every node hangs off the root ...
    parent[0] = -1
    parent[300:384] = np.arange(299, 383)                    # ... except a chain 299 -> 300 -> ... -> 383
    anc = anc_from_parent(parent, B, B)
    scale = 1.0
    rows = [(v, h) for v in (0, 1, 127, 128, 200, 255, 256, 299, 300, 383, 384, 400, 415, 416, 500, 511) for h in (0, 3)]
    ref, rlse = tree_attn_rows_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale,
                                   rows)
    assert rlse.max() < -150                                 # every visible score is far below zero
    out, lse, st = H.run_tree_attn(x["q"][None], None, None, None, [L], x["tree_k"][None], x["tree_v"][None],
                                   anc[None], [B], scale, max_seq_len=0)
    assert st == 0 and not np.isnan(out).any()
    got = np.stack([out[0, v, h] for v, h in rows])
    err = np.abs(got - ref)
    assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR, (err.max(), err.mean())
    got_lse = np.array([lse[0, h, v] for v, h in rows])
    assert np.abs(got_lse - rlse).max() <= 1e-3 * np.abs(rlse).max()


@pytest.mark.parametrize("mt,force", [("1", "2"), ("1", "2,g"), ("1", "2,h"), ("1", "4"), ("2", "1"), ("2", "2"),
                                      ("2", "4,g"), ("2", "4,h")])
def test_adversarial_scores_under_forced_slicings(mt, force):
    """The launch plan decides where the key slices begin, and with it which rows meet an empty first tile.  The
    library reads JET_FORCE_MT / JET_FORCE_SPLIT once per process, so the adversarial-score tests run again in
    a child process under one or two query tiles per CTA and 1, 2 or 4 key slices (merged in a cluster or through
    the workspace)."""
    import os
    import subprocess
    import sys
    if os.environ.get("JET_FORCE_SPLIT"):
        pytest.skip("already inside a forced run")
    env = dict(os.environ, JET_FORCE_MT=mt, JET_FORCE_SPLIT=force)
    r = subprocess.run([sys.executable, "-m", "pytest", __file__, "-m", "gpu", "-x", "-q", "-k",
                        "very_negative or far_above"], env=env, capture_output=True, text=True,
                       cwd=os.path.dirname(os.path.dirname(os.path.abspath(__file__))), timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


@pytest.mark.parametrize("B", [16, 32])
def test_small_budgets_at_the_full_prefix(B):
    """Few query rows per KV head (one query tile per KV head): the key range is cut into as many slices as
    the device has room for (more than a cluster can hold, merged through the workspace; the last slices own
    no rows to combine)."""
    import jet_harness as H
    Hq, Hkv, D, L = 32, 8, 128, 4096
    rng = np.random.default_rng(600 + B)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(B, rng)
    anc = anc_from_parent(parent, B, B)
    scale = 1.0 / np.sqrt(D)
    ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L],
                                   x["tree_k"][None], x["tree_v"][None], anc[None], [B], scale)
    assert st == 0
    _check(out[0], lse[0], ref, rlse, B)


@pytest.mark.parametrize("mt,split", [("1", "1"), ("1", "3"), ("1", "6"), ("1", "9,g"), ("1", "16,g"), ("1", "18,g"),
                                      ("1", "9,h"), ("1", "4,h"), ("1", "18,h"), ("2", "1"), ("2", "2"), ("2", "4,g"),
                                      ("2", "4,h")])
def test_every_kind_of_launch_plan(mt, split):
    """The planner picks one plan per shape; the others (query tiles per CTA, number of key slices, merge through
    a cluster, through the workspace inside the launch (",g") or through the workspace with a second launch
    (",h")) must compute the same thing.  Runs the benchmark-shape test, the tile
    boundary tests and the tree-shape tests in a child process under a forced plan (a forced plan the device
    cannot hold is ignored by the library, i.e. falls back to the planner's)."""
    import os
    import subprocess
    import sys
    if os.environ.get("JET_FORCE_SPLIT") or os.environ.get("JET_FORCE_MT"):
        pytest.skip("already inside a forced run")
    env = dict(os.environ, JET_FORCE_MT=mt, JET_FORCE_SPLIT=split)
    r = subprocess.run([sys.executable, "-m", "pytest", __file__, "-m", "gpu", "-x", "-q", "-k",
                        "qwen3_8b_config or tile_boundaries or tree_shapes or padding_nodes or small_budgets"],
                       env=env, capture_output=True, text=True,
                       cwd=os.path.dirname(os.path.dirname(os.path.abspath(__file__))), timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_cta_pair_form():
    """The CTA-pair form of the key loop (consecutive query tiles of a work item on two SMs that share every K/V
    tile through tcgen05 cta_group::2): never the planner's choice, so it is forced in a child process, where the
    plan query must report it and the benchmark-shape, tile-boundary, tree-shape, padding, adversarial-score and
    ragged paged batch tests must pass with it."""
    import os
    import subprocess
    import sys
    if os.environ.get("JET_FORCE_SPLIT") or os.environ.get("JET_FORCE_MT") or os.environ.get("JET_FORCE_PAIR"):
        pytest.skip("already inside a forced run")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, JET_FORCE_MT="1", JET_FORCE_PAIR="1")
    code = ("import paper_2606_18394_b200 as jet\n"
            "p = jet.jet_tree_verify_attn_plan(1, 64, 32, 8, 128, 4096)\n"
            "assert p['pair'] and p['query_tiles_per_cta'] == 1, p\n"
            "q = jet.jet_tree_verify_attn_plan(1, 16, 32, 8, 128, 4096)\n"
            "assert not q['pair'], q\n")           # one query tile per KV head: nothing to pair
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    r = subprocess.run([sys.executable, "-m", "pytest", __file__, "-m", "gpu", "-x", "-q", "-k",
                        "qwen3_8b_config or tile_boundaries or tree_shapes or padding_nodes or very_negative or "
                        "far_above or batched_paged_ragged or sweep_16k"],
                       env=env, capture_output=True, text=True, cwd=root, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_the_planner_never_picks_the_pair_form():
    import paper_2606_18394_b200 as jet
    import os
    if os.environ.get("JET_FORCE_PAIR"):
        pytest.skip("inside a forced run")
    for B, L in ((64, 4096), (128, 4096), (256, 16384), (512, 32768)):
        assert not jet.jet_tree_verify_attn_plan(1, B, 32, 8, 128, L)["pair"]


def test_sweep_16k_sampled_rows():
    """Long prefix (sweep shape, B=128): the oracle checks a seeded sample of (node, head) rows."""
    import jet_harness as H
    c = CONFIGS["sweep_16k"]
    B, Hq, Hkv, D, L = 128, c["Hq"], c["Hkv"], c["D"], c["L"]
    rng = np.random.default_rng(3000)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(B, rng, max_depth=12)
    anc = anc_from_parent(parent, B, B)
    scale = 1.0 / np.sqrt(D)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L],
                                   x["tree_k"][None], x["tree_v"][None], anc[None], [B], scale)
    assert st == 0 and not np.isnan(out).any()
    rows = [(int(rng.integers(0, B)), int(rng.integers(0, Hq))) for _ in range(96)] + [(0, 0), (B - 1, Hq - 1)]
    ref, rlse = tree_attn_rows_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale,
                                   rows)
    got = np.stack([out[0, v, h] for v, h in rows])
    err = np.abs(got - ref)
    assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR
    assert np.abs(np.array([lse[0, h, v] for v, h in rows]) - rlse).max() <= LSE_ERR


def test_moe_30b_full_size_sampled_rows():
    """Largest single-sequence shape (8 query heads per KV head, prefix 32768, 512-node tree, depth 12): the
    launch configuration the planner picks at full size; the oracle checks a seeded sample of rows."""
    import jet_harness as H
    c = CONFIGS["moe_30b"]
    B, Hq, Hkv, D, L = 512, c["Hq"], c["Hkv"], c["D"], c["L"]
    rng = np.random.default_rng(5000)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(B, rng, max_depth=c["N"])
    anc = anc_from_parent(parent, B, B)
    scale = 1.0 / np.sqrt(D)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L],
                                   x["tree_k"][None], x["tree_v"][None], anc[None], [B], scale)
    assert st == 0 and not np.isnan(out).any()
    rows = [(int(rng.integers(0, B)), int(rng.integers(0, Hq))) for _ in range(64)] + [(0, 0), (B - 1, Hq - 1)]
    ref, rlse = tree_attn_rows_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale,
                                   rows)
    got = np.stack([out[0, v, h] for v, h in rows])
    err = np.abs(got - ref)
    assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR
    assert np.abs(np.array([lse[0, h, v] for v, h in rows]) - rlse).max() <= LSE_ERR


def test_batched_paged_full_size_sampled_rows():
    """The serving shape at full size (32 sequences, prefixes 1024..8192, paged, shuffled page table): the
    configuration in which sequences are launched longest first and CTAs take two query tiles; the oracle
    checks a seeded sample of rows of the shortest, the longest and one more sequence."""
    import jet_harness as H
    c = CONFIGS["batched_paged"]
    batch, B, Hq, Hkv, D = c["batch"], c["B"], c["Hq"], c["Hkv"], c["D"]
    rng = np.random.default_rng(4500)
    seq = rng.integers(c["L_range"][0], c["L_range"][1] + 1, size=batch).astype(np.int32)
    kp, vp, table = make_paged_cache(rng, seq, 16, Hkv, D, reserve=9)
    n_nodes = np.full(batch, B, np.int32)
    n_nodes[3] = 17
    qs, tks, tvs, ancs = [], [], [], []
    for b in range(batch):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, 0)
        parent, _, _ = random_tree(int(n_nodes[b]), rng, max_depth=c["N"])
        qs.append(x["q"]); tks.append(x["tree_k"]); tvs.append(x["tree_v"])
        ancs.append(anc_from_parent(parent, int(n_nodes[b]), B))
    scale = 1.0 / np.sqrt(D)
    out, lse, st = H.run_tree_attn(np.stack(qs), kp, vp, table, seq, np.stack(tks), np.stack(tvs), np.stack(ancs),
                                   n_nodes, scale)
    assert st == 0 and not np.isnan(out).any()
    for b in sorted({int(np.argmin(seq)), int(np.argmax(seq)), 3}):
        n = int(n_nodes[b])
        kpre = gather_paged_prefix(kp, table[b], int(seq[b]))
        vpre = gather_paged_prefix(vp, table[b], int(seq[b]))
        rows = [(int(rng.integers(0, n)), int(rng.integers(0, Hq))) for _ in range(24)] + [(0, 0), (n - 1, Hq - 1)]
        ref, rlse = tree_attn_rows_ref(qs[b], kpre, vpre, tks[b], tvs[b], ancs[b], n, scale, rows)
        got = np.stack([out[b, v, h] for v, h in rows])
        err = np.abs(got - ref)
        assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR, b
        assert np.abs(np.array([lse[b, h, v] for v, h in rows]) - rlse).max() <= LSE_ERR
        assert (out[b, n:] == 0).all()


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("batch,B,Hq,Hkv,D", [(3, 16, 8, 2, 64), (5, 64, 8, 2, 128), (32, 64, 32, 8, 128)])
def test_batched_paged_ragged(batch, B, Hq, Hkv, D, flags):
    import jet_harness as H
    rng = np.random.default_rng(4000 + batch)
    if batch == 32:
        seq = rng.integers(100, 600, size=batch).astype(np.int32)      # shape of the serving case, shorter
    else:
        seq = rng.integers(0, 400, size=batch).astype(np.int32)
        seq[0] = 16 * 5
        seq[1] = 0
    kp, vp, table = make_paged_cache(rng, seq, 16, Hkv, D, reserve=9)
    # rows past each sequence's length are junk: poison them
    for b in range(batch):
        for pos in range(int(seq[b]), (int(seq[b]) + 9 + 15) // 16 * 16):
            kp[table[b, pos // 16], pos % 16] = NAN_BITS
            vp[table[b, pos // 16], pos % 16] = NAN_BITS
    n_nodes = rng.integers(1, B + 1, size=batch)
    n_nodes[0] = B
    qs, tks, tvs, ancs = [], [], [], []
    for b in range(batch):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, 0)
        parent, _, _ = random_tree(int(n_nodes[b]), rng, max_depth=8)
        qs.append(x["q"]); tks.append(x["tree_k"]); tvs.append(x["tree_v"])
        ancs.append(anc_from_parent(parent, int(n_nodes[b]), B))
    scale = 1.0 / np.sqrt(D)
    out, lse, st = H.run_tree_attn(np.stack(qs), kp, vp, table, seq, np.stack(tks), np.stack(tvs), np.stack(ancs),
                                   n_nodes, scale, flags=flags)
    assert st == 0
    check = range(batch) if batch <= 5 else (0, 7, 31)
    for b in check:
        kpre = gather_paged_prefix(kp, table[b], int(seq[b]))
        vpre = gather_paged_prefix(vp, table[b], int(seq[b]))
        ref, rlse = tree_attn_ref(qs[b], kpre, vpre, tks[b], tvs[b], ancs[b], int(n_nodes[b]), scale)
        _check(out[b], lse[b], ref, rlse, int(n_nodes[b]))


def test_batched_contiguous_with_batch_stride():
    import jet_harness as H
    rng = np.random.default_rng(99)
    batch, B, Hq, Hkv, D, Lmax = 3, 32, 8, 2, 128, 300
    seq = np.array([300, 17, 128], dtype=np.int32)
    kc = np.full((batch, Lmax, Hkv, D), NAN_BITS, np.uint16); vc = np.full_like(kc, NAN_BITS)
    xs, ancs = [], []
    for b in range(batch):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, int(seq[b]))
        kc[b, :seq[b]], vc[b, :seq[b]] = x["k_prefix"], x["v_prefix"]
        parent, _, _ = random_tree(B, rng)
        xs.append(x); ancs.append(anc_from_parent(parent, B, B))
    scale = 1.0 / np.sqrt(D)
    out, lse, st = H.run_tree_attn(np.stack([x["q"] for x in xs]), kc, vc, None, seq,
                                   np.stack([x["tree_k"] for x in xs]), np.stack([x["tree_v"] for x in xs]),
                                   np.stack(ancs), [B] * batch, scale, max_seq_len=Lmax)
    assert st == 0
    for b in range(batch):
        x = xs[b]
        ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], ancs[b], B, scale)
        _check(out[b], lse[b], ref, rlse, B)


def test_argument_errors():
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    t = torch.zeros(1 << 16, dtype=torch.bfloat16, device=H.DEV)
    i32 = torch.ones(64, dtype=torch.int32, device=H.DEV)
    ws = H.workspace(1 << 20)
    args = dict(q=t, k_cache=t, v_cache=t, page_table=None, max_pages_per_seq=0, page_size=0, num_pages=0,
                seq_len=i32, max_seq_len=16, tree_k=t, tree_v=t, anc_mask=i32, n_nodes=i32, batch=1, B=8, Hq=8,
                Hkv=2, D=128, kv_batch_stride=0, softmax_scale=0.1, out=t, lse=None, device_status=None,
                workspace=ws, check=False)
    assert jet.jet_tree_verify_attn(**{**args, "D": 96}) == jet.JET_ERR_UNSUPPORTED
    assert jet.jet_tree_verify_attn(**{**args, "Hq": 6, "Hkv": 2}) == jet.JET_ERR_UNSUPPORTED
    assert jet.jet_tree_verify_attn(**{**args, "Hq": 7}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_verify_attn(**{**args, "B": 513}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_verify_attn(**{**args, "q": None}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_verify_attn(**{**args, "workspace": None}) == jet.JET_ERR_WORKSPACE
    assert jet.jet_tree_verify_attn(**{**args, "softmax_scale": -0.1}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_verify_attn(**{**args, "softmax_scale": float("nan")}) == jet.JET_ERR_INVALID_ARG
    assert jet.jet_tree_verify_attn(**{**args, "page_table": i32, "page_size": 32, "max_pages_per_seq": 4,
                                       "num_pages": 4}) == jet.JET_ERR_UNSUPPORTED


def test_workspace_counters_are_left_clean_across_repeated_calls():
    """The slice exchange through the workspace counts arrivals in the workspace head; every call must
    leave the counters at zero so that the same workspace serves the next call (here: 5 calls, two shapes)."""
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    rng = np.random.default_rng(5)
    B, Hq, Hkv, D, L = 64, 32, 8, 128, 4096
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(B, rng)
    anc = anc_from_parent(parent, B, B)
    scale = 1.0 / np.sqrt(D)
    ref, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
    nbytes = jet.jet_tree_verify_attn_workspace_bytes(1, B, Hq, Hkv, D, L)
    assert nbytes > 4096, "this shape is expected to use the workspace exchange"
    ws = torch.zeros(nbytes, dtype=torch.uint8, device=H.DEV)
    d = dict(q=H.dev_bf16(x["q"][None]), k=H.dev_bf16(x["k_prefix"][None]), v=H.dev_bf16(x["v_prefix"][None]),
             tk=H.dev_bf16(x["tree_k"][None]), tv=H.dev_bf16(x["tree_v"][None]), anc=H.dev(anc[None].view(np.int32)),
             n=H.dev(np.array([B], np.int32)), seq=H.dev(np.array([L], np.int32)))
    status = torch.zeros(1, dtype=torch.int32, device=H.DEV)
    for it in range(5):
        out = torch.full((1, B, Hq, D), float("nan"), dtype=torch.bfloat16, device=H.DEV)
        jet.jet_tree_verify_attn(d["q"], d["k"], d["v"], None, 0, 0, 0, d["seq"], L, d["tk"], d["tv"], d["anc"], d["n"],
                                 1, B, Hq, Hkv, D, L * Hkv * D, float(scale), out, None, status, ws)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        err = np.abs(H.bf16_to_f64(out)[0] - ref)
        assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR, it
        assert int(ws[:4096].view(torch.int32).abs().sum().item()) == 0, "counters not reset"


def test_two_streams_with_their_own_workspaces():
    """Calls that may overlap on the device are allowed as long as each has its own workspace: two streams
    run the benchmark shape back to back, interleaved, and every result matches the oracle."""
    import torch
    import jet_harness as H
    import paper_2606_18394_b200 as jet
    rng = np.random.default_rng(8)
    B, Hq, Hkv, D, L = 64, 32, 8, 128, 4096
    scale = 1.0 / np.sqrt(D)
    cases = []
    for _ in range(2):
        x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
        parent, _, _ = random_tree(B, rng)
        anc = anc_from_parent(parent, B, B)
        ref, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
        d = dict(q=H.dev_bf16(x["q"][None]), k=H.dev_bf16(x["k_prefix"][None]), v=H.dev_bf16(x["v_prefix"][None]),
                 tk=H.dev_bf16(x["tree_k"][None]), tv=H.dev_bf16(x["tree_v"][None]),
                 anc=H.dev(anc[None].view(np.int32)), n=H.dev(np.array([B], np.int32)),
                 seq=H.dev(np.array([L], np.int32)),
                 ws=torch.zeros(jet.jet_tree_verify_attn_workspace_bytes(1, B, Hq, Hkv, D, L), dtype=torch.uint8,
                                device=H.DEV),
                 status=torch.zeros(1, dtype=torch.int32, device=H.DEV),
                 outs=[torch.full((1, B, Hq, D), float("nan"), dtype=torch.bfloat16, device=H.DEV) for _ in range(6)],
                 stream=torch.cuda.Stream())
        cases.append((d, ref))
    torch.cuda.synchronize()
    for it in range(6):
        for d, _ in cases:
            jet.jet_tree_verify_attn(d["q"], d["k"], d["v"], None, 0, 0, 0, d["seq"], L, d["tk"], d["tv"], d["anc"],
                                     d["n"], 1, B, Hq, Hkv, D, L * Hkv * D, float(scale), d["outs"][it], None,
                                     d["status"], d["ws"], stream=d["stream"])
    torch.cuda.synchronize()
    for d, ref in cases:
        assert int(d["status"].item()) == 0
        for out in d["outs"]:
            err = np.abs(H.bf16_to_f64(out)[0] - ref)
            assert err.max() <= MAX_ERR and err.mean() <= MEAN_ERR


def test_two_query_tiles_per_cta_variant():
    """The planner picks the kernel variant with two query tiles per CTA for batched shapes only;
    JET_FORCE_MT=2 selects it for these single-sequence shapes too (read once per process, hence the
    child process)."""
    import os
    import subprocess
    import sys
    code = r'''
import sys, os
sys.path.insert(0, os.getcwd()); sys.path.insert(0, os.path.join(os.getcwd(), "tests"))
import numpy as np
import jet_harness as H
from jet_inputs import make_attn_inputs, random_tree
from oracle import anc_from_parent, tree_attn_ref
for B, Hq, Hkv, D, L, n in ((96, 8, 2, 128, 700, 96), (64, 8, 2, 64, 300, 50), (256, 8, 2, 128, 140, 256)):
    rng = np.random.default_rng(B + L)
    x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
    parent, _, _ = random_tree(n, rng)
    anc = anc_from_parent(parent, n, B)
    scale = 1.0 / np.sqrt(D)
    ref, rlse = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, n, scale)
    out, lse, st = H.run_tree_attn(x["q"][None], x["k_prefix"][None], x["v_prefix"][None], None, [L], x["tree_k"][None],
                                   x["tree_v"][None], anc[None], [n], scale)
    err = np.abs(out[0] - ref)
    assert st == 0 and err.max() <= 2e-2 and err.mean() <= 2e-3, (B, st, err.max(), err.mean())
    assert (out[0][n:] == 0).all() and np.abs(lse[0][:, :n] - rlse[:, :n]).max() <= 1e-3
print("ok")
'''
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, JET_FORCE_MT="2")
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "ok" in res.stdout, res.stdout + res.stderr


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_library_usable():
    """Failure made on the host: the workspace's arrival counter of the first work item is preset to a value from
    which the key slices can never count up to their number (a dirty workspace is a caller error the header
    describes).  With the poll limit of the workspace exchange shortened (test hook), every CTA of that work
    item gives up within milliseconds: the call returns, device_status reads JET_ERR_TIMEOUT, nothing hangs or
    faults, and the next call on a re-zeroed workspace is correct (TMEM was released, no barrier left armed)."""
    import os
    import subprocess
    import sys
    code = r'''
import sys, os
sys.path.insert(0, os.getcwd()); sys.path.insert(0, os.path.join(os.getcwd(), "tests"))
import numpy as np, torch
import jet_harness as H
import paper_2606_18394_b200 as jet
from jet_inputs import make_attn_inputs, random_tree
from oracle import anc_from_parent, tree_attn_ref
B, Hq, Hkv, D, L = 32, 8, 2, 128, 600
rng = np.random.default_rng(3)
x = make_attn_inputs(rng, B, Hq, Hkv, D, L)
parent, _, _ = random_tree(B, rng)
anc = anc_from_parent(parent, B, B)
scale = 1.0 / np.sqrt(D)
ref, _ = tree_attn_ref(x["q"], x["k_prefix"], x["v_prefix"], x["tree_k"], x["tree_v"], anc, B, scale)
nbytes = jet.jet_tree_verify_attn_workspace_bytes(1, B, Hq, Hkv, D, L)
assert nbytes > 4096, "the forced plan must exchange through the workspace"
ws = torch.zeros(nbytes, dtype=torch.uint8, device=H.DEV)
d = dict(q=H.dev_bf16(x["q"][None]), k=H.dev_bf16(x["k_prefix"][None]), v=H.dev_bf16(x["v_prefix"][None]),
         tk=H.dev_bf16(x["tree_k"][None]), tv=H.dev_bf16(x["tree_v"][None]), anc=H.dev(anc[None].view(np.int32)),
         n=H.dev(np.array([B], np.int32)), seq=H.dev(np.array([L], np.int32)))
def call(out, status):
    return jet.jet_tree_verify_attn(d["q"], d["k"], d["v"], None, 0, 0, 0, d["seq"], L, d["tk"], d["tv"], d["anc"],
                                    d["n"], 1, B, Hq, Hkv, D, L * Hkv * D, float(scale), out, None, status, ws,
                                    check=False)
status = torch.zeros(1, dtype=torch.int32, device=H.DEV)
out = torch.full((1, B, Hq, D), float("nan"), dtype=torch.bfloat16, device=H.DEV)
ws[:4096].view(torch.int32)[0] = -1000          # the first work item's arrival count can never reach its slice count
assert call(out, status) == jet.JET_OK          # the call itself is asynchronous and has nothing to report yet
torch.cuda.synchronize()                        # returns: every wait was bounded
assert int(status.item()) == jet.JET_ERR_TIMEOUT, int(status.item())
# second call, workspace zeroed again: correct, and the status word is only ever set, never cleared, by the library
ws.zero_(); status.zero_()
out2 = torch.full((1, B, Hq, D), float("nan"), dtype=torch.bfloat16, device=H.DEV)
assert call(out2, status) == jet.JET_OK
torch.cuda.synchronize()
assert int(status.item()) == 0
err = np.abs(H.bf16_to_f64(out2)[0] - ref)
assert not np.isnan(H.bf16_to_f64(out2)).any() and err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
assert int(ws[:4096].view(torch.int32).abs().sum().item()) == 0
print("ok")
'''
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, JET_FORCE_MT="1", JET_FORCE_SPLIT="2,g", JET_TEST_POLL_LIMIT="2000")
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "ok" in res.stdout, res.stdout[-2000:] + res.stderr[-3000:]
