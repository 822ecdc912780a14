"""Pins for log_softmax_ref / tree_build_logits_ref (draft log-probabilities from raw logits, Section 3.3).

The log-softmax is checked against scipy's routine, closed forms and the properties that define it; the
tree from logits against properties of the softmax (shift invariance) and against tree_build_ref fed with
log-probabilities that scipy computed -- none of them re-types the oracle's formula.
"""
import math

import numpy as np
import pytest
from scipy.special import log_softmax, logsumexp

from jet_inputs import make_draft_logits
from oracle import log_softmax_ref, tree_build_logits_ref, tree_build_ref


def _same_tree(a, b):
    return (a["n_nodes"] == b["n_nodes"] and all(np.array_equal(a[k], b[k]) for k in ("parent", "depth", "token", "anc_mask")))


@pytest.mark.parametrize("sigma,offset", [(1.0, 0.0), (3.0, 0.0), (3.0, 50.0), (8.0, -200.0)])
def test_against_scipy(sigma, offset):
    rng = np.random.default_rng(int(sigma * 10 + offset + 300))
    z = make_draft_logits(rng, 5, 7001, sigma, offset=offset)
    lp, lse = log_softmax_ref(z)
    assert lp.dtype == np.float32 and lse.dtype == np.float64
    ref = log_softmax(z.astype(np.float64), axis=1)
    assert np.abs(lse - logsumexp(z.astype(np.float64), axis=1)).max() < 1e-11
    # the float32 result is the rounding of the float64 one: at most one ulp from scipy's value rounded
    ref32 = ref.astype(np.float32)
    assert np.abs(lp.view(np.int32).astype(np.int64) - ref32.view(np.int32).astype(np.int64)).max() <= 1
    assert np.abs(lp.astype(np.float64) - ref).max() <= np.spacing(np.abs(ref32)).max()


def test_closed_forms():
    V = 4096
    lp, lse = log_softmax_ref(np.full((1, V), 3.25, np.float32))
    assert abs(lse[0] - (3.25 + math.log(V))) < 1e-12
    assert (lp == np.float32(-math.log(V))).all()
    z = np.full((1, V), -np.inf, np.float32)
    z[0, 7], z[0, 100] = math.log(3.0), 0.0          # probabilities 3/4 and 1/4
    lp, lse = log_softmax_ref(z)
    assert abs(lse[0] - math.log(4.0)) < 1e-7          # log(3) was rounded to float32 on the way in
    assert abs(lp[0, 7] - math.log(0.75)) < 1e-6 and abs(lp[0, 100] - math.log(0.25)) < 1e-6
    assert np.isneginf(lp[0, 0])


def test_rows_sum_to_one_and_shift_invariance():
    rng = np.random.default_rng(9)
    z = make_draft_logits(rng, 3, 20000, 3.0, peaked_p=0.7)
    lp, lse = log_softmax_ref(z)
    assert np.abs(np.exp(lp.astype(np.float64)).sum(axis=1) - 1.0).max() < 1e-5
    # shift every logit by 64 (each entry then moves by 64 up to its float32 rounding): the log-probabilities
    # follow the shift each entry really got, minus the shift of lse
    z2 = (z.astype(np.float64) + 64.0).astype(np.float32)
    lp2, lse2 = log_softmax_ref(z2)
    exact = (z2.astype(np.float64) - z.astype(np.float64))      # the shift each entry really got
    assert np.abs((lse2 - lse) - 64.0).max() < 1e-4                 # entries moved by 64 up to their float32 rounding
    assert np.abs(lp2.astype(np.float64) - lp.astype(np.float64) - (exact - (lse2 - lse)[:, None])).max() < 4e-6


@pytest.mark.parametrize("mode,alpha", [("accum_logp", 0.0), ("entropy", 0.0), ("hybrid", 1.0)])
@pytest.mark.parametrize("seed", range(3))
def test_tree_from_logits_equals_tree_from_scipy_log_probs(mode, alpha, seed):
    rng = np.random.default_rng(70 + seed)
    N, W, B, V = 6, 5, 48, 3000
    z = make_draft_logits(rng, N, V, 2.5, peaked_p=0.6 if seed else None, offset=10.0 * seed)
    a = tree_build_logits_ref(z, 4, N, W, B, score_mode=mode, alpha=alpha)
    lp = log_softmax(z.astype(np.float64), axis=1).astype(np.float32)
    b = tree_build_ref(lp, 4, N, W, B, score_mode=mode, alpha=alpha)
    assert _same_tree(a, b)
    # scores may differ by an ulp per add where scipy's lse differs in its last bits
    assert np.abs(a["score"][:a["n_nodes"]] - b["score"][:b["n_nodes"]]).max() < 1e-5
    assert np.abs(a["depth_lse"] - logsumexp(z.astype(np.float64), axis=1)).max() < 1e-5


def test_tree_is_invariant_under_a_per_row_shift_by_a_power_of_two():
    """softmax(z + c) = softmax(z): with c a power of two far below the logits' ulp range the shifted logits
    are exact, lse moves by exactly c, and the whole tree (scores included) is unchanged bit for bit."""
    rng = np.random.default_rng(5)
    N, W, B, V = 5, 4, 40, 2000
    z = (np.round(make_draft_logits(rng, N, V, 2.0).astype(np.float64) * 1024) / 1024).astype(np.float32)   # 10 fractional bits
    shift = np.array([0.0, 8.0, -16.0, 32.0, 4.0])[:, None]
    z2 = (z.astype(np.float64) + shift).astype(np.float32)
    assert np.array_equal(z2.astype(np.float64), z.astype(np.float64) + shift)       # exact
    a = tree_build_logits_ref(z, 1, N, W, B)
    b = tree_build_logits_ref(z2, 1, N, W, B)
    assert _same_tree(a, b)
    assert np.abs(a["score"] - b["score"]).max() < 1e-5
    assert np.abs((b["depth_lse"] - a["depth_lse"]) - shift[:, 0]).max() < 1e-5


def test_collapsing_logits_tie_to_the_lower_token():
    """Two different logits whose log-probabilities round to the same float32 are ranked by token id (the
    ranking is taken on the rounded log-probabilities)."""
    V = 64
    z = np.full((1, V), -30.0, np.float32)
    z[0, 40] = np.float32(1.0)
    z[0, 10] = np.nextafter(np.float32(1.0), np.float32(0.0))       # one ulp below, lower token id
    z[0, 5] = 20.0                                                   # pushes lse up: log-probs near -19 have coarser ulps
    lp, _ = log_softmax_ref(z)
    assert lp[0, 40] == lp[0, 10]
    t = tree_build_logits_ref(z, 0, 1, 3, 4)
    assert t["token"].tolist() == [0, 5, 10, 40]
