"""Pins for lm_head_argmax_ref (the target's greedy prediction from its final hidden states, Section 3.3 /
Appendix E): exact integer arithmetic by brute force, one-hot hidden states, ties, sign flip, widening of the
bfloat16 inputs."""
import numpy as np

from jet_inputs import f32_to_bf16_bits
from oracle import lm_head_argmax_ref


def test_small_integers_against_brute_force_sums():
    rng = np.random.default_rng(1)
    R, d, V = 5, 7, 11
    h = rng.integers(-4, 5, size=(R, d))
    w = rng.integers(-4, 5, size=(V, d))
    want_logits = [[sum(int(h[r, k]) * int(w[t, k]) for k in range(d)) for t in range(V)] for r in range(R)]
    want_tgt = [min(range(V), key=lambda t: (-row[t], t)) for row in want_logits]         # largest, then lowest id
    for hh, ww in ((h.astype(np.float64), w.astype(np.float64)),
                   (f32_to_bf16_bits(h.astype(np.float32)), f32_to_bf16_bits(w.astype(np.float32)))):   # small ints are exact in bf16
        got = lm_head_argmax_ref(hh, ww)
        assert np.array_equal(got["logits"], np.array(want_logits, dtype=np.float64))
        assert got["tgt"].tolist() == want_tgt
        want_abs = [[sum(abs(int(h[r, k]) * int(w[t, k])) for k in range(d)) for t in range(V)] for r in range(R)]
        assert np.array_equal(got["abs_dot"], np.array(want_abs, dtype=np.float64))


def test_one_hot_hidden_state_selects_a_weight_column():
    rng = np.random.default_rng(2)
    V, d = 9, 6
    w = rng.normal(size=(V, d))
    for k in range(d):
        h = np.zeros((1, d))
        h[0, k] = 2.0
        got = lm_head_argmax_ref(h, w)
        assert got["tgt"][0] == int(np.argmax(w[:, k]))
        np.testing.assert_allclose(got["logits"][0], 2.0 * w[:, k], rtol=0, atol=0)
        # a transposed weight matrix would pick the arg-max of a ROW of w here
    assert lm_head_argmax_ref(np.eye(d)[:1], w.copy())["logits"].shape == (1, V)


def test_ties_go_to_the_lowest_token_and_negation_gives_the_arg_min():
    w = np.array([[1.0, 0.0], [3.0, 1.0], [3.0, 1.0], [-5.0, 2.0], [3.0, 1.0]])
    h = np.array([[1.0, 0.0], [0.0, 1.0], [-1.0, 0.0]])
    got = lm_head_argmax_ref(h, w)
    assert got["tgt"].tolist() == [1, 3, 3]            # row 0: tokens 1, 2, 4 tie at 3 -> 1; row 2: -(-5) = 5 -> 3
    rng = np.random.default_rng(3)
    w2, h2 = rng.normal(size=(20, 8)), rng.normal(size=(4, 8))
    a, b = lm_head_argmax_ref(h2, w2), lm_head_argmax_ref(-h2, w2)
    assert np.array_equal(b["tgt"], np.argmin(a["logits"], axis=1))
    assert np.array_equal(a["abs_dot"], b["abs_dot"])


def test_bf16_inputs_are_widened_exactly():
    hb = np.array([[0x3F80, 0xC000, 0x3FC0]], dtype=np.uint16)          # 1.0, -2.0, 1.5
    wb = np.array([[0x4000, 0x3F80, 0x0000], [0x3F00, 0xBF80, 0x4080]], dtype=np.uint16)   # (2, 1, 0), (0.5, -1, 4)
    got = lm_head_argmax_ref(hb, wb)
    assert got["logits"].tolist() == [[0.0, 8.5]]
    assert got["tgt"].tolist() == [1]
