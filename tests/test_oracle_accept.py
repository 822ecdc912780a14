"""Pins for the greedy-acceptance oracle (Section 3.3 / Appendix E).

Checked against a hand-worked example, the expected-token closed form of
Eq. (1) on chains (Monte Carlo), an independent ancestor-bitmask formulation,
planted paths and degenerate cases.
"""
import json
import os

import numpy as np
import pytest

from jet_inputs import chain_tree, make_logp, make_target_logits, plant_path, random_tree
from oracle import anc_from_parent, tree_accept_ref, tree_build_ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _logits_with_argmax(tgt, V):
    logits = np.zeros((len(tgt), V), dtype=np.float32)
    for v, t in enumerate(tgt):
        logits[v, t] = 1.0
    return logits


def test_handworked_example():
    g = json.load(open(os.path.join(GOLDEN, "tree_accept_handworked.json")))
    B = len(g["parent"])
    parent = np.array(g["parent"])
    depth = np.zeros(B, dtype=np.int32)
    for v in range(1, B):
        depth[v] = depth[parent[v]] + 1
    r = tree_accept_ref(_logits_with_argmax(g["tgt"], 100), np.array(g["token"]), parent, depth, B, g["N"])
    assert r["tgt"].tolist() == g["tgt"]
    assert r["accept_len"] == g["accept_len"]
    assert r["path"].tolist() == g["path"]
    assert r["out_tokens"].tolist() == g["out_tokens"]


def test_argmax_takes_first_maximum():
    logits = np.array([[0.0, 3.0, 3.0, -1.0], [5.0, 5.0, 5.0, 5.0]], dtype=np.float32)
    parent, depth, token = np.array([-1, 0]), np.array([0, 1]), np.array([9, 1])
    r = tree_accept_ref(logits, token, parent, depth, 2, 1)
    assert r["tgt"].tolist() == [1, 0]
    assert r["accept_len"] == 1 and r["out_tokens"].tolist() == [1, 0]


def test_expected_tokens_closed_form_on_chains():
    """Eq. (1): with i.i.d. per-token acceptance alpha on a chain of N draft tokens,
    E[#tokens advanced] = (1 - alpha^(N+1)) / (1 - alpha)."""
    rng = np.random.default_rng(2024)
    N, V, trials = 6, 50, 20000
    parent, depth, token = chain_tree(N + 1)
    token = (np.arange(N + 1) % (V - 1)).astype(np.int32)
    for alpha in (0.3, 0.8):
        total = 0
        for _ in range(trials):
            ok = rng.random(N + 1) < alpha
            # node v's target prediction equals the child's token with probability alpha
            tgt = [int(token[v + 1]) if (v < N and ok[v]) else V - 1 for v in range(N + 1)]
            r = tree_accept_ref(_logits_with_argmax(tgt, V), token, parent, depth, N + 1, N)
            total += r["accept_len"] + 1
        expect = (1 - alpha ** (N + 1)) / (1 - alpha)
        sigma = 2.5 / np.sqrt(trials)               # generous bound on the std of the mean
        assert abs(total / trials - expect) < 4 * sigma


@pytest.mark.parametrize("seed", range(8))
def test_bitmask_formulation_agrees(seed):
    """acc[v] = all of Anc(v)+{v} match  <=>  (anc[v] & ~match_bits) == 0; deepest accepted node wins."""
    rng = np.random.default_rng(seed)
    B, V, N = 40, 6, 7
    parent, depth, token = random_tree(B, rng, V=V, max_depth=N)
    logits = make_target_logits(rng, B, V, 1.0)
    r = tree_accept_ref(logits, token, parent, depth, B, N)
    tgt = logits.argmax(1)
    match = 1
    for v in range(1, B):
        if token[v] == tgt[parent[v]]:
            match |= 1 << v
    anc = anc_from_parent(parent, B, B)
    best = (0, 0)
    for v in range(B):
        row = int(anc[v, 0]) | (int(anc[v, 1]) << 32)
        if row & ~match == 0 and (depth[v] > best[0]):
            best = (int(depth[v]), v)
    assert r["accept_len"] == best[0]
    assert r["end_node"] == best[1]
    assert r["out_tokens"][r["accept_len"]] == tgt[r["end_node"]]
    assert [int(x) for x in r["path"] if x >= 0][-1] == r["end_node"]


@pytest.mark.parametrize("seed", range(4))
def test_planted_path_is_recovered(seed):
    rng = np.random.default_rng(300 + seed)
    N, W, B, V = 6, 4, 32, 2000
    logp = make_logp(rng, N, V, 2.0, peaked_p=0.7)
    t = tree_build_ref(logp, 1, N, W, B)
    for want in (0, 1, 3, 6):
        logits = make_target_logits(rng, B, V, 2.0)
        end, eff = plant_path(logits, t["token"], t["parent"], t["depth"], t["n_nodes"], want, rng)
        r = tree_accept_ref(logits, t["token"], t["parent"], t["depth"], t["n_nodes"], N)
        assert r["accept_len"] == eff == t["depth"][end]
        assert r["end_node"] == end
        assert r["out_tokens"][:eff].tolist() == [int(t["token"][v]) for v in r["path"][1:eff + 1]]


def test_all_mismatch_and_full_chain():
    N, V = 5, 30
    parent, depth, token = chain_tree(N + 1)
    token = np.arange(10, 10 + N + 1).astype(np.int32)
    r = tree_accept_ref(_logits_with_argmax([0] * (N + 1), V), token, parent, depth, N + 1, N)
    assert r["accept_len"] == 0 and r["out_tokens"].tolist() == [0] + [-1] * N and r["path"][0] == 0
    tgt = [int(token[v + 1]) for v in range(N)] + [3]
    r = tree_accept_ref(_logits_with_argmax(tgt, V), token, parent, depth, N + 1, N)
    assert r["accept_len"] == N and r["out_tokens"].tolist() == tgt
    assert r["path"].tolist() == list(range(N + 1))


def test_duplicate_sibling_tokens_take_smallest_end_node_and_padding_ignored():
    parent = np.array([-1, 0, 0, -1]); depth = np.array([0, 1, 1, -1]); token = np.array([1, 7, 7, -1])
    logits = _logits_with_argmax([7, 2, 3, 0], 10)
    r = tree_accept_ref(logits, token, parent, depth, 3, 2)
    assert r["accept_len"] == 1 and r["end_node"] == 1 and r["out_tokens"].tolist() == [7, 2, -1]
    assert r["tgt"][3] == -1
