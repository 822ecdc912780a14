"""Pins for the non-greedy acceptance oracle (Section 3.3, Eq. nongreedy_specdec).

The rule is pinned by what the mathematics fixes: on a chain whose tokens were drawn from the draft
distribution, the emitted tokens are distributed exactly as under the target model (the defining property of
speculative sampling); the expected accepted length has a closed form; q == p accepts everything; a token the
target gives no mass is never accepted nor emitted as correction; and the deepest-accepted-node selection is
cross-checked by brute force over leaves."""
import numpy as np

from oracle import target_probs_ref, tree_accept_sample_ref


def _log_softmax(x):
    x = np.asarray(x, np.float64)
    x = x - x.max(axis=-1, keepdims=True)
    return x - np.log(np.exp(x).sum(axis=-1, keepdims=True))


def _chain(tokens):
    n = len(tokens) + 1
    token = np.array([0] + list(tokens), np.int32)
    parent = np.arange(-1, n - 1, dtype=np.int32)
    depth = np.arange(n, dtype=np.int32)
    return token, parent, depth, n


def test_first_emitted_token_is_distributed_as_the_target():
    rng = np.random.default_rng(11)
    V, trials = 6, 40000
    p_logits = rng.normal(size=V).astype(np.float32) * 1.5
    q_logp = _log_softmax(rng.normal(size=(1, V)) * 1.5)
    p = target_probs_ref(p_logits, 1.0)
    q = np.exp(q_logp[0])
    counts = np.zeros(V)
    accepted = 0
    for _ in range(trials):
        y = int(rng.choice(V, p=q))
        token, parent, depth, n = _chain([y])
        logits = np.stack([p_logits, rng.normal(size=V).astype(np.float32)])
        r = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, n, 1, rng.random(n), rng.random())
        counts[r["out_tokens"][0]] += 1
        accepted += r["accept_len"]
    freq = counts / trials
    sigma = np.sqrt(p * (1 - p) / trials)
    assert np.all(np.abs(freq - p) < 5 * sigma + 1e-9), (freq, p)
    # acceptance rate of one draft token: sum_x min(p, q)
    rate = np.minimum(p, q).sum()
    assert abs(accepted / trials - rate) < 5 * np.sqrt(rate * (1 - rate) / trials)


def test_second_token_follows_the_target_conditional():
    rng = np.random.default_rng(12)
    V, trials = 4, 40000
    root_logits = rng.normal(size=V).astype(np.float32)
    cond_logits = rng.normal(size=(V, V)).astype(np.float32) * 1.5        # target row after first token a
    q_logp = _log_softmax(rng.normal(size=(2, V)))
    counts = np.zeros((V, V))
    for _ in range(trials):
        y1, y2 = int(rng.choice(V, p=np.exp(q_logp[0]))), int(rng.choice(V, p=np.exp(q_logp[1])))
        token, parent, depth, n = _chain([y1, y2])
        logits = np.stack([root_logits, cond_logits[y1], rng.normal(size=V).astype(np.float32)])
        r = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, n, 2, rng.random(n), rng.random())
        if r["accept_len"] >= 1:
            counts[r["out_tokens"][0], r["out_tokens"][1]] += 1
    for a in range(V):
        n_a = counts[a].sum()
        if n_a < 2000:
            continue
        p = target_probs_ref(cond_logits[a], 1.0)
        sigma = np.sqrt(p * (1 - p) / n_a)
        assert np.all(np.abs(counts[a] / n_a - p) < 5 * sigma + 1e-9), a


def test_expected_accepted_length_closed_form():
    rng = np.random.default_rng(13)
    V, N, trials = 8, 4, 30000
    tokens = [1, 2, 3, 4]
    alphas = [0.9, 0.5, 0.7, 0.3]
    q_logp = np.full((N, V), np.log(1.0 / V))
    logits = np.zeros((N + 1, V), np.float32)
    for t in range(N):                     # p(token) = alpha / V, the rest of the mass on token 0
        p = np.full(V, 0.0)
        p[tokens[t]] = alphas[t] / V
        p[0] = 1.0 - p[tokens[t]]
        logits[t] = np.log(np.maximum(p, 1e-300)).astype(np.float32)
    token, parent, depth, n = _chain(tokens)
    total = 0
    for _ in range(trials):
        r = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, n, N, rng.random(n), rng.random())
        total += r["accept_len"]
    expect = sum(np.prod(alphas[: k + 1]) for k in range(N))
    assert abs(total / trials - expect) < 0.03


def test_equal_distributions_accept_the_whole_chain_and_bonus_comes_from_the_target():
    rng = np.random.default_rng(14)
    V, N = 16, 5
    rows = rng.normal(size=(N + 1, V)).astype(np.float32)
    q_logp = _log_softmax(rows[:N])
    tokens = [int(rng.integers(V)) for _ in range(N)]
    token, parent, depth, n = _chain(tokens)
    for _ in range(50):
        u_s = rng.random()
        r = tree_accept_sample_ref(rows, 1.0, q_logp, token, parent, depth, n, N, rng.random(n), u_s)
        assert r["accept_len"] == N and not r["residual_used"]
        cdf = np.cumsum(target_probs_ref(rows[N], 1.0))
        assert r["correction"] == int(np.searchsorted(cdf, u_s * cdf[-1], side="right"))


def test_token_without_target_mass_is_rejected_and_never_emitted():
    rng = np.random.default_rng(15)
    V = 10
    logits = rng.normal(size=(2, V)).astype(np.float32)
    logits[0, 3] = -np.inf
    q_logp = _log_softmax(rng.normal(size=(1, V)))
    token, parent, depth, n = _chain([3])
    for _ in range(200):
        r = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, n, 1, rng.random(n), rng.random())
        assert r["accept_len"] == 0 and r["correction"] != 3 and r["residual_used"]
        assert r["dist"][r["correction"]] > 0


def test_inverse_cdf_end_points_and_temperature():
    V = 5
    logits = np.array([[0.0, -np.inf, 1.0, 2.0, -np.inf]], np.float32)
    token, parent, depth = np.array([0], np.int32), np.array([-1], np.int32), np.array([0], np.int32)
    q_logp = np.zeros((1, V))
    first = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, 1, 1, np.zeros(1), 0.0)
    last = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, 1, 1, np.zeros(1), 1.0 - 1e-12)
    assert first["correction"] == 0 and last["correction"] == 3        # never a token without mass
    cold = tree_accept_sample_ref(logits, 0.05, q_logp, token, parent, depth, 1, 1, np.zeros(1), 0.5)
    assert cold["correction"] == 3                                      # low temperature concentrates on the arg-max
    assert np.isclose(target_probs_ref(logits[0], 2.0)[2] / target_probs_ref(logits[0], 2.0)[0], np.exp(0.5))


def test_deepest_accepted_node_matches_brute_force_over_leaves():
    rng = np.random.default_rng(16)
    V, N, B = 12, 4, 24
    for trial in range(200):
        parent = np.full(B, -1, np.int32)
        depth = np.zeros(B, np.int32)
        for v in range(1, B):
            cands = [u for u in range(v) if depth[u] < N]
            parent[v] = int(rng.choice(cands))
            depth[v] = depth[parent[v]] + 1
        token = rng.integers(0, V, size=B).astype(np.int32)
        logits = rng.normal(size=(B, V)).astype(np.float32)
        q_logp = _log_softmax(rng.normal(size=(N, V)))
        u = rng.random(B)
        r = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, B, N, u, rng.random())
        # brute force: walk every root-to-leaf path, stop at the first rejected node
        best_len, best_end = 0, 0
        for leaf in range(B):
            chain, v = [], leaf
            while v != -1:
                chain.append(v)
                v = int(parent[v])
            chain.reverse()
            k = 0
            for t in range(1, len(chain)):
                if r["ok"][chain[t]]:
                    k = t
                else:
                    break
            end = chain[k]
            if k > best_len or (k == best_len and end < best_end):
                best_len, best_end = k, end
        assert (r["accept_len"], r["end_node"]) == (best_len, best_end)
        assert list(r["path"][: best_len + 1]) == [int(x) for x in r["path"][: best_len + 1]]
        assert r["path"][0] == 0 and r["path"][best_len] == best_end


def test_branched_tree_applies_the_rule_per_branch_and_is_not_target_distributed():
    """The reading taken for several siblings (the paper gives the per-branch rule only): every sibling is tested
    on its own against the same target distribution and the deepest passing branch wins, lowest index first.
    That is exact on chains (tests above) and NOT distribution-preserving on branched trees -- the header of the
    library says so.  Pinned here so that the behaviour cannot drift unnoticed: with q == p two siblings both
    pass whatever the random numbers are, so the first emitted token is always the lower-indexed sibling's,
    where the target would emit it with probability p only."""
    rng = np.random.default_rng(5)
    V = 5
    p_logits = np.log(np.array([0.4, 0.3, 0.15, 0.1, 0.05])).astype(np.float32)
    q_logp = _log_softmax(p_logits[None].astype(np.float64))          # q == p at depth 0
    token = np.array([0, 1, 0], np.int32)                              # root, two children: tokens 1 and 0
    parent = np.array([-1, 0, 0], np.int32)
    depth = np.array([0, 1, 1], np.int32)
    logits = np.stack([p_logits, rng.normal(size=V).astype(np.float32), rng.normal(size=V).astype(np.float32)])
    firsts = set()
    for _ in range(200):
        r = tree_accept_sample_ref(logits, 1.0, q_logp, token, parent, depth, 3, 1, rng.random(3), rng.random())
        assert r["accept_len"] == 1 and r["path"][1] == 1              # sibling with the lower node index
        firsts.add(int(r["out_tokens"][0]))
    assert firsts == {1}                                               # always token 1; the target gives it 0.3
    # a sibling that fails its own test does not stop the other one
    q2 = _log_softmax(np.log(np.array([[0.02, 0.9, 0.02, 0.03, 0.03]])))    # token 1 over-proposed: alpha = 0.3 / 0.9
    r = tree_accept_sample_ref(logits, 1.0, q2, token, parent, depth, 3, 1, np.array([0.0, 0.9, 0.5]), 0.3)
    assert r["accept_len"] == 1 and r["path"][1] == 2 and r["out_tokens"][0] == 0
