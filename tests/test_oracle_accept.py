"""Pins for the oracle's lossless tree acceptance.

 * hand-worked decision traces at vocabulary 4 (tests/golden/accept_hand_cases.json)
 * greedy == naive comparison over every root-to-node path
 * rejection sampling is lossless: the exact distribution of the first emitted
   token, obtained by enumerating every ordered child tuple at vocabulary 8 and
   measuring the oracle's accept thresholds and bonus intervals as a black box,
   equals the target softmax computed here in numpy
 * special cases with closed forms (q == p, point-mass q, single child)
"""
import itertools
import json
import os

import numpy as np
import pytest

import oracle
from paper_2408_15562_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "accept_hand_cases.json")


def _cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"])
def test_hand_worked_cases(case):
    parent = np.asarray([case["parent"]], np.int32)
    N = parent.shape[1]
    if "target_logits" in case:
        logits = np.asarray([case["target_logits"]], np.float32)
    else:
        with np.errstate(divide="ignore"):
            logits = np.log(np.asarray([case["target_probs"]], np.float64)).astype(np.float32)
    dp = np.asarray([case["draft_probs"]], np.float32) if "draft_probs" in case else None
    r = oracle.tree_accept(logits, dp, np.asarray([case["draft_tokens"]], np.int32), parent,
                           np.asarray([case["temperature"]], np.float32),
                           np.asarray([case["uniforms"]], np.float32))
    k = int(r["n_accepted"][0])
    assert list(r["accepted_path"][0, :k]) == case["accepted_path"]
    assert (r["accepted_path"][0, k:] == -1).all()
    assert int(r["bonus_token"][0]) == case["bonus_token"]
    assert N == len(case["draft_tokens"])


# ---------------------------------------------------------------------------
# greedy
# ---------------------------------------------------------------------------
def _naive_greedy(logits, tokens, parent):
    """Mark every node whose whole root path matches the target argmax; the
    accepted path is the walk through marked nodes taking the lowest index."""
    N = len(parent)
    arg = [int(np.argmax(logits[i])) for i in range(N)]     # np.argmax: first maximum
    ok = [False] * N
    ok[0] = True
    for i in range(1, N):
        ok[i] = ok[parent[i]] and tokens[i] == arg[parent[i]]
    path = [0]
    while True:
        nxt = [c for c in range(N) if parent[c] == path[-1] and ok[c]]
        if not nxt:
            break
        path.append(min(nxt))
    return path, arg[path[-1]]


@pytest.mark.parametrize("seed", range(6))
def test_greedy_equals_naive_per_path(seed):
    rng = np.random.default_rng(100 + seed)
    B, N, V = 3, 20, 12                      # small vocab: duplicate sibling tokens and ties occur
    parent = np.stack([synth.pruned_tree(rng, N, 5, 3) for _ in range(B)]).astype(np.int32)
    logits = rng.integers(-3, 4, size=(B, N, V)).astype(np.float32)   # integer logits: many exact ties
    tokens = np.zeros((B, N), np.int32)
    for b in range(B):
        for i in range(1, N):
            a = int(np.argmax(logits[b, parent[b, i]]))
            tokens[b, i] = a if rng.random() < 0.6 else int(rng.integers(V))
    r = oracle.tree_accept(logits, None, tokens, parent, np.zeros(B, np.float32), None)
    for b in range(B):
        path, bonus = _naive_greedy(logits[b], tokens[b], parent[b])
        k = int(r["n_accepted"][b])
        assert list(r["accepted_path"][b, :k]) == path
        assert int(r["bonus_token"][b]) == bonus


def test_greedy_chain_is_textbook_prefix_match():
    rng = np.random.default_rng(3)
    N, V = 9, 50
    parent = synth.chain_tree(N)[None]
    logits = rng.standard_normal((1, N, V)).astype(np.float32)
    arg = logits[0].argmax(1)
    for n_match in range(N):
        tokens = np.zeros((1, N), np.int32)
        for i in range(1, N):
            tokens[0, i] = arg[i - 1] if i <= n_match else (arg[i - 1] + 1) % V
        r = oracle.tree_accept(logits, None, tokens, parent, np.zeros(1, np.float32), None)
        assert int(r["n_accepted"][0]) == n_match + 1
        assert int(r["bonus_token"][0]) == arg[n_match]


def test_row_stats_against_numpy():
    rng = np.random.default_rng(4)
    x = (rng.standard_normal((5, 1000)) * 3).astype(np.float32)
    x[2, 17] = x[2].max()                     # duplicate maximum: lowest index wins
    x[2, 400] = x[2, 17]
    for T in (1.0, 0.7):
        m, s, a = oracle.row_stats(x, T)
        xd = x.astype(np.float64)
        np.testing.assert_array_equal(m, xd.max(1))
        np.testing.assert_array_equal(a, xd.argmax(1))
        np.testing.assert_allclose(s, np.exp((xd - xd.max(1, keepdims=True)) / T).sum(1), rtol=1e-13)
    assert a[2] == 17


# ---------------------------------------------------------------------------
# rejection sampling: exact distribution by enumeration
# ---------------------------------------------------------------------------
def _softmax(x, T=1.0):
    z = x.astype(np.float64) / T
    z -= z.max()
    e = np.exp(z)
    return e / e.sum()


def _random_dist(rng, V, n_zero):
    w = rng.random(V) + 0.05
    if n_zero:
        w[rng.choice(V, n_zero, replace=False)] = 0.0
    return w / w.sum()


def _one_level_first_token_distribution(logits_row, q_row, m, T):
    """Exact P(first emitted token) for a root with m children drawn without
    replacement from q_row. The oracle is probed as a black box: one batch
    entry per ordered child tuple; accept thresholds come from its decision
    trace and are confirmed by flipping the uniform around them; the bonus
    distribution is walked interval by interval through the inverse CDF."""
    V = len(q_row)
    N = m + 1
    tuples = [t for t in itertools.permutations(range(V), m) if all(q_row[x] > 0 for x in t)]
    weight = []
    for t in tuples:
        wgt, rem = 1.0, 1.0
        for x in t:
            wgt *= q_row[x] / rem
            rem -= q_row[x]
        weight.append(wgt)
    weight = np.asarray(weight)
    assert abs(weight.sum() - 1.0) < 1e-12 or m > np.count_nonzero(q_row)
    B = len(tuples)
    parent = np.tile(synth.star_tree(N), (B, 1)).astype(np.int32)
    logits = np.tile(logits_row.astype(np.float32), (B, N, 1))
    dp = np.tile(q_row.astype(np.float32), (B, N, 1))
    tokens = np.zeros((B, N), np.int32)
    tokens[:, 1:] = np.asarray(tuples, np.int32)
    temp = np.full(B, T, np.float32)
    q32 = q_row.astype(np.float32).astype(np.float64)

    # accept probability of child k given children < k were rejected
    acc = np.zeros((B, m))
    for k in range(1, N):
        force = np.full((B, N), -1, np.int32)
        force[:, 1:k] = 0
        un = np.full((B, N + 1), 0.5, np.float32)
        r = oracle.tree_accept(logits, dp, tokens, parent, temp, un, force)
        p_x = r["trace_p"][:, k]
        q_x = r["trace_rq"][:, k] / 0.5
        a = np.where(q_x > 0, np.minimum(1.0, p_x / np.where(q_x > 0, q_x, 1.0)), (p_x > 0) * 1.0)
        acc[:, k - 1] = a
        # the decision really flips at that threshold
        for sign, expect_accept in ((-1, True), (+1, False)):
            un2 = un.copy()
            probe = a * (1 + sign * 1e-3)
            sel = (a > 1e-3) & (a < 0.998)
            un2[:, k] = np.where(sel, probe, 0.5).astype(np.float32)
            r2 = oracle.tree_accept(logits, dp, tokens, parent, temp, un2, force)
            took = (r2["n_accepted"] == 2) & (r2["accepted_path"][:, 1] == k)
            assert (took[sel] == expect_accept).all()

    # bonus distribution given every child rejected
    force = np.full((B, N), -1, np.int32)
    force[:, 1:] = 0
    bonus = np.zeros((B, V))
    u = np.zeros(B)
    done = np.zeros(B, bool)
    for _ in range(V + 1):
        un = np.full((B, N + 1), 0.5, np.float32)
        un[:, N] = np.minimum(u, 1 - 2.0 ** -24).astype(np.float32)
        r = oracle.tree_accept(logits, dp, tokens, parent, temp, un, force)
        info = r["bonus_info"]
        for b in range(B):
            if done[b]:
                continue
            t = int(r["bonus_token"][b])
            assert bonus[b, t] == 0.0
            bonus[b, t] = (info[b, 2] - info[b, 1]) / info[b, 3]
            if info[b, 5] < 0:
                done[b] = True
            else:
                u[b] = info[b, 2] / info[b, 3] + 1e-6
        if done.all():
            break
    assert done.all()
    np.testing.assert_allclose(bonus.sum(1), 1.0, atol=1e-12)

    dist = np.zeros(V)
    for b, t in enumerate(tuples):
        alive = 1.0
        for k, x in enumerate(t):
            dist[x] += weight[b] * alive * acc[b, k]
            alive *= 1.0 - acc[b, k]
        dist += weight[b] * alive * bonus[b]
    return dist, q32


@pytest.mark.parametrize("m", [1, 2, 3])
@pytest.mark.parametrize("zeros", [(0, 0), (2, 0), (0, 2), (2, 2)])
def test_rejection_sampling_is_lossless_vocab8(m, zeros):
    rng = np.random.default_rng(1000 + 10 * m + zeros[0] * 3 + zeros[1])
    V = 8
    p = _random_dist(rng, V, zeros[0])
    q = _random_dist(rng, V, zeros[1])
    q = q.astype(np.float32).astype(np.float64)       # the oracle sees fp32 draft probabilities
    with np.errstate(divide="ignore"):
        logits = np.log(p).astype(np.float32)          # -inf for zero target mass
    dist, _ = _one_level_first_token_distribution(logits, q / q.sum(), m, 1.0)
    np.testing.assert_allclose(dist, _softmax(logits), atol=2e-7)


def test_rejection_sampling_lossless_at_other_temperature():
    rng = np.random.default_rng(77)
    V = 8
    logits = (rng.standard_normal(V) * 2).astype(np.float32)
    q = _random_dist(rng, V, 0).astype(np.float32).astype(np.float64)
    dist, _ = _one_level_first_token_distribution(logits, q / q.sum(), 2, 0.6)
    np.testing.assert_allclose(dist, _softmax(logits, 0.6), atol=2e-7)


def test_second_level_follows_the_accepted_childs_row():
    """After child c is accepted the walk restarts from c's own rows: the
    first token emitted below c is distributed as softmax(logits[c])."""
    rng = np.random.default_rng(78)
    V = 8
    # tree: root -> {1, 2}; node 2 -> {3, 4}.  Force acceptance of node 2 and
    # enumerate node 2's children exactly as in the one-level case.
    row2 = (rng.standard_normal(V) * 2).astype(np.float32)
    q2 = _random_dist(rng, V, 1).astype(np.float32).astype(np.float64)
    q2 /= q2.sum()
    tuples = [t for t in itertools.permutations(range(V), 2) if all(q2[x] > 0 for x in t)]
    B, N = len(tuples), 5
    parent = np.tile(np.array([-1, 0, 0, 2, 2], np.int32), (B, 1))
    logits = (rng.standard_normal((1, N, V)) * 2).astype(np.float32).repeat(B, 0)
    logits[:, 2] = row2
    dp = np.tile(_random_dist(rng, V, 0).astype(np.float32), (B, N, 1))
    dp[:, 2] = q2.astype(np.float32)
    tokens = np.zeros((B, N), np.int32)
    tokens[:, 1], tokens[:, 2] = 5, 6
    tokens[:, 3:] = np.asarray(tuples, np.int32)
    temp = np.ones(B, np.float32)
    weight = np.asarray([q2[a] * q2[b] / (1 - q2[a]) for a, b in tuples])
    acc = np.zeros((B, 2))
    for k in (3, 4):
        force = np.full((B, N), -1, np.int32)
        force[:, 1], force[:, 2] = 0, 1
        force[:, 3:k] = 0
        un = np.full((B, N + 1), 0.5, np.float32)
        r = oracle.tree_accept(logits, dp, tokens, parent, temp, un, force)
        p_x, q_x = r["trace_p"][:, k], r["trace_rq"][:, k] / 0.5
        acc[:, k - 3] = np.where(q_x > 0, np.minimum(1.0, p_x / np.where(q_x > 0, q_x, 1)), p_x > 0)
    force = np.full((B, N), -1, np.int32)
    force[:, 1], force[:, 2], force[:, 3], force[:, 4] = 0, 1, 0, 0
    bonus = np.zeros((B, V))
    u = np.zeros(B)
    done = np.zeros(B, bool)
    for _ in range(V + 1):
        un = np.full((B, N + 1), 0.5, np.float32)
        un[:, N] = u.astype(np.float32)
        r = oracle.tree_accept(logits, dp, tokens, parent, temp, un, force)
        assert (r["accepted_path"][:, :2] == [0, 2]).all() and (r["n_accepted"] == 2).all()
        for b in range(B):
            if done[b]:
                continue
            info = r["bonus_info"][b]
            bonus[b, int(r["bonus_token"][b])] = (info[2] - info[1]) / info[3]
            done[b] = info[5] < 0
            u[b] = info[2] / info[3] + 1e-6
    dist = np.zeros(V)
    for b, t in enumerate(tuples):
        alive = 1.0
        for k, x in enumerate(t):
            dist[x] += weight[b] * alive * acc[b, k]
            alive *= 1 - acc[b, k]
        dist += weight[b] * alive * bonus[b]
    np.testing.assert_allclose(dist, _softmax(row2), atol=2e-7)


def test_closed_form_special_cases():
    rng = np.random.default_rng(79)
    V = 8
    logits = (rng.standard_normal(V) * 2).astype(np.float32)
    p = _softmax(logits)
    parent = synth.star_tree(2)[None]
    temp = np.ones(1, np.float32)
    lg = np.tile(logits, (1, 2, 1))
    # q == p (to fp32): the first child is accepted for every uniform below ~1
    dp = np.tile(p.astype(np.float32), (1, 2, 1))
    for x in range(V):
        for r in (0.0, 0.5, 0.99):
            out = oracle.tree_accept(lg, dp, np.array([[0, x]], np.int32), parent, temp,
                                     np.array([[0, r, 0.3]], np.float32))
            assert int(out["n_accepted"][0]) == 2
    # point-mass q on x: accepted iff r < p(x); after a reject p(x) becomes 0
    for x in range(V):
        dpm = np.zeros((1, 2, V), np.float32)
        dpm[:, :, x] = 1.0
        for r in (p[x] * 0.99, p[x] * 1.01):
            out = oracle.tree_accept(lg, dpm, np.array([[0, x]], np.int32), parent, temp,
                                     np.array([[0, r, 0.3]], np.float32))
            assert (int(out["n_accepted"][0]) == 2) == (r < p[x])
            if r > p[x]:
                assert int(out["bonus_token"][0]) != x
    # single child, general q: residual is norm(max(p-q,0)) -- bonus support check
    q = _random_dist(rng, V, 0)
    dpq = np.tile(q.astype(np.float32), (1, 2, 1))
    x = int(np.argmax(q - p))                        # q(x) > p(x): rejectable
    support = set(np.nonzero(p - q.astype(np.float32) > 0)[0])
    seen = set()
    for u in np.linspace(0, 0.999, 200):
        out = oracle.tree_accept(lg, dpq, np.array([[0, x]], np.int32), parent, temp,
                                 np.array([[0, 0.9999, u]], np.float32))
        assert int(out["n_accepted"][0]) == 1
        seen.add(int(out["bonus_token"][0]))
    assert seen <= support and len(seen) >= 1


def test_leaf_root_only_tree():
    """N = 1: path is [root] and the bonus is drawn from the root's own row."""
    logits = np.log(np.array([[[0.1, 0.2, 0.3, 0.4]]])).astype(np.float32)
    for u, tok in ((0.05, 0), (0.25, 1), (0.5, 2), (0.95, 3)):
        r = oracle.tree_accept(logits, np.full((1, 1, 4), 0.25, np.float32), np.zeros((1, 1), np.int32),
                               np.array([[-1]], np.int32), np.ones(1, np.float32),
                               np.array([[0.0, u]], np.float32))
        assert int(r["n_accepted"][0]) == 1 and int(r["bonus_token"][0]) == tok
    r = oracle.tree_accept(logits, None, np.zeros((1, 1), np.int32), np.array([[-1]], np.int32),
                           np.zeros(1, np.float32), None)
    assert int(r["bonus_token"][0]) == 3
