"""Pins of the sampled-acceptance oracle (CPU only), against what the paper and the mathematics fix:

* hand-worked two-sibling example (tests/golden/sampled_two_siblings.json): the thresholds of the uniforms at which
  the decisions flip, and the bonus token once both siblings are rejected;
* p = p^: every first child is kept (ratio 1), so the path is the first-child chain;
* one-hot draft distribution: keep probability is p(x), the residual is p with x removed;
* the draw of the bonus token against numpy's cumulative sum + searchsorted;
* losslessness (the property Sec. 3.1 states: the output follows the target model's distribution): on a two-level
  tree whose children are drawn i.i.d. from p^, the emitted token pair follows p(x1) * p(x2 | x1), checked by
  Monte-Carlo on a 5-token vocabulary at 5 standard deviations;
* malformed sequences are flagged, not walked."""
import json
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sampled_two_siblings.json")


def _one(draft_ids, parents, p_rows, ph_rows, ua, ub):
    path, alen, bonus, bad = oracle.accept_sampled([draft_ids], [parents], np.asarray([p_rows], np.float32),
                                                   np.asarray([ph_rows], np.float32), [ua], [ub])
    assert bad == 0
    return list(path[0][:alen[0]]), int(bonus[0])


def test_hand_worked_two_sibling_thresholds():
    g = json.load(open(GOLDEN))
    ph = [g["p_hat"]] * 3
    for case in g["cases"]:
        p = [case["p"]] * 3
        t1, t2 = case["first_threshold"], case["second_threshold"]
        e = 1e-4
        assert _one(case["draft_ids"], g["parents"], p, ph, [0, t1 - e, 0.99], 0.5)[0] == [0, 1]
        if t2 > 0:
            assert _one(case["draft_ids"], g["parents"], p, ph, [0, t1 + e, t2 - e], 0.5)[0] == [0, 2]
        for ub in (0.0, 0.3, 0.999):
            path, bonus = _one(case["draft_ids"], g["parents"], p, ph, [0, t1 + e, t2 + e], ub)
            assert path == [0] and bonus == case["bonus_after_both"]


def test_equal_distributions_keep_every_first_child():
    rng = np.random.Generator(np.random.Philox(5))
    V, N = 50, 7
    parents = [-1, 0, 0, 1, 1, 3, 2]                     # first-child chain: 0 -> 1 -> 3 -> 5
    p = rng.dirichlet(np.ones(V), size=N).astype(np.float32)
    ids = rng.integers(0, V, size=N)
    for trial in range(20):
        ua = rng.random(N, dtype=np.float32)
        ub = float(rng.random(dtype=np.float32))
        path, bonus = _one(ids, parents, p, p, ua, ub)
        assert path == [0, 1, 3, 5]
        cdf = np.cumsum(p[5].astype(np.float64))
        assert bonus == int(np.searchsorted(cdf, ub * cdf[-1], side="right"))


def test_one_hot_draft_keeps_with_probability_p_and_resamples_from_p_without_the_token():
    V = 6
    p = np.array([0.05, 0.35, 0.2, 0.1, 0.25, 0.05], dtype=np.float32)
    x = 1
    ph = np.zeros(V, dtype=np.float32); ph[x] = 1.0
    for u in np.linspace(0.0, 0.999, 50):
        path, bonus = _one([0, x], [-1, 0], [p, p], [ph, ph], [0, u], 0.5)
        assert (path == [0, 1]) == (u < float(p[x]))
    rest = p.astype(np.float64).copy(); rest[x] = 0.0
    cdf = np.cumsum(rest)
    for ub in np.linspace(0.0, 0.999, 97):
        ub = float(np.float32(ub))
        path, bonus = _one([0, x], [-1, 0], [p, p], [ph, ph], [0, 0.9], ub)
        assert path == [0] and bonus == int(np.searchsorted(cdf, ub * cdf[-1], side="right")) and bonus != x


def test_leaf_root_draws_from_the_target_row_like_numpy():
    rng = np.random.Generator(np.random.Philox(6))
    V = 1000
    p = rng.dirichlet(np.full(V, 0.3), size=1).astype(np.float32)
    p[0, rng.integers(0, V, size=300)] = 0.0              # zero-weight tokens are never drawn
    cdf = np.cumsum(p[0].astype(np.float64))
    for ub in rng.random(200, dtype=np.float32):
        path, bonus = _one([3], [-1], p, p, [0], float(ub))
        assert path == [0] and bonus == int(np.searchsorted(cdf, float(ub) * cdf[-1], side="right")) and p[0, bonus] > 0


def test_output_follows_the_target_distribution_on_a_two_level_tree():
    rng = np.random.Generator(np.random.Philox(7))
    V, K1, K2, B = 5, 3, 2, 400_000
    N = 1 + K1 + K1 * K2
    p_root, ph_root = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
    p_next, ph_next = rng.dirichlet(np.ones(V), size=V), rng.dirichlet(np.ones(V), size=V)   # by first token
    parents = np.array([-1] + [0] * K1 + [1 + c for c in range(K1) for _ in range(K2)], dtype=np.int32)
    ids = np.zeros((B, N), dtype=np.int32)
    ids[:, 1:1 + K1] = rng.choice(V, size=(B, K1), p=ph_root)
    for c in range(K1):
        cdf = np.cumsum(ph_next[ids[:, 1 + c]], axis=1)
        for j in range(K2):
            u = rng.random(B)[:, None]
            ids[:, 1 + K1 + c * K2 + j] = np.minimum((u > cdf).sum(axis=1), V - 1)
    p = np.zeros((B, N, V), dtype=np.float32); ph = np.zeros_like(p)
    p[:, 0], ph[:, 0] = p_root, ph_root
    for c in range(K1):
        p[:, 1 + c], ph[:, 1 + c] = p_next[ids[:, 1 + c]], ph_next[ids[:, 1 + c]]
    # second-level nodes are leaves here; their rows give the third token, which this test does not look at
    p[:, 1 + K1:] = 1.0 / V; ph[:, 1 + K1:] = 1.0 / V
    ua = rng.random((B, N), dtype=np.float32); ub = rng.random(B, dtype=np.float32)
    path, alen, bonus, bad = oracle.accept_sampled(ids, np.tile(parents, (B, 1)), p, ph, ua, ub)
    assert bad == 0
    rows = np.arange(B)
    first = np.where(alen >= 2, ids[rows, path[:, 1]], bonus)
    # the second emitted token exists within this cycle only when the first was a kept draft
    has2 = alen >= 2
    second = np.where(alen >= 3, ids[rows, np.maximum(path[:, 2], 0)], bonus)
    f1 = np.bincount(first, minlength=V) / B
    assert np.all(np.abs(f1 - p_root) < 5 * np.sqrt(p_root * (1 - p_root) / B))
    for x in range(V):
        sel = has2 & (first == x)
        n = sel.sum()
        assert n > 2000
        f2 = np.bincount(second[sel], minlength=V) / n
        assert np.all(np.abs(f2 - p_next[x]) < 5 * np.sqrt(p_next[x] * (1 - p_next[x]) / n))
    # and the tree helps: more than one draft level is kept in a fair share of the cycles
    assert (alen >= 3).mean() > 0.05


def test_malformed_sequences_are_flagged_and_not_walked():
    V = 4
    p = np.full((3, 3, V), 0.25, dtype=np.float32)
    ids = np.array([[0, 1, 2], [0, 7, 1], [0, 1, 1]], dtype=np.int32)          # sequence 1: token 7 >= V
    parents = np.array([[-1, 0, 1], [-1, 0, 0], [-1, 2, 0]], dtype=np.int32)   # sequence 2: parent 2 of node 1
    path, alen, bonus, bad = oracle.accept_sampled(ids, parents, p, p, np.zeros((3, 3), np.float32), np.zeros(3, np.float32))
    assert bad == 2 and list(alen) == [3, 0, 0] and list(bonus[1:]) == [-1, -1]
    assert np.all(path[1:] == -1) and list(path[0]) == [0, 1, 2]
