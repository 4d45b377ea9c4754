"""Pins for the oracle's token scoring (Appendix D.1) and its TopK."""
import itertools

import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads


def brute_topk(values, k):
    """Selection by repeated scan: the largest value, lowest position first."""
    vals = list(values)
    taken = []
    for _ in range(min(k, len(vals))):
        best = None
        for p, v in enumerate(vals):
            if p in taken:
                continue
            if best is None or v > vals[best]:
                best = p
        taken.append(best)
    return sorted(taken)


def test_topk_matches_brute_force_with_ties():
    rng = np.random.default_rng(1)
    for n, k in itertools.product([1, 2, 7, 33], [1, 3, 7, 40]):
        v = rng.integers(0, 4, size=n).astype(np.float64)      # many exact ties
        assert fo.topk_ascending(v, k).tolist() == brute_topk(v, k)


def test_topk_ties_lowest_index_and_identity():
    v = np.array([1.0, 5.0, 5.0, 5.0, 0.0, 5.0])
    assert fo.topk_ascending(v, 2).tolist() == [1, 2]
    assert fo.topk_ascending(v, 3).tolist() == [1, 2, 3]
    assert fo.topk_ascending(v, 6).tolist() == [0, 1, 2, 3, 4, 5]
    assert fo.topk_ascending(v, 99).tolist() == [0, 1, 2, 3, 4, 5]
    out = fo.topk_ascending(np.random.default_rng(0).random(100), 17)
    assert np.all(np.diff(out) > 0)


def test_token_score_closed_forms():
    eps = 1e-6
    u = np.zeros((1, 8)); u[0, 3] = 1.0                         # unit vector
    for a, b in [(2.0, 0.5), (-3.0, 1.0), (1.0, 1.0)]:
        s = fo.token_scores(b * u, a * u, np.array([0]), eps)[0]
        assert s == pytest.approx(abs(a - b) / (abs(a) + eps), rel=1e-14)
    # 3-4-5 triangle: previous state zero, current (3,4) -> 5 / (5 + eps)
    s = fo.token_scores(np.zeros((1, 2)), np.array([[3.0, 4.0]]), np.array([0]), eps)[0]
    assert s == pytest.approx(5.0 / (5.0 + eps), rel=1e-14)
    # the denominator is the norm of the CURRENT state (the more recent one)
    s = fo.token_scores(np.array([[10.0, 0.0]]), np.array([[1.0, 0.0]]), np.array([0]), 0.0)[0]
    assert s == pytest.approx(9.0)
    # unchanged rows score exactly zero
    g = np.random.default_rng(0).standard_normal((5, 16))
    assert np.all(fo.token_scores(g, g, np.arange(5), eps) == 0.0)
    # scale invariance as eps -> 0
    g2 = g + 0.1 * np.random.default_rng(1).standard_normal((5, 16))
    s1 = fo.token_scores(g, g2, np.arange(5), 0.0)
    s2 = fo.token_scores(7.0 * g, 7.0 * g2, np.arange(5), 0.0)
    np.testing.assert_allclose(s1, s2, rtol=1e-13)


def test_token_scores_use_candidate_rows_only():
    rng = np.random.default_rng(3)
    g1, g2 = rng.standard_normal((10, 4)), rng.standard_normal((10, 4))
    cand = np.array([2, 5, 9])
    s = fo.token_scores(g1, g2, cand, 1e-6)
    for t, i in enumerate(cand):
        ref = np.linalg.norm(g2[i] - g1[i]) / (np.linalg.norm(g2[i]) + 1e-6)
        assert s[t] == pytest.approx(ref, rel=1e-13)


def test_planted_rows_are_selected_config1(c1_inputs):
    """Generator ground truth: the 25% rows that received the large update are exactly the top 25%."""
    w = c1_inputs.workload
    s, act = fo.select_tokens(c1_inputs.G[0], c1_inputs.G[1], np.arange(w.L), w.k_tokens, w.eps)
    assert act.tolist() == c1_inputs.changed_rows[0].tolist()
    planted = np.zeros(w.L, bool); planted[c1_inputs.changed_rows[0]] = True
    assert s[planted].min() > 0.3 and s[~planted].max() < 0.01


def test_nested_sets_and_constant_budget():
    w = workloads.config2(L=256, n_heads=1)
    x = workloads.make_layer_inputs(w, seed=2)
    orc = fo.LayerOracle(w.L, w.n_heads, w.head_dim, 64, 4, 128, w.eps, w.sm_scale)
    sets, _ = orc.token_sets(x.G, [w.k_tokens] * 3)
    assert set(sets[1]) <= set(sets[0]) and set(sets[2]) <= set(sets[1])
    assert len(sets[0]) == w.k_tokens and sets[1].tolist() == sets[0].tolist()   # k >= |A^(r-1)| keeps all
    sets2, _ = orc.token_sets(x.G, [40, 20, 10])
    assert [len(s) for s in sets2] == [40, 20, 10]
    assert set(sets2[2]) <= set(sets2[1]) <= set(sets2[0])
    slot = fo.slot_map(sets2[0], w.L)
    assert (slot >= 0).sum() == 40 and slot[sets2[0]].tolist() == list(range(40))
