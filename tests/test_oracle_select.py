"""Pins for the selection / advantage oracle: each test ties it to something the paper or
mathematics fixes (the definition by brute force, Lemma 3.1, Algorithm 2's update rule,
Theorem 2, the zero-total-advantage remark of Appendix A.3, library mean/std)."""
from fractions import Fraction
from itertools import combinations
from math import comb

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20250413)


def _tiny_cases():
    """(rewards fp32 [n], m) over random and adversarial reward patterns, n <= 10."""
    cases = []
    for n in range(1, 11):
        for m in range(1, n + 1):
            if comb(n, m) > 260:
                continue
            cases.append((RNG.normal(0, 1, n).astype(np.float32), m))                       # continuous
            cases.append((RNG.integers(0, 2, n).astype(np.float32), m))                     # binary
            cases.append((RNG.choice([0.0, 0.5, 1.0], n).astype(np.float32), m))            # ternary ties
            cases.append((RNG.choice([-2.0, -0.25, 0.0, 0.25, 3.0], n).astype(np.float32), m))  # negatives
            cases.append((np.full(n, 0.75, np.float32), m))                                 # all equal
            cases.append(((RNG.integers(0, 2, n) + 0.1 * RNG.integers(0, 2, n)
                           + RNG.normal(0, 0.05, n)).astype(np.float32), m))                # mixed (config 3)
    return cases


def _stable_order(r):
    return sorted(range(len(r)), key=lambda i: (float(r[i]) + 0.0, i))


def _split(order, n, m, k):
    return sorted(order[: m - k] + order[n - k:])


def test_variance_helper_matches_library_variance():
    for _ in range(20):
        x = RNG.normal(0, 3, RNG.integers(1, 9)).astype(np.float32)
        assert float(oracle.variance_exact(x)) == pytest.approx(np.var(x.astype(np.float64)), rel=1e-12, abs=1e-15)


def test_algorithm2_attains_the_definition_by_brute_force():
    """Section 3.3: S = argmax over all m-subsets of Var.  Exact comparison."""
    for r, m in _tiny_cases():
        best, argbest = oracle.max_variance_subsets(r, m)
        out = oracle.select(r[None, :], m)
        S = tuple(int(i) for i in out["idx"][0])
        assert len(set(S)) == m and all(0 <= i < len(r) for i in S)
        assert oracle.variance_exact(r[list(S)]) == best, (r, m, S)
        assert S in argbest


def test_lemma31_structure_and_smallest_k():
    """Lemma 3.1: optimum = k highest + (m-k) lowest of the sorted order; Algorithm 2 starts at
    k = 0 and replaces only on a strictly larger variance, so the smallest maximiser wins."""
    for r, m in _tiny_cases():
        n = len(r)
        order = _stable_order(r)
        out = oracle.select(r[None, :], m)
        k = int(out["k"][0])
        assert list(out["idx"][0]) == _split(order, n, m, k)
        scores = [oracle.variance_exact(r[_split(order, n, m, kk)]) for kk in range(m + 1)]
        assert k == min(kk for kk in range(m + 1) if scores[kk] == max(scores))


def test_theorem2_binary_rewards_closed_form():
    """Theorem 2: binary rewards, m even: m/2 highest + m/2 lowest maximises the variance.  With c
    ones in the group the kept subset holds ones = clamp(m/2, m-(n-c), c) and Var = p(1-p)."""
    for n in (4, 8, 16, 33, 64):
        for m in (2, 4, 8, 16):
            if m > n:
                continue
            for c in range(n + 1):
                r = np.zeros(n, np.float32)
                r[RNG.permutation(n)[:c]] = 1.0
                out = oracle.select(r[None, :], m)
                ones = int(r[out["idx"][0]].sum())
                want = min(max(m // 2, m - (n - c)), c)
                assert ones == want, (n, m, c)
                p = Fraction(ones, m)
                assert oracle.variance_exact(r[out["idx"][0]]) == p * (1 - p)


def test_exact_tie_between_splits_prefers_smallest_k():
    # two zeros, four ones, m = 4: k = 0 keeps the 4 lowest = 2 zeros + 2 ones, the same multiset of
    # rewards as k = 1 and k = 2.  The update is strict, so the first (k = 0) stays.
    r = np.array([1, 0, 1, 1, 0, 1], np.float32)
    out = oracle.select(r[None, :], 4)
    assert int(out["k"][0]) == 0
    assert list(out["idx"][0]) == [0, 1, 2, 4]


def test_stable_argsort_breaks_reward_ties_by_index_and_signed_zero():
    r = np.array([0.0, -0.0, 1.0, 0.0, 1.0, -0.0], np.float32)
    out = oracle.select(r[None, :], 2)
    # sorted order is 0,1,3,5 (zeros by index) then 2,4; best split is 1 low + 1 high = {0} U {4}
    assert list(out["idx"][0]) == [0, 4] and int(out["k"][0]) == 1


def test_degenerate_groups():
    r = np.full((3, 7), 2.5, np.float32)
    out = oracle.select(r, 3)
    assert (out["k"] == 0).all() and (out["idx"] == np.arange(3)).all() and (out["adv"] == 0).all()
    r1 = RNG.normal(size=(5, 9)).astype(np.float32)
    one = oracle.select(r1, 1)        # a single rollout has zero variance for every k: k = 0, the lowest
    assert (one["k"] == 0).all() and (one["adv"] == 0).all()
    assert (one["idx"][:, 0] == np.argmin(r1, axis=1)).all()
    r = RNG.normal(size=(4, 6)).astype(np.float32)
    full = oracle.select(r, 6)
    assert (full["idx"] == np.arange(6)).all()
    with pytest.raises(ValueError):
        oracle.select(r, 7)
    with pytest.raises(ValueError):
        oracle.select(r, 0)


def test_m_equals_n_is_plain_grpo_normalisation():
    """Section 3.1: a_i = (r_i - mu)/sigma over the whole group (library mean/std, population)."""
    r = RNG.normal(0.3, 1.0, size=(16, 12)).astype(np.float32)
    out = oracle.select(r, 12)
    r64 = r.astype(np.float64)
    want = (r64 - r64.mean(axis=1, keepdims=True)) / r64.std(axis=1, keepdims=True)
    np.testing.assert_allclose(out["adv"], want, rtol=1e-12, atol=1e-14)


def test_kept_advantages_use_subset_statistics_and_sum_to_zero():
    """Section 3.2 / Appendix A.3: statistics of the kept subset, total advantage 0, unit variance."""
    r = (RNG.integers(0, 2, size=(64, 32)) + RNG.normal(0, 0.05, size=(64, 32))).astype(np.float32)
    m = 8
    out = oracle.select(r, m)
    kept = np.take_along_axis(r.astype(np.float64), out["idx"].astype(np.int64), axis=1)
    want = (kept - kept.mean(axis=1, keepdims=True)) / kept.std(axis=1, keepdims=True)
    np.testing.assert_allclose(out["adv"], want, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(out["adv"].sum(axis=1), 0.0, atol=1e-12)
    np.testing.assert_allclose((out["adv"] ** 2).sum(axis=1), m, rtol=1e-12)


def test_binary_advantages_closed_form():
    r = np.array([[1, 1, 1, 0, 0, 0, 0, 0, 0, 0, 0, 0]], np.float32)       # 3 ones, m = 8 -> 3 ones kept
    out = oracle.select(r, 8)
    p = 3 / 8
    kept = r[0, out["idx"][0]]
    want = np.where(kept == 1, (1 - p), -p) / np.sqrt(p * (1 - p))
    np.testing.assert_allclose(out["adv"][0], want, rtol=1e-14)


def test_before_variant_and_sample_std():
    """Appendix A.3 'Before': statistics of the full group, then down-sample."""
    r = RNG.normal(size=(8, 16)).astype(np.float32)
    base = oracle.select(r, 4)
    before = oracle.select(r, 4, flags=oracle.FLAG_ADV_BEFORE)
    assert (before["idx"] == base["idx"]).all()
    r64 = r.astype(np.float64)
    full = (r64 - r64.mean(axis=1, keepdims=True)) / r64.std(axis=1, keepdims=True)
    np.testing.assert_allclose(before["adv"], np.take_along_axis(full, base["idx"].astype(np.int64), 1), rtol=1e-12)
    samp = oracle.select(r, 4, flags=oracle.FLAG_STD_SAMPLE)
    np.testing.assert_allclose(samp["adv"], base["adv"] * np.sqrt(3 / 4), rtol=1e-12)


def test_affine_invariance_with_exact_arithmetic():
    r = RNG.integers(-8, 9, size=(32, 24)).astype(np.float32) / 4
    a = oracle.select(r, 6)
    b = oracle.select(r * 8 + 3, 6)
    assert (a["idx"] == b["idx"]).all() and (a["k"] == b["k"]).all()
    np.testing.assert_allclose(a["adv"], b["adv"], rtol=1e-13, atol=1e-15)


def test_gap_reports_distance_to_runner_up():
    r = np.array([[0, 0, 0, 1, 1, 1]], np.float32)
    out = oracle.select(r, 2)     # scores m^2 Var: k=0 -> 0, k=1 -> 1, k=2 -> 0
    assert out["gap"][0] == 1.0
    assert np.isinf(oracle.select(np.ones((1, 5), np.float32), 2)["gap"][0])


def test_philox_known_answers(request):
    path = request.config.rootpath / "tests" / "golden" / "philox4x32_10_kat.txt"
    rows = [ln.split() for ln in open(path) if not ln.startswith("#") and ln.strip()]
    assert len(rows) == 3
    for h in rows:
        v = [int(x, 16) for x in h]
        assert list(oracle.philox4x32_10(v[:4], v[4:6])) == v[6:]


def test_max_reward_rule_is_top_m():
    r = RNG.normal(size=(16, 20)).astype(np.float32)
    out = oracle.select(r, 5, rule=oracle.RULE_MAXREWARD)
    for g in range(16):
        assert sorted(r[g, out["idx"][g]]) == sorted(np.sort(r[g])[-5:])
    assert (out["k"] == 5).all()


def test_percentile_rule_positions():
    """Section 3.2: the (j+0.5)/m quantiles; n = 8, m = 4 -> sorted positions 1, 3, 5, 7."""
    r = np.array([[7, 3, 5, 1, 0, 2, 6, 4]], np.float32)      # value v sits at sorted position v
    out = oracle.select(r, 4, rule=oracle.RULE_PERCENTILE)
    assert sorted(r[0, out["idx"][0]]) == [1, 3, 5, 7]
    out = oracle.select(np.arange(10, dtype=np.float32)[None, :], 3, rule=oracle.RULE_PERCENTILE)
    assert list(out["idx"][0]) == [1, 5, 8]                    # floor(10/6), floor(30/6), floor(50/6)


def test_random_rule_is_a_seeded_uniform_subset():
    G, n, m = 20000, 10, 3
    r = np.zeros((G, n), np.float32)
    a = oracle.select(r, m, rule=oracle.RULE_RANDOM, seed=123)
    b = oracle.select(r, m, rule=oracle.RULE_RANDOM, seed=123)
    c = oracle.select(r, m, rule=oracle.RULE_RANDOM, seed=124)
    assert (a["idx"] == b["idx"]).all() and (a["idx"] != c["idx"]).any()
    assert (np.diff(a["idx"], axis=1) > 0).all() and a["idx"].min() >= 0 and a["idx"].max() < n
    freq = np.bincount(a["idx"].ravel(), minlength=n) / G          # each index kept with prob m/n
    assert np.abs(freq - m / n).max() < 4 * np.sqrt(0.3 * 0.7 / G)
    pairs = {}
    for row in a["idx"]:
        for p in combinations(row, 2):
            pairs[p] = pairs.get(p, 0) + 1
    assert len(pairs) == comb(n, 2)                                # every pair occurs
