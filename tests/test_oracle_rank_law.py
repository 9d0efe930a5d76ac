"""Pins for oracle.rank_law: Lemma 1 (law of the threshold rank) checked by listing
every possible sample, and the two tail identities used by the plan."""
from math import comb

import numpy as np
import pytest
from scipy import stats

from oracle import rank_law


@pytest.mark.parametrize("N,S,t", [(7, 3, 1), (7, 3, 3), (10, 4, 2), (12, 5, 3), (12, 12, 7), (13, 1, 1)])
def test_pmf_mean_variance_against_enumeration(N, S, t):
    pmf = rank_law.enumerate_rank_pmf(N, S, t)
    formula = np.array([rank_law.nhg_pmf(N, S, t, r) for r in range(N + 1)])
    assert np.allclose(pmf, formula, atol=1e-15)
    support = np.flatnonzero(pmf > 0)
    assert support.min() == t and support.max() == N - S + t          # r in [t, N-S+t]
    r = np.arange(N + 1)
    mean = float((r * pmf).sum())
    var = float(((r - mean) ** 2 * pmf).sum())
    assert mean == pytest.approx(rank_law.nhg_mean(N, S, t), rel=1e-12)
    assert var == pytest.approx(rank_law.nhg_var(N, S, t), rel=1e-10, abs=1e-12)


@pytest.mark.parametrize("N,S,t", [(10, 4, 2), (12, 5, 3), (11, 6, 1)])
def test_failure_events_are_hypergeometric_tails(N, S, t):
    pmf = rank_law.enumerate_rank_pmf(N, S, t)
    for k in range(1, N + 1):
        assert pmf[:k].sum() == pytest.approx(rank_law.p_recall_fail_srs(N, S, t, k), abs=1e-13)
    for M in range(1, N + 1):
        assert pmf[M + 1:].sum() == pytest.approx(rank_law.p_overflow_srs(N, S, t, M), abs=1e-13)


def test_pmf_sums_to_one_and_matches_moments_at_moderate_size():
    N, S, t = 5000, 300, 7
    r = np.arange(t, N - S + t + 1)
    pmf = np.array([rank_law.nhg_pmf(N, S, t, int(x)) for x in r])
    assert pmf.sum() == pytest.approx(1.0, rel=1e-12)
    mean = float((r * pmf).sum())
    assert mean == pytest.approx(rank_law.nhg_mean(N, S, t), rel=1e-10)
    assert float(((r - mean) ** 2 * pmf).sum()) == pytest.approx(rank_law.nhg_var(N, S, t), rel=1e-9)
    # the same law through SciPy's negative hypergeometric: walking down the ranks, R - t
    # unsampled elements ("successes", N - S of them) are met before the t-th sampled one
    alt = stats.nhypergeom.pmf(r - t, N, N - S, t)
    assert np.allclose(pmf, alt, rtol=1e-9, atol=1e-300)


def test_binomial_bounds_dominate_the_exact_tails():
    # Stratified sampling on an exchangeable input has exactly the hypergeometric law;
    # the binomial bound used by the plan must never be below it.
    for N, S in [(1 << 20, 32768), (1 << 26, 32768), (1_000_003, 4096), (50_331_648, 131072)]:
        for k in (2, 33, 4097):
            for t in (1, 3, 9, 40):
                assert rank_law.p_recall_fail_bound(N, S, t, k) >= rank_law.p_recall_fail_srs(N, S, t, k) * (1 - 1e-7)
        for t in (1, 3, 9, 40):
            for M in (100, 10_000, 300_000):
                assert rank_law.p_overflow_bound(N, S, t, M) >= rank_law.p_overflow_srs(N, S, t, M) * (1 - 1e-7)
    assert rank_law.p_recall_fail_bound(1000, 10, 1, 1) == 0.0          # the single best element cannot be missed
    assert rank_law.p_overflow_bound(1000, 10, 3, 1000) == 0.0          # a buffer as large as the input cannot overflow


def test_bound_matches_direct_enumeration_of_a_tiny_stratified_sample():
    # N = 12, S = 3 strata of 4; top-(k-1) ranks placed on positions {0, 5, 6}.
    # X = number of sampled positions among them = Bern(1/4) + Bern(2/4) + Bern(0).
    p = [0.25, 0.5, 0.0]
    exact_ge1 = 1 - (1 - p[0]) * (1 - p[1])
    exact_ge2 = p[0] * p[1]
    # Hoeffding: beyond the mean (0.75) the binomial with the same mean is heavier-tailed
    assert stats.binom.sf(1, 3, 0.25) >= exact_ge2
    assert rank_law.p_recall_fail_bound(12, 3, 2, 4) == pytest.approx(stats.binom.sf(1, 3, 3 / 12))
    assert rank_law.p_recall_fail_bound(12, 3, 2, 4) >= exact_ge2
    assert exact_ge1 <= 1.0
    assert comb(12, 3) == 220
