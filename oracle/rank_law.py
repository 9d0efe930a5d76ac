"""Law of the threshold rank and the exact failure probabilities.  TEST INFRASTRUCTURE ONLY.

Lemma 1 of the paper: S indices are drawn uniformly without replacement from
N; tau is the t-th largest sampled value and R its rank in the whole input
(rank 1 = largest).  R is negative hypergeometric, Eq. (nhg_pmf), with the mean
and variance of Eq. (nhg_mean_var).  The two failure events of Section 4,
R < k and R > M, become tails of an ordinary hypergeometric count:

    R < k   <=>  at least t of the S draws fall among the top k-1 ranks,
    R > M   <=>  at most t-1 of the S draws fall among the top M ranks.

Pins (tests/test_oracle_rank_law.py): exhaustive enumeration of all C(N,S)
samples for small N (pmf, support, mean, variance, both tail identities) and
agreement of the pmf with the closed-form mean and variance at larger sizes.
"""
from __future__ import annotations

from math import comb

import numpy as np
from scipy import stats


def nhg_pmf(N: int, S: int, t: int, r: int) -> float:
    """Pr(R = r), Eq. (nhg_pmf); zero outside r in [t, N-S+t].  Exact integers."""
    if r < t or r > N - S + t:
        return 0.0
    return comb(r - 1, t - 1) * comb(N - r, S - t) / comb(N, S)


def nhg_mean(N: int, S: int, t: int) -> float:
    """E[R] = (N+1) t / (S+1), Eq. (nhg_mean_var)."""
    return (N + 1) * t / (S + 1)


def nhg_var(N: int, S: int, t: int) -> float:
    """Var(R) = t (S-t+1) (N+1) (N-S) / ((S+1)^2 (S+2)), Eq. (nhg_mean_var)."""
    return t * (S - t + 1) * (N + 1) * (N - S) / ((S + 1) ** 2 * (S + 2))


def p_recall_fail_srs(N: int, S: int, t: int, k: int) -> float:
    """Pr(R < k) under simple random sampling: Hypergeom(N, k-1, S) >= t."""
    if k <= 1:
        return 0.0
    return float(stats.hypergeom.sf(t - 1, N, k - 1, S))


def p_overflow_srs(N: int, S: int, t: int, M: int) -> float:
    """Pr(R > M) under simple random sampling: Hypergeom(N, M, S) <= t-1."""
    if M >= N:
        return 0.0
    return float(stats.hypergeom.cdf(t - 1, N, M, S))


# --- the stratified scheme the library samples with -------------------------------------
#
# The paper does not say how to draw "S indices without replacement" on a GPU.
# This build draws one index from each of S disjoint strata
#     [floor(j N / S), floor((j+1) N / S)),  j = 0..S-1,
# uniformly inside the stratum and independently across strata.  The number X of
# draws that land in any fixed set of c ranks is then a sum of S independent
# Bernoulli variables whose mean mu lies in [c / ceil(N/S), c / floor(N/S)]
# (a stratum holds floor(N/S) or ceil(N/S) elements).  Hoeffding (1956, Theorem 4)
# compares such a sum with the binomial of the same mean:
#     Pr(X >= t) <= Pr(Bin(S, mu/S) >= t)   whenever t - 1 >= mu,
#     Pr(X <= t-1) <= Pr(Bin(S, mu/S) <= t-1) whenever t <= mu,
# and a binomial tail is monotone in p, so the end of the interval for mu that
# makes the failure likelier gives a bound.  Outside those ranges the bounds
# below fall back to Markov's inequality (upper tail) or to 1 (lower tail).

def p_recall_fail_bound(N: int, S: int, t: int, k: int) -> float:
    """Upper bound on Pr(R < k) for the stratified scheme.

    X = draws among the top k-1 ranks, mean <= mu = S pA, pA = min(1, (k-1) / (S floor(N/S))).
    Bin(S, pA) >= t when t - 1 >= mu, else Markov's min(1, mu / t)."""
    if k <= 1:
        return 0.0
    pa = min(1.0, (k - 1) / (S * (N // S)))
    mu = S * pa
    if t - 1 >= mu:
        return float(stats.binom.sf(t - 1, S, pa))
    return min(1.0, mu / t)


def p_overflow_bound(N: int, S: int, t: int, M: int) -> float:
    """Upper bound on Pr(R > M) for the stratified scheme; zero when M >= N.

    Y = draws among the top M ranks, mean >= mu = S pB, pB = min(1, M / (S ceil(N/S))).
    Bin(S, pB) <= t-1 when t <= mu, else 1 (no statement)."""
    if M >= N:
        return 0.0
    pb = min(1.0, M / (S * (-(-N // S))))
    if t <= S * pb:
        return float(stats.binom.cdf(t - 1, S, pb))
    return 1.0


def enumerate_rank_pmf(N: int, S: int, t: int) -> np.ndarray:
    """Pr(R = r) for r = 0..N by listing every S-subset of ranks 1..N (tiny N only)."""
    from itertools import combinations

    counts = np.zeros(N + 1, dtype=np.int64)
    for sample in combinations(range(1, N + 1), S):
        counts[sample[t - 1]] += 1      # ranks ascending: the t-th smallest rank is the t-th largest value
    return counts / counts.sum()
