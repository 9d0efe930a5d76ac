"""Parameter selection (S, t, M).  TEST INFRASTRUCTURE ONLY (see package header).

Two plans are written out here.

`plan_paper` is Algorithm 1 of the paper taken literally, step by step, built
from the equations of Section 4: Eq. (t_choice), Eq. (c_0), Eq. (c), Eq. (M),
Eq. (optimal_S) and the clamp S in [S_min, S_max] = [32768, 2^17].

`plan_guarded` is the plan the library returns.  It keeps Algorithm 1's sample
size and Theorem 1's contract (total failure probability at most eps, split
eps/2 + eps/2) but replaces two things that do not meet that contract:

  * Algorithm 1's last step sets t = 1 whenever alpha S < -ln(eps/2).  With
    t = 1 the threshold is the sample maximum, the highest threshold there is:
    recall then fails as soon as one of the top k-1 elements is sampled, which
    happens with probability about 1 - exp(-alpha S), not exp(-alpha S); and
    Eq. (M) was derived for the Gaussian t, so the buffer overflows as well.
    The guarded plan never applies that step.
  * The Gaussian closed forms Eq. (t_choice) and Eq. (M) are slightly
    optimistic for finite S (they ignore the skew of the count and use
    q(1-q) ~ alpha(1-alpha)).  The guarded plan takes t as the smallest rank
    whose recall-failure bound is at most eps/2 and the capacity as the larger
    of Eq. (M) and the smallest M whose overflow bound is at most eps/2; both
    bounds are the binomial bounds of `rank_law` for the stratified sampler.

Readings of points the paper leaves open:
`log k` in Eq. (cost_model) / Eq. (optimal_S) is log2 (Algorithm 1 says so); the
rounding of S* is half away from zero; S is also capped at N; relaxed recall
rho < 1 means "accept k_rho = ceil(rho k) survivors", i.e. the recall bound is
taken for k_rho instead of k while the capacity still follows k (the buffer has
to hold the k requested outputs) -- the paper gives no formula for that mode,
so it is pinned by what the mathematics fixes: Lemma 1's exact tail
Pr(R < k_rho) <= eps/2, minimality of the rank, and a Monte Carlo of both
failure events with k_rho as the accepted count; when the buffer would hold half the input or the
sample would be half the input the filter is pointless and the plan says
mode = 1 (direct exact selection).

Pins (tests/test_oracle_plan.py): the constants the paper prints (z ~ 6.58 for
eps = 1e-3, (kN)^(1/3) ~ 4,600 for N = 1e9, k = 100, the order of magnitude of
M for N = 2^29, k = 64, the SAE shape arithmetic), M = c k through Eq. (c_0) and
Eq. (c), the arg-min of the cost model, the 1/3 slope of S*, the exact tails,
and Monte Carlo failure rates (<= eps for the guarded plan, far above eps for
Algorithm 1's t = 1 step).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

from scipy import stats

from . import rank_law

S_MIN_DEFAULT = 32768        # "S_min = 32768 avoids high-variance threshold estimates"
S_MAX_DEFAULT = 1 << 17      # "e.g. S_max = 2^17 = 131,072"
EPS_DEFAULT = 1e-3           # Algorithm 1, default failure budget
COST_RATIO_DEFAULT = 1.0     # tau_B / tau_A, Algorithm 1 default


# ----------------------------------------------------------------------------- equations
def z_one_sided(eps_part: float) -> float:
    """z_A = Phi^{-1}(1 - eps_A) (Section 4, 'Controlling insufficient recall').

    Evaluated as the upper-tail quantile of eps_A, which is the same number without the
    rounding of 1 - eps_A (that rounding costs ~1e-11 of z at eps = 1e-6)."""
    return float(stats.norm.isf(eps_part))


def z_total(eps: float) -> float:
    """Algorithm 1 step 1: z = Phi^{-1}(1 - eps/2) + Phi^{-1}(1 - eps/2)."""
    return 2.0 * z_one_sided(eps / 2.0)


def fpc(N: int, S: int) -> float:
    """Finite-population correction f = 1 - S/N (Lemma 2)."""
    return 1.0 - S / N


def eq_t_choice(N: int, k: int, S: int, z_a: float) -> int:
    """Eq. (t_choice): t = ceil(S alpha + z_A sqrt(S alpha (1-alpha) f)), at least 1."""
    alpha = k / N
    return max(1, math.ceil(S * alpha + z_a * math.sqrt(S * alpha * (1.0 - alpha) * fpc(N, S))))


def eq_c0(N: int, k: int, S: int, z_a: float) -> float:
    """Eq. (c_0): nominal buffer multiplier 1 + z_A / sqrt(S) * sqrt((1-alpha)/alpha f)."""
    alpha = k / N
    return 1.0 + z_a / math.sqrt(S) * math.sqrt((1.0 - alpha) / alpha * fpc(N, S))


def eq_c(N: int, k: int, S: int, z_a: float, z_b: float) -> float:
    """Eq. (c): c = c_0 + z_B sqrt((1-alpha) f / (alpha S))."""
    alpha = k / N
    return eq_c0(N, k, S, z_a) + z_b * math.sqrt((1.0 - alpha) * fpc(N, S) / (alpha * S))


def eq_M(N: int, k: int, S: int, z: float) -> float:
    """Eq. (M), Corollary 1: M = k + z sqrt(k (N-k) / S * (1 - S/N)) (not yet rounded)."""
    return k + z * math.sqrt(k * (N - k) / S * fpc(N, S))


def cost_model(N: int, k: int, S: float, z: float, cost_ratio: float) -> float:
    """Eq. (cost_model) with f = 1 and tau_A = 1: C = S + (tau_B/tau_A) M log2 k."""
    M = k + z * math.sqrt(k * (N - k) / S)
    return S + cost_ratio * M * math.log2(k)


def optimal_S(N: int, k: int, z: float, cost_ratio: float = COST_RATIO_DEFAULT) -> float:
    """Eq. (optimal_S), Theorem 2, with log = log2 as in Algorithm 1 step 3."""
    return (z * cost_ratio * math.log2(k) / 2.0) ** (2.0 / 3.0) * (k * (N - k)) ** (1.0 / 3.0)


def round_half_away(x: float) -> int:
    """The 'round to nearest' of Algorithm 1 step 4 for x >= 0."""
    return int(math.floor(x + 0.5))


def sample_size(N: int, k: int, eps: float, s_min: int = S_MIN_DEFAULT,
                s_max: int = S_MAX_DEFAULT, cost_ratio: float = COST_RATIO_DEFAULT) -> int:
    """Algorithm 1 steps 1-4, then S <= N (a sample cannot exceed the input)."""
    s_star = optimal_S(N, k, z_total(eps), cost_ratio)
    return min(N, min(s_max, max(s_min, round_half_away(s_star))))


# ----------------------------------------------------------------------------- Algorithm 1
def plan_paper(N: int, k: int, eps: float = EPS_DEFAULT, s_min: int = S_MIN_DEFAULT,
               s_max: int = S_MAX_DEFAULT, cost_ratio: float = COST_RATIO_DEFAULT,
               apply_sparse_rule: bool = True) -> tuple[int, int, int]:
    """Algorithm 1 as printed: returns (S, t, M).

    `apply_sparse_rule=False` drops only the last step (t <- 1 when
    alpha S < -ln(eps/2)), leaving the Gaussian t of Eq. (t_choice).
    """
    z = z_total(eps)                                           # step 1
    alpha = k / N                                              # step 2
    S = sample_size(N, k, eps, s_min, s_max, cost_ratio)       # steps 3-4
    t = eq_t_choice(N, k, S, z / 2.0)                          # steps 5-6
    M = math.ceil(eq_M(N, k, S, z))                            # step 7
    if apply_sparse_rule and alpha * S < -math.log(eps / 2.0):  # step 8
        t = 1
    return S, t, M


# ----------------------------------------------------------------------------- guarded plan
@dataclass(frozen=True)
class Plan:
    m: int                # sample size S
    r: int                # sample rank t (1-based, t-th largest sampled value)
    capacity: int         # buffer capacity M
    k_accept: int         # k, or ceil(recall k) in relaxed mode
    mode: int             # 0 = sample/filter/refine, 1 = direct exact selection
    z: float
    alpha: float
    p_recall_fail: float  # bound on Pr(R < k_accept) for (m, r)
    p_overflow: float     # bound on Pr(R > capacity) for (m, r)
    r_tight: int = 0      # second-chance rank after an overflow (0 = none), see second_chance_ranks
    r_loose: int = 0      # second-chance rank after a recall failure (0 = none)


def accept_count(k: int, recall: float) -> int:
    """k_rho = ceil(rho k), guarded against rho k landing a hair above an integer."""
    return min(k, max(1, math.ceil(recall * k - 1e-9)))


def guarded_rank(N: int, S: int, k_accept: int, eps_a: float) -> int:
    """Smallest t in [1, S] whose recall-failure bound is <= eps_a (S if none)."""
    lo, hi = 1, S
    if rank_law.p_recall_fail_bound(N, S, hi, k_accept) > eps_a:
        return S
    while lo < hi:                       # the bound is non-increasing in t
        mid = (lo + hi) // 2
        if rank_law.p_recall_fail_bound(N, S, mid, k_accept) <= eps_a:
            hi = mid
        else:
            lo = mid + 1
    return lo


def guarded_capacity(N: int, S: int, t: int, k: int, eps_b: float) -> int:
    """Smallest M in [k, N] whose overflow bound is <= eps_b (the bound is 0 at M = N)."""
    lo, hi = k, N
    while lo < hi:                       # the bound is non-increasing in M
        mid = (lo + hi) // 2
        if rank_law.p_overflow_bound(N, S, t, mid) <= eps_b:
            hi = mid
        else:
            lo = mid + 1
    return lo


def second_chance_ranks(N: int, k: int, S: int, t: int, capacity: int) -> tuple[int, int]:
    """Ranks for one more filtering pass before the exact fallback (a reading: Section 3, "Refinement", and the
    appendix "Fallback as a Safety Mechanism" only say that a failed row falls back to an exact top-k of the input).

    The sample outlives the failure.  Seen from a threshold of rank t that kept just over M elements, the threshold of
    a tighter rank t' keeps about M t'/t of them (the sampled ranks below a given one are spread like uniform order
    statistics); aiming midway between k and M gives r_tight = floor(t (k + M) / (2 M)).  Seen from one that kept just
    under k, each further sample rank adds about N/S survivors; midway again: r_loose = t + ceil((M - k) S / (2 N)).
    A rank that does not exist (r_tight < 1 or not below t; r_loose above S or not above t) is reported as 0."""
    tight = t * (k + capacity) // (2 * capacity)
    loose = t + -(-((capacity - k) * S) // (2 * N))
    return (tight if 1 <= tight < t else 0), (loose if t < loose <= S else 0)


def plan_guarded(N: int, k: int, eps: float = EPS_DEFAULT, recall: float = 1.0,
                 s_min: int = S_MIN_DEFAULT, s_max: int = S_MAX_DEFAULT,
                 cost_ratio: float = COST_RATIO_DEFAULT) -> Plan:
    """The plan of the library's `profk_plan` (see the module header for the reading)."""
    if not (1 <= k <= N) or not (0.0 < eps < 1.0) or not (0.0 < recall <= 1.0):
        raise ValueError("need 1 <= k <= N, 0 < eps < 1, 0 < recall <= 1")
    z = z_total(eps)
    S = sample_size(N, k, eps, s_min, s_max, cost_ratio)
    k_acc = accept_count(k, recall)
    t = guarded_rank(N, S, k_acc, eps / 2.0)
    m_exact = guarded_capacity(N, S, t, k, eps / 2.0)
    m_paper = math.ceil(eq_M(N, k, S, z))
    capacity = min(N, max(m_exact, m_paper))
    mode = 1 if (2 * capacity >= N or N <= 2 * S) else 0
    r_tight, r_loose = second_chance_ranks(N, k, S, t, capacity)
    return Plan(m=S, r=t, capacity=capacity, k_accept=k_acc, mode=mode, z=z, alpha=k / N,
                p_recall_fail=rank_law.p_recall_fail_bound(N, S, t, k_acc),
                p_overflow=rank_law.p_overflow_bound(N, S, t, capacity), r_tight=r_tight, r_loose=r_loose)
