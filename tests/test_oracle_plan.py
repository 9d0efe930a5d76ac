"""Pins for oracle.plan: the constants and worked numbers the paper prints, the algebra
that links its equations, and the contract of Theorem 1 for the guarded plan."""
import math

import numpy as np
import pytest
from scipy import optimize, stats

from oracle import plan, rank_law


def test_printed_constants(golden):
    assert plan.z_total(1e-3) == pytest.approx(golden["z_eps_1e-3"][0], abs=5e-3)
    assert plan.EPS_DEFAULT == golden["eps_default"][0]
    assert plan.COST_RATIO_DEFAULT == golden["cost_ratio_default"][0]
    assert plan.S_MIN_DEFAULT == golden["s_min"][0]
    assert plan.S_MAX_DEFAULT == golden["s_max"][0] == 2 ** 17
    # standard normal quantiles from tables: Phi^{-1}(0.995), Phi^{-1}(0.9995), Phi^{-1}(0.99995)
    assert plan.z_one_sided(0.005) == pytest.approx(2.5758293, abs=1e-6)
    assert plan.z_one_sided(0.0005) == pytest.approx(3.2905267, abs=1e-6)
    assert plan.z_one_sided(0.00005) == pytest.approx(3.8905919, abs=1e-6)


def test_sae_shape_arithmetic(golden):
    assert golden["sae_batch"][0] * golden["sae_dict"][0] == golden["sae_N"][0]
    assert golden["sae_batch"][0] * golden["sae_k"][0] == golden["sae_K"][0]


def test_worked_example_of_the_sample_size(golden):
    # The text's "S* ~ 4,600" for N = 1e9, k = 100 is the bare scaling factor (kN)^(1/3).
    N, k = int(golden["s_star_example_N"][0]), int(golden["s_star_example_k"][0])
    assert (k * N) ** (1 / 3) == pytest.approx(golden["s_star_example"][0], rel=0.01)
    z = plan.z_total(1e-3)
    ratio = plan.optimal_S(N, k, z) / (k * (N - k)) ** (1 / 3)
    assert ratio == pytest.approx((z * math.log2(k) / 2) ** (2 / 3), rel=1e-12)   # Eq. (optimal_S)


def test_sample_size_scales_with_the_cube_root_of_kN():
    z = plan.z_total(1e-3)
    k = 64
    Ns = np.array([2.0 ** e for e in range(22, 31)])
    s = np.array([plan.optimal_S(int(n), k, z) for n in Ns])
    slope = np.polyfit(np.log(Ns * k), np.log(s), 1)[0]
    assert slope == pytest.approx(1 / 3, abs=1e-4)


@pytest.mark.parametrize("N,k", [(2 ** 28, 1024), (2 ** 24, 37), (10 ** 9, 100)])
def test_optimal_sample_size_minimises_the_cost_model(N, k):
    z = plan.z_total(1e-3)
    res = optimize.minimize_scalar(lambda s: plan.cost_model(N, k, s, z, 1.0), bounds=(16, N / 4), method="bounded",
                                   options={"xatol": 1e-3})
    assert res.x == pytest.approx(plan.optimal_S(N, k, z), rel=1e-4)              # Theorem 2


def test_clamps_and_rounding():
    assert plan.sample_size(2 ** 20, 64, 1e-3) == 32768                            # S* ~ 2,968 -> S_min
    assert plan.sample_size(2 ** 29, 131072, 1e-3) == 131072                       # S* ~ 604k -> S_max
    assert plan.sample_size(2 ** 26, 4096, 1e-2) == plan.round_half_away(plan.optimal_S(2 ** 26, 4096, plan.z_total(1e-2)))
    assert plan.sample_size(2 ** 30, 1, 1e-3) == 32768                             # log2(1) = 0 -> S* = 0
    assert plan.sample_size(1000, 10, 1e-3) == 1000                                # never more than N
    assert plan.round_half_away(2.5) == 3 and plan.round_half_away(2.49) == 2


@pytest.mark.parametrize("N,k,S", [(2 ** 26, 4096, 65536), (2 ** 29, 131072, 131072), (10 ** 6, 5000, 40000)])
def test_buffer_closed_form_is_c_times_k(N, k, S):
    za, zb = plan.z_one_sided(3e-4), plan.z_one_sided(7e-4)                        # unequal split on purpose
    assert plan.eq_c(N, k, S, za, zb) * k == pytest.approx(plan.eq_M(N, k, S, za + zb), rel=1e-12)   # Corollary 1
    # c_0 k is the expected number of survivors N q for q of Eq. (t_choice)
    alpha = k / N
    q = alpha + za * math.sqrt(alpha * (1 - alpha) * plan.fpc(N, S) / S)
    assert plan.eq_c0(N, k, S, za) * k == pytest.approx(N * q, rel=1e-12)
    assert plan.eq_t_choice(N, k, S, za) == math.ceil(S * q - 1e-9)


def test_buffer_example_order_of_magnitude(golden):
    # "M ~ 5,000" for N = 2^29, k = 64: Eq. (M) gives a few thousand for S between 2^15 and 2^17.
    z = plan.z_total(1e-3)
    ms = [plan.eq_M(2 ** 29, 64, s, z) for s in (2 ** 15, 2 ** 16, 2 ** 17)]
    assert ms[0] > golden["m_example"][0] > ms[2]
    assert ms[1] == pytest.approx(golden["m_example"][0], rel=0.05)


def test_excess_buffer_scales_with_cube_root_when_S_is_optimal():
    z = plan.z_total(1e-3)
    k = 256
    Ns = [2 ** e for e in range(24, 31)]
    excess = [plan.eq_M(n, k, plan.optimal_S(n, k, z), z) - k for n in Ns]
    slope = np.polyfit(np.log([n * k for n in Ns]), np.log(excess), 1)[0]
    assert slope == pytest.approx(1 / 3, abs=2e-3)                                 # M - k = O((kN)^(1/3))


def test_algorithm_1_literal_steps():
    # alpha S = 2 < -ln(5e-4) = 7.6  ->  last step forces t = 1
    S, t, M = plan.plan_paper(2 ** 20, 64, 1e-3)
    assert (S, t) == (32768, 1)
    z = plan.z_total(1e-3)
    assert M == math.ceil(64 + z * math.sqrt(64 * (2 ** 20 - 64) / 32768 * (1 - 32768 / 2 ** 20)))
    # dense regime: alpha S = 32 > 7.6 -> Gaussian t kept
    S, t, M = plan.plan_paper(2 ** 29, 131072, 1e-3)
    assert S == 131072 and t == math.ceil(32 + z / 2 * math.sqrt(32 * (1 - 2 ** -12) * (1 - 2 ** -12)))
    assert plan.plan_paper(2 ** 20, 64, 1e-3, apply_sparse_rule=False)[1] == plan.eq_t_choice(2 ** 20, 64, 32768, z / 2)


SHAPES = [(2 ** 20, 64, 1e-3), (2 ** 26, 16, 1e-2), (2 ** 26, 256, 1e-4), (2 ** 26, 4096, 1e-4), (2 ** 20, 32, 1e-3),
          (2 ** 29, 131072, 1e-3), (2 ** 30, 1, 1e-3), (2 ** 30, 65536, 1e-3), (50331648, 131072, 1e-3), (1_000_003, 77, 1e-3)]


@pytest.mark.parametrize("N,k,eps", SHAPES)
def test_guarded_plan_contract(N, k, eps):
    p = plan.plan_guarded(N, k, eps)
    assert p.m == plan.sample_size(N, k, eps) and 1 <= p.r <= p.m and k <= p.capacity <= N
    # Theorem 1's contract, with eps/2 for each failure mode
    assert p.p_recall_fail <= eps / 2 and p.p_overflow <= eps / 2
    assert rank_law.p_recall_fail_srs(N, p.m, p.r, k) <= eps / 2
    assert rank_law.p_overflow_srs(N, p.m, p.r, p.capacity) <= eps / 2
    # minimality of both choices
    if p.r > 1:
        assert rank_law.p_recall_fail_bound(N, p.m, p.r - 1, k) > eps / 2
    m_paper = math.ceil(plan.eq_M(N, k, p.m, p.z))
    assert p.capacity >= m_paper                                                   # never below Eq. (M)
    if p.capacity > m_paper:
        assert rank_law.p_overflow_bound(N, p.m, p.r, p.capacity - 1) > eps / 2
    # the guarded rank is never below the Gaussian one of Eq. (t_choice) by more than rounding, and close to it
    t_gauss = plan.eq_t_choice(N, k, p.m, p.z / 2)
    assert t_gauss - 1 <= p.r <= t_gauss + 6


RELAXED_SHAPES = [(2 ** 26, 4096, 1e-2, 0.5), (2 ** 26, 4096, 1e-2, 0.9), (2 ** 26, 4096, 1e-2, 0.95), (2 ** 26, 256, 1e-4, 0.5),
                  (2 ** 20, 64, 1e-3, 0.9), (2 ** 18, 64, 1e-2, 0.9), (2 ** 29, 131072, 1e-3, 0.95), (1_000_003, 77, 1e-3, 0.9)]


@pytest.mark.parametrize("N,k,eps,recall", RELAXED_SHAPES)
def test_guarded_plan_contract_in_relaxed_mode(N, k, eps, recall):
    """Relaxed recall (the abstract's "recovering 95% of the true top-k"): the paper gives no formula, the
    mathematics does.  With k_rho = ceil(rho k) accepted survivors Theorem 1's budget reads
    Pr(R < k_rho) <= eps/2 and Pr(R > M) <= eps/2, the rank is the smallest that meets the first, and the
    buffer still has to hold the k requested outputs, so the capacity follows k, not k_rho."""
    p = plan.plan_guarded(N, k, eps, recall=recall)
    exact = plan.plan_guarded(N, k, eps)
    k_rho = math.ceil(recall * k)
    assert p.k_accept == k_rho < k and p.m == exact.m
    # the recall half of the budget, for k_rho: the plan's own bound and Lemma 1's exact tail
    assert p.p_recall_fail <= eps / 2
    assert p.p_recall_fail == rank_law.p_recall_fail_bound(N, p.m, p.r, k_rho)
    assert rank_law.p_recall_fail_srs(N, p.m, p.r, k_rho) <= eps / 2
    # minimality: one rank less breaks the bound for k_rho (a plan that took the rank for k would sit above it)
    if p.r > 1:
        assert rank_law.p_recall_fail_bound(N, p.m, p.r - 1, k_rho) > eps / 2
    assert p.r <= exact.r
    # the overflow half of the budget, and a capacity derived from k: never below Eq. (M) for k, and minimal above it
    assert p.p_overflow <= eps / 2 and rank_law.p_overflow_srs(N, p.m, p.r, p.capacity) <= eps / 2
    m_paper = math.ceil(plan.eq_M(N, k, p.m, p.z))
    assert p.capacity >= m_paper >= k
    if p.capacity > m_paper:
        assert rank_law.p_overflow_bound(N, p.m, p.r, p.capacity - 1) > eps / 2
    # a lower rank keeps fewer elements: the capacity does not grow
    assert p.capacity <= exact.capacity


def test_relaxed_rank_differs_from_the_exact_one_where_the_pins_can_see_it():
    # (shapes on which taking the rank for k instead of k_rho, or the reverse, changes the plan)
    for N, k, eps, recall in RELAXED_SHAPES[:4]:
        assert plan.plan_guarded(N, k, eps, recall=recall).r < plan.plan_guarded(N, k, eps).r


def test_guarded_capacity_approaches_the_closed_form_in_the_gaussian_regime():
    ratios = []
    for k in (2 ** 12, 2 ** 15, 2 ** 18, 2 ** 21):                                 # alpha S = 8 .. 4096 at S = 2^17
        N = 2 ** 26
        p = plan.plan_guarded(N, k, 1e-3, s_min=2 ** 17, s_max=2 ** 17)
        ratios.append((p.capacity - k) / (plan.eq_M(N, k, p.m, p.z) - k))
    assert all(r >= 1 for r in ratios)
    assert ratios == sorted(ratios, reverse=True) and ratios[-1] < 1.03


def test_relaxed_mode_and_direct_mode():
    p = plan.plan_guarded(2 ** 26, 4096, 1e-2, recall=0.95)
    assert p.k_accept == math.ceil(0.95 * 4096) == 3892
    assert p.r <= plan.plan_guarded(2 ** 26, 4096, 1e-2).r and p.capacity >= 4096
    assert plan.accept_count(20, 0.95) == 19 and plan.accept_count(16, 0.95) == 16 and plan.accept_count(5, 0.01) == 1
    assert plan.plan_guarded(50000, 10, 1e-3).mode == 1                            # sample would be the whole input
    assert plan.plan_guarded(2 ** 20, 2 ** 19, 1e-3).mode == 1                     # buffer would hold half the input
    assert plan.plan_guarded(2 ** 20, 64, 1e-3).mode == 0
    with pytest.raises(ValueError):
        plan.plan_guarded(10, 11)


@pytest.mark.parametrize("N,k,eps", SHAPES)
def test_second_chance_ranks_aim_between_k_and_the_capacity(N, k, eps):
    """The ranks of the second filtering pass: integers on either side of t whose survivor counts, by Lemma 1's mean
    E[R] = (N+1) r / (S+1), lie inside [k, M] -- a second pass that starts from there can pass the check."""
    p = plan.plan_guarded(N, k, eps)
    tight, loose = plan.second_chance_ranks(N, k, p.m, p.r, p.capacity)
    assert (p.r_tight, p.r_loose) == (tight, loose)
    assert tight == 0 or 1 <= tight < p.r
    assert loose == 0 or p.r < loose <= p.m
    assert tight == p.r * (k + p.capacity) // (2 * p.capacity) or tight == 0
    if tight:
        assert k <= rank_law.nhg_mean(N, p.m, tight) * 1.0 or tight == 1          # mean count of the tighter rank is not below k ...
        assert rank_law.nhg_mean(N, p.m, tight) <= p.capacity                      # ... and fits the buffer
    if loose:
        mean = rank_law.nhg_mean(N, p.m, loose)
        assert k <= mean <= p.capacity + N / p.m                                   # within one stratum of the buffer at most
    if p.r == 1:
        assert tight == 0                                                          # nothing is tighter than the sample maximum
