"""Monte Carlo pins: the guarded plan keeps Theorem 1's budget; Algorithm 1's t = 1 step does not."""
import numpy as np
import pytest

from oracle import mc, plan, rank_law


def test_simulated_rank_follows_lemma_1():
    rng = np.random.default_rng(0)
    N, S, t = 4096, 64, 3
    R = mc.simulate_ranks(N, S, t, 4000, rng)
    assert R.mean() == pytest.approx(rank_law.nhg_mean(N, S, t), rel=0.03)
    assert R.var() == pytest.approx(rank_law.nhg_var(N, S, t), rel=0.12)
    assert R.min() >= t and R.max() <= N - S + t


def test_guarded_plan_meets_the_budget_on_small_rows():
    rng = np.random.default_rng(1)
    N, k, eps = 1 << 16, 64, 2e-2                                   # large eps so a few thousand trials resolve it
    p = plan.plan_guarded(N, k, eps, s_min=2048, s_max=2048)
    for placement in ("random", "sorted"):
        R = mc.simulate_ranks(N, p.m, p.r, 3000, rng, placement)
        rate = np.mean((R < k) | (R > p.capacity))
        assert rate <= eps + 3 * np.sqrt(eps / 3000)


def test_literal_sparse_rule_breaks_the_budget():
    rng = np.random.default_rng(2)
    N, k, eps = 1 << 16, 64, 1e-3
    S, t, M = plan.plan_paper(N, k, eps, s_min=2048, s_max=2048)
    assert t == 1                                                    # alpha S = 2 < -ln(eps/2)
    R = mc.simulate_ranks(N, S, t, 500, rng)
    assert np.mean(R < k) > 0.5                                      # ~ 1 - exp(-alpha S) = 0.86, not exp(-alpha S)


@pytest.mark.parametrize("N,k,eps", [(1 << 20, 64, 1e-3), (1 << 26, 256, 1e-2), (1 << 26, 4096, 1e-2), (1 << 29, 131072, 1e-3)])
def test_failure_rates_at_the_benchmark_shapes(N, k, eps):
    rng = np.random.default_rng(3)
    trials = 400_000
    p = plan.plan_guarded(N, k, eps)
    fa, fb = mc.failure_rate_exchangeable(N, p.m, p.r, k, p.capacity, trials, rng)
    sigma = np.sqrt(eps / trials)
    assert fa + fb <= eps + 4 * sigma
    assert fa == pytest.approx(rank_law.p_recall_fail_srs(N, p.m, p.r, k), abs=4 * sigma)
    assert fb == pytest.approx(rank_law.p_overflow_srs(N, p.m, p.r, p.capacity), abs=4 * sigma)
    # Algorithm 1 as printed, same shape: at least one of its failure modes is far over budget
    S, t, M = plan.plan_paper(N, k, eps)
    ga, gb = mc.failure_rate_exchangeable(N, S, t, k, M, 20_000, rng)
    assert ga + gb > eps


@pytest.mark.parametrize("N,k,eps,recall", [(1 << 26, 4096, 1e-2, 0.5), (1 << 26, 4096, 1e-2, 0.9), (1 << 26, 4096, 1e-2, 0.95)])
def test_relaxed_plan_meets_the_budget_for_the_accepted_count_and_no_lower_rank_does(N, k, eps, recall):
    """Relaxed recall by simulation: the failure events are R < k_rho and R > M.  The plan keeps their total
    within eps, and its rank is minimal -- at one rank less the simulated recall failure alone exceeds eps/2."""
    rng = np.random.default_rng(5)
    trials = 400_000
    p = plan.plan_guarded(N, k, eps, recall=recall)
    assert p.k_accept == int(np.ceil(recall * k)) and p.r > 1
    fa, fb = mc.failure_rate_exchangeable(N, p.m, p.r, p.k_accept, p.capacity, trials, rng)
    sigma = np.sqrt(eps / trials)
    assert fa + fb <= eps + 4 * sigma
    assert fa == pytest.approx(rank_law.p_recall_fail_srs(N, p.m, p.r, p.k_accept), abs=4 * sigma)
    ga, _ = mc.failure_rate_exchangeable(N, p.m, p.r - 1, p.k_accept, p.capacity, trials, rng)
    assert ga > eps / 2 + 4 * sigma
    # against the full k the same rank would be over budget: the plan really is the one for k_rho
    ha, _ = mc.failure_rate_exchangeable(N, p.m, p.r, k, p.capacity, trials, rng)
    assert ha > eps / 2 + 4 * sigma if recall < 0.95 else ha > fa


def test_record_threshold_keeps_the_budget_on_rows_full_of_ties():
    """The four stages run on rows whose values repeat thousands of times: with the threshold taken as a
    (value, index) record the count check fails no more often than the budget allows, as on distinct values;
    with the filter as printed the copies of tau overflow the buffer on every run."""
    from oracle import stages
    rng = np.random.default_rng(4)
    N, k, eps = 1 << 15, 16, 5e-2
    p = plan.plan_guarded(N, k, eps, s_min=1024, s_max=1024)
    rows = {"constant": np.full(N, 3.0, dtype=np.float32),
            "four values": rng.integers(0, 4, size=N).astype(np.float32),
            "relu": np.maximum(rng.standard_normal(N), 0.0).astype(np.float32)}
    trials = 400
    for name, x in rows.items():
        by_record = sum(stages.run_row(x, k, p.m, p.r, p.capacity, p.k_accept, seed=s, composite=True).status != stages.STATUS_OK
                        for s in range(trials))
        assert by_record <= trials * eps + 3 * np.sqrt(trials * eps), name
        if name != "relu":                                           # (relu: the top of the row is distinct values)
            literal = sum(stages.run_row(x, k, p.m, p.r, p.capacity, p.k_accept, seed=s).status == stages.STATUS_OVERFLOW
                          for s in range(40))
            assert literal == 40, name
