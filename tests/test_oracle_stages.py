"""Pins for oracle.stages: the four stages of Section 3 run on NumPy arrays."""
import numpy as np
import pytest

from oracle import philox, stages, topk


def test_success_branch_returns_the_exact_topk():
    rng = np.random.default_rng(0)
    hits = 0
    for seed in range(40):
        x = rng.standard_normal(4096).astype(np.float32)
        res = stages.run_row(x, k=20, m=256, r=4, capacity=400, k_accept=20, seed=seed)
        v, i = topk.topk_row(x, 20)
        assert np.array_equal(res.idx, i) and np.array_equal(res.vals, v)          # always exact, whichever branch
        if res.status == stages.STATUS_OK:
            hits += 1
            assert 20 <= res.survivors <= 400
    assert hits > 20


def test_survivor_count_is_the_rank_of_tau():
    x = np.random.default_rng(1).permutation(5000).astype(np.float32)              # distinct values
    s_idx = philox.sample_indices(5000, 100, seed=9)
    tau = stages.threshold(x, s_idx, 3)
    assert tau == np.sort(x[s_idx])[::-1][2]
    R = stages.count_survivors(x, tau)
    assert R == int(np.flatnonzero(np.sort(x)[::-1] == tau)[0]) + 1                # Lemma 1's R: rank 1 = largest
    assert np.array_equal(stages.survivor_set(x, tau), np.flatnonzero(x >= tau))


def test_failure_branches_by_construction():
    x = np.arange(1000, dtype=np.float32)
    # capacity too small for the survivors of a low threshold -> overflow
    res = stages.run_row(x, k=5, m=10, r=10, capacity=5, k_accept=5, seed=1)
    assert res.status == stages.STATUS_OVERFLOW and res.survivors > 5
    assert np.array_equal(res.idx, np.arange(999, 994, -1))
    # threshold = sample maximum, k larger than what survives -> insufficient recall
    res = stages.run_row(x, k=400, m=10, r=1, capacity=1000, k_accept=400, seed=1)
    assert res.status == stages.STATUS_RECALL and res.survivors < 400
    assert np.array_equal(res.idx, np.arange(999, 599, -1))
    # all-equal input: every element passes "x >= tau" -> overflow, answer = lowest indices
    z = np.zeros(300, dtype=np.float32)
    res = stages.run_row(z, k=7, m=20, r=2, capacity=50, k_accept=7, seed=3)
    assert res.status == stages.STATUS_OVERFLOW and res.survivors == 300
    assert np.array_equal(res.idx, np.arange(7))
    # direct mode
    res = stages.run_row(x, k=3, m=0, r=0, capacity=0, k_accept=3, seed=0, mode=1)
    assert res.status == stages.STATUS_DIRECT and res.idx.tolist() == [999, 998, 997]


def test_relaxed_mode_returns_a_padded_prefix():
    x = np.arange(1000, dtype=np.float32)
    for seed in range(20):
        res = stages.run_row(x, k=100, m=50, r=3, capacity=1000, k_accept=20, seed=seed)
        if res.status == stages.STATUS_OK and res.survivors < 100:
            R = res.survivors
            assert np.array_equal(res.idx[:R], np.arange(999, 999 - R, -1))        # prefix of the exact answer
            assert np.all(res.idx[R:] == -1) and np.all(np.isneginf(res.vals[R:]))
            return
    pytest.fail("no seed produced a short buffer")


def test_bf16_rows_and_nan_are_kept():
    rng = np.random.default_rng(3)
    f = rng.standard_normal(2000).astype(np.float32)
    b = (f.view(np.uint32) >> 16).astype(np.uint16)
    res = stages.run_row(b, k=10, m=64, r=4, capacity=2000, k_accept=10, seed=5)
    v, i = topk.topk_row(b, 10)
    assert np.array_equal(res.idx, i) and np.array_equal(res.vals, v)
    g = f.copy(); g[17] = np.nan
    tau = np.float32(1.0)
    assert 17 in stages.survivor_set(g, tau)                                       # not (NaN < tau)


# ----------------------------------------------------------------------------- tie-proof variant (records)
def _records_desc(x):
    """All (value, index) records of the row in the order (value descending, index ascending), by brute force."""
    return sorted(range(len(x)), key=lambda i: (-float(x[i]), i))


def test_record_threshold_on_distinct_values_changes_nothing():
    x = np.random.default_rng(3).permutation(4000).astype(np.float32)
    s_idx = philox.sample_indices(4000, 64, seed=2)
    tau, tau_idx = stages.threshold_record(x, s_idx, 5)
    assert tau == stages.threshold(x, s_idx, 5) and x[tau_idx] == tau and tau_idx in set(s_idx.tolist())
    assert np.array_equal(stages.survivor_set_record(x, tau, tau_idx), stages.survivor_set(x, tau))
    for seed in range(10):
        a = stages.run_row(x, 20, 64, 3, 600, 20, seed=seed)
        b = stages.run_row(x, 20, 64, 3, 600, 20, seed=seed, composite=True)
        assert (a.status, a.survivors) == (b.status, b.survivors) and np.array_equal(a.idx, b.idx)


def test_record_threshold_with_ties_is_the_rank_of_the_threshold_record():
    rng = np.random.default_rng(4)
    x = rng.integers(0, 4, size=600).astype(np.float32)                # four values, 150 copies each
    order = _records_desc(x)
    for seed in range(8):
        s_idx = philox.sample_indices(600, 40, seed=seed)
        for t in (1, 3, 10, 40):
            tau, tau_idx = stages.threshold_record(x, s_idx, t)
            # brute force: the t-th sampled record in the full order of records
            sampled_in_order = [i for i in order if i in set(s_idx.tolist())]
            assert tau_idx == sampled_in_order[t - 1] and tau == x[tau_idx]
            kept = stages.survivor_set_record(x, tau, tau_idx)
            rank = order.index(tau_idx) + 1                             # Lemma 1's R for distinct records
            assert kept.size == rank and set(kept.tolist()) == set(order[:rank])
            # the literal filter keeps every copy of tau: at least as many, usually far more
            assert stages.count_survivors(x, tau) >= rank


def test_record_filter_on_a_constant_row_follows_the_rank_law():
    # All elements equal: the literal filter keeps the whole row (R = N, certain overflow); on records the row is
    # as good as sorted by index, R = tau_idx + 1, and its mean is Lemma 1's t (N + 1) / (S + 1).
    n, S, t = 20_000, 200, 7
    x = np.full(n, 2.5, dtype=np.float32)
    Rs = []
    for seed in range(300):
        s_idx = philox.sample_indices(n, S, seed=seed)
        tau, tau_idx = stages.threshold_record(x, s_idx, t)
        assert tau_idx == np.sort(s_idx)[t - 1]
        R = stages.survivor_set_record(x, tau, tau_idx).size
        assert R == tau_idx + 1
        Rs.append(R)
        assert stages.count_survivors(x, tau) == n
    # (stratified sampling: the t-th smallest index lies in stratum t - 1, uniformly: mean (t - 1/2) N / S + 1/2)
    assert abs(np.mean(Rs) - ((t - 0.5) * n / S + 0.5)) < 3 * (n / S) / np.sqrt(12 * 300)
    res = stages.run_row(x, k=50, m=S, r=t, capacity=2000, k_accept=50, seed=1, composite=True)
    assert res.status == stages.STATUS_OK and np.array_equal(res.idx, np.arange(50))
    assert stages.run_row(x, k=50, m=S, r=t, capacity=2000, k_accept=50, seed=1).status == stages.STATUS_OVERFLOW


def test_record_filter_keeps_the_topk_whenever_enough_survive():
    rng = np.random.default_rng(5)
    for seed in range(30):
        x = rng.integers(0, 8, size=3000).astype(np.float32)           # heavy ties
        res = stages.run_row(x, k=25, m=128, r=4, capacity=500, k_accept=25, seed=seed, composite=True)
        v, i = topk.topk_row(x, 25)
        assert np.array_equal(res.idx, i) and np.array_equal(res.vals, v)


# ----------------------------------------------------------------------------- the filter's comparison on special values
def _f32(bits_list):
    return np.array(bits_list, dtype=np.uint32).view(np.float32)


def test_filter_comparison_is_the_total_order_on_zeros_and_nans():
    NEG_NAN, POS_NAN = 0xFFC00000, 0x7FC00000
    x = _f32([NEG_NAN, NEG_NAN, NEG_NAN, 0x3F800000, 0x3F000000, 0x3E4CCCCD, 0x00000000, 0x80000000, POS_NAN])
    #          -nan     -nan     -nan     1.0         0.5         0.2         +0.0        -0.0        +nan
    one, zero, neg_zero = x[3], x[6], x[7]
    # floating point would call the three sign-bit NaNs "not below 1.0"; in the total order they rank lowest
    assert stages.survivor_set(x, one).tolist() == [3, 8] and stages.count_survivors(x, one) == 2
    assert stages.survivor_set(x, zero).tolist() == [3, 4, 5, 6, 8]          # -0.0 ranks below +0.0
    assert stages.survivor_set(x, neg_zero).tolist() == [3, 4, 5, 6, 7, 8]
    # whatever the threshold, the kept elements are the R largest of the row: the buffer's top-k is the row's
    for tau in x:
        kept = stages.survivor_set(x, tau)
        R = kept.size
        _, want = topk.topk_row(x, R)
        assert sorted(kept.tolist()) == sorted(want.tolist())
    # a run through all four stages on a row with sign-bit NaNs: the count check passes and the answer is exact
    rng = np.random.default_rng(9)
    y = rng.standard_normal(5000).astype(np.float32)
    y[::7] = _f32([NEG_NAN])[0]
    v, i = topk.topk_row(y, 10)
    statuses = set()
    for seed in range(20):
        # threshold = the sample maximum: fewer than ten elements rank at or above it, though 715 NaNs are "not below" it
        res = stages.run_row(y, k=10, m=64, r=1, capacity=2000, k_accept=10, seed=seed)
        assert np.array_equal(res.idx, i)
        statuses.add(res.status)
    assert stages.STATUS_RECALL in statuses


# ----------------------------------------------------------------------------- second chance before the exact fallback
def test_second_chance_ranks_and_the_second_filtering_pass_by_hand():
    """A row built by hand, N = 64, sample of S = 16 (one index per stratum of four).  The thresholds of the three
    ranks are read off the sorted sample, the survivor counts by counting, and the branch taken follows from them."""
    from oracle import philox
    rng = np.random.default_rng(21)
    x = rng.permutation(64).astype(np.float32)                       # distinct values 0..63
    s_idx = philox.sample_indices(64, 16, seed=9, row=0)
    sample_desc = np.sort(x[s_idx])[::-1]
    count = lambda tau: int(np.count_nonzero(x >= tau))              # distinct values: R is a plain count
    k = 6
    # overflow with rank 8, buffer of 20: the tighter rank 3 must bring the count back into [k, 20]
    R8, R3 = count(sample_desc[7]), count(sample_desc[2])
    assert R8 > 20 and k <= R3 <= 20, (R8, R3)                       # (the hand-picked seed makes it so)
    res = stages.run_row(x, k, 16, 8, 20, k, seed=9, r_tight=3)
    assert res.status == stages.STATUS_OVERFLOW_REFILTERED and res.survivors == R3 and res.tau == sample_desc[2]
    ov, oi = topk.topk_brute(x, k)
    assert np.array_equal(res.idx, oi) and np.array_equal(res.vals, ov)
    # without a tighter rank, or with one that still overflows, the exact fallback answers, reporting the first pass
    for tight in (0, 7):
        res = stages.run_row(x, k, 16, 8, 20, k, seed=9, r_tight=tight)
        assert res.status == stages.STATUS_OVERFLOW and res.survivors == R8 and res.tau == sample_desc[7]
        assert np.array_equal(res.idx, oi)
    # recall failure with rank 1 (the sample maximum) and k = 12: the looser rank 5 repairs it, rank 2 does not
    k = 12
    R1, R2, R5 = count(sample_desc[0]), count(sample_desc[1]), count(sample_desc[4])
    assert R1 < k and R2 < k and k <= R5 <= 40, (R1, R2, R5)
    ov, oi = topk.topk_brute(x, k)
    res = stages.run_row(x, k, 16, 1, 40, k, seed=9, r_loose=5)
    assert res.status == stages.STATUS_RECALL_REFILTERED and res.survivors == R5 and res.tau == sample_desc[4]
    assert np.array_equal(res.idx, oi) and np.array_equal(res.vals, ov)
    res = stages.run_row(x, k, 16, 1, 40, k, seed=9, r_loose=2)
    assert res.status == stages.STATUS_RECALL and res.survivors == R1 and np.array_equal(res.idx, oi)
    # the tie-proof variant takes the same branches on distinct values
    res = stages.run_row(x, k, 16, 1, 40, k, seed=9, r_loose=5, composite=True)
    assert res.status == stages.STATUS_RECALL_REFILTERED and res.survivors == R5 and np.array_equal(res.idx, oi)
    # relaxed mode: the second pass is checked against the full k
    res = stages.run_row(x, 12, 16, 1, 40, 3, seed=9, r_loose=2)     # k_accept = 3: R1 decides
    assert (res.status == stages.STATUS_OK) == (R1 >= 3)
