"""The second filtering pass before the exact fallback (profk_plan_t.r_tight / r_loose): a row that fails the count
check is filtered once more with the threshold of a tighter or looser sample rank; only if that fails too is it
selected exactly.  Outputs are bit-exact either way; status, threshold and survivor count follow the oracle's run of
the same stages (oracle/stages.py)."""
import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
from oracle import stages as o_stages
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    profk.lib()
    torch.cuda.set_device(0)


def bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def check(x, k, pl, seed, want_status=None):
    """One call under plan `pl`: exact output, and per-row status / tau / R equal to the oracle's."""
    v, i = profk.topk(x.cuda(), k, plan_override=pl, seed=seed)
    torch.cuda.synchronize()
    xn = workloads.as_numpy(x)
    xn2 = xn[None, :] if xn.ndim == 1 else xn
    ov, oi = o_topk.topk(xn2, k)
    assert np.array_equal(i.cpu().numpy().reshape(ov.shape[0], k), oi), "indices differ from the oracle"
    assert np.array_equal(bits(workloads.as_numpy(v)).reshape(ov.shape[0], k), bits(ov)), "values differ from the oracle"
    stats = profk.read_stats(xn2.shape[0])
    for r in range(xn2.shape[0]):
        res = o_stages.run_row(xn2[r], k, pl.m, pl.r, pl.capacity, pl.k_accept, seed=seed, row=r, composite=pl.tie_rule == profk.TIES_BY_INDEX,
                               r_tight=pl.r_tight, r_loose=pl.r_loose)
        tau_bits, R, cap, status = stats[r]
        assert status == res.status, (r, status, res.status)
        assert tau_bits == int(bits(np.asarray([res.tau]))[0]), r
        assert R == res.survivors or (res.survivors > cap and R > cap), (r, R, res.survivors)
        if want_status is not None:
            assert status == want_status, (r, status)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,n", [(1, 1 << 22), (3, 1_000_003), (12, 300_001)])
def test_overflow_then_the_tighter_rank(dtype, rows, n):
    x = workloads.normal(rows, n, seed=80, dtype=dtype)
    k = 64
    m, r = 4096, 40                                                           # about 40 n / 4096 survivors
    cap = 25 * n // 4096                                                      # too small for them, enough for rank 20
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_tight=20), seed=1, want_status=profk.ROW_OVERFLOW_REFILTERED)
    # a rank that is hardly tighter overflows again: the exact selection answers
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_tight=39), seed=1, want_status=profk.ROW_OVERFLOW)
    # no tighter rank named: as before
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0), seed=1, want_status=profk.ROW_OVERFLOW)
    # the filter as printed (value-only threshold) takes the same route
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_tight=20, tie_rule=profk.TIES_KEEP_ALL), seed=2)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,n", [(1, 1 << 22), (4, 1_000_003), (9, 300_001)])
def test_recall_failure_then_the_looser_rank(dtype, rows, n):
    x = workloads.normal(rows, n, seed=81, dtype=dtype)
    k = 1000
    m = 32768                                                                 # rank 1: about n / 32768 survivors, far fewer than k
    cap = 5 * k
    loose = -(-5 * k * m // (2 * n))                                          # about 2.5 k survivors expected
    check(x, k, profk.Plan(m=m, r=1, capacity=cap, k_accept=k, mode=0, r_loose=loose), seed=3, want_status=profk.ROW_RECALL_REFILTERED)
    check(x, k, profk.Plan(m=m, r=1, capacity=cap, k_accept=k, mode=0, r_loose=2), seed=3, want_status=profk.ROW_RECALL)
    check(x, k, profk.Plan(m=m, r=1, capacity=cap, k_accept=k, mode=0), seed=3, want_status=profk.ROW_RECALL)


def test_ties_and_special_values_in_the_second_pass():
    n, k = 1 << 21, 200
    rows = {"constant": torch.full((n,), 3.0), "few values": workloads.few_values(n, seed=82, distinct=4),
            "relu bf16": workloads.relu_gaussian(n, seed=83, dtype=torch.bfloat16)}
    special = workloads.normal(1, n, seed=84)[0]
    special[::1000] = float("nan")
    special[1::1000] = -float("nan")
    special[2::3000] = float("inf")
    special[3::5000] = -0.0
    rows["special"] = special
    for name, x in rows.items():
        for rule in (profk.TIES_BY_INDEX, profk.TIES_KEEP_ALL):
            check(x, k, profk.Plan(m=4096, r=60, capacity=40 * n // 4096, k_accept=k, mode=0, r_tight=25, tie_rule=rule), seed=4)
            check(x, k, profk.Plan(m=65536, r=1, capacity=20_000, k_accept=k, mode=0, r_loose=200, tie_rule=rule), seed=5)


def test_the_librarys_own_plan_names_the_ranks_and_the_largest_samples_of_many_rows_skip_them():
    pl = profk.plan(1 << 26, 256, 1e-4)
    assert 0 < pl.r_tight < pl.r < pl.r_loose
    # more than four rows and a sample above 131072: the keys are not kept, the exact selection answers at once
    x = workloads.normal(6, 1 << 20, seed=85)
    pl = profk.Plan(m=262144, r=2560, capacity=8000, k_accept=64, mode=0, r_tight=1280)
    v, i = profk.topk(x.cuda(), 64, plan_override=pl, seed=6)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(workloads.as_numpy(x), 64)
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(v.cpu().numpy()), bits(ov))
    assert all(s[3] == profk.ROW_OVERFLOW for s in profk.read_stats(6))


def test_a_billion_element_row_overflows_and_is_repaired_in_one_more_scan():
    n, k = 1 << 30, 64
    xd = workloads.cauchy(n, 4, device="cuda")
    xn = xd.cpu().numpy()
    keys = o_topk.order_key(xn)
    pl = profk.plan(n, k, 1e-3)
    tight = profk.Plan(m=pl.m, r=8 * pl.r, capacity=pl.capacity, k_accept=k, mode=0, r_tight=pl.r)      # rank 8 t overflows M, rank t fits
    v, i = profk.topk(xd, k, plan_override=tight, seed=7)
    torch.cuda.synchronize()
    assert o_topk.verify_topk(xn, k, v.cpu().numpy(), i.cpu().numpy(), keys=keys) == []
    assert profk.read_stats(1)[0][3] == profk.ROW_OVERFLOW_REFILTERED
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = {}
    for name, plan in (("second pass", tight), ("exact selection", profk.Plan(m=pl.m, r=8 * pl.r, capacity=pl.capacity, k_accept=k, mode=0))):
        for _ in range(2):
            profk.topk(xd, k, plan_override=plan, seed=7)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(5):
            profk.topk(xd, k, plan_override=plan, seed=7)
        e1.record()
        torch.cuda.synchronize()
        times[name] = e0.elapsed_time(e1) / 5
    print("forced overflow at 2^30, ms per call:", times)
    assert times["second pass"] < 0.6 * times["exact selection"]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_batches_repaired_by_the_grid_wide_kernel_take_the_second_pass_too(dtype):
    """More than 18 rows: failed rows are repaired by the grid-wide kernel, one after the other when fewer than eight
    failed.  A capacity just above the expected survivor count makes a few rows of the batch overflow; the tighter rank
    brings most of them back, and every row's status, threshold and count follow the oracle."""
    rows, n, k = 40, 1 << 18, 64
    x = workloads.normal(rows, n, seed=86, dtype=dtype)
    xn = workloads.as_numpy(x)
    m, r = 2048, 16                                                           # 2048 survivors expected, sigma 512
    found = None
    for cap in (2560, 2688, 2816, 2944, 3072):                                # pick a capacity that 1..7 rows exceed
        pl = profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_tight=8)
        first = [o_stages.run_row(xn[row], k, m, r, cap, k, seed=21, row=row, composite=True).status for row in range(rows)]
        if 1 <= sum(s != o_stages.STATUS_OK for s in first) <= 7:
            found = pl
            break
    assert found is not None, "no capacity with 1..7 failing rows: change the seed"
    check(x, k, found, seed=21)
    stats = profk.read_stats(rows)
    assert any(s[3] == profk.ROW_OVERFLOW_REFILTERED for s in stats)
    # recall failures in a few rows: rank 4 of 2048 keeps about 512, k = 250 is within reach of bad luck
    k2 = 250
    found = None
    for r2 in (4, 3):
        pl = profk.Plan(m=m, r=r2, capacity=4000, k_accept=k2, mode=0, r_loose=12)
        first = [o_stages.run_row(xn[row], k2, m, r2, 4000, k2, seed=22, row=row, composite=True).status for row in range(rows)]
        if 1 <= sum(s != o_stages.STATUS_OK for s in first) <= 7:
            found = pl
            break
    assert found is not None, "no rank with 1..7 failing rows: change the seed"
    check(x, k2, found, seed=22)
    assert any(s[3] == profk.ROW_RECALL_REFILTERED for s in profk.read_stats(rows))
    # eight or more failed rows are dealt out one per CTA and selected exactly at once: statuses 1 / 2 as before
    pl = profk.Plan(m=m, r=r, capacity=1024, k_accept=k, mode=0, r_tight=8)
    v, i = profk.topk(x.cuda(), k, plan_override=pl, seed=23)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(xn, k)
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(workloads.as_numpy(v)), bits(ov))
    assert all(s[3] == profk.ROW_OVERFLOW for s in profk.read_stats(rows))


def _btk_forms(xn, k, out):
    """The BatchTopK forms in `out` against the oracle's kept set of the host row xn."""
    want = o_topk.kept_mask(xn, k)
    idx = out["indices"].cpu().numpy()
    assert np.array_equal(np.sort(idx), np.flatnonzero(want)), "kept indices differ from the oracle's set"
    assert np.array_equal(bits(workloads.as_numpy(out["values"])), bits(xn[idx]))
    assert np.array_equal(out["mask"].cpu().numpy().view(np.uint32), o_topk.pack_mask(want))
    dense = np.zeros_like(xn)
    dense[want] = xn[want]
    assert np.array_equal(bits(workloads.as_numpy(out["dense"]).reshape(-1)), bits(dense))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_large_selections_from_one_row_take_the_second_pass_inside_their_fused_kernels(dtype):
    """k beyond what one CTA orders: the ordering kernel of `profk_topk_*` and the emit kernel of `profk_batchtopk_*`
    repair their single row themselves, with the same second filtering pass before the exact selection."""
    n, k, m = 3_000_001, 20_000, 65536                                        # a sample rank keeps about 45.8 elements
    x = workloads.normal(1, n, seed=87, dtype=dtype)[0]
    xn = workloads.as_numpy(x)
    cap = 34_000
    cases = [
        (profk.Plan(m=m, r=1000, capacity=cap, k_accept=k, mode=0, r_tight=600), profk.ROW_OVERFLOW_REFILTERED),   # 45.8 K, then 27.5 K
        (profk.Plan(m=m, r=1000, capacity=cap, k_accept=k, mode=0, r_tight=990), profk.ROW_OVERFLOW),              # overflows again
        (profk.Plan(m=m, r=1000, capacity=cap, k_accept=k, mode=0), profk.ROW_OVERFLOW),                           # no rank named
        (profk.Plan(m=m, r=300, capacity=cap, k_accept=k, mode=0, r_loose=600), profk.ROW_RECALL_REFILTERED),      # 13.7 K, then 27.5 K
        (profk.Plan(m=m, r=300, capacity=cap, k_accept=k, mode=0, r_loose=310), profk.ROW_RECALL),                 # too few again
        (profk.Plan(m=m, r=1000, capacity=cap, k_accept=k, mode=0, r_tight=600, tie_rule=profk.TIES_KEEP_ALL), None),
    ]
    for seed, (pl, want) in enumerate(cases):
        check(x, k, pl, seed=30 + seed, want_status=want)
        ordered = profk.read_stats(1)[0]
        out = profk.batchtopk(x.cuda(), k, seed=30 + seed, want_pairs=True, want_mask=True, want_dense=True, plan_override=pl)
        torch.cuda.synchronize()
        _btk_forms(xn, k, out)
        assert profk.read_stats(1)[0] == ordered                             # same stages, same threshold, count and status
    # in place: the second pass and the exact selection read the input before the dense form overwrites it
    xc = x.cuda().clone()
    out = profk.batchtopk(xc, k, seed=30, want_pairs=True, want_mask=True, in_place=True, plan_override=cases[0][0])
    torch.cuda.synchronize()
    _btk_forms(xn, k, out)
    assert profk.read_stats(1)[0][3] == profk.ROW_OVERFLOW_REFILTERED


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_large_selections_from_a_few_rows_take_the_second_pass_in_the_repair_kernel(dtype):
    """Two to four rows with k beyond what one CTA orders: the grid-wide repair kernel between the two phases of the large
    refine filters a failed row once more; the second phase orders what that pass left."""
    rows, n, k, m = 3, 2_000_003, 20_000, 65536                               # a sample rank keeps about 30.5 elements
    x = workloads.normal(rows, n, seed=88, dtype=dtype)
    cap = 34_000
    check(x, k, profk.Plan(m=m, r=1500, capacity=cap, k_accept=k, mode=0, r_tight=900), seed=40, want_status=profk.ROW_OVERFLOW_REFILTERED)
    check(x, k, profk.Plan(m=m, r=1500, capacity=cap, k_accept=k, mode=0, r_tight=1490), seed=41, want_status=profk.ROW_OVERFLOW)
    check(x, k, profk.Plan(m=m, r=450, capacity=cap, k_accept=k, mode=0, r_loose=900), seed=42, want_status=profk.ROW_RECALL_REFILTERED)
    check(x, k, profk.Plan(m=m, r=450, capacity=cap, k_accept=k, mode=0), seed=43, want_status=profk.ROW_RECALL)
    # a mix: one row's own capacity problem only (the others pass): a capacity between the rows' survivor counts
    pl = profk.Plan(m=m, r=1000, capacity=cap, k_accept=k, mode=0, r_tight=800)        # about 30.5 K survivors: all pass
    check(x, k, pl, seed=44, want_status=profk.ROW_OK)


@pytest.mark.parametrize("dtype,n", [(torch.bfloat16, 500_009), (torch.float32, (1 << 24) + 5)])
def test_large_selections_from_up_to_eighteen_rows_take_the_second_pass_when_the_sample_is_small(dtype, n):
    """Five to eighteen rows whose k (above 8192) the grid refines -- bf16 at any row length, fp32 from 2^24 elements on:
    the second pass is taken when the sample has at most 131072 keys, the exact selection otherwise."""
    rows, k, m = 6, 9000, 32768
    x = workloads.normal(rows, n, seed=89, dtype=dtype)
    per = n / m                                                               # survivors per sample rank
    r, cap = int(30_000 / per) + 1, 22_000                                    # about 30 K survivors: too many
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_tight=int(15_000 / per) + 1), seed=50,
          want_status=profk.ROW_OVERFLOW_REFILTERED)
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0), seed=50, want_status=profk.ROW_OVERFLOW)
    r = max(int(4_000 / per), 1)                                              # about 4 K survivors: too few
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_loose=int(15_000 / per) + 1), seed=51,
          want_status=profk.ROW_RECALL_REFILTERED)
    # 262144 keys are not kept: the exact selection answers
    pl = profk.Plan(m=8 * m, r=8 * r, capacity=cap, k_accept=k, mode=0, r_loose=8 * int(15_000 / per) + 8)
    v, i = profk.topk(x.cuda(), k, plan_override=pl, seed=52)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(workloads.as_numpy(x), k)
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(workloads.as_numpy(v)), bits(ov))
    assert all(s[3] == profk.ROW_RECALL for s in profk.read_stats(rows))


def test_a_few_rows_of_a_grid_ordered_call_fail_and_the_others_pass():
    """Seven rows, k above what one CTA orders for them: the groups of the grid order the rows that pass, then the whole
    grid repairs the others -- some by the second pass, one (no room even for the tighter rank) exactly."""
    rows, n, k, m = 7, 400_003, 9000, 32768
    x = workloads.normal(rows, n, seed=90, dtype=torch.bfloat16)
    xn = workloads.as_numpy(x)
    per = n / m
    r = int(20_000 / per) + 1
    tight = int(14_000 / per) + 1
    first = sorted(o_stages.run_row(xn[i], k, m, r, n, k, seed=60, row=i, composite=True).survivors for i in range(rows))
    cap = (first[2] + first[3]) // 2                                          # three rows fit, four overflow
    assert first[2] < cap < first[3]
    pl = profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, r_tight=tight)
    check(x, k, pl, seed=60)
    got = sorted(s[3] for s in profk.read_stats(rows))
    assert got == [profk.ROW_OK] * 3 + [profk.ROW_OVERFLOW_REFILTERED] * 4
    # no tighter rank named: the four rows are selected exactly
    check(x, k, profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0), seed=60)
    assert sorted(s[3] for s in profk.read_stats(rows)) == [profk.ROW_OK] * 3 + [profk.ROW_OVERFLOW] * 4


def test_twelve_long_rows_with_the_largest_kept_sample():
    """12 rows of 2^22 under a 131072-key sample: one CTA orders each row, its clusters take the second pass."""
    rows, n, k, m = 12, 1 << 22, 256, 131072
    x = workloads.normal(rows, n, seed=91)
    per = n / m                                                               # 32 survivors per sample rank
    check(x, k, profk.Plan(m=m, r=200, capacity=4000, k_accept=k, mode=0, r_tight=60), seed=70, want_status=profk.ROW_OVERFLOW_REFILTERED)
    check(x, k, profk.Plan(m=m, r=2, capacity=4000, k_accept=k, mode=0, r_loose=40), seed=71, want_status=profk.ROW_RECALL_REFILTERED)
