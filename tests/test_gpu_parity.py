"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
from oracle import philox as o_philox
from oracle import plan as o_plan
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


def bits(a: np.ndarray) -> np.ndarray:
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def gpu_topk(x: torch.Tensor, k: int, **kw):
    v, i = profk.topk(x.cuda(), k, **kw)
    torch.cuda.synchronize()
    return workloads.as_numpy(v), i.cpu().numpy()


def assert_exact(x: torch.Tensor, k: int, v: np.ndarray, i: np.ndarray):
    xn = workloads.as_numpy(x)
    ov, oi = o_topk.topk(xn, k)
    assert np.array_equal(i, oi), "indices differ from the oracle"
    assert np.array_equal(bits(v), bits(ov)), "values differ from the oracle"


def assert_stats_match(x: torch.Tensor, k: int, pl, seed: int, stats, rows=None):
    """Threshold, survivor count and outcome of the count check, row by row, against the oracle's run of the four
    stages under the same plan, seed and tie rule."""
    xn = workloads.as_numpy(x)
    xn = xn[None, :] if xn.ndim == 1 else xn
    for r in (range(xn.shape[0]) if rows is None else rows):
        tau_bits, R, cap, status = stats[r]
        # A row repaired by the second filtering pass (statuses 4 and 5; only calls whose refine kernel repairs rows
        # itself take it) is compared with the oracle's run of that pass, any other row with the run without it.
        second = status in (profk.ROW_RECALL_REFILTERED, profk.ROW_OVERFLOW_REFILTERED)
        res = o_stages.run_row(xn[r], k, pl.m, pl.r, pl.capacity, pl.k_accept, seed=seed, row=r,
                               composite=getattr(pl, "tie_rule", profk.TIES_BY_INDEX) == profk.TIES_BY_INDEX,
                               r_tight=getattr(pl, "r_tight", 0) if second else 0, r_loose=getattr(pl, "r_loose", 0) if second else 0)
        assert cap == pl.capacity
        assert tau_bits == int(bits(np.asarray([res.tau]))[0]), f"row {r}: threshold differs"     # same sample, same threshold
        assert status == res.status, f"row {r}: status {status}, oracle {res.status}"
        assert R == res.survivors or (res.survivors > cap and R > cap), f"row {r}: R = {R}, oracle {res.survivors}"


# ----------------------------------------------------------------------------- whole call
def test_config1_uniform_2p20_k64():
    x = workloads.uniform(1 << 20, seed=0)
    v, i = gpu_topk(x, 64, eps=1e-3, seed=0)
    assert_exact(x, 64, v, i)
    pl = o_plan.plan_guarded(1 << 20, 64, 1e-3, **profk.default_tuning(1 << 20))     # the oracle's plan on the library's tuning inputs
    assert_stats_match(x, 64, pl, 0, profk.read_stats(1))


@pytest.mark.parametrize("seed", range(6))
def test_result_does_not_depend_on_the_seed(seed):
    x = workloads.normal(1, 1 << 18, seed=77)[0]
    v, i = gpu_topk(x, 100, eps=1e-3, seed=seed)
    assert_exact(x, 100, v, i)


@pytest.mark.parametrize("n,k", [(1, 1), (2, 2), (5, 3), (33, 33), (1000, 1), (4097, 17), (65537, 256), (262145, 1000),
                                 (1_000_003, 77), (3_000_001, 2999)])
def test_ragged_sizes(n, k):
    x = workloads.normal(1, n, seed=n)[0]
    v, i = gpu_topk(x, k, eps=1e-3, seed=1)
    assert_exact(x, k, v, i)


def test_unaligned_base_pointer_and_odd_row_stride():
    big = workloads.normal(1, 3 * 100_003 + 8, seed=5)[0].cuda()
    for off in (1, 2, 3):
        x = big[off: off + 3 * 100_003].view(3, 100_003)                     # rows start at odd element offsets
        v, i = profk.topk(x, 50, eps=1e-3, seed=2)
        torch.cuda.synchronize()
        assert_exact(x.cpu(), 50, v.cpu().numpy(), i.cpu().numpy())
    xb = big.to(torch.bfloat16)
    for off in (1, 3, 7):
        x = xb[off: off + 3 * 100_003].view(3, 100_003)
        v, i = profk.topk(x, 50, eps=1e-3, seed=2)
        torch.cuda.synchronize()
        assert_exact(x.cpu(), 50, workloads.as_numpy(v), i.cpu().numpy())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_batched_rows(dtype):
    x = workloads.normal(24, 1 << 17, seed=2, dtype=dtype)
    v, i = gpu_topk(x, 32, eps=1e-3, seed=9)
    assert_exact(x, 32, v, i)
    stats = profk.read_stats(24)
    pl = o_plan.plan_guarded(1 << 17, 32, 1e-3, **profk.default_tuning(1 << 17))
    assert_stats_match(x, 32, pl, 9, stats)                  # (bf16 rows hold many copies of their threshold)
    # the same rows with the filter as printed: every copy of the threshold value survives
    literal = profk.Plan(m=pl.m, r=pl.r, capacity=pl.capacity, k_accept=pl.k_accept, mode=0, tie_rule=profk.TIES_KEEP_ALL)
    v, i = profk.topk(x.cuda(), 32, plan_override=literal, seed=9)
    torch.cuda.synchronize()
    assert_exact(x, 32, workloads.as_numpy(v), i.cpu().numpy())
    assert_stats_match(x, 32, literal, 9, profk.read_stats(24))


# ----------------------------------------------------------------------------- forced failures
def _forced(x, k, plan):
    v, i = profk.topk(x.cuda(), k, plan_override=plan, seed=3)
    torch.cuda.synchronize()
    rows = 1 if x.dim() == 1 else x.shape[0]
    return workloads.as_numpy(v), i.cpu().numpy(), profk.read_stats(rows)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_forced_overflow_recall_failure_and_direct_mode(dtype):
    x = workloads.normal(5, 200_000, seed=11, dtype=dtype)
    k = 64
    # capacity == k: every row overflows
    v, i, st = _forced(x, k, profk.Plan(m=4096, r=40, capacity=k, k_accept=k, mode=0))
    assert_exact(x, k, v, i)
    assert all(s[3] == profk.ROW_OVERFLOW for s in st)
    # threshold = sample maximum: (almost) nothing survives
    v, i, st = _forced(x, k, profk.Plan(m=65536, r=1, capacity=4096, k_accept=k, mode=0))
    assert_exact(x, k, v, i)
    assert all(s[3] == profk.ROW_RECALL and s[1] < k for s in st)
    # direct exact selection
    v, i, st = _forced(x, k, profk.Plan(m=0, r=0, capacity=k, k_accept=k, mode=1))
    assert_exact(x, k, v, i)
    assert all(s[3] == profk.ROW_DIRECT for s in st)


def test_mixed_rows_some_fail():
    # rows 0 and 2 hold many copies of their maximum: with the filter as printed their buffers overflow, the others do not
    x = workloads.normal(4, 150_000, seed=12)
    x[0, ::3] = 9.0
    x[2, 1::2] = 7.5
    pl = profk.Plan(m=2048, r=4, capacity=2000, k_accept=40, mode=0, tie_rule=profk.TIES_KEEP_ALL)
    v, i, st = _forced(x, 40, pl)
    assert_exact(x, 40, v, i)
    assert [s[3] for s in st] == [profk.ROW_OVERFLOW, profk.ROW_OK, profk.ROW_OVERFLOW, profk.ROW_OK]
    assert_stats_match(x, 40, pl, 3, st)
    # with the threshold as a record only the copies up to the threshold's index survive: no row fails
    pl = profk.Plan(m=2048, r=4, capacity=2000, k_accept=40, mode=0)
    v, i, st = _forced(x, 40, pl)
    assert_exact(x, 40, v, i)
    assert_stats_match(x, 40, pl, 3, st)
    assert [s[3] for s in st] == [profk.ROW_OK] * 4


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_threshold_record_on_rows_full_of_copies(dtype):
    # constant rows, rows of a few values, a row whose copies of the threshold straddle tile and row ends, under
    # both tie rules and for ranks that take the candidate ranking (small t) and the radix path (deep t)
    n = 400_003
    g = torch.Generator().manual_seed(31)
    x = torch.stack([torch.full((n,), 1.25), torch.randint(0, 3, (n,), generator=g).float(),
                     torch.relu(torch.randn(n, generator=g) - 1.0), torch.zeros(n),
                     torch.randint(0, 200, (n,), generator=g).float() / 8]).to(dtype)
    x[3, -5:] = 1.0
    for m, r, cap in ((4096, 6, 3000), (4096, 200, 40_000), (32768, 3000, 60_000), (1024, 1024, n // 2)):
        for rule in (profk.TIES_BY_INDEX, profk.TIES_KEEP_ALL):
            pl = profk.Plan(m=m, r=r, capacity=cap, k_accept=50, mode=0, tie_rule=rule)
            v, i, st = _forced(x, 50, pl)
            assert_exact(x, 50, v, i)
            assert_stats_match(x, 50, pl, 3, st)
    # one long row: the sample is gathered by its own kernel and selected by a 16-CTA cluster
    y = torch.randint(0, 4, (6_000_000,), generator=g).float().to(dtype)
    for m, r in ((131072, 40), (131072, 5000), (16384, 128)):
        pl = profk.Plan(m=m, r=r, capacity=600_000, k_accept=100, mode=0)
        v, i, st = _forced(y, 100, pl)
        assert_exact(y, 100, v, i)
        assert_stats_match(y, 100, pl, 3, st)


def test_k_equals_n_and_plan_direct_mode():
    x = workloads.normal(1, 5000, seed=13)[0]
    v, i = gpu_topk(x, 5000)
    assert_exact(x, 5000, v, i)
    x = workloads.normal(3, 2_000, seed=14)                                  # N <= 2 S: plan says mode 1
    assert profk.plan(2_000, 10).mode == 1
    v, i = gpu_topk(x, 10)
    assert_exact(x, 10, v, i)
    x = workloads.normal(3, 40_000, seed=14)                                 # k so large that the buffer would hold half the row
    assert profk.plan(40_000, 15_000).mode == 1
    v, i = gpu_topk(x, 15_000)
    assert_exact(x, 15_000, v, i)


# ----------------------------------------------------------------------------- ties and special values
def test_ties_and_degenerate_inputs():
    n = 300_000
    for name in ("few_values", "spikes"):
        recipe, seed = workloads.ADVERSARIAL[name]
        x = recipe(n, seed)
        for k in (1, 64, 1000):
            v, i = gpu_topk(x, k, eps=1e-3, seed=4)
            assert_exact(x, k, v, i)
    x = torch.zeros(n)
    v, i = gpu_topk(x, 100)
    assert np.array_equal(i, np.arange(100))                                 # all equal: lowest indices win
    x = workloads.sorted_uniform(n, 6)
    v, i = gpu_topk(x, 500, eps=1e-3)
    assert_exact(x, 500, v, i)
    v, i = gpu_topk(torch.flip(x, [0]), 500, eps=1e-3)
    assert_exact(torch.flip(x, [0]), 500, v, i)


def test_nan_inf_and_signed_zero_follow_the_total_order():
    x = workloads.normal(1, 100_000, seed=15)[0]
    x[5] = float("nan"); x[77] = float("inf"); x[78] = float("inf"); x[99] = -float("inf")
    x[1000:1010] = 0.0; x[2000:2010] = -0.0
    for k in (1, 3, 5000, 8192, 50_000, 100_000):
        v, i = gpu_topk(x, k)
        assert_exact(x, k, v, i)
    xb = x.to(torch.bfloat16)
    v, i = gpu_topk(xb, 1000)
    assert_exact(xb, 1000, v, i)


def test_failure_rate_on_rows_full_of_ties_stays_within_the_budget():
    # 256 rows x 8 seeds of a ReLU-Gaussian in bf16 (half the row is one value, the rest repeats by the hundred) and of a
    # four-valued row: the library's plan at eps = 1e-2, counted over 2048 row-calls each
    eps, k, n = 1e-2, 64, 1 << 18
    g = torch.Generator().manual_seed(35)
    inputs = {"relu bf16": torch.relu(torch.randn((256, n), generator=g)).to(torch.bfloat16),
              "four values": torch.randint(0, 4, (256, n), generator=g).to(torch.float32)}
    for name, x in inputs.items():
        xd = x.cuda()
        ov, oi = o_topk.topk(workloads.as_numpy(x), k)
        failed = 0
        for seed in range(8):
            v, i = profk.topk(xd, k, eps=eps, seed=seed)
            torch.cuda.synchronize()
            assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(workloads.as_numpy(v)), bits(ov)), (name, seed)
            failed += sum(1 for st in profk.read_stats(256) if st[3] != profk.ROW_OK)
        calls = 8 * 256
        assert failed <= calls * eps + 4 * np.sqrt(calls * eps), (name, failed)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_batch_with_the_largest_sample_of_the_small_threshold_kernel(dtype):
    # 80 rows, one 256-thread CTA each, 4096 samples: every sample is a candidate's worth of shared memory
    x = workloads.normal(80, 100_000, seed=33, dtype=dtype)
    for r in (1, 20, 32):
        pl = profk.Plan(m=4096, r=r, capacity=8000, k_accept=16, mode=0)
        v, i, st = _forced(x, 16, pl)
        assert_exact(x, 16, v, i)
        assert_stats_match(x, 16, pl, 3, st, rows=(0, 41, 79))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_survivors_are_counted_in_the_total_order(dtype):
    # NaNs with the sign bit set rank lowest and -0.0 ranks below +0.0: floating point would count them as
    # "not below" a threshold they do not reach, and the count check would pass on a buffer without the top-k
    x = workloads.normal(3, 200_000, seed=19).to(dtype)
    raw = x.view(torch.int32 if dtype == torch.float32 else torch.int16)
    neg_nan = -(1 << 22) if dtype == torch.float32 else -(1 << 6)            # 0xFFC00000 / 0xFFC0
    raw[0, ::7] = neg_nan
    x[1] = torch.relu(x[1])
    x[1, ::5] = -0.0                                                          # floods of +0.0 and of -0.0
    raw[2, ::3] = neg_nan
    x[2, 1::3] = float("nan")
    for m, r, cap in ((64, 1, 50_000), (4096, 3000, 190_000), (4096, 2000, 150_000), (2048, 40, 100_000)):
        for rule in (profk.TIES_BY_INDEX, profk.TIES_KEEP_ALL):
            pl = profk.Plan(m=m, r=r, capacity=cap, k_accept=10, mode=0, tie_rule=rule)
            v, i, st = _forced(x, 10, pl)
            assert_exact(x, 10, v, i)
            assert_stats_match(x, 10, pl, 3, st)


# ----------------------------------------------------------------------------- large selections
def test_large_k_uses_the_cluster_sort():
    x = workloads.normal(1, 1 << 22, seed=21)[0]
    for k in (8193, 20_000, 100_000):
        v, i = gpu_topk(x, k, eps=1e-3, seed=2)
        assert_exact(x, k, v, i)
    xb = workloads.relu_gaussian(1 << 22, seed=3)                      # bf16, thousands of copies of each value
    for k in (10_000, 65_536):
        v, i = gpu_topk(xb, k, eps=1e-3, seed=5)
        assert_exact(xb, k, v, i)


def test_large_k_batched_forced_failures_and_direct_mode():
    x = workloads.normal(3, 300_000, seed=22)
    k = 10_000
    v, i = gpu_topk(x, k, eps=1e-3, seed=1)
    assert_exact(x, k, v, i)
    v, i, st = _forced(x, k, profk.Plan(m=8192, r=400, capacity=k, k_accept=k, mode=0))      # every row overflows
    assert_exact(x, k, v, i)
    assert all(s[3] == profk.ROW_OVERFLOW for s in st)
    v, i, st = _forced(x, k, profk.Plan(m=8192, r=100, capacity=60_000, k_accept=k, mode=0))  # too few survivors
    assert_exact(x, k, v, i)
    assert all(s[3] == profk.ROW_RECALL for s in st)
    v, i, st = _forced(x, k, profk.Plan(m=0, r=0, capacity=k, k_accept=k, mode=1))
    assert_exact(x, k, v, i)
    y = workloads.normal(1, 70_000, seed=23)[0]
    v, i = gpu_topk(y, 70_000)                                          # k = N
    assert_exact(y, 70_000, v, i)


# ----------------------------------------------------------------------------- stages on their own
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sample_indices_and_threshold_match_the_oracle(dtype):
    n, m, r = 1_000_003, 5000, 7
    x = workloads.normal(3, n, seed=16, dtype=dtype)
    tau, sidx = profk.sample_threshold(x.cuda(), m, r, seed=0xABCDEF0123, want_indices=True)
    torch.cuda.synchronize()
    xn = workloads.as_numpy(x)
    for row in range(3):
        want_idx = o_philox.sample_indices(n, m, 0xABCDEF0123, row)
        assert np.array_equal(sidx[row].cpu().numpy().astype(np.int64) & 0xFFFFFFFF, want_idx)
        want_tau = o_stages.threshold(xn[row], want_idx, r)
        assert bits(workloads.as_numpy(tau[row:row + 1]))[0] == bits(np.asarray([want_tau]))[0]
    # ranks beyond 128 that the cluster still bounds from its group maxima (up to 128 per CTA)
    for m2, r2 in ((131072, 405), (131072, 2048), (40000, 129), (65536, 1500)):
        tau = profk.sample_threshold(x[:1].cuda(), m2, r2, seed=6)
        torch.cuda.synchronize()
        want = o_stages.threshold(xn[0], o_philox.sample_indices(n, m2, 6, 0), r2)
        assert bits(workloads.as_numpy(tau))[0] == bits(np.asarray([want]))[0], (m2, r2)
    # large sample spread over an 8-CTA cluster, deep rank
    tau = profk.sample_threshold(x[:1].cuda(), 131072, 9000, seed=5)
    torch.cuda.synchronize()
    want = o_stages.threshold(xn[0], o_philox.sample_indices(n, 131072, 5, 0), 9000)
    assert bits(workloads.as_numpy(tau))[0] == bits(np.asarray([want]))[0]


@pytest.mark.parametrize("rows", [12, 20, 40, 80])
def test_threshold_of_mid_ranks_in_clusters_of_every_size(rows):
    # 8-, 4-, 2- and 1-CTA clusters per row; ranks on both sides of the switch to the cluster-wide bound, and beyond 128
    n = 300_007
    x = workloads.normal(rows, n, seed=36)
    xn = workloads.as_numpy(x)
    for m, r in ((8192, 15), (8192, 16), (8192, 100), (20000, 128), (20000, 300)):
        tau = profk.sample_threshold(x.cuda(), m, r, seed=11)
        torch.cuda.synchronize()
        got = bits(workloads.as_numpy(tau))
        for row in (0, rows // 2, rows - 1):
            want = o_stages.threshold(xn[row], o_philox.sample_indices(n, m, 11, row), r)
            assert got[row] == bits(np.asarray([want]))[0], (m, r, row)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_filter_keeps_exactly_the_survivor_set(dtype):
    n = 777_777
    x = workloads.normal(2, n, seed=17, dtype=dtype)
    xn = workloads.as_numpy(x)
    tau = torch.tensor([2.5, 3.0]).to(dtype)
    buf, counts = profk.filter_pass(x.cuda(), tau.cuda(), capacity=20_000)
    torch.cuda.synchronize()
    for row in range(2):
        want = o_stages.survivor_set(xn[row], workloads.as_numpy(tau)[row])
        c = int(counts[row])
        assert c == want.size
        rec = buf[row, :c].cpu().numpy().view(np.uint64)
        got_idx = np.sort((rec & np.uint64(0xFFFFFFFF)).astype(np.int64))
        assert np.array_equal(got_idx, want)                                  # same set, any order
        keys = (~(rec >> np.uint64(32))).astype(np.uint32)
        okeys = o_topk.order_key(xn[row])
        okeys32 = okeys.astype(np.uint32)                                    # a bf16 key sits in the low 16 bits
        order = np.argsort(rec & np.uint64(0xFFFFFFFF))
        assert np.array_equal(keys[order], okeys32[want])
    # overflow: the counter only has to exceed the capacity
    buf, counts = profk.filter_pass(x.cuda(), torch.tensor([-10.0, -10.0]).to(dtype).cuda(), capacity=1000)
    torch.cuda.synchronize()
    assert int(counts[0]) > 1000 and int(counts[1]) > 1000


# ----------------------------------------------------------------------------- relaxed recall
def test_relaxed_recall_returns_a_padded_prefix():
    x = workloads.normal(1, 1 << 20, seed=18)[0]
    k = 512
    ov, oi = o_topk.topk_row(workloads.as_numpy(x), k)
    short = 0
    for seed in range(12):
        # a plan whose threshold is often too high for k but fine for k_accept
        pl = profk.Plan(m=8192, r=3, capacity=4096, k_accept=128, mode=0)
        v, i = profk.topk(x.cuda(), k, plan_override=pl, seed=seed)
        torch.cuda.synchronize()
        v, i = v.cpu().numpy(), i.cpu().numpy()
        _, R, _, status = profk.read_stats(1)[0]
        n_real = min(k, R) if status == profk.ROW_OK else k
        assert np.array_equal(i[:n_real], oi[:n_real]) and np.array_equal(bits(v[:n_real]), bits(ov[:n_real]))
        assert np.all(i[n_real:] == -1) and np.all(np.isneginf(v[n_real:]))
        short += n_real < k
    assert short > 0, "no seed exercised the short-buffer branch"
    pl = profk.plan(1 << 20, k, 1e-2, recall=0.95)
    v, i = gpu_topk(x, k, eps=1e-2, recall=0.95, seed=1)
    _, R, _, status = profk.read_stats(1)[0]
    n_real = min(k, R) if status == profk.ROW_OK else k
    assert n_real >= pl.k_accept
    assert np.array_equal(i[:n_real], oi[:n_real])


# ----------------------------------------------------------------------------- stream order
def test_input_produced_on_the_stream_just_before_the_call():
    # The first kernel of a call may be staged behind the work before it on the stream and must wait for that work
    # before it reads the input: here the input is overwritten by a kernel queued right before every call, on a
    # side stream, with no synchronisation in between.
    n, k = 1 << 22, 100
    side = torch.cuda.Stream()
    x = torch.empty(n, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(7)
    outs, snaps = [], []
    with torch.cuda.stream(side):
        for it in range(6):
            x.normal_(generator=g)                   # producer kernel
            v, i = profk.topk(x, k, seed=it)         # consumer, same stream
            outs.append((v.clone(), i.clone()))
            snaps.append(x.clone())                  # what the consumer must have seen
    side.synchronize()
    for (v, i), snap in zip(outs, snaps):
        assert_exact(snap.cpu(), k, workloads.as_numpy(v), i.cpu().numpy())


def test_call_captured_in_a_cuda_graph():
    # All launches of a call (cluster launches, programmatic dependents, the cooperative kernels of the many-row
    # and large-k paths) can be captured once and replayed on new data.
    for rows, n, k in [(1, 1 << 22, 128), (64, 1 << 16, 16), (1, 1 << 22, 20000)]:
        x = torch.empty((rows, n), device="cuda")
        out = (torch.empty((rows, k), device="cuda"), torch.empty((rows, k), dtype=torch.int64, device="cuda"))
        g = torch.Generator(device="cuda").manual_seed(rows + k)
        x.normal_(generator=g)
        profk.topk(x, k, out=out)                    # first use of the shape (workspace, attributes) outside the capture
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                profk.topk(x, k, out=out, seed=3)
        for _ in range(2):
            x.normal_(generator=g)
            graph.replay()
            torch.cuda.synchronize()
            assert_exact(x.cpu(), k, workloads.as_numpy(out[0]), out[1].cpu().numpy())


# ----------------------------------------------------------------------------- dense survivors: the deferring build of the filter
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_dense_survivors_noted_in_shared_memory_and_decided_after_streaming(dtype):
    """Plans with one to a dozen survivors per warp-tile (rank / sample size): the filter only notes candidate vectors
    while it streams and decides them afterwards.  Ragged and unaligned rows, batches and single rows, floods of copies
    of the threshold (the list in shared memory fills up and the warps fall back to the direct slow path), both tie
    rules; status, threshold and survivor count follow the oracle."""
    k = 40
    cases = []
    for rows, n in ((1, 1 << 22), (1, 3_000_001), (7, 300_001), (40, 1 << 17)):
        cases.append((f"normal {rows}x{n}", workloads.normal(rows, n, seed=90 + rows, dtype=dtype)))
    cases.append(("constant", torch.full((3, 1 << 19), 1.25).to(dtype)))
    cases.append(("few values", workloads.few_values(1 << 21, seed=91, distinct=4).to(dtype).view(1, -1)))
    cases.append(("relu", workloads.relu_gaussian(1 << 21, seed=92, dtype=torch.float32).to(dtype).view(2, -1)))
    for name, x in cases:
        rows, n = x.shape
        for m, r in ((2048, 24), (1024, 6)):                 # 12 / 6 expected survivors per bf16 warp-tile, half of that for fp32
            cap = min(n // 2 - 1, 3 * r * (n // m))
            for rule in (profk.TIES_BY_INDEX, profk.TIES_KEEP_ALL):
                pl = profk.Plan(m=m, r=r, capacity=cap, k_accept=k, mode=0, tie_rule=rule)
                v, i = profk.topk(x.cuda(), k, plan_override=pl, seed=13)
                torch.cuda.synchronize()
                assert_exact(x, k, workloads.as_numpy(v), i.cpu().numpy())
                assert_stats_match(x, k, pl, 13, profk.read_stats(rows))
    # an unaligned view of a batch
    big = workloads.normal(1, 5 * 100_003 + 8, seed=93, dtype=dtype)[0].cuda()
    for off in (1, 3):
        x = big[off: off + 5 * 100_003].view(5, 100_003)
        pl = profk.Plan(m=1024, r=12, capacity=4000, k_accept=k, mode=0)
        v, i = profk.topk(x, k, plan_override=pl, seed=14)
        torch.cuda.synchronize()
        assert_exact(x.cpu(), k, workloads.as_numpy(v), i.cpu().numpy())
        assert_stats_match(x.cpu(), k, pl, 14, profk.read_stats(5))
