"""GPU parity of the exact replacement of failed rows (Section 3, "Refinement"): plans that force the
count check to fail, on shapes that send the row through every variant of the exact selection -- a
row cut into several segments (one cluster each, merged by the last to finish), one cluster per row,
and the grid-wide kernel used for many rows -- against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
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


def forced(xg: torch.Tensor, k: int, plan):
    v, i = profk.topk(xg, k, plan_override=plan, seed=5)
    torch.cuda.synchronize()
    rows = 1 if xg.dim() == 1 else xg.shape[0]
    return workloads.as_numpy(v), i.cpu().numpy(), profk.read_stats(rows)


def assert_exact(x: torch.Tensor, k: int, v: np.ndarray, i: np.ndarray):
    ov, oi = o_topk.topk(workloads.as_numpy(x), k)
    assert np.array_equal(i, oi), "indices differ from the oracle"
    assert np.array_equal(bits(v), bits(ov)), "values differ from the oracle"


def overflow_plan(k):      # capacity == k and a low threshold: every row overflows
    return profk.Plan(m=4096, r=400, capacity=k, k_accept=k, mode=0)


def recall_plan(k):        # threshold = the sample maximum: (almost) nothing survives
    return profk.Plan(m=65536, r=1, capacity=max(4096, k), k_accept=k, mode=0)


@pytest.mark.parametrize("k", [1, 64, 1000, 8192])
def test_long_row_cut_into_segments(k):
    x = workloads.normal(1, 3_000_001, seed=21)[0]
    v, i, st = forced(x.cuda(), k, overflow_plan(k))
    assert st[0][3] == profk.ROW_OVERFLOW
    assert_exact(x, k, v, i)
    v, i, st = forced(x.cuda(), k, recall_plan(k))
    if k >= 1000:                                                # about N / m = 46 survivors: too few for these k
        assert st[0][3] == profk.ROW_RECALL
    assert_exact(x, k, v, i)


def test_unaligned_row_start():
    base = workloads.normal(1, 2_500_003, seed=22)[0].cuda()
    for off in (1, 2, 3):
        xg = base[off:]
        v, i, _ = forced(xg, 300, overflow_plan(300))
        assert_exact(xg.cpu(), 300, v, i)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_two_long_rows(dtype):
    x = workloads.normal(2, 5_000_000 + 7, seed=23, dtype=dtype)      # odd row length: the second row is unaligned
    for plan in (overflow_plan(500), recall_plan(500)):
        v, i, st = forced(x.cuda(), 500, plan)
        assert all(s[3] in (profk.ROW_OVERFLOW, profk.ROW_RECALL) for s in st)     # 76 survivors expected, 500 wanted
        assert_exact(x, 500, v, i)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_constant_row_is_decided_by_the_index(dtype):
    n = 2_000_000
    x = torch.full((n,), 1.5, dtype=dtype)
    for k in (1, 100, 5000):
        v, i, st = forced(x.cuda(), k, overflow_plan(k))
        assert st[0][3] == profk.ROW_OVERFLOW
        assert np.array_equal(i, np.arange(k))
        assert np.array_equal(bits(v), bits(workloads.as_numpy(x[:k])))


def test_ties_across_segment_boundaries():
    recipe, seed = workloads.ADVERSARIAL["few_values"]
    x = recipe(4_000_000, seed)
    for k in (64, 5000):
        v, i, _ = forced(x.cuda(), k, overflow_plan(k))
        assert_exact(x, k, v, i)
    recipe, seed = workloads.ADVERSARIAL["spikes"]
    x = recipe(4_000_000, seed)
    v, i, _ = forced(x.cuda(), 200, overflow_plan(200))        # more outputs than spikes: zeros by index after them
    assert_exact(x, 200, v, i)


def test_answer_in_one_segment():
    n = 3_000_000
    asc = torch.arange(n, dtype=torch.float32)
    for x in (asc, asc.flip(0)):                                # the top-k sits at the very end / the very start
        v, i, _ = forced(x.cuda(), 1000, recall_plan(1000))
        assert_exact(x, 1000, v, i)


@pytest.mark.parametrize("rows", [3, 9, 10, 18, 19, 40])
def test_row_counts_around_the_switch_to_the_grid_kernel(rows):
    x = workloads.normal(rows, 300_000 + rows, seed=24)
    x[rows // 2, ::2] = 6.0                                      # one row with many copies of its maximum
    v, i, st = forced(x.cuda(), 50, overflow_plan(50))
    assert all(s[3] == profk.ROW_OVERFLOW for s in st)
    assert_exact(x, 50, v, i)
    # mixed: only the tie-heavy row fails
    v, i, st = forced(x.cuda(), 50, profk.Plan(m=2048, r=4, capacity=2000, k_accept=50, mode=0, tie_rule=profk.TIES_KEEP_ALL))
    assert st[rows // 2][3] == profk.ROW_OVERFLOW
    assert_exact(x, 50, v, i)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_direct_mode_with_clusters(dtype):
    x = workloads.normal(2, 150_001, seed=25, dtype=dtype)
    for k in (10, 3000):
        v, i, st = forced(x.cuda(), k, profk.Plan(m=0, r=0, capacity=k, k_accept=k, mode=1))
        assert all(s[3] == profk.ROW_DIRECT for s in st)
        assert_exact(x, k, v, i)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_direct_mode_and_failures_of_many_rows(dtype):
    # many rows at once: the grid-wide kernel deals them out one per CTA
    x = workloads.normal(300, 70_001, seed=27, dtype=dtype)
    for k in (5, 2000):
        v, i, st = forced(x.cuda(), k, profk.Plan(m=0, r=0, capacity=k, k_accept=k, mode=1))
        assert all(s[3] == profk.ROW_DIRECT for s in st)
        assert_exact(x, k, v, i)
    v, i, st = forced(x.cuda(), 100, overflow_plan(100))
    assert all(s[3] == profk.ROW_OVERFLOW for s in st)
    assert_exact(x, 100, v, i)
    x = torch.zeros((200, 50_000), dtype=dtype)                  # every row a flood of ties: lowest indices win
    v, i, st = forced(x.cuda(), 64, overflow_plan(64))
    assert np.array_equal(i, np.tile(np.arange(64), (200, 1)))
    # the library's own plan for short rows of this kind
    x = workloads.normal(2048, 1 << 16, seed=28, dtype=dtype)
    v, i = profk.topk(x.cuda(), 8)
    torch.cuda.synchronize()
    assert_exact(x, 8, workloads.as_numpy(v), i.cpu().numpy())


def test_special_values_in_the_exact_path():
    x = workloads.normal(1, 1_000_000, seed=26)[0]
    x[5] = float("nan"); x[77] = float("inf"); x[99_999] = float("inf"); x[123_456] = -float("inf")
    x[200_000] = torch.tensor(np.array([0x7FC00001], dtype=np.uint32).view(np.float32))[0]     # a second NaN pattern
    xg = x.cuda()
    v, i, _ = forced(xg, 20, overflow_plan(20))
    assert_exact(x, 20, v, i)
