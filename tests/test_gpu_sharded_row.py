"""One row split over G shards, run on ONE GPU shard after shard through the library's real stage calls, the two
exchanges made by local copies: bit-exact against the oracle, and the threshold is the unsharded call's."""
import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, sharding, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    profk.lib()
    torch.cuda.set_device(0)


def bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def run_sharded(x, shards, k, **kw):
    n = x.numel()
    layout = sharding.shard_layout(n, k, shards, kw.get("eps", 1e-3), kw.get("recall", 1.0))
    assert layout[0][0] == 0 and layout[-1][1] == n and all(a[1] == b[0] for a, b in zip(layout, layout[1:]))
    xd = x.cuda()
    local = {g: xd[lo:hi].clone() for g, (lo, hi) in enumerate(layout)}       # each shard in memory of its own
    v, i, info = sharding.topk_one_row(local, shards, n, k, gather=sharding.local_gather(shards), **kw)
    torch.cuda.synchronize()
    return workloads.as_numpy(v), i.cpu().numpy(), info


@pytest.mark.parametrize("shards", [2, 4, 8])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sharded_row_equals_the_oracle_and_shares_the_threshold(shards, dtype):
    n, k = 1 << 22, 100
    x = workloads.normal(1, n, seed=70, dtype=dtype)[0]
    xn = workloads.as_numpy(x)
    ov, oi = o_topk.topk_row(xn, k)
    for seed in (0, 1, 2):
        v, i, info = run_sharded(x, shards, k, eps=1e-3, seed=seed)
        assert info["status"] == profk.ROW_OK and not info["repaired"]
        assert np.array_equal(i, oi) and np.array_equal(bits(v), bits(ov)), (shards, seed)
        # the unsharded call with the same seed: same threshold, same survivor count
        profk.topk(x.cuda(), k, eps=1e-3, seed=seed)
        tau_bits, R, cap, status = profk.read_stats(1)[0]
        assert status == profk.ROW_OK
        thr = info["threshold_record"].cpu().numpy().view(np.uint32)
        assert int(thr[0]) == tau_bits, "the sharded call selected another threshold"
        assert info["survivors"] == R and sum(info["shard_counts"]) == R


@pytest.mark.parametrize("n,k,shards", [(3_000_001, 2999, 3), (1_000_003, 77, 5), (1 << 24, 20_000, 4), (1 << 20, 1, 16)])
def test_ragged_lengths_large_k_and_odd_shard_counts(n, k, shards):
    x = workloads.normal(1, n, seed=71)[0]
    ov, oi = o_topk.topk_row(workloads.as_numpy(x), k)
    v, i, info = run_sharded(x, shards, k, eps=1e-3, seed=5)
    assert np.array_equal(i, oi) and np.array_equal(bits(v), bits(ov))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_ties_across_shard_boundaries(dtype):
    """Rows full of copies of the threshold value: the threshold record's index decides which copies survive, and the
    shards before, at and behind that index each treat their copies accordingly."""
    n, k, shards = 1 << 22, 500, 4
    cases = {"constant": torch.full((n,), 2.5), "few values": workloads.few_values(n, seed=72, distinct=8),
             "relu": workloads.relu_gaussian(n, seed=73, dtype=torch.float32)}
    for name, x in cases.items():
        x = x.to(dtype)
        ov, oi = o_topk.topk_row(workloads.as_numpy(x), k)
        for seed in (0, 1):
            v, i, info = run_sharded(x, shards, k, eps=1e-3, seed=seed)
            assert np.array_equal(i, oi) and np.array_equal(bits(v), bits(ov)), (name, seed)
            if name != "relu":
                assert info["status"] == profk.ROW_OK, (name, info["status"])      # counted by rank: no flood, no repair


def test_relaxed_mode_and_the_repair_path(monkeypatch):
    n, k, shards = 1 << 21, 64, 4
    x = workloads.normal(1, n, seed=74)[0]
    ov, oi = o_topk.topk_row(workloads.as_numpy(x), k)
    v, i, info = run_sharded(x, shards, k, eps=1e-2, recall=0.9, seed=1)
    n_real = k if info["repaired"] else min(k, info["survivors"])
    assert n_real >= info["plan"].k_accept
    assert np.array_equal(i[:n_real], oi[:n_real]) and np.array_equal(bits(v[:n_real]), bits(ov[:n_real]))
    assert np.all(i[n_real:] == -1)

    # a plan whose buffer is far too small: the count check fails and every shard's exact top-k is merged instead
    class TightStages(sharding.CudaStages):
        def plan(self, n, k, eps, recall):
            pl = profk.plan(n, k, eps, recall)
            return profk.Plan(m=pl.m, r=pl.m // 8, capacity=k, k_accept=k, mode=0, tie_rule=pl.tie_rule)

    layout = sharding.shard_layout(n, k, shards, stages=TightStages())
    xd = x.cuda()
    local = {g: xd[lo:hi].clone() for g, (lo, hi) in enumerate(layout)}
    v, i, info = sharding.topk_one_row(local, shards, n, k, seed=2, stages=TightStages(), gather=sharding.local_gather(shards))
    torch.cuda.synchronize()
    assert info["status"] == profk.ROW_OVERFLOW and info["repaired"]
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(v.cpu().numpy()), bits(ov))
    # ... and one whose threshold is the sample maximum: too few candidates
    class HighStages(sharding.CudaStages):
        def plan(self, n, k, eps, recall):
            pl = profk.plan(n, k, eps, recall)
            return profk.Plan(m=65536, r=1, capacity=pl.capacity, k_accept=k, mode=0, tie_rule=pl.tie_rule)

    layout = sharding.shard_layout(n, k, shards, stages=HighStages())         # another sample size, other strata
    local = {g: xd[lo:hi].clone() for g, (lo, hi) in enumerate(layout)}
    v, i, info = sharding.topk_one_row(local, shards, n, k, seed=3, stages=HighStages(), gather=sharding.local_gather(shards))
    torch.cuda.synchronize()
    assert info["status"] == profk.ROW_RECALL and info["repaired"]
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(v.cpu().numpy()), bits(ov))


def test_direct_mode_row():
    n, k, shards = 2_000, 10, 4                                                  # the sample would be half the row: no filter
    x = workloads.normal(1, n, seed=75)[0]
    ov, oi = o_topk.topk_row(workloads.as_numpy(x), k)
    v, i, info = run_sharded(x, shards, k, eps=1e-3, seed=0)
    assert info["status"] == profk.ROW_DIRECT
    assert np.array_equal(i, oi) and np.array_equal(bits(v), bits(ov))
