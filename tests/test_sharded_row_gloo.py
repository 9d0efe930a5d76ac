"""One row over several ranks, on CPU: the exchange and offset logic of `sharding.topk_one_row` with two (and three)
`gloo` ranks.  The library's stage calls need a GPU, so a small NumPy stand-in written on top of the oracle takes
their place here; what is under test is the driver -- shard layout, padded all-gathers, global indices, the count
check's outcome and the repair path -- whose results must equal the oracle's full sort on every rank."""
import os
import socket
from types import SimpleNamespace

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import philox as o_philox
from oracle import plan as o_plan
from oracle import topk as o_topk
from paper_2608_12573_b200 import sharding


class NumpyStages:
    """Stand-in for `sharding.CudaStages`: the same interface on CPU tensors (float32 only)."""

    def __init__(self, capacity=None, rank_override=None):
        self.capacity, self.rank_override = capacity, rank_override

    def plan(self, n, k, eps, recall):
        p = o_plan.plan_guarded(n, k, eps, recall, s_min=512, s_max=512)
        return SimpleNamespace(m=p.m, r=self.rank_override or p.r, capacity=self.capacity or p.capacity, k_accept=p.k_accept,
                               mode=p.mode, tie_rule=1)

    def bounds(self, n, m, shards, g):
        pairs = (m + 1) // 2
        lo = 2 * (pairs * g // shards)
        hi = m if g + 1 == shards else 2 * (pairs * (g + 1) // shards)
        return lo, hi, lo * n // m, hi * n // m

    def sample_keys(self, shard, base, n, m, j_lo, j_hi, seed):
        idx = o_philox.sample_indices(n, m, seed, 0)[j_lo:j_hi]
        assert idx.min() >= base and idx.max() < base + shard.numel()        # a shard's strata lie inside the shard
        return torch.from_numpy(o_topk.order_key(shard.numpy()[idx - base]).view(np.int32).copy())

    def threshold(self, keys, dtype, n, m, r, seed, tie_rule):
        k32 = keys.numpy().view(np.uint32)
        order = np.lexsort((np.arange(m), ~k32))                             # key descending, sample number ascending
        j = order[r - 1]
        tau_idx = int(o_philox.sample_indices(n, m, seed, 0)[j])
        return torch.tensor([int(k32[j]), 0, tau_idx, 0], dtype=torch.int64)  # {key of tau, -, index of the record, -}

    def filter(self, shard, base, thr, capacity):
        keys = o_topk.order_key(shard.numpy()).astype(np.int64)
        tau_key, tau_idx = int(thr[0]), int(thr[2])
        gidx = np.arange(shard.numel()) + base
        kept = np.flatnonzero((keys > tau_key) | ((keys == tau_key) & (gidx <= tau_idx)))
        recs = ((0xFFFFFFFF - keys[kept]) << 32) | kept                      # ascending records = value descending, index ascending
        out = torch.zeros(capacity, dtype=torch.int64)
        out[:min(capacity, recs.size)] = torch.from_numpy(recs[:capacity])
        state = torch.zeros(8, dtype=torch.int32)
        state[0] = int(kept.size)
        return out, state

    def refine(self, records, states, bases, thr, dtype, capacity, k, k_accept):
        counts = states[:, 0].tolist()
        total = sum(counts)
        status = 2 if (total > capacity or any(c > records.shape[1] for c in counts)) else 1 if total < k_accept else 0
        vals = torch.full((k,), -float("inf"))
        idx = torch.full((k,), -1, dtype=torch.int64)
        if status == 0:
            merged = np.sort(np.concatenate([records[g, :c].numpy() + bases[g] for g, c in enumerate(counts)]))[:k]
            keys = (0xFFFFFFFF - (merged >> 32)).astype(np.uint32)
            bits = np.where(keys & 0x80000000, keys & 0x7FFFFFFF, ~keys).astype(np.uint32)
            vals[:merged.size] = torch.from_numpy(bits.view(np.float32).copy())
            idx[:merged.size] = torch.from_numpy(merged & 0xFFFFFFFF)
        return vals, idx, torch.tensor([status, total], dtype=torch.int32)

    def exact_topk(self, row, k):
        v, i = o_topk.topk_row(row.numpy(), k)
        return torch.from_numpy(v), torch.from_numpy(i)


def _row(n, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(n, generator=g)
    x[::97] = 1.75                                                            # ties, also across shard boundaries
    return x


CASES = [  # (n, k, stages kwargs, expected status)
    (200_003, 40, {}, 0),
    (200_003, 40, {"capacity": 40}, 2),                                       # overflow -> repair
    (200_003, 2000, {"rank_override": 1}, 1),                                 # threshold = sample maximum: too few candidates -> repair
    (900, 20, {}, 3),                                                         # direct mode: no sampling
]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        results = []
        for n, k, kw, _ in CASES:
            x = _row(n, 5)
            stages = NumpyStages(**kw)
            lo, hi = sharding.shard_layout(n, k, world, stages=stages)[rank]
            v, i, info = sharding.topk_one_row({rank: x[lo:hi].clone()}, world, n, k, seed=3, stages=stages,
                                               gather=sharding.dist_gather(world, rank))
            results.append((v.numpy().copy(), i.numpy().copy(), info["status"]))
        out.put((rank, results))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_ranks_agree_with_the_oracle(world):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for c, (n, k, kw, want_status) in enumerate(CASES):
        ov, oi = o_topk.topk_row(_row(n, 5).numpy(), k)
        for rank in range(world):
            v, i, status = got[rank][c]
            assert status == want_status, (c, rank, status)
            assert np.array_equal(i, oi) and np.array_equal(v.view(np.uint32), ov.view(np.uint32)), (c, rank)


def test_all_shards_in_one_process_give_the_same():
    for n, k, kw, want_status in CASES:
        x = _row(n, 5)
        stages = NumpyStages(**kw)
        for shards in (1, 2, 5):
            layout = sharding.shard_layout(n, k, shards, stages=stages)
            assert layout[0][0] == 0 and layout[-1][1] == n and all(a[1] == b[0] for a, b in zip(layout, layout[1:]))
            local = {g: x[lo:hi].clone() for g, (lo, hi) in enumerate(layout)}
            v, i, info = sharding.topk_one_row(local, shards, n, k, seed=3, stages=stages, gather=sharding.local_gather(shards))
            ov, oi = o_topk.topk_row(x.numpy(), k)
            assert info["status"] == want_status
            assert np.array_equal(i.numpy(), oi) and np.array_equal(v.numpy().view(np.uint32), ov.view(np.uint32))
