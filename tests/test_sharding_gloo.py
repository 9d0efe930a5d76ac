"""The N > 1 host logic on CPU: two `gloo` ranks shard rows, take the maximum of their timings and agree on
the whole-job rate (no GPU, no data-path collective)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_12573_b200 import sharding


def test_shard_rows_partitions_every_row_once():
    for rows in (0, 1, 7, 512, 513):
        for world in (1, 2, 3, 8):
            blocks = [sharding.shard_rows(rows, world, r) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == rows
            assert all(a[1] == b[0] for a, b in zip(blocks, blocks[1:]))
            sizes = [b - a for a, b in blocks]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_rows(4, 2, 2)
    assert sharding.whole_job_rate(1 << 26, 8, 0.064) == pytest.approx(8 * (1 << 26) / 64e-6)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        start, stop = sharding.shard_rows(513, world, rank)
        mine = torch.zeros(513, dtype=torch.int64)
        mine[start:stop] = 1
        dist.all_reduce(mine)                                   # every row owned by exactly one rank
        slowest = sharding.max_over_ranks(10.0 + 5.0 * rank)     # rank 1 is slower
        dist.barrier()
        out.put((rank, int(mine.min()), int(mine.max()), slowest, sharding.rank_seed_offset(rank)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == [0, 1]
    assert all(r[1] == 1 and r[2] == 1 for r in results)
    assert all(r[3] == 15.0 for r in results)                    # both ranks see the slower rank's time
    assert results[0][4] != results[1][4]
