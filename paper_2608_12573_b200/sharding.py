"""Host-side helpers for running the hot path on several GPUs of one node.

Rows are independent problems (the method is applied to every batch element on its own), so the work is
split by rows with no collective on the data path: each rank answers its own rows on its own GPU.  The only
communication is bookkeeping -- a barrier around the timed region and the maximum of the per-rank timings.
"""
from __future__ import annotations


def shard_rows(rows: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous block of rows for `rank`: [start, stop).  Blocks differ in size by at most one row."""
    if not (0 <= rank < world) or rows < 0:
        raise ValueError("need 0 <= rank < world and rows >= 0")
    base, extra = divmod(rows, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def rank_seed_offset(rank: int) -> int:
    """Offset added to a workload's seed so that every rank of a weak-scaling run draws its own data."""
    return 7919 * rank


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank timing over the process group (identity without a group)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_per_step_max: float) -> float:
    """Throughput of the whole job: the units all ranks processed per second of the slowest rank."""
    return world * units_per_rank / (ms_per_step_max * 1e-3)
