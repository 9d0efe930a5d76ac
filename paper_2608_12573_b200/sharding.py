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


# ---------------------------------------------------------------------------------------------------------------
# One row split over several GPUs.
#
# The paper runs on one GPU and leaves distributed settings to future work (Section "Limitations").  The four stages
# of Section 3 need two exchanges when a single row is cut into contiguous shards, one per GPU:
#   stage 1  every GPU gathers the sample keys of ITS strata                 -> all-gather of the S keys
#   stage 2  every GPU selects the same threshold record from the S keys
#   stage 3  every GPU filters its shard into a local candidate buffer        -> all-gather of (count, records)
#   stage 4  the count check on the summed counts and the refinement of the merged records, replicated
# Shards are made of whole sampling strata, so the sample -- hence the threshold -- is the one the unsharded call
# draws for the same seed.  A row that fails the count check is repaired by the exact top-k of every shard, gathered
# and selected from once more (the top-k of a union is the top-k of the union of the parts' top-k).
#
# `topk_one_row` is written over "the shards this process holds" and a `gather` callable, so the same code runs
#   * one shard per process, `gather` = an all-gather through torch.distributed (NCCL on GPUs, gloo on CPU): every
#     exchange lands in local memory; no kernel is ever handed another GPU's memory;
#   * all shards in one process, `gather` = local concatenation: the whole path on ONE GPU, shard after shard,
#     which is how it is tested without several GPUs.
# The arithmetic is in the stage calls (`CudaStages`: the C ABI); this file only moves their results around.


class CudaStages:
    """The library's stage calls on the current CUDA device (see `include/profk.h`, "one row split over several GPUs")."""

    def plan(self, n, k, eps, recall):
        import paper_2608_12573_b200 as profk

        return profk.plan(n, k, eps, recall)

    def bounds(self, n, m, shards, g):
        import paper_2608_12573_b200 as profk

        return profk.shard_bounds(n, m, shards, g)

    def sample_keys(self, shard, base, n, m, j_lo, j_hi, seed):
        import paper_2608_12573_b200 as profk

        return profk.shard_sample_keys(shard, base, n, m, j_lo, j_hi, seed)

    def threshold(self, keys, dtype, n, m, r, seed, tie_rule):
        import paper_2608_12573_b200 as profk

        return profk.threshold_from_keys(keys, dtype, n, m, r, seed, tie_rule)

    def filter(self, shard, base, thr, capacity):
        import paper_2608_12573_b200 as profk

        return profk.filter_shard(shard, base, thr, capacity)

    def refine(self, records, states, bases, thr, dtype, capacity, k, k_accept):
        import paper_2608_12573_b200 as profk

        return profk.refine_gathered(records, states, bases, thr, dtype, capacity, k, k_accept)

    def exact_topk(self, row, k):
        """Exact top-k of a 1-D tensor: (values, positions), ties to the lowest position."""
        import paper_2608_12573_b200 as profk

        return profk.topk(row, k)


def local_gather(shards: int):
    """`gather` for a process that holds every shard: pieces {g: tensor} -> [tensor of shard 0, ..., of shard G-1]."""
    def gather(pieces, sizes):
        return [pieces[g][:sizes[g]] for g in range(shards)]
    return gather


def dist_gather(shards: int, rank: int, group=None):
    """`gather` for one shard per rank: an all-gather through torch.distributed into local tensors.  Pieces may differ
    in length by a few elements, so each is padded to the longest before the exchange and trimmed after it."""
    import torch
    import torch.distributed as dist

    def gather(pieces, sizes):
        mine = pieces[rank]
        longest = max(sizes)
        padded = mine
        if mine.shape[0] < longest:
            padded = torch.zeros((longest,) + tuple(mine.shape[1:]), dtype=mine.dtype, device=mine.device)
            padded[:mine.shape[0]] = mine
        outs = [torch.empty_like(padded) for _ in range(shards)]
        dist.all_gather(outs, padded.contiguous(), group=group)
        return [outs[g][:sizes[g]] for g in range(shards)]
    return gather


def topk_one_row(local: dict, shards: int, n: int, k: int, eps: float = 1e-3, recall: float = 1.0, seed: int = 0,
                 stages=None, gather=None):
    """Top-k of ONE row of length n held as `shards` contiguous shards (see `shard_layout`).

    local   {g: 1-D tensor} -- the shards this process holds (one per process with `dist_gather`, all of them with
            `local_gather`)
    Returns (values (k,), indices (k,) into the whole row, info dict).  The result is the exact top-k (relaxed mode:
    a prefix of it, then padding) on every process.  One 8-byte device-to-host read per call (the count check's
    outcome decides whether the repair runs)."""
    import torch

    stages = stages if stages is not None else CudaStages()
    gather = gather if gather is not None else local_gather(shards)
    pl = stages.plan(n, k, eps, recall)
    dtype = next(iter(local.values())).dtype
    if pl.mode != 0:
        bounds = even_layout(n, shards)
        return _repair(local, bounds, shards, k, stages, gather) + ({"status": 3, "survivors": 0, "repaired": True, "plan": pl},)
    bounds = [stages.bounds(n, pl.m, shards, g) for g in range(shards)]
    for g, x in local.items():
        if x.dim() != 1 or x.numel() != bounds[g][3] - bounds[g][2]:
            raise ValueError(f"shard {g} must hold elements [{bounds[g][2]}, {bounds[g][3]}) of the row")
    # stage 1, exchange 1
    keys = {g: stages.sample_keys(x, bounds[g][2], n, pl.m, bounds[g][0], bounds[g][1], seed) for g, x in local.items()}
    keys_all = torch.cat(gather(keys, [b[1] - b[0] for b in bounds]))
    # stage 2 (replicated)
    thr = stages.threshold(keys_all, dtype, n, pl.m, pl.r, seed, pl.tie_rule)
    # stage 3, exchange 2
    filtered = {g: stages.filter(x, bounds[g][2], thr, pl.capacity) for g, x in local.items()}
    records = torch.stack(gather({g: f[0] for g, f in filtered.items()}, [pl.capacity] * shards))
    states = torch.stack(gather({g: f[1] for g, f in filtered.items()}, [8] * shards))
    # stage 4 (replicated)
    vals, idx, status = stages.refine(records, states, [b[2] for b in bounds], thr, dtype, pl.capacity, k, pl.k_accept)
    code, survivors = (int(v) for v in status.tolist())
    info = {"status": code, "survivors": survivors & 0xFFFFFFFF, "repaired": code != 0, "plan": pl, "threshold_record": thr,
            "shard_counts": [int(c) for c in states[:, 0].tolist()]}
    if code == 0:
        return vals, idx, info
    vals, idx = _repair(local, [(0, 0, b[2], b[3]) for b in bounds], shards, k, stages, gather)
    return vals, idx, info


def even_layout(n: int, shards: int):
    """Shard bounds (0, 0, elem_lo, elem_hi) for a row that is not sampled at all (direct mode): equal parts."""
    return [(0, 0, n * g // shards, n * (g + 1) // shards) for g in range(shards)]


def shard_layout(n: int, k: int, shards: int, eps: float = 1e-3, recall: float = 1.0, stages=None):
    """[(elem_lo, elem_hi)] of the shards `topk_one_row` expects for this problem: whole pairs of sampling strata."""
    stages = stages if stages is not None else CudaStages()
    pl = stages.plan(n, k, eps, recall)
    if pl.mode != 0:
        return [(b[2], b[3]) for b in even_layout(n, shards)]
    return [stages.bounds(n, pl.m, shards, g)[2:] for g in range(shards)]


def _repair(local, bounds, shards, k, stages, gather):
    """Exact answer without the filter: every shard's exact top-k, gathered; the top-k of their union."""
    import torch

    lens = [min(k, b[3] - b[2]) for b in bounds]
    tops = {g: stages.exact_topk(x, lens[g]) for g, x in local.items()}
    vals = torch.cat(gather({g: t[0] for g, t in tops.items()}, lens))
    idx = torch.cat([i + bounds[g][2] for g, i in enumerate(gather({g: t[1] for g, t in tops.items()}, lens))])
    # Shards are in index order and each list is ordered (value descending, index ascending), so among equal values
    # a lower position in the concatenation is a lower index in the row: the tie rule carries over.
    out_vals, pos = stages.exact_topk(vals, k)
    return out_vals, idx[pos]
