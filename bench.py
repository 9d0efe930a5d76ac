#!/usr/bin/env python
"""Benchmark of the Prof-K hot path on B200.

One step = one call of the whole hot path (sample -> threshold -> filter -> count check ->
refine) over one batch of synthetic input.  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

Workloads (`--config`): "cfg2" (default; single row N = 2^26 fp32 N(0,1), k = 256, eps = 1e-4),
"cfg2_k16", "cfg2_k4096", "cfg1", "cfg3_f32", "cfg3_bf16", ... (see CONFIGS).  The headline line is that one
workload; at N = 1 the default run also times every other benchmark configuration briefly (a few dozen calls
each, inputs drawn on the device) and lists them under `extra.configs` (`--no-extra-configs` skips that).
With N > 1 GPUs (torchrun) every rank runs the same workload on its own data (weak scaling,
no data-path collective: rows are independent problems).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

CONFIGS = {
    # name: (rows, N, dtype, recipe, seed, k, eps, recall)
    "cfg1": (1, 1 << 20, "f32", "uniform", 0, 64, 1e-3, 1.0),
    "cfg2": (1, 1 << 26, "f32", "normal", 1, 256, 1e-4, 1.0),
    "cfg2_k16": (1, 1 << 26, "f32", "normal", 1, 16, 1e-4, 1.0),
    "cfg2_k4096": (1, 1 << 26, "f32", "normal", 1, 4096, 1e-4, 1.0),
    "cfg2_relaxed": (1, 1 << 26, "f32", "normal", 1, 4096, 1e-2, 0.95),
    "cfg3_f32": (512, 1 << 20, "f32", "normal", 2, 32, 1e-3, 1.0),
    "cfg3_bf16": (512, 1 << 20, "bf16", "normal", 2, 32, 1e-3, 1.0),
    "cfg4": (1, 1 << 29, "bf16", "relu_gaussian", 3, 32 * 4096, 1e-3, 1.0),
    # the shape of Section 5's sparse-autoencoder measurement: N = 50,331,648 flattened activations, K = 131,072
    "cfg4_sae_f32": (1, 50331648, "f32", "relu_gaussian", 3, 131072, 1e-3, 1.0),
    "cfg4_sae_bf16": (1, 50331648, "bf16", "relu_gaussian", 3, 131072, 1e-3, 1.0),
    # a few rows whose selection the whole grid orders (one cooperative launch after the filter): for launch lists
    "rows4_bf16_k8192": (4, 1 << 24, "bf16", "normal", 9, 8192, 1e-3, 1.0),
    "cfg5_cauchy_k64": (1, 1 << 30, "f32", "cauchy", 4, 64, 1e-3, 1.0),
    "cfg5_cauchy_k65536": (1, 1 << 30, "f32", "cauchy", 4, 65536, 1e-3, 1.0),
    "cfg5_pareto_k1": (1, 1 << 30, "f32", "pareto", 5, 1, 1e-3, 1.0),
    "cfg5_pareto_k1024": (1, 1 << 30, "f32", "pareto", 5, 1024, 1e-3, 1.0),
    "cfg5_sorted_k1024": (1, 1 << 30, "f32", "sorted", 6, 1024, 1e-3, 1.0),
    "cfg5_few_values_k64": (1, 1 << 30, "f32", "few_values", 7, 64, 1e-3, 1.0),
    "cfg5_spikes_k64": (1, 1 << 30, "f32", "spikes", 8, 64, 1e-3, 1.0),
    "cfg5_spikes_k1024": (1, 1 << 30, "f32", "spikes", 8, 1024, 1e-3, 1.0),
}

# DRAM bytes (read + write) of one filter launch at cfg2, from the ncu capture summarised in
# profiles/filter_kernel_f32_2p26.md (dram__bytes_read.sum + dram__bytes_write.sum).
FILTER_TRAFFIC_BYTES = {"cfg2": 272.20e6}

L2_BYTES = 126 * 1024 * 1024


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def make_input(cfg, seed_offset=0, device="cpu"):
    """One batch of the workload (rows x N).  Inputs of 2^29 elements and more are drawn on the GPU."""
    import torch

    from paper_2608_12573_b200 import workloads

    rows, n, dt, recipe, seed, *_ = cfg
    dtype = torch.float32 if dt == "f32" else torch.bfloat16
    seed = seed + seed_offset
    if recipe == "uniform":
        return workloads.uniform(n, seed, device).view(1, n)
    if recipe == "normal":
        return workloads.normal(rows, n, seed, dtype=dtype, device=device)
    if recipe == "relu_gaussian":
        return workloads.relu_gaussian(n, seed, dtype=dtype, device=device).view(1, n)
    fn, _ = workloads.ADVERSARIAL[recipe]
    return fn(n, seed, device=device).view(1, n)


class ClockSampler:
    """nvidia-smi clock / throttle sampling in the background during the timed region."""

    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.lines: list[str] = []
        self.times: list[float] = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())
            self.times.append(time.time())          # arrival time of the sample on this host's clock

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        self.samples = []                            # (arrival time, SM MHz)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln, when in zip(self.lines, self.times):
            f = [s.strip() for s in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            self.samples.append((when, float(f[1])))
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def inside(self, windows) -> list[float]:
        """SM clocks of the samples that arrived inside one of the (start, end) host-time windows."""
        return [mhz for when, mhz in getattr(self, "samples", []) if any(a <= when <= b for a, b in windows)]


def time_oracle(cfg, sample_elems: int, steps: int, warmup: int, x=None):
    """The CPU oracle as it stands (full stable sort per row), on a bounded sample of the workload."""
    import numpy as np

    from oracle import topk as o_topk
    from paper_2608_12573_b200 import workloads

    rows, n, dt, recipe, seed, k, eps, recall = cfg
    if x is None:
        x = make_input(cfg) if rows * n < (1 << 29) else make_input((rows, sample_elems) + tuple(cfg[2:]))
    xn = workloads.as_numpy(x)
    per_row = min(n, sample_elems)
    n_rows = max(1, min(rows, sample_elems // per_row))
    sample = np.ascontiguousarray(xn[:n_rows, :per_row])
    kk = min(k, per_row)
    for _ in range(warmup):
        o_topk.topk(sample, kk)
    t0 = time.perf_counter()
    for _ in range(steps):
        o_topk.topk(sample, kk)
    dt_s = (time.perf_counter() - t0) / steps
    return n_rows * per_row / dt_s, dt_s, f"{n_rows} row(s) x {per_row} elements of the workload, k={kk}, 1 thread"


def run_reference(args, cfg, name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # The oracle sorts roughly 7e6 elements/s on one core: size each step's sample so that the
    # whole run (warm-up + steps) stays near one minute.
    total_budget = 4e8
    sample_elems = int(min(1 << 24, max(1 << 14, total_budget / (args.steps + max(args.warmup, 1)))))
    value, dt_s, sample = time_oracle(cfg, sample_elems, args.steps, max(args.warmup, 1))
    rows, n, dt, recipe, seed, k, eps, recall = cfg
    line = {
        "impl": "reference", "metric": "top-k elements/s", "value": value, "unit": "elements/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": dt, "data": "synthetic",
        "config": {"workload": describe(name, cfg) + f"; each step of this arm sorts a bounded sample of it: {sample}"},
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def describe(name, cfg):
    rows, n, dt, recipe, seed, k, eps, recall = cfg
    mode = "exact" if recall >= 1.0 else f"relaxed recall {recall}"
    return f"{name}: {rows} row(s) x N={n} {dt}, {recipe} seed {seed}, k={k}, eps={eps}, {mode}"


def count_fallbacks(profk, inputs, rows, k, eps, recall, out, n_calls, seed0=10_000):
    """Rows (over n_calls calls, each with its own seed) whose count check failed and were repaired (by a second filtering
    pass or by the exact selection)."""
    failed = 0
    for s in range(n_calls):
        profk.topk(inputs[s % len(inputs)], k, eps=eps, recall=recall, seed=seed0 + s, out=out)
        failed += sum(1 for st in profk.read_stats(rows) if (st[3] & 0xFF) in (profk.ROW_RECALL, profk.ROW_OVERFLOW, profk.ROW_RECALL_REFILTERED,
                                                                               profk.ROW_OVERFLOW_REFILTERED))
    return failed


def time_filter_alone(profk, torch, inputs, rows, n, dt, pl, launches, warmup):
    """The dominant kernel alone: the filter pass through its stage-level entry point, same launch configuration,
    `launches` launches back to back with a zeroed counter each, one pair of CUDA events on the launching stream.
    Returns None in direct mode, else a dict (ms_per_launch, algorithmic bytes, GB/s; GB/s None if the buffer overflowed)."""
    import ctypes

    if pl.mode != 0:
        return None
    dev = inputs[0].device
    elem = 4 if dt == "f32" else 2
    taus = [profk.sample_threshold(x, pl.m, pl.r, seed=0) for x in inputs]       # every input copy with its own thresholds
    buf = torch.empty((rows, pl.capacity), dtype=torch.int64, device=dev)
    stride = profk.FILTER_COUNT_STRIDE           # one counter per 32 bytes
    many = torch.zeros(((launches + warmup) * rows, stride), dtype=torch.int32, device=dev)
    fn = getattr(profk.lib(), "profk_filter_f32" if dt == "f32" else "profk_filter_bf16")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def launch(i):
        code = fn(ctypes.c_void_p(inputs[i % len(inputs)].data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n),
                  ctypes.c_void_p(taus[i % len(inputs)].data_ptr()), ctypes.c_int64(pl.capacity), ctypes.c_void_p(buf.data_ptr()),
                  ctypes.c_void_p(many.data_ptr() + 4 * stride * i * rows), stream)
        assert code == 0

    for i in range(warmup):
        launch(launches + i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(launches):
        launch(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / launches
    survivors = float(many[:launches * rows, 0].sum().item()) / launches        # per launch, averaged over the launches
    # The stand-alone filter takes the threshold as a value alone: on a row flooded with copies of tau its buffer
    # overflows and the launch stops early, so its duration is not that of a scan.
    overflowed = bool((many[:launches * rows, 0] > pl.capacity).any().item())
    algo = rows * n * elem + survivors * 8            # read every element once + one 8-byte record per survivor
    return {"ms_per_launch": ms, "algorithmic_bytes": algo, "overflowed": overflowed, "survivors_per_launch": survivors,
            "GBps": None if overflowed else algo / (ms * 1e-3) / 1e9}


EXTRA_CONFIGS = ["cfg1", "cfg2_k16", "cfg2_k4096", "cfg2_relaxed", "cfg3_f32", "cfg3_bf16", "cfg4", "cfg4_sae_f32",
                 "cfg4_sae_bf16", "cfg5_cauchy_k64", "cfg5_few_values_k64"]


def measure_extra_config(profk, torch, name, dev, peak):
    """One of the other benchmark configurations, briefly: inputs drawn on the device (seeded), a few dozen calls."""
    cfg = CONFIGS[name]
    rows, n, dt, recipe, seed, k, eps, recall = cfg
    elem = 4 if dt == "f32" else 2
    in_bytes = rows * n * elem
    copies = max(2, min(8, -(-3 * L2_BYTES // in_bytes)))
    inputs = [make_input(cfg, seed_offset=1000 * c, device=str(dev)) for c in range(copies)]
    pl = profk.plan(n, k, eps, recall, rows=rows)
    profk.ensure_workspace(rows, pl.capacity, k, dev)
    out = (torch.empty((rows, k), dtype=inputs[0].dtype, device=dev), torch.empty((rows, k), dtype=torch.int64, device=dev))
    calls = 40 if in_bytes <= (1 << 30) else 20
    # warm-up: at least 5 calls and 50 ms of them (the GPU idled while the CPU baseline ran: a short configuration timed
    # right after it met clocks that had not come back up -- 28 us instead of 16.7 for config 1)
    t_warm, warm = time.time(), 0
    while warm < 5 or time.time() - t_warm < 0.05:
        profk.topk(inputs[warm % copies], k, eps=eps, recall=recall, seed=warm % 5, out=out)
        warm += 1
        if warm % 64 == 0:
            torch.cuda.synchronize()
    launches = profk.last_launch_count()
    torch.cuda.synchronize()
    calls = max(calls, min(400, int(2e-3 * warm / max(time.time() - t_warm, 1e-6))))      # a timed window of 2 ms at least
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(calls):
        profk.topk(inputs[i % copies], k, eps=eps, recall=recall, seed=5 + i, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / calls
    n_seeds = 20 if rows == 1 else 2
    failed = count_fallbacks(profk, inputs, rows, k, eps, recall, out, n_seeds)
    filt = time_filter_alone(profk, torch, inputs, rows, n, dt, pl, launches=20, warmup=3)
    gbs = in_bytes / (ms * 1e-3) / 1e9
    res = {"name": name, "workload": describe(name, cfg), "plan": {"m": pl.m, "r": pl.r, "capacity": pl.capacity, "mode": pl.mode},
           "calls": calls, "ms_per_call": ms, "elements_per_s": rows * n / (ms * 1e-3), "whole_call_GBps": gbs,
           "frac_of_8TBps_read_once": gbs / 8000.0, "frac_of_measured_peak": gbs / peak, "launches_per_call": launches,
           "fallback_rows": failed, "row_calls_checked": n_seeds * rows, "input_copies_rotated": copies,
           "filter_ms_per_launch": filt["ms_per_launch"] if filt else None,
           "filter_GBps": filt["GBps"] if filt else None,
           "filter_frac_of_measured_peak": (filt["GBps"] / peak) if filt and filt["GBps"] else None}
    if name.startswith("cfg4"):
        # The same selection through the BatchTopK consumer entry point (Section 5, "Application"): the kept set
        # without ordering -- as unordered (value, index) pairs, with the bit mask, and as a dense array.
        forms = {"pairs": dict(want_pairs=True), "pairs_and_mask": dict(want_pairs=True, want_mask=True),
                 "dense": dict(want_pairs=False, want_dense=True)}
        res["batchtopk_ms_per_call"] = {}
        for form, kw in forms.items():
            for i in range(3):
                profk.batchtopk(inputs[i % copies], k, eps=eps, seed=i, **kw)
            torch.cuda.synchronize()
            e0.record()
            for i in range(calls):
                profk.batchtopk(inputs[i % copies], k, eps=eps, seed=5 + i, **kw)
            e1.record()
            torch.cuda.synchronize()
            res["batchtopk_ms_per_call"][form] = e0.elapsed_time(e1) / calls
        res["batchtopk_launches_per_call"] = profk.last_launch_count()
        res["batchtopk_note"] = ("outputs are allocated through torch inside the timed loop (caching allocator); the dense form also "
                                 "writes N elements of zeros")
    if k > 8192 and rows <= 4:
        res["filter_note"] = ("the stand-alone filter launch takes the build of the kernel that the call takes at this density of survivors, "
                              "without the histogram the call's own launch also makes for the kernel behind it")
    del inputs, out
    torch.cuda.empty_cache()
    return res


def run_one_row_sharded(args, cfg, profk, sharding, torch, dev, rank, world):
    """Strong scaling of one long row: every rank holds one shard (drawn on its GPU, seeded by the shard), each step is
    one `sharding.topk_one_row` call (stage 1, all-gather of the sample keys, stage 2, stage 3, all-gather of the
    candidate buffers, stage 4).  Timed with CUDA events, max over ranks; each call ends with an 8-byte read of the count
    check's outcome, which is inside the timed region."""
    rows, n, dt, recipe, seed, k, eps, recall = cfg
    assert rows == 1, "--one-row-sharded needs a single-row configuration"
    elem = 4 if dt == "f32" else 2
    lo, hi = sharding.shard_layout(n, k, world, eps, recall)[rank]
    shard_cfg = (1, hi - lo) + tuple(cfg[2:])
    copies = 2
    shards = [make_input(shard_cfg, seed_offset=1000 * c + 31 * rank, device=str(dev)).view(-1) for c in range(copies)]
    gather = sharding.dist_gather(world, rank) if world > 1 else sharding.local_gather(1)
    warmup, steps = max(args.warmup, 3), args.steps

    def step(i):
        return sharding.topk_one_row({rank: shards[i % copies]}, world, n, k, eps, recall, seed=i, gather=gather)

    repaired = 0
    for i in range(warmup):
        step(i)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        repaired += int(step(warmup + i)[2]["repaired"])
    e1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ms = sharding.max_over_ranks(e0.elapsed_time(e1), dev) / steps
    if rank != 0:
        return
    gbs = n * elem / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "top-k elements/s", "value": n / (ms * 1e-3), "unit": "elements/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": dt, "data": "synthetic",
        "config": {"workload": describe(args.config, cfg) + f"; ONE row cut into {world} shard(s), one per GPU",
                   "parallelism": f"{world} shard(s) of one row; two all-gathers per call (sample keys, candidate buffers)"},
        "extra": {"whole_row_GBps": gbs, "frac_of_8TBps_read_once_per_gpu": gbs / world / 8000.0, "calls_repaired": repaired}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="cfg2", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="profk", choices=["profk", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-configs", action="store_true", help="skip the brief timing of the other configurations")
    ap.add_argument("--blocks", type=int, default=25, help="timed blocks of --steps calls (the first is the headline)")
    ap.add_argument("--one-row-sharded", action="store_true",
                    help="strong scaling instead of replicas: ONE row of the configuration's length cut into one shard per GPU "
                         "(sharding.topk_one_row: two all-gathers per call); with --gpus 1 the same path on a single shard")
    ap.add_argument("--entry", default="topk", choices=["topk", "batchtopk"],
                    help="with --hot-path-only: the entry point a step calls (batchtopk: the kept set as unordered pairs; single-row configurations)")
    ap.add_argument("--hot-path-only", action="store_true",
                    help="run only warm-up + timed steps of the hot path (for profiler captures) and exit")
    ap.add_argument("--rows", type=int, default=0,
                    help="override the configuration's number of rows (a smaller case of the same kernels for a profiler capture)")
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    if args.rows > 0:
        cfg = (args.rows,) + cfg[1:]
    if args.impl == "reference":
        run_reference(args, cfg, args.config)
        return

    import torch

    import paper_2608_12573_b200 as profk
    from paper_2608_12573_b200 import _build, sharding

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    _build.build()
    profk.lib()

    rows, n, dt, recipe, seed, k, eps, recall = cfg
    elem = 4 if dt == "f32" else 2
    in_bytes = rows * n * elem
    warmup = max(args.warmup, 3)
    steps = args.steps
    if args.one_row_sharded:
        run_one_row_sharded(args, cfg, profk, sharding, torch, dev, rank, world)
        if world > 1:
            dist.destroy_process_group()
        return

    # Inputs: enough distinct copies that no step finds its input in L2 (126 MB).
    copies = max(2, min(8, -(-3 * L2_BYTES // in_bytes)))
    big = rows * n >= (1 << 29)
    if big:        # drawn on the device (seeded); one pinned host copy serves the end-to-end leg
        dev_inputs = [make_input(cfg, seed_offset=1000 * c + sharding.rank_seed_offset(rank), device=str(dev)) for c in range(copies)]
        host_inputs = [dev_inputs[0].cpu().pin_memory()]
    else:
        host_inputs = [make_input(cfg, seed_offset=1000 * c + sharding.rank_seed_offset(rank)).pin_memory() for c in range(copies)]
        dev_inputs = [h.to(dev) for h in host_inputs]
    pl = profk.plan(n, k, eps, recall, rows=rows)
    profk.ensure_workspace(rows, pl.capacity, k, dev)
    out_vals = torch.empty((rows, k), dtype=dev_inputs[0].dtype, device=dev)
    out_idx = torch.empty((rows, k), dtype=torch.int64, device=dev)
    host_vals = torch.empty((rows, k), dtype=dev_inputs[0].dtype).pin_memory()
    host_idx = torch.empty((rows, k), dtype=torch.int64).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step(i):
        if args.hot_path_only and args.entry == "batchtopk":
            profk.batchtopk(dev_inputs[i % copies], k, eps=eps, seed=i, want_pairs=True)
        else:
            profk.topk(dev_inputs[i % copies], k, eps=eps, recall=recall, seed=i, out=(out_vals, out_idx))

    # ---- device-resident timing: the headline value ----
    sampler = ClockSampler(local_rank)
    if rank == 0 and not args.hot_path_only:
        sampler.start()
        time.sleep(0.5)            # let nvidia-smi come up; it keeps sampling until the filter loop is done
    for i in range(warmup):
        step(i)
    launches_per_step = profk.last_launch_count()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    windows = []                   # host-time windows of the timed blocks, for the clock samples
    t_host = time.time()
    ev0.record()
    for i in range(steps):
        step(warmup + i)
    ev1.record()
    barrier()
    windows.append((t_host, time.time()))
    ms_total = ev0.elapsed_time(ev1)
    if args.hot_path_only:
        if rank == 0:
            print(json.dumps({"hot_path_only": True, "ms_per_step": ms_total / steps, "launches_per_step": launches_per_step}))
        return
    ms_total = sharding.max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / steps
    value = sharding.whole_job_rate(rows * n, world, ms_per_step)

    # The same block of `steps` calls again, blocks - 1 more times: how steady the headline is (median / min / max).
    block_ms = [ms_per_step]
    for b in range(1, max(1, args.blocks)):
        barrier()
        t_host = time.time()
        ev0.record()
        for i in range(steps):
            step(warmup + b * steps + i)
        ev1.record()
        barrier()
        windows.append((t_host, time.time()))
        block_ms.append(sharding.max_over_ranks(ev0.elapsed_time(ev1), dev) / steps)

    # fallback rate observed over a separate run of seeds (statistics read-back synchronises, so not timed):
    # at least 1000 row-calls for inputs up to 2^26 elements
    if rows * n <= (1 << 26):
        n_seeds = max(2, -(-1000 // rows))
    else:
        n_seeds = (40 if big else 200) if rows == 1 else max(2, 200 // rows)
    fallbacks = count_fallbacks(profk, dev_inputs, rows, k, eps, recall, (out_vals, out_idx), n_seeds)
    fallback_rate = fallbacks / (n_seeds * rows)

    # ---- end to end: pinned host input -> device -> call -> result back on the host ----
    stage = torch.empty_like(dev_inputs[0])

    def e2e_step(i):
        stage.copy_(host_inputs[i % len(host_inputs)], non_blocking=True)
        profk.topk(stage, k, eps=eps, recall=recall, seed=i, out=(out_vals, out_idx))
        host_vals.copy_(out_vals, non_blocking=True)
        host_idx.copy_(out_idx, non_blocking=True)

    e2e_steps = max(3, min(steps, 20))
    for i in range(2):
        e2e_step(i)
    barrier()
    ev0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    ev1.record()
    barrier()
    e2e_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dev) / e2e_steps
    e2e_value = sharding.whole_job_rate(rows * n, world, e2e_ms)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- the dominant kernel alone: the filter pass, same launch configuration, CUDA events ----
    t_host = time.time()
    filt = time_filter_alone(profk, torch, dev_inputs, rows, n, dt, pl, launches=steps, warmup=warmup)
    windows.append((t_host, time.time()))
    clocks = sampler.stop()
    inside = sampler.inside(windows)
    clocks["samples_inside_timed_blocks"] = len(inside)
    clocks["sm_mhz_inside_timed_blocks"] = {"min": min(inside), "median": sorted(inside)[len(inside) // 2], "max": max(inside)} if inside else None
    peak, peak_kind = measured_peak_gbs()
    roofline = None
    if filt is not None:
        roofline = {"bound": "hbm", "kernel": "filter_kernel", "achieved": filt["GBps"], "peak": peak, "unit": "GB/s",
                    "frac": filt["GBps"] / peak if filt["GBps"] else None, "peak_kind": f"of {peak_kind}",
                    "traffic": FILTER_TRAFFIC_BYTES.get(args.config),
                    "traffic_source": ("profiles/filter_kernel_f32_2p26.md: ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch "
                                       "of this workload (a stored capture, not measured in this run)") if args.config in FILTER_TRAFFIC_BYTES else None,
                    "ms_per_launch": filt["ms_per_launch"], "algorithmic_bytes": filt["algorithmic_bytes"],
                    "achieved_from": "algorithmic bytes of this run (rows x N x sizeof(dtype) + 8 bytes per survivor, survivors read back) / CUDA-event duration"}
        if filt["overflowed"]:
            roofline["note"] = ("stand-alone filter launch overflowed its buffer (value-only threshold on a tie-flooded row) "
                                "and stopped early")

    # ---- context: torch.topk on the same GPU ----
    for i in range(3):
        torch.topk(dev_inputs[i % copies], k, dim=-1)
    torch.cuda.synchronize()
    ev0.record()
    reps = 5
    for i in range(reps):
        torch.topk(dev_inputs[i % copies], k, dim=-1)
    ev1.record()
    torch.cuda.synchronize()
    torch_topk_ms = ev0.elapsed_time(ev1) / reps

    cpu_baseline = None
    if not args.no_cpu_baseline:
        cpu_sample = 1 << 26          # about ten seconds of the oracle on one core
        v, dt_s, sample = time_oracle(cfg, cpu_sample, 1, 0, x=host_inputs[0])
        cpu_baseline = {"value": v, "unit": "elements/s", "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                        "sample": sample, "seconds": dt_s}

    # ---- the other benchmark configurations, briefly (single GPU only; the headline's inputs are freed first) ----
    extra_configs = None
    if world == 1 and not args.no_extra_configs:
        del dev_inputs, host_inputs, stage
        torch.cuda.empty_cache()
        extra_configs = []
        for name in EXTRA_CONFIGS:
            if name == args.config:
                continue
            try:
                extra_configs.append(measure_extra_config(profk, torch, name, dev, peak))
            except Exception as exc:            # reported, never hidden: a configuration that could not be timed says why
                extra_configs.append({"name": name, "error": f"{type(exc).__name__}: {exc}"})

    whole_call_gbs = in_bytes / (ms_per_step * 1e-3) / 1e9
    sorted_blocks = sorted(block_ms)
    line = {
        "metric": "top-k elements/s", "value": value, "unit": "elements/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dt, "data": "synthetic",
        "config": {"workload": describe(args.config, cfg), "plan": {"m": pl.m, "r": pl.r, "capacity": pl.capacity, "mode": pl.mode},
                   "l2": f"{copies} distinct input copies of {in_bytes >> 20} MiB rotated so no step re-reads L2-resident data",
                   "parallelism": f"{world} independent replica(s), one per GPU"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "elements/s", "h2d_bytes_per_step": in_bytes,
                "d2h_bytes_per_step": rows * k * (elem + 8), "ms_per_step": e2e_ms},
        "gpu_launches": launches_per_step * steps,
        "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "extra": {"whole_call_GBps": whole_call_gbs, "frac_of_8TBps_read_once": whole_call_gbs / 8000.0,
                  "frac_of_measured_peak": whole_call_gbs / peak,
                  "blocks": {"count": len(block_ms), "steps_each": steps, "ms_per_step_median": sorted_blocks[len(sorted_blocks) // 2],
                             "ms_per_step_min": sorted_blocks[0], "ms_per_step_max": sorted_blocks[-1],
                             "note": "block 0 is the headline; `value` and `ms_per_step` come from it alone"},
                  "fallback_rate_observed": fallback_rate, "fallback_row_calls": n_seeds * rows, "fallback_rate_budget": eps,
                  "torch_topk_ms_same_gpu": torch_topk_ms, "launches_per_step": launches_per_step,
                  "configs": extra_configs,
                  "configs_note": "other benchmark configurations, timed briefly in this run: inputs drawn on the device with the "
                                  "seeded CUDA generator, 5 warm-up + 20-40 timed calls, CUDA events, distinct input copies rotated"},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
