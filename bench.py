#!/usr/bin/env python
"""Benchmark of the Prof-K hot path on B200.

One step = one call of the whole hot path (sample -> threshold -> filter -> count check ->
refine) over one batch of synthetic input.  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

Workloads (`--config`): "cfg2" (default; single row N = 2^26 fp32 N(0,1), k = 256, eps = 1e-4),
"cfg2_k16", "cfg2_k4096", "cfg1", "cfg3_f32", "cfg3_bf16".
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
FILTER_TRAFFIC_BYTES = {"cfg2": 272.39e6}

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

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.lines: list[str] = []
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

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [s.strip() for s in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


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
        "config": {"workload": describe(name, cfg)},
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def describe(name, cfg):
    rows, n, dt, recipe, seed, k, eps, recall = cfg
    mode = "exact" if recall >= 1.0 else f"relaxed recall {recall}"
    return f"{name}: {rows} row(s) x N={n} {dt}, {recipe} seed {seed}, k={k}, eps={eps}, {mode}"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="cfg2", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="profk", choices=["profk", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
    fallbacks = 0
    ev0.record()
    for i in range(steps):
        step(warmup + i)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    if args.hot_path_only:
        if rank == 0:
            print(json.dumps({"hot_path_only": True, "ms_per_step": ms_total / steps, "launches_per_step": launches_per_step}))
        return
    ms_total = sharding.max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / steps
    value = sharding.whole_job_rate(rows * n, world, ms_per_step)

    # fallback rate observed over a separate run of seeds (statistics read-back synchronises, so not timed)
    n_seeds = (40 if big else 200) if rows == 1 else max(1, 200 // rows)
    for s in range(n_seeds):
        profk.topk(dev_inputs[s % copies], k, eps=eps, recall=recall, seed=10_000 + s, out=(out_vals, out_idx))
        fallbacks += sum(1 for st in profk.read_stats(rows) if (st[3] & 0xFF) in (profk.ROW_RECALL, profk.ROW_OVERFLOW))
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
    taus = profk.sample_threshold(dev_inputs[0], pl.m, pl.r, seed=0) if pl.mode == 0 else None
    roofline = None
    if taus is not None:
        buf = torch.empty((rows, pl.capacity), dtype=torch.int64, device=dev)
        counts = torch.zeros(rows, dtype=torch.int32, device=dev)
        lib = profk.lib()
        import ctypes

        fn = getattr(lib, "profk_filter_f32" if dt == "f32" else "profk_filter_bf16")
        stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

        def filt(i):
            counts.zero_()
            code = fn(ctypes.c_void_p(dev_inputs[i % copies].data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n),
                      ctypes.c_void_p(taus.data_ptr()), ctypes.c_int64(pl.capacity), ctypes.c_void_p(buf.data_ptr()),
                      ctypes.c_void_p(counts.data_ptr()), stream)
            assert code == 0

        for i in range(warmup):
            filt(i)
        torch.cuda.synchronize()
        # `steps` launches back to back, each with its own zeroed counter, bracketed by one pair of events:
        # the average is the kernel's duration plus the ~1 us gap between queued launches.
        many = torch.zeros(steps * rows, dtype=torch.int32, device=dev)
        fe0, fe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fe0.record()
        for i in range(steps):
            code = fn(ctypes.c_void_p(dev_inputs[i % copies].data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n),
                      ctypes.c_void_p(taus.data_ptr()), ctypes.c_int64(pl.capacity), ctypes.c_void_p(buf.data_ptr()),
                      ctypes.c_void_p(many.data_ptr() + 4 * i * rows), stream)
        fe1.record()
        torch.cuda.synchronize()
        filt_ms = fe0.elapsed_time(fe1) / steps
        survivors = float(many[:rows].sum().item())
        # The stand-alone filter takes the threshold as a value alone: on a row flooded with copies of tau its buffer
        # overflows and the launch stops early, so its duration is not that of a scan.
        filter_overflowed = bool((many[:rows] > pl.capacity).any().item())
    clocks = sampler.stop()
    if taus is not None:
        algo_bytes = in_bytes + survivors * 8            # read every element once + one 8-byte record per survivor
        peak, peak_kind = measured_peak_gbs()
        achieved = algo_bytes / (filt_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "filter_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": FILTER_TRAFFIC_BYTES.get(args.config),
                    "ms_per_launch": filt_ms, "algorithmic_bytes": algo_bytes}
        if filter_overflowed:
            roofline.update({"achieved": None, "frac": None,
                             "note": "stand-alone filter launch overflowed its buffer (value-only threshold on a tie-flooded row) and stopped early"})

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
        cpu_baseline = {"value": v, "unit": "elements/s", "cores": 1, "kind": "oracle", "sample": sample,
                        "seconds": dt_s}

    whole_call_gbs = in_bytes / (ms_per_step * 1e-3) / 1e9
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
                  "frac_of_measured_peak": whole_call_gbs / measured_peak_gbs()[0],
                  "fallback_rate_observed": fallback_rate, "fallback_rate_budget": eps,
                  "torch_topk_ms_same_gpu": torch_topk_ms, "launches_per_step": launches_per_step},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
