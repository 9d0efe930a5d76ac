"""Prof-K one-pass probabilistic top-k for NVIDIA B200: thin Python binding of the C ABI.

Every function here only marshals arguments (torch tensors -> device pointers, the
current CUDA stream) into the `extern "C"` entry points declared in `include/profk.h`;
all arithmetic of the method runs inside the CUDA library `libprofk.so`, which is built
in-tree by `paper_2608_12573_b200._build.build()`.  There is no CPU fallback: a call
raises when the library is missing or reports an error.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_LIB = None
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libprofk.so")

EXPORTS = [
    "profk_plan", "profk_plan_batch", "profk_plan_ex", "profk_default_tuning", "profk_default_tuning_batch", "profk_workspace_bytes", "profk_set_workspace",
    "profk_topk_f32", "profk_topk_bf16", "profk_topk_planned_f32", "profk_topk_planned_bf16",
    "profk_filter_f32", "profk_filter_bf16", "profk_sample_threshold_f32", "profk_sample_threshold_bf16",
    "profk_read_stats", "profk_last_launch_count", "profk_strerror", "profk_topk_noalloc_f32",
    "profk_debug_set_prefetch_wait_polls",
    "profk_batchtopk_workspace_bytes", "profk_batchtopk_f32", "profk_batchtopk_bf16", "profk_batchtopk_planned_f32",
    "profk_batchtopk_planned_bf16",
    "profk_shard_bounds", "profk_shard_sample_keys_f32", "profk_shard_sample_keys_bf16", "profk_threshold_from_keys_f32",
    "profk_threshold_from_keys_bf16", "profk_filter_shard_f32", "profk_filter_shard_bf16", "profk_refine_gathered_f32",
    "profk_refine_gathered_bf16",
]

FILTER_COUNT_STRIDE = 8      # PROFK_FILTER_COUNT_STRIDE: uint32 words per row in the counts array of profk_filter_*
ROW_OK, ROW_RECALL, ROW_OVERFLOW, ROW_DIRECT = 0, 1, 2, 3
ROW_RECALL_REFILTERED, ROW_OVERFLOW_REFILTERED = 4, 5    # repaired by a second filtering pass (plan.r_loose / plan.r_tight)
TIES_KEEP_ALL, TIES_BY_INDEX = 0, 1      # profk_plan_t.tie_rule: the filter as printed / the threshold as a (value, index) record


class ProfkError(RuntimeError):
    pass


class _PlanStruct(ctypes.Structure):
    _fields_ = [("m", ctypes.c_int64), ("r", ctypes.c_int64), ("capacity", ctypes.c_int64),
                ("k_accept", ctypes.c_int64), ("mode", ctypes.c_int32), ("tie_rule", ctypes.c_int32),
                ("z", ctypes.c_double), ("alpha", ctypes.c_double),
                ("p_recall_fail", ctypes.c_double), ("p_overflow", ctypes.c_double),
                ("r_tight", ctypes.c_int64), ("r_loose", ctypes.c_int64)]


class _TuningStruct(ctypes.Structure):
    _fields_ = [("s_min", ctypes.c_int64), ("s_max", ctypes.c_int64), ("cost_ratio", ctypes.c_double)]


class _StatsStruct(ctypes.Structure):
    _fields_ = [("tau_bits", ctypes.c_uint32), ("survivors", ctypes.c_uint32),
                ("capacity", ctypes.c_uint32), ("status", ctypes.c_uint32)]


@dataclass
class Plan:
    m: int
    r: int
    capacity: int
    k_accept: int
    mode: int
    z: float = 0.0
    alpha: float = 0.0
    p_recall_fail: float = 0.0
    p_overflow: float = 0.0
    tie_rule: int = TIES_BY_INDEX
    r_tight: int = 0      # second-chance ranks: 0 = none (a row that fails the count check is selected exactly at once)
    r_loose: int = 0

    def _struct(self) -> _PlanStruct:
        return _PlanStruct(self.m, self.r, self.capacity, self.k_accept, self.mode, self.tie_rule,
                           self.z, self.alpha, self.p_recall_fail, self.p_overflow, self.r_tight, self.r_loose)


def lib() -> ctypes.CDLL:
    """The loaded CUDA library; raises if it has not been built."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(_LIB_PATH):
            raise ProfkError(f"{_LIB_PATH} is missing: run paper_2608_12573_b200._build.build() "
                             "(there is no fallback implementation)")
        _LIB = ctypes.CDLL(_LIB_PATH)
        _LIB.profk_strerror.restype = ctypes.c_char_p
        _LIB.profk_strerror.argtypes = [ctypes.c_int]
        for name in EXPORTS:
            getattr(_LIB, name)          # fail now if a symbol is absent
    return _LIB


def _check(code: int, what: str) -> None:
    if code != 0:
        raise ProfkError(f"{what}: {lib().profk_strerror(code).decode()} ({code})")


_plan_cache: dict = {}


PAPER_TUNING = dict(s_min=32768, s_max=131072, cost_ratio=1.0)     # Section 4's values of the tuning inputs


def default_tuning(N: int, rows: int = 1) -> dict:
    """`profk_default_tuning_batch`: the tuning inputs `plan` uses when none are given (the paper's, with the
    floor on the sample size following the row length for short rows and the cost ratio growing with it)."""
    t = _TuningStruct(0, 0, 0.0)
    _check(lib().profk_default_tuning_batch(ctypes.c_int64(rows), ctypes.c_int64(N), ctypes.byref(t)), "profk_default_tuning_batch")
    return dict(s_min=int(t.s_min), s_max=int(t.s_max), cost_ratio=float(t.cost_ratio))


def plan(N: int, k: int, eps: float = 1e-3, recall: float = 1.0, s_min: int | None = None,
         s_max: int | None = None, cost_ratio: float | None = None, rows: int = 1) -> Plan:
    """`profk_plan_batch` / `profk_plan_ex`: the parameters (S, t, M) for rows of length N.  Without tuning
    inputs: the library's defaults for a call with `rows` rows (`default_tuning`);
    `plan(N, k, eps, recall, **PAPER_TUNING)` gives the paper's."""
    key = (N, k, eps, recall, s_min, s_max, cost_ratio, rows)
    hit = _plan_cache.get(key)
    if hit is not None:
        return hit
    res = _plan_uncached(N, k, eps, recall, s_min, s_max, cost_ratio, rows)
    if len(_plan_cache) > 4096:
        _plan_cache.clear()
    _plan_cache[key] = res
    return res


def _plan_uncached(N, k, eps, recall, s_min, s_max, cost_ratio, rows) -> Plan:
    out = _PlanStruct()
    if s_min is None and s_max is None and cost_ratio is None:
        code = lib().profk_plan_batch(ctypes.c_int64(rows), ctypes.c_int64(N), ctypes.c_int64(k), ctypes.c_double(eps),
                                      ctypes.c_double(recall), ctypes.byref(out))
    else:
        tun = _TuningStruct(32768 if s_min is None else s_min, 131072 if s_max is None else s_max,
                            1.0 if cost_ratio is None else cost_ratio)
        code = lib().profk_plan_ex(ctypes.c_int64(N), ctypes.c_int64(k), ctypes.c_double(eps),
                                   ctypes.c_double(recall), ctypes.byref(tun), ctypes.byref(out))
    _check(code, "profk_plan")
    return Plan(out.m, out.r, out.capacity, out.k_accept, out.mode, out.z, out.alpha,
                out.p_recall_fail, out.p_overflow, out.tie_rule, out.r_tight, out.r_loose)


def workspace_bytes(rows: int, capacity: int, k: int) -> int:
    n = ctypes.c_size_t()
    _check(lib().profk_workspace_bytes(ctypes.c_int64(rows), ctypes.c_int64(capacity), ctypes.c_int64(k),
                                       ctypes.byref(n)), "profk_workspace_bytes")
    return int(n.value)


_workspaces: dict = {}     # device index -> torch tensor kept alive while registered
_workspace_ok: set = set()  # (device, rows, capacity, k) shapes known to fit the registered workspace


def ensure_workspace(rows: int, capacity: int, k: int, device) -> None:
    """Allocate (through torch) and register a workspace large enough for the shape."""
    import torch

    dev = torch.device(device)
    idx = dev.index if dev.index is not None else torch.cuda.current_device()
    if (idx, rows, capacity, k) in _workspace_ok:
        return
    need = workspace_bytes(rows, capacity, k)
    cur = _workspaces.get(idx)
    if cur is not None and cur.numel() >= need:
        _workspace_ok.add((idx, rows, capacity, k))
        return
    with torch.cuda.device(idx):
        buf = torch.empty(max(need, 1 << 20), dtype=torch.uint8, device=dev)
        _check(lib().profk_set_workspace(ctypes.c_void_p(buf.data_ptr()), ctypes.c_size_t(buf.numel())),
               "profk_set_workspace")
    _workspaces[idx] = buf
    _workspace_ok.clear()
    _workspace_ok.add((idx, rows, capacity, k))


def _stream_ptr():
    import torch

    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _suffix(x) -> str:
    import torch

    if x.dtype == torch.float32:
        return "f32"
    if x.dtype == torch.bfloat16:
        return "bf16"
    raise ProfkError(f"unsupported dtype {x.dtype}: float32 and bfloat16 only")


def _rows_view(x):
    if not x.is_cuda:
        raise ProfkError("input must be a CUDA tensor")
    if x.dim() == 1:
        x = x.unsqueeze(0)
    if x.dim() != 2 or not x.is_contiguous():
        raise ProfkError("input must be a contiguous (N,) or (rows, N) tensor")
    return x


def topk(x, k: int, eps: float = 1e-3, recall: float = 1.0, seed: int = 0, plan_override: Plan | None = None,
         out=None):
    """`profk_topk_*` / `profk_topk_planned_*` on the current stream.

    x: CUDA tensor (N,) or (rows, N), float32 or bfloat16.  Returns (values, indices) with
    shapes (rows, k) (or (k,) for 1-D input); nothing is synchronised.
    """
    import torch

    one_d = x.dim() == 1
    x2 = _rows_view(x)
    rows, n = x2.shape
    pl = plan_override if plan_override is not None else plan(n, k, eps, recall, rows=rows)
    ensure_workspace(rows, pl.capacity, k, x2.device)
    if out is None:
        vals = torch.empty((rows, k), dtype=x2.dtype, device=x2.device)
        idx = torch.empty((rows, k), dtype=torch.int64, device=x2.device)
    else:
        vals, idx = out
    sfx = _suffix(x2)
    with torch.cuda.device(x2.device):
        if plan_override is None:
            fn = getattr(lib(), f"profk_topk_{sfx}")
            code = fn(ctypes.c_void_p(x2.data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n), ctypes.c_int64(k),
                      ctypes.c_double(eps), ctypes.c_double(recall), ctypes.c_uint64(seed), _stream_ptr(),
                      ctypes.c_void_p(vals.data_ptr()), ctypes.c_void_p(idx.data_ptr()))
        else:
            st = pl._struct()
            fn = getattr(lib(), f"profk_topk_planned_{sfx}")
            code = fn(ctypes.c_void_p(x2.data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n), ctypes.c_int64(k),
                      ctypes.byref(st), ctypes.c_uint64(seed), _stream_ptr(),
                      ctypes.c_void_p(vals.data_ptr()), ctypes.c_void_p(idx.data_ptr()))
    _check(code, "profk_topk")
    if one_d:
        return vals[0], idx[0]
    return vals, idx


def batchtopk_workspace_bytes(capacity: int, k: int) -> int:
    n = ctypes.c_size_t()
    _check(lib().profk_batchtopk_workspace_bytes(ctypes.c_int64(capacity), ctypes.c_int64(k), ctypes.byref(n)),
           "profk_batchtopk_workspace_bytes")
    return int(n.value)


def _ensure_bytes(need: int, device) -> None:
    """Register a workspace of at least `need` bytes on `device` (allocated through torch)."""
    import torch

    dev = torch.device(device)
    idx = dev.index if dev.index is not None else torch.cuda.current_device()
    cur = _workspaces.get(idx)
    if cur is not None and cur.numel() >= need:
        return
    with torch.cuda.device(idx):
        buf = torch.empty(max(need, 1 << 20), dtype=torch.uint8, device=dev)
        _check(lib().profk_set_workspace(ctypes.c_void_p(buf.data_ptr()), ctypes.c_size_t(buf.numel())),
               "profk_set_workspace")
    _workspaces[idx] = buf
    _workspace_ok.clear()


def batchtopk(x, k: int, eps: float = 1e-3, seed: int = 0, want_pairs: bool = True, want_mask: bool = False,
              want_dense: bool = False, in_place: bool = False, plan_override: Plan | None = None):
    """`profk_batchtopk_*` on the current stream: the K largest entries of the flattened tensor `x` as a set.

    Returns a dict with the forms asked for: "values", "indices" (K each, in no particular order), "mask"
    (int32 words, bit i % 32 of word i // 32), "dense" (a tensor shaped like `x`; `in_place=True` overwrites
    `x` itself and returns it).  Nothing is synchronised."""
    import torch

    if not x.is_cuda or not x.is_contiguous():
        raise ProfkError("input must be a contiguous CUDA tensor")
    flat = x.view(-1)
    n = flat.numel()
    pl = plan_override if plan_override is not None else plan(n, k, eps, 1.0)
    _ensure_bytes(batchtopk_workspace_bytes(pl.capacity, k), flat.device)
    out = {}
    vals = idx = mask = dense = None
    if want_pairs:
        vals = torch.empty(k, dtype=flat.dtype, device=flat.device)
        idx = torch.empty(k, dtype=torch.int64, device=flat.device)
        out["values"], out["indices"] = vals, idx
    if want_mask:
        mask = torch.empty((n + 31) // 32, dtype=torch.int32, device=flat.device)
        out["mask"] = mask
    if want_dense or in_place:
        dense = flat if in_place else torch.empty_like(flat)
        out["dense"] = dense.view(x.shape)

    def ptr(t):
        return ctypes.c_void_p(t.data_ptr() if t is not None else None)

    sfx = _suffix(flat)
    with torch.cuda.device(flat.device):
        if plan_override is None:
            code = getattr(lib(), f"profk_batchtopk_{sfx}")(ptr(flat), ctypes.c_int64(n), ctypes.c_int64(k), ctypes.c_double(eps),
                                                          ctypes.c_uint64(seed), _stream_ptr(), ptr(vals), ptr(idx), ptr(mask), ptr(dense))
        else:
            st = pl._struct()
            code = getattr(lib(), f"profk_batchtopk_planned_{sfx}")(ptr(flat), ctypes.c_int64(n), ctypes.c_int64(k), ctypes.byref(st),
                                                                  ctypes.c_uint64(seed), _stream_ptr(), ptr(vals), ptr(idx), ptr(mask),
                                                                  ptr(dense))
    _check(code, "profk_batchtopk")
    return out


# ---- one row over several GPUs: the stage calls (argument marshalling only; sharding.py makes the exchanges) ----
def shard_bounds(n: int, m: int, shards: int, shard: int) -> tuple[int, int, int, int]:
    """`profk_shard_bounds`: (j_lo, j_hi, elem_lo, elem_hi) of shard `shard` of `shards`: whole pairs of sampling strata."""
    out = [ctypes.c_int64() for _ in range(4)]
    _check(lib().profk_shard_bounds(ctypes.c_int64(n), ctypes.c_int64(m), ctypes.c_int64(shards), ctypes.c_int64(shard),
                                    *[ctypes.byref(o) for o in out]), "profk_shard_bounds")
    return tuple(int(o.value) for o in out)


def shard_sample_keys(shard, shard_base: int, n: int, m: int, j_lo: int, j_hi: int, seed: int):
    """`profk_shard_sample_keys_*`: uint32 order keys (as an int32 tensor) of the samples of strata [j_lo, j_hi)."""
    import torch

    keys = torch.empty(j_hi - j_lo, dtype=torch.int32, device=shard.device)
    fn = getattr(lib(), f"profk_shard_sample_keys_{_suffix(shard)}")
    with torch.cuda.device(shard.device):
        _check(fn(ctypes.c_void_p(shard.data_ptr()), ctypes.c_int64(shard_base), ctypes.c_int64(shard.numel()), ctypes.c_int64(n),
                  ctypes.c_int64(m), ctypes.c_int64(j_lo), ctypes.c_int64(j_hi), ctypes.c_uint64(seed),
                  ctypes.c_void_p(keys.data_ptr()), _stream_ptr()), "profk_shard_sample_keys")
    return keys


def threshold_from_keys(keys, dtype, n: int, m: int, r: int, seed: int, tie_rule: int = TIES_BY_INDEX):
    """`profk_threshold_from_keys_*`: the 4-word threshold record (int32 tensor) from the m gathered keys."""
    import torch

    thr = torch.empty(4, dtype=torch.int32, device=keys.device)
    sfx = "f32" if dtype == torch.float32 else "bf16"
    with torch.cuda.device(keys.device):
        _check(getattr(lib(), f"profk_threshold_from_keys_{sfx}")(ctypes.c_void_p(keys.data_ptr()), ctypes.c_int64(n), ctypes.c_int64(m),
                                                                ctypes.c_int64(r), ctypes.c_uint64(seed), ctypes.c_int(tie_rule),
                                                                ctypes.c_void_p(thr.data_ptr()), _stream_ptr()), "profk_threshold_from_keys")
    return thr


def filter_shard(shard, shard_base: int, thr, capacity: int):
    """`profk_filter_shard_*`: (records int64 (capacity,), state int32 (8,)) -- indices local to the shard."""
    import torch

    records = torch.empty(capacity, dtype=torch.int64, device=shard.device)
    state = torch.empty(8, dtype=torch.int32, device=shard.device)
    fn = getattr(lib(), f"profk_filter_shard_{_suffix(shard)}")
    with torch.cuda.device(shard.device):
        _check(fn(ctypes.c_void_p(shard.data_ptr()), ctypes.c_int64(shard_base), ctypes.c_int64(shard.numel()), ctypes.c_void_p(thr.data_ptr()),
                  ctypes.c_int64(capacity), ctypes.c_void_p(records.data_ptr()), ctypes.c_void_p(state.data_ptr()), _stream_ptr()),
               "profk_filter_shard")
    return records, state


def refine_gathered(records, states, bases, thr, dtype, capacity: int, k: int, k_accept: int):
    """`profk_refine_gathered_*`: records (shards, shard_capacity) int64, states (shards, 8) int32, bases: list of int.
    Returns (values (k,), indices (k,), status int32 (2,) = [PROFK_ROW_*, R]); nothing is synchronised."""
    import torch

    shards, shard_cap = records.shape
    ensure_workspace(1, capacity, k, records.device)
    vals = torch.empty(k, dtype=dtype, device=records.device)
    idx = torch.empty(k, dtype=torch.int64, device=records.device)
    status = torch.empty(2, dtype=torch.int32, device=records.device)
    arr = (ctypes.c_int64 * shards)(*[int(b) for b in bases])
    sfx = "f32" if dtype == torch.float32 else "bf16"
    with torch.cuda.device(records.device):
        _check(getattr(lib(), f"profk_refine_gathered_{sfx}")(ctypes.c_void_p(records.data_ptr()), ctypes.c_void_p(states.data_ptr()), arr,
                                                            ctypes.c_int64(shards), ctypes.c_int64(shard_cap), ctypes.c_void_p(thr.data_ptr()),
                                                            ctypes.c_int64(capacity), ctypes.c_int64(k), ctypes.c_int64(k_accept),
                                                            ctypes.c_void_p(vals.data_ptr()), ctypes.c_void_p(idx.data_ptr()),
                                                            ctypes.c_void_p(status.data_ptr()), _stream_ptr()), "profk_refine_gathered")
    return vals, idx, status


def topk_noalloc(x, k: int, eps: float = 1e-3, recall: float = 1.0, seed: int = 0, out=None):
    """`profk_topk_noalloc_f32`: top-k with the library's built-in scratch, for callers that must not
    allocate.  The output tensors are the caller's (`out=(values, indices)`); when `out` is omitted this
    convenience wrapper allocates them through torch, which the C entry point itself never does.
    float32 only; shapes whose workspace exceeds 16 MiB raise ProfkError."""
    import torch

    one_d = x.dim() == 1
    x2 = _rows_view(x)
    if x2.dtype != torch.float32:
        raise ProfkError("topk_noalloc: float32 only")
    rows, n = x2.shape
    if out is None:
        out = (torch.empty((rows, k), dtype=x2.dtype, device=x2.device),
               torch.empty((rows, k), dtype=torch.int64, device=x2.device))
    vals, idx = out
    with torch.cuda.device(x2.device):
        code = lib().profk_topk_noalloc_f32(ctypes.c_void_p(x2.data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n),
                                            ctypes.c_int64(k), ctypes.c_double(eps), ctypes.c_double(recall),
                                            ctypes.c_uint64(seed), _stream_ptr(), ctypes.c_void_p(vals.data_ptr()),
                                            ctypes.c_void_p(idx.data_ptr()))
    _check(code, "profk_topk_noalloc_f32")
    return (vals[0], idx[0]) if one_d else (vals, idx)


def filter_pass(x, tau, capacity: int):
    """`profk_filter_*`: stage 3 alone.  Returns (records uint64 as int64 tensor (rows, capacity), counts int32 (rows,))."""
    import torch

    x2 = _rows_view(x)
    rows, n = x2.shape
    tau = tau.reshape(rows).contiguous()
    buf = torch.empty((rows, capacity), dtype=torch.int64, device=x2.device)
    counts = torch.zeros((rows, FILTER_COUNT_STRIDE), dtype=torch.int32, device=x2.device)       # one counter per 32 bytes
    fn = getattr(lib(), f"profk_filter_{_suffix(x2)}")
    with torch.cuda.device(x2.device):
        code = fn(ctypes.c_void_p(x2.data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n), ctypes.c_void_p(tau.data_ptr()),
                  ctypes.c_int64(capacity), ctypes.c_void_p(buf.data_ptr()), ctypes.c_void_p(counts.data_ptr()), _stream_ptr())
    _check(code, "profk_filter")
    return buf, counts[:, 0]


def sample_threshold(x, m: int, r: int, seed: int, want_indices: bool = False):
    """`profk_sample_threshold_*`: stages 1-2 alone.  Returns tau (rows,) and optionally the sampled indices."""
    import torch

    x2 = _rows_view(x)
    rows, n = x2.shape
    tau = torch.empty(rows, dtype=x2.dtype, device=x2.device)
    sidx = torch.empty((rows, m), dtype=torch.int32, device=x2.device) if want_indices else None
    fn = getattr(lib(), f"profk_sample_threshold_{_suffix(x2)}")
    with torch.cuda.device(x2.device):
        code = fn(ctypes.c_void_p(x2.data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n), ctypes.c_int64(m),
                  ctypes.c_int64(r), ctypes.c_uint64(seed), ctypes.c_void_p(tau.data_ptr()),
                  ctypes.c_void_p(sidx.data_ptr() if want_indices else None), _stream_ptr())
    _check(code, "profk_sample_threshold")
    return (tau, sidx) if want_indices else tau


def read_stats(rows: int):
    """`profk_read_stats`: list of (tau_bits, survivors, capacity, status) for the last call; synchronises."""
    arr = (_StatsStruct * rows)()
    _check(lib().profk_read_stats(_stream_ptr(), ctypes.c_int64(rows), arr), "profk_read_stats")
    return [(s.tau_bits, s.survivors, s.capacity, s.status) for s in arr]


def last_launch_count() -> int:
    return int(lib().profk_last_launch_count())
