"""The four stages of the method run literally on one row.  TEST INFRASTRUCTURE ONLY.

Section 3 of the paper, "The Prof-K algorithm":
  1. Sampling: S indices (here: `philox.sample_indices`).
  2. Threshold estimation: sort the sampled values in descending order and take
     tau = s_t, the t-th largest.
  3. Filtering: one pass over the row, keeping every element with x_i >= tau in a
     buffer of capacity M; R = |{i : x_i >= tau}|.
  4. Refinement: exact top-k of the buffer; if fewer than k candidates were kept,
     or the buffer overflowed, exact top-k of the whole row instead.

Readings: "descending order" is the total order of `topk.order_key`; the filter
predicate is "not (x_i < tau)" in floating point, which equals x_i >= tau on
inputs without NaN and keeps NaN otherwise (a superset of the key-order set, so
no top-k member is lost); in relaxed mode the acceptance test is
k_accept <= R <= M and a short buffer is returned as it is, followed by padding
(value -inf, index -1).

Tie-proof variant (`composite=True`; not in the paper, whose analysis assumes distinct
ranks): the threshold is the t-th sample as a RECORD under (value descending, index
ascending) -- its value tau and its index tau_idx -- and the filter drops the elements
that have exactly tau's value (the same order key) and an index above tau_idx.  Records
are distinct, so R is the rank of the threshold record among all records of the row and
Lemma 1's law holds for any input, ties included; on rows without ties at tau nothing
changes.

Status codes mirror the library's per-row statistics.

Pins (tests/test_oracle_stages.py): whenever k <= R <= M the refined answer
equals the exact top-k (the design goal stated after the four stages); R equals
the rank of tau in the sorted row for distinct values (Lemma 1's R); the failure
branches are reached with hand-built inputs.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import philox, topk

STATUS_OK = 0            # k_accept <= R <= M: answer came from the buffer
STATUS_RECALL = 1        # R < k_accept: fewer candidates than needed -> exact selection
STATUS_OVERFLOW = 2      # R > M: buffer too small -> exact selection
STATUS_DIRECT = 3        # plan mode 1: exact selection without sampling


@dataclass
class StageResult:
    sample_idx: np.ndarray      # the S sampled indices
    tau: object                 # threshold, an element of the row (same dtype / bit pattern)
    survivors: int              # R
    status: int
    vals: np.ndarray            # k values (padded in relaxed mode)
    idx: np.ndarray             # k indices, int64, -1 = padding


def _as_float(x: np.ndarray) -> np.ndarray:
    """Numeric view for the comparison: bf16 bit patterns widen exactly to float32."""
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return x


def threshold(x: np.ndarray, sample_idx: np.ndarray, t: int):
    """Stage 2: the t-th largest sampled value (ties in value are the same value)."""
    sampled = x[sample_idx]
    order = np.argsort(~topk.order_key(sampled), kind="stable")
    return sampled[order[t - 1]]


def count_survivors(x: np.ndarray, tau) -> int:
    """Stage 3's R = |{i : x_i >= tau}| with the predicate not (x_i < tau)."""
    xf = _as_float(x)
    tf = _as_float(np.asarray([tau], dtype=x.dtype))[0]
    return int(np.count_nonzero(~(xf < tf)))


def survivor_set(x: np.ndarray, tau) -> np.ndarray:
    """Indices kept by stage 3, ascending."""
    xf = _as_float(x)
    tf = _as_float(np.asarray([tau], dtype=x.dtype))[0]
    return np.flatnonzero(~(xf < tf))


def threshold_record(x: np.ndarray, sample_idx: np.ndarray, t: int):
    """Stage 2 on records: the t-th sample under (value descending, index ascending), as (value, index)."""
    sampled = x[sample_idx]
    order = np.lexsort((sample_idx, ~topk.order_key(sampled)))      # last key is the primary one
    j = order[t - 1]
    return sampled[j], int(sample_idx[j])


def survivor_set_record(x: np.ndarray, tau, tau_idx: int) -> np.ndarray:
    """Indices kept by the tie-proof stage 3, ascending: not (x_i < tau), minus the elements with tau's own
    order key and an index above tau_idx."""
    xf = _as_float(x)
    tf = _as_float(np.asarray([tau], dtype=x.dtype))[0]
    same = topk.order_key(x) == topk.order_key(np.asarray([tau], dtype=x.dtype))[0]
    late = np.arange(x.shape[0]) > tau_idx
    return np.flatnonzero(~(xf < tf) & ~(same & late))


def run_row(x: np.ndarray, k: int, m: int, r: int, capacity: int, k_accept: int,
            seed: int, row: int = 0, mode: int = 0, composite: bool = False) -> StageResult:
    """All four stages on one row with an explicit plan (m, r, capacity, k_accept)."""
    n = x.shape[0]
    if mode == 1:
        vals, idx = topk.topk_row(x, k)
        return StageResult(np.empty(0, np.int64), None, 0, STATUS_DIRECT, vals, idx)
    s_idx = philox.sample_indices(n, m, seed, row)                  # stage 1
    if composite:
        tau, tau_idx = threshold_record(x, s_idx, r)                 # stage 2, on records
        kept = survivor_set_record(x, tau, tau_idx)                  # stage 3, tie-proof
    else:
        tau = threshold(x, s_idx, r)                                 # stage 2
        kept = survivor_set(x, tau)                                  # stage 3
    R = int(kept.size)
    if R > capacity:                                                 # stage 4, failure branches
        vals, idx = topk.topk_row(x, k)
        return StageResult(s_idx, tau, R, STATUS_OVERFLOW, vals, idx)
    if R < k_accept:
        vals, idx = topk.topk_row(x, k)
        return StageResult(s_idx, tau, R, STATUS_RECALL, vals, idx)
    kk = min(k, R)                                                   # stage 4 on the buffer
    bvals, bpos = topk.topk_row(x[kept], kk)
    vals = np.empty(k, dtype=x.dtype)
    idx = np.full(k, -1, dtype=np.int64)
    vals[:kk] = bvals
    idx[:kk] = kept[bpos]
    if kk < k:                                                       # relaxed mode only
        vals[kk:] = np.float32(-np.inf) if x.dtype == np.float32 else np.uint16(0xFF80)
    return StageResult(s_idx, tau, R, STATUS_OK, vals, idx)
