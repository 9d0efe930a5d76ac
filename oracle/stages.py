"""The four stages of the method run literally on one row.  TEST INFRASTRUCTURE ONLY.

Section 3 of the paper, "The Prof-K algorithm":
  1. Sampling: S indices (here: `philox.sample_indices`).
  2. Threshold estimation: sort the sampled values in descending order and take
     tau = s_t, the t-th largest.
  3. Filtering: one pass over the row, keeping every element with x_i >= tau in a
     buffer of capacity M; R = |{i : x_i >= tau}|.
  4. Refinement: exact top-k of the buffer; if fewer than k candidates were kept,
     or the buffer overflowed, exact top-k of the whole row instead.

Readings: "descending order" is the total order of `topk.order_key`, and the
filter's "x_i >= tau" is read in that same order (key(x_i) >= key(tau)), so the
kept elements are exactly the R largest of the row and the count check
k <= R <= M says what it is meant to say.  On ordinary values this is the
floating-point comparison; it differs only where the two orders do (-0.0 ranks
below +0.0; a NaN with the sign bit set ranks lowest and one without it highest,
whereas floating point calls the zeros equal and a NaN unordered -- counting a
lowest-ranked NaN among the survivors would let the check pass without the
top-k in the buffer).  In relaxed mode the acceptance test is
k_accept <= R <= M and a short buffer is returned as it is, followed by padding
(value -inf, index -1).

Tie-proof variant (`composite=True`; not in the paper, whose analysis assumes distinct
ranks): the threshold is the t-th sample as a RECORD under (value descending, index
ascending) -- its value tau and its index tau_idx -- and the filter drops the elements
that have exactly tau's value (the same order key) and an index above tau_idx.  Records
are distinct, so R is the rank of the threshold record among all records of the row and
Lemma 1's law holds for any input, ties included; on rows without ties at tau nothing
changes.

Second chance before the exact fallback (`r_tight`, `r_loose`; a reading of "Refinement": the
paper sends a failed row straight to an exact top-k of the full input): the sample is still there,
so a row whose buffer overflowed is filtered once more with the threshold of the tighter sample rank
r_tight, a row with too few candidates with that of the looser rank r_loose -- same buffer, same
tie rule, and the check k <= R' <= M (the full k also in relaxed mode).  If it passes, the answer is
refined from that pass (it is the same exact top-k) and the status says so; if not, or if the plan
names no such rank (0), the exact top-k of the whole row replaces it as before.

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
STATUS_RECALL_REFILTERED = 4      # R < k_accept, then k <= R' <= M under the looser rank: answer from the second pass
STATUS_OVERFLOW_REFILTERED = 5    # R > M, then k <= R' <= M under the tighter rank: answer from the second pass


@dataclass
class StageResult:
    sample_idx: np.ndarray      # the S sampled indices
    tau: object                 # threshold, an element of the row (same dtype / bit pattern)
    survivors: int              # R
    status: int
    vals: np.ndarray            # k values (padded in relaxed mode)
    idx: np.ndarray             # k indices, int64, -1 = padding


def threshold(x: np.ndarray, sample_idx: np.ndarray, t: int):
    """Stage 2: the t-th largest sampled value (ties in value are the same value)."""
    sampled = x[sample_idx]
    order = np.argsort(~topk.order_key(sampled), kind="stable")
    return sampled[order[t - 1]]


def _key_of(x: np.ndarray, tau):
    return topk.order_key(np.asarray([tau], dtype=x.dtype))[0]


def count_survivors(x: np.ndarray, tau) -> int:
    """Stage 3's R = |{i : x_i >= tau}|, the comparison taken in the total order."""
    return int(np.count_nonzero(topk.order_key(x) >= _key_of(x, tau)))


def survivor_set(x: np.ndarray, tau) -> np.ndarray:
    """Indices kept by stage 3, ascending."""
    return np.flatnonzero(topk.order_key(x) >= _key_of(x, tau))


def threshold_record(x: np.ndarray, sample_idx: np.ndarray, t: int):
    """Stage 2 on records: the t-th sample under (value descending, index ascending), as (value, index)."""
    sampled = x[sample_idx]
    order = np.lexsort((sample_idx, ~topk.order_key(sampled)))      # last key is the primary one
    j = order[t - 1]
    return sampled[j], int(sample_idx[j])


def survivor_set_record(x: np.ndarray, tau, tau_idx: int) -> np.ndarray:
    """Indices kept by the tie-proof stage 3, ascending: the elements above tau, and those equal to tau (the same
    order key) with an index up to tau_idx."""
    keys, tk = topk.order_key(x), _key_of(x, tau)
    return np.flatnonzero((keys > tk) | ((keys == tk) & (np.arange(x.shape[0]) <= tau_idx)))


def _filter_with_rank(x: np.ndarray, s_idx: np.ndarray, rank: int, composite: bool):
    """Stages 2 and 3 for one sample rank: (tau, indices kept)."""
    if composite:
        tau, tau_idx = threshold_record(x, s_idx, rank)              # stage 2, on records
        return tau, survivor_set_record(x, tau, tau_idx)             # stage 3, tie-proof
    tau = threshold(x, s_idx, rank)                                  # stage 2
    return tau, survivor_set(x, tau)                                 # stage 3


def run_row(x: np.ndarray, k: int, m: int, r: int, capacity: int, k_accept: int,
            seed: int, row: int = 0, mode: int = 0, composite: bool = False,
            r_tight: int = 0, r_loose: int = 0) -> StageResult:
    """All four stages on one row with an explicit plan (m, r, capacity, k_accept[, r_tight, r_loose])."""
    n = x.shape[0]
    if mode == 1:
        vals, idx = topk.topk_row(x, k)
        return StageResult(np.empty(0, np.int64), None, 0, STATUS_DIRECT, vals, idx)
    s_idx = philox.sample_indices(n, m, seed, row)                  # stage 1
    tau, kept = _filter_with_rank(x, s_idx, r, composite)            # stages 2 and 3
    R = int(kept.size)
    if R > capacity or R < k_accept:                                 # stage 4, failure branches
        failed = STATUS_OVERFLOW if R > capacity else STATUS_RECALL
        second = r_tight if R > capacity else r_loose
        if second:                                                   # one more filtering pass with the other rank
            tau2, kept2 = _filter_with_rank(x, s_idx, second, composite)
            if k <= kept2.size <= capacity:
                bvals, bpos = topk.topk_row(x[kept2], k)
                status = STATUS_OVERFLOW_REFILTERED if failed == STATUS_OVERFLOW else STATUS_RECALL_REFILTERED
                return StageResult(s_idx, tau2, int(kept2.size), status, bvals, kept2[bpos].astype(np.int64))
        vals, idx = topk.topk_row(x, k)
        return StageResult(s_idx, tau, R, failed, vals, idx)
    kk = min(k, R)                                                   # stage 4 on the buffer
    bvals, bpos = topk.topk_row(x[kept], kk)
    vals = np.empty(k, dtype=x.dtype)
    idx = np.full(k, -1, dtype=np.int64)
    vals[:kk] = bvals
    idx[:kk] = kept[bpos]
    if kk < k:                                                       # relaxed mode only
        vals[kk:] = np.float32(-np.inf) if x.dtype == np.float32 else np.uint16(0xFF80)
    return StageResult(s_idx, tau, R, STATUS_OK, vals, idx)
