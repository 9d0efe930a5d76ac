"""Exact top-k by definition.  TEST INFRASTRUCTURE ONLY (see package header).

Section 3 (problem setup) of the paper: given x in R^N and k >= 1, return the k
largest entries of x together with their indices; batched input is handled row
by row.  The paper does not say how equal values are ordered; this build fixes
"value descending, then index ascending", which makes the answer unique.

Values are compared through the usual order-preserving integer key of an IEEE
bit pattern, which extends "<" to a total order
    -NaN < -inf < ... < -0.0 < +0.0 < ... < +inf < +NaN.
On inputs without NaN and without -0.0 this is plain numeric order.

bfloat16 has no NumPy dtype: a bf16 array is passed as its uint16 bit patterns.

The flattened BatchTopK of Section 5 ("Application: BatchTopK sparse
autoencoders") keeps the K largest entries of the flattened activation matrix
and sets the rest to zero: `kept_mask`, `kept_dense` and `pack_mask` state that
result in the three forms the library emits, all derived from `topk_row`.

Pins (tests/test_oracle_topk.py): brute force on tiny inputs with ties, the
special case k = N (a stable descending sort), the prefix property in k, and
the checker `verify_topk` accepting the true answer and rejecting every single
corruption tried; for the BatchTopK forms, brute force on tiny tied inputs, a
hand example, the defining properties of the kept set and NumPy's `packbits`.
"""
from __future__ import annotations

import numpy as np


def order_key(x: np.ndarray) -> np.ndarray:
    """Unsigned integer key whose numeric order is the total order on values.

    float32 in -> uint32 out; uint16 (bf16 bit patterns) in -> uint16 out.
    A non-negative pattern gets its sign bit set; a negative pattern is
    complemented (so more negative values get smaller keys).
    """
    if x.dtype == np.float32:
        b = x.view(np.uint32)
        neg = (b >> np.uint32(31)).astype(bool)
        return np.where(neg, ~b, b | np.uint32(0x80000000)).astype(np.uint32)
    if x.dtype == np.uint16:
        neg = (x >> np.uint16(15)).astype(bool)
        return np.where(neg, ~x, x | np.uint16(0x8000)).astype(np.uint16)
    raise TypeError(f"order_key: unsupported dtype {x.dtype}")


def topk_row(x: np.ndarray, k: int) -> tuple[np.ndarray, np.ndarray]:
    """Top-k of one row by a full sort.  Returns (values[k], indices[k] int64).

    A stable ascending sort of the complemented key lists indices by value
    descending and, inside a run of equal values, by index ascending.
    """
    n = x.shape[0]
    if not (1 <= k <= n):
        raise ValueError("need 1 <= k <= N")
    inv = ~order_key(x)
    order = np.argsort(inv, kind="stable")[:k]
    return x[order].copy(), order.astype(np.int64)


def topk(x: np.ndarray, k: int) -> tuple[np.ndarray, np.ndarray]:
    """Row-wise top-k of a (rows, N) or (N,) array; see `topk_row`."""
    if x.ndim == 1:
        return topk_row(x, k)
    vals = np.empty((x.shape[0], k), dtype=x.dtype)
    idx = np.empty((x.shape[0], k), dtype=np.int64)
    for r in range(x.shape[0]):
        vals[r], idx[r] = topk_row(x[r], k)
    return vals, idx


def kept_mask(x: np.ndarray, k: int) -> np.ndarray:
    """BatchTopK's kept set as a boolean mask over the flattened input: entry i is True iff i is among the
    top-k of the flattened array (ties at the k-th value go to the lowest indices)."""
    flat = x.reshape(-1)
    _, idx = topk_row(flat, k)
    mask = np.zeros(flat.shape[0], dtype=bool)
    mask[idx] = True
    return mask


def kept_dense(x: np.ndarray, k: int) -> np.ndarray:
    """BatchTopK's result as a dense array: the kept entries bit for bit at their positions, +0.0 elsewhere
    (the all-zero bit pattern in either element type).  Same shape as x."""
    flat = x.reshape(-1)
    mask = kept_mask(flat, k)
    out = np.zeros_like(flat)
    out[mask] = flat[mask]
    return out.reshape(x.shape)


def pack_mask(mask: np.ndarray) -> np.ndarray:
    """Boolean mask -> uint32 words, bit (i % 32) of word (i // 32) = mask[i]; the last word is zero-padded."""
    n = mask.shape[0]
    words = np.zeros((n + 31) // 32, dtype=np.uint32)
    pos = np.flatnonzero(mask)
    np.bitwise_or.at(words, pos // 32, (np.uint32(1) << (pos % 32).astype(np.uint32)))
    return words


def topk_brute(x: np.ndarray, k: int) -> tuple[np.ndarray, np.ndarray]:
    """k rounds of arg-max with the lowest index winning ties.  Tiny inputs only."""
    keys = [int(v) for v in order_key(x)]
    taken = [False] * len(keys)
    out = []
    for _ in range(k):
        best = -1
        for i, key in enumerate(keys):
            if not taken[i] and (best < 0 or key > keys[best]):
                best = i
        taken[best] = True
        out.append(best)
    idx = np.asarray(out, dtype=np.int64)
    return x[idx].copy(), idx


def _first_positions(keys: np.ndarray, value, count: int, chunk: int = 1 << 24) -> np.ndarray:
    """The `count` lowest positions where keys == value (scanned chunk by chunk to bound memory)."""
    found: list[np.ndarray] = []
    have = 0
    for start in range(0, keys.shape[0], chunk):
        if have >= count:
            break
        hit = np.flatnonzero(keys[start:start + chunk] == value) + start
        found.append(hit[:count - have])
        have += found[-1].size
    return np.concatenate(found) if found else np.empty(0, dtype=np.int64)


def verify_topk(x: np.ndarray, k: int, vals: np.ndarray, idx: np.ndarray, keys: np.ndarray | None = None) -> list[str]:
    """Check a claimed top-k of one row against the definition in O(N).
    (`keys` = order_key(x), if the caller already has it.)

    The claimed answer equals the unique correct one iff all of these hold:
      1. idx are k distinct in-range indices and vals[j] is bitwise x[idx[j]];
      2. the list is ordered by (key descending, index ascending);
      3. every element whose key exceeds the k-th key is in the list
         (their number equals the number of listed keys above the k-th key);
      4. the listed elements that tie with the k-th key are the lowest-indexed
         elements of x with that key.
    Returns a list of violated conditions (empty = correct).
    """
    bad: list[str] = []
    n = x.shape[0]
    idx = np.asarray(idx)
    if idx.shape != (k,) or vals.shape != (k,):
        return ["shape"]
    if idx.min() < 0 or idx.max() >= n:
        return ["index out of range"]
    if np.unique(idx).size != k:
        bad.append("duplicate index")
    bits = np.uint32 if x.dtype == np.float32 else np.uint16
    if not np.array_equal(x[idx].view(bits), np.ascontiguousarray(vals).view(bits)):
        bad.append("value != x[index]")
    if keys is None:
        keys = order_key(x)
    lk = keys[idx].astype(np.int64)
    dk = np.diff(lk)
    di = np.diff(idx.astype(np.int64))
    if np.any(dk > 0) or np.any((dk == 0) & (di <= 0)):
        bad.append("order")
    kth = keys.dtype.type(lk[-1])
    above_all = int(np.count_nonzero(keys > kth))
    above_listed = int(np.count_nonzero(lk > int(kth)))
    if above_all != above_listed:
        bad.append("missing a larger element")
    n_tie = k - above_listed
    ties_expected = _first_positions(keys, kth, n_tie)
    ties_listed = np.sort(idx[lk == int(kth)])
    if not np.array_equal(ties_expected, ties_listed):
        bad.append("ties are not the lowest indices")
    return bad
