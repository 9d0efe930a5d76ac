"""Philox4x32-10 and the sample-index recipe.  TEST INFRASTRUCTURE ONLY.

Stage 1 of the method (Section 3, "Sampling") draws S indices uniformly without
replacement; the paper does not say how.  This build's reading, which the CUDA
path implements a second time on its own:

  * the index range [0, N) is cut into S disjoint strata
        [lo_j, hi_j) = [floor(j N / S), floor((j+1) N / S)),   j = 0 .. S-1;
  * stratum j contributes exactly one index, lo_j + floor(u_j (hi_j - lo_j) / 2^64),
    where u_j is a 64-bit word from the counter-based generator Philox4x32-10
    (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
    SC'11) with key = (seed low word, seed high word).  One generator block of
    four words serves two strata: block b has counter (b, row low word, row high
    word, 0); stratum 2b takes u = word0 + 2^32 word1, stratum 2b+1 takes
    u = word2 + 2^32 word3.

Indices are distinct by construction and every element of a stratum is equally
likely.  The random numbers are a function of (seed, row, j) only, so the two
implementations can be compared index for index.

Pins (tests/test_oracle_philox.py): the generator is compared word for word
with the Philox4x32-10 host generator of the cuRAND library (a CPU routine, no
GPU involved); the index recipe is checked for range, distinctness, one index
per stratum and uniformity inside a stratum.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_LO = np.uint64(0xFFFFFFFF)
_32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on arrays of counters; returns four uint32 arrays.

    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 as 64-bit products;
    the new counter is (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0).  The key is
    advanced by the Weyl constants (W0, W1) between rounds (nine times in all).
    """
    c0 = np.asarray(c0, dtype=np.uint64) & _LO
    c1 = np.broadcast_to(np.asarray(c1, dtype=np.uint64) & _LO, c0.shape)
    c2 = np.broadcast_to(np.asarray(c2, dtype=np.uint64) & _LO, c0.shape)
    c3 = np.broadcast_to(np.asarray(c3, dtype=np.uint64) & _LO, c0.shape)
    k0 &= 0xFFFFFFFF
    k1 &= 0xFFFFFFFF
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _W0) & 0xFFFFFFFF
            k1 = (k1 + _W1) & 0xFFFFFFFF
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _32, p0 & _LO
        hi1, lo1 = p1 >> _32, p1 & _LO
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
    return tuple(w.astype(np.uint32) for w in (c0, c1, c2, c3))


def stratum_bounds(N: int, S: int) -> tuple[np.ndarray, np.ndarray]:
    """lo_j = floor(j N / S) and hi_j = floor((j+1) N / S) as int64 arrays."""
    j = np.arange(S + 1, dtype=object) * N // S          # exact integers, any size
    b = np.asarray(j, dtype=np.int64)
    return b[:-1], b[1:]


def sample_indices(N: int, S: int, seed: int, row: int = 0) -> np.ndarray:
    """The S sample indices of one row (int64, ascending because strata are ordered)."""
    if not (1 <= S <= N):
        raise ValueError("need 1 <= S <= N")
    lo, hi = stratum_bounds(N, S)
    j = np.arange(S, dtype=np.uint64)
    b0, b1, b2, b3 = philox4x32_10(j >> np.uint64(1), row & 0xFFFFFFFF, (row >> 32) & 0xFFFFFFFF, 0,
                                   seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    odd = (j & np.uint64(1)).astype(bool)
    w0 = np.where(odd, b2, b0)
    w1 = np.where(odd, b3, b1)
    width = (hi - lo).astype(np.uint64)                   # < 2^32 always (N < 2^32)
    # floor(u * width / 2^64) with u = w0 + 2^32 w1, in 64-bit pieces:
    #   u * width = w1*width * 2^32 + w0*width
    t_lo = w0.astype(np.uint64) * width                   # < 2^64
    t_hi = w1.astype(np.uint64) * width                   # < 2^64
    off = (t_hi + (t_lo >> _32)) >> _32
    return lo + off.astype(np.int64)
