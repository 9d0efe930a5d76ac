"""Pins for oracle.topk: the definition of top-k (Section 3) with the tie rule
"value descending, then index ascending"."""
import numpy as np
import pytest

from oracle import topk


def _cases():
    rng = np.random.default_rng(11)
    yield np.zeros(9, np.float32)                                     # all equal
    yield np.array([1, 0, 1, 0, 0, 1, 1], np.float32)                 # two values
    yield np.array([3, 3, 2, 5, 5, 5, -1, 2, 3, 0], np.float32)
    for n in (1, 2, 7, 16, 33):
        yield rng.integers(-3, 4, n).astype(np.float32)               # many ties
        yield rng.standard_normal(n).astype(np.float32)               # distinct values
    yield np.array([0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, 0.0, -0.0], np.float32)


@pytest.mark.parametrize("x", list(_cases()), ids=lambda a: f"n{a.size}")
def test_full_sort_equals_brute_force_for_every_k(x):
    for k in range(1, x.size + 1):
        v, i = topk.topk_row(x, k)
        bv, bi = topk.topk_brute(x, k)
        assert np.array_equal(i, bi)
        assert np.array_equal(v.view(np.uint32), bv.view(np.uint32))


def test_k_equals_n_is_a_stable_descending_sort():
    rng = np.random.default_rng(5)
    x = rng.integers(0, 50, 2000).astype(np.float32)
    v, i = topk.topk_row(x, x.size)
    assert np.array_equal(v, np.sort(x)[::-1])                        # textbook: descending sort
    same = v[1:] == v[:-1]
    assert np.all(i[1:][same] > i[:-1][same])                         # ties by ascending index
    assert np.array_equal(np.sort(i), np.arange(x.size))


def test_prefix_property_and_hand_example():
    x = np.array([0.5, 2.0, 2.0, -1.0, 7.0, 2.0, 0.5], np.float32)
    v, i = topk.topk_row(x, 5)
    assert i.tolist() == [4, 1, 2, 5, 0]                              # worked by hand
    assert v.tolist() == [7.0, 2.0, 2.0, 2.0, 0.5]
    rng = np.random.default_rng(2)
    y = rng.integers(0, 9, 500).astype(np.float32)
    v9, i9 = topk.topk_row(y, 90)
    for k in (1, 17, 89):
        vk, ik = topk.topk_row(y, k)
        assert np.array_equal(ik, i9[:k]) and np.array_equal(vk, v9[:k])


def test_total_order_on_special_values():
    nan = np.float32(np.nan)
    neg_nan = np.array([0xFFC00000], np.uint32).view(np.float32)[0]
    x = np.array([1.0, -0.0, 0.0, nan, -np.inf, neg_nan, np.inf, -2.0], np.float32)
    _, i = topk.topk_row(x, x.size)
    # +NaN > +inf > 1 > +0 > -0 > -2 > -inf > -NaN
    assert i.tolist() == [3, 6, 0, 2, 1, 7, 4, 5]
    keys = topk.order_key(np.array([-1.5, -1.0, -0.0, 0.0, 1e-40, 1.0, 1.5], np.float32))
    assert np.all(np.diff(keys.astype(np.int64)) > 0)                 # key order == numeric order


def test_bf16_bit_patterns():
    # bf16 = upper half of the fp32 pattern: 1.0 = 0x3F80, 2.0 = 0x4000, -1.0 = 0xBF80, 0.5 = 0x3F00
    x = np.array([0x3F80, 0x4000, 0xBF80, 0x3F00, 0x4000, 0x0000], np.uint16)
    v, i = topk.topk_row(x, 4)
    assert i.tolist() == [1, 4, 0, 3]
    assert v.tolist() == [0x4000, 0x4000, 0x3F80, 0x3F00]
    f = np.random.default_rng(3).standard_normal(300).astype(np.float32)
    b = (f.view(np.uint32) >> 16).astype(np.uint16)                   # truncate to bf16
    _, ib = topk.topk_row(b, 300)
    wide = (b.astype(np.uint32) << 16).view(np.float32)
    _, iw = topk.topk_row(wide, 300)
    assert np.array_equal(ib, iw)                                     # same order as the widened floats


def test_batched_rows_are_independent():
    rng = np.random.default_rng(9)
    x = rng.integers(0, 20, (5, 64)).astype(np.float32)
    v, i = topk.topk(x, 7)
    for r in range(5):
        vr, ir = topk.topk_brute(x[r], 7)
        assert np.array_equal(i[r], ir) and np.array_equal(v[r], vr)


def test_checker_accepts_truth_and_rejects_corruptions():
    rng = np.random.default_rng(4)
    x = rng.integers(0, 12, 400).astype(np.float32)                   # heavy ties at the boundary
    for k in (1, 5, 40, 399, 400):
        v, i = topk.topk_row(x, k)
        assert topk.verify_topk(x, k, v, i) == []
    k = 40
    v, i = topk.topk_row(x, k)
    kth = v[-1]
    ties = np.flatnonzero(x == kth)
    assert ties.size > int(np.count_nonzero(v == kth)), "test needs unused ties"
    # a later tie instead of the lowest-indexed one
    i2 = i.copy(); i2[-1] = ties[-1]
    assert "ties are not the lowest indices" in topk.verify_topk(x, k, x[i2], i2)
    # swapped order
    i3 = i.copy(); i3[[0, 1]] = i3[[1, 0]]
    assert "order" in topk.verify_topk(x, k, x[i3], i3)
    # a smaller element in place of a top one
    i4 = i.copy(); i4[0] = int(np.argmin(x)); o = np.lexsort((i4, -x[i4])); i4 = i4[o]
    assert topk.verify_topk(x, k, x[i4], i4) != []
    # value not matching the index
    v5 = v.copy(); v5[3] += 1
    assert "value != x[index]" in topk.verify_topk(x, k, v5, i)
    # duplicate index
    i6 = i.copy(); i6[1] = i6[0]
    assert topk.verify_topk(x, k, x[i6], i6) != []


# ----------------------------------------------------------------------------- BatchTopK forms (Section 5, "Application")
def test_kept_set_equals_brute_force_on_tiny_tied_inputs():
    rng = np.random.default_rng(11)
    for n in (1, 2, 7, 33, 64):
        for trial in range(6):
            x = rng.integers(0, 4, size=n).astype(np.float32)           # heavy ties
            if trial == 0:
                x[:] = 2.0                                               # all equal: the kept set is the first k indices
            for k in sorted({1, n // 2 or 1, n}):
                mask = topk.kept_mask(x, k)
                _, bi = topk.topk_brute(x, k)
                want = np.zeros(n, dtype=bool)
                want[bi] = True
                assert np.array_equal(mask, want), (n, trial, k)
                if trial == 0:
                    assert np.array_equal(np.flatnonzero(mask), np.arange(k))
                # the defining properties: k kept; no dropped entry beats a kept one; ties at the k-th value go to the lowest indices
                keys = topk.order_key(x).astype(np.int64)
                assert mask.sum() == k
                if k < n:
                    kth = keys[mask].min()
                    assert keys[~mask].max() <= kth
                    tied = np.flatnonzero(keys == kth)
                    n_tied_kept = int(mask[tied].sum())
                    assert np.array_equal(tied[:n_tied_kept], tied[mask[tied]])


def test_kept_dense_and_packed_mask():
    x = np.array([[0.5, -1.0, 3.0, 0.5], [0.5, 2.0, -0.0, 0.5]], dtype=np.float32)       # a 2 x 4 "activation matrix"
    dense = topk.kept_dense(x, 4)                                       # top 4 of the 8 flattened entries: 3.0, 2.0, then the two first 0.5
    assert dense.shape == x.shape
    assert np.array_equal(dense, np.array([[0.5, 0.0, 3.0, 0.5], [0.0, 2.0, 0.0, 0.0]], dtype=np.float32))
    assert not np.signbit(dense).any()                                  # dropped entries are +0.0, also where the input held -0.0
    mask = topk.kept_mask(x, 4)
    assert np.flatnonzero(mask).tolist() == [0, 2, 3, 5]
    assert topk.pack_mask(mask).tolist() == [0b101101]
    # bf16 bit patterns: zero is the all-zero pattern there too
    xb = np.array([0x3F80, 0x4000, 0xBF80, 0x3F80], dtype=np.uint16)    # 1, 2, -1, 1
    assert topk.kept_dense(xb, 2).tolist() == [0x3F80, 0x4000, 0, 0]
    # packing against NumPy's own bit packing (little-endian bit order inside little-endian words)
    rng = np.random.default_rng(12)
    for n in (1, 31, 32, 33, 1000):
        m = rng.random(n) < 0.3
        padded = np.zeros((n + 31) // 32 * 32, dtype=bool)
        padded[:n] = m
        assert np.array_equal(topk.pack_mask(m), np.packbits(padded, bitorder="little").view("<u4"))
