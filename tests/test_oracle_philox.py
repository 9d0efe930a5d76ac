"""Pins for oracle.philox: the generator against cuRAND's CPU ("host") Philox4x32-10
generator, and the properties of the stratified index recipe."""
import ctypes
import ctypes.util
import glob

import numpy as np
import pytest

from oracle import philox

_CURAND_PHILOX = 161        # curandRngType_t: CURAND_RNG_PHILOX4_32_10
_HOST_LANES = 65536         # the host generator interleaves this many subsequences


def _load_curand():
    names = [ctypes.util.find_library("curand")] + sorted(glob.glob("/usr/local/cuda*/targets/*/lib/libcurand.so.*")) \
        + sorted(glob.glob("/usr/local/cuda*/lib64/libcurand.so.*"))
    for n in names:
        if n:
            try:
                return ctypes.CDLL(n)
            except OSError:
                pass
    return None


def _curand_host(lib, seed, offset, n):
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), _CURAND_PHILOX) == 0
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    out = np.zeros(n, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n)) == 0
    lib.curandDestroyGenerator(gen)
    return out


def test_generator_matches_curand_host_philox():
    lib = _load_curand()
    if lib is None:
        pytest.skip("libcurand not found")
    # cuRAND's host generator emits 4 words per counter; output quad q comes from
    # counter (q // 65536 as a 64-bit value in words 0-1, q % 65536 in word 2, 0) and key = seed.
    for seed in (0, 1, 0x123456789ABCDEF, 0xFEDCBA9876543210):
        k0, k1 = seed & 0xFFFFFFFF, seed >> 32
        got = _curand_host(lib, seed, 0, 4 * 3000).reshape(-1, 4)
        ours = np.stack(philox.philox4x32_10(np.zeros(3000, np.uint64), 0, np.arange(3000), 0, k0, k1), 1)
        assert np.array_equal(got, ours)
        for c0, c1, c2 in [(1, 0, 0), (3, 5, 7), (0xFFFFFFFF, 0x3FFF, 1), (123456789, 9, 65535)]:
            offset = (((c1 << 32) + c0) * _HOST_LANES + c2) * 4
            got = _curand_host(lib, seed, offset, 4)
            ours = np.array([w[0] for w in philox.philox4x32_10(np.array([c0]), c1, c2, 0, k0, k1)])
            assert np.array_equal(got, ours), (seed, c0, c1, c2)


def test_counter_words_all_matter():
    base = philox.philox4x32_10(np.array([5]), 6, 7, 8, 9, 10)
    for args in [(4, 6, 7, 8, 9, 10), (5, 0, 7, 8, 9, 10), (5, 6, 0, 8, 9, 10), (5, 6, 7, 0, 9, 10), (5, 6, 7, 8, 0, 10),
                 (5, 6, 7, 8, 9, 0)]:
        other = philox.philox4x32_10(np.array([args[0]]), *args[1:])
        assert all(int(a[0]) != int(b[0]) for a, b in zip(base, other))


@pytest.mark.parametrize("N,S", [(1 << 20, 32768), (1_000_003, 4096), (100, 100), (101, 7), (2 ** 32 - 1, 1 << 17)])
def test_one_distinct_index_per_stratum(N, S):
    lo, hi = philox.stratum_bounds(N, S)
    assert lo[0] == 0 and hi[-1] == N and np.array_equal(lo[1:], hi[:-1])          # strata tile [0, N)
    w = hi - lo
    assert w.min() == N // S and w.max() == -(-N // S)
    idx = philox.sample_indices(N, S, seed=42, row=3)
    assert idx.dtype == np.int64 and idx.shape == (S,)
    assert np.all(idx >= lo) and np.all(idx < hi)
    assert np.unique(idx).size == S
    again = philox.sample_indices(N, S, seed=42, row=3)
    assert np.array_equal(idx, again)
    assert not np.array_equal(idx, philox.sample_indices(N, S, seed=43, row=3)) or N == S
    assert not np.array_equal(idx, philox.sample_indices(N, S, seed=42, row=4)) or N == S


def test_offsets_are_uniform_inside_a_stratum():
    N, S = 1 << 22, 1 << 16                       # strata of exactly 64 elements
    counts = np.zeros(64, dtype=np.int64)
    for seed in range(8):
        idx = philox.sample_indices(N, S, seed)
        counts += np.bincount(idx % 64, minlength=64)
    expected = counts.sum() / 64
    chi2 = float(((counts - expected) ** 2 / expected).sum())
    assert chi2 < 120.0                           # 63 degrees of freedom; 120 is beyond the 1e-5 tail
    # 64-bit scaling: the offset is floor(u * width / 2^64), so width 3 with extreme words gives 0 and 2
    assert philox.sample_indices(3, 1, 0).item() in (0, 1, 2)
