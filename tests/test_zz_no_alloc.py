"""The allocation-free entry point.  This file sorts last on purpose: if it fails, a run that stops at
the first failure has already run every other test.

`profk_topk_noalloc_f32` serves callers that cannot call cudaMalloc (or any allocator) at the moment
they need a top-k -- code inside an allocator callback, a plug-in that was handed all its buffers up
front, a process whose device memory already belongs to another pool.  Its scratch is a fixed array
inside the library, so the test checks three things through the C ABI: that it returns exactly what
the ordinary entry point returns (and what the CPU oracle's full sort returns), that it still does so
on a second call in a row (the array then holds the first call's leftovers), and that it refuses
shapes that do not fit instead of overrunning.  The shapes reach every layout the scratch can take:
a few rows (the refine kernel's clusters and their exact-selection scratch), a batch of more than 18
rows (the per-CTA scratch of the grid-wide exact selection), and a selection beyond 8192 (bins,
partitioned append counters and a doubled row pitch).
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, workloads

pytestmark = pytest.mark.gpu


def _call(fn, x, k, eps, seed, vals, idx):
    rows, n = x.shape
    return fn(ctypes.c_void_p(x.data_ptr()), ctypes.c_int64(rows), ctypes.c_int64(n), ctypes.c_int64(k),
              ctypes.c_double(eps), ctypes.c_double(1.0), ctypes.c_uint64(seed),
              ctypes.c_void_p(torch.cuda.current_stream().cuda_stream),
              ctypes.c_void_p(vals.data_ptr()), ctypes.c_void_p(idx.data_ptr()))


def test_noalloc_entry_matches_the_ordinary_one_twice_in_a_row():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    lib = profk.lib()
    torch.cuda.set_device(0)
    shapes = [(1, 1 << 22, 100), (6, 300_001, 17), (64, 1 << 18, 32), (1, 1 << 22, 10_000), (2, 1 << 20, 9_000)]
    for rows, n, k in shapes:
        xs = [workloads.normal(rows, n, seed=40 + r).cuda() for r in range(2)]      # two different inputs, two calls in a row
        # reference: the existing entry point, with a registered workspace
        pl = profk.plan(n, k, 1e-3, rows=rows)
        profk.ensure_workspace(rows, pl.capacity, k, xs[0].device)
        want = []
        for r, x in enumerate(xs):
            v = torch.empty((rows, k), dtype=torch.float32, device="cuda")
            i = torch.empty((rows, k), dtype=torch.int64, device="cuda")
            assert _call(lib.profk_topk_f32, x, k, 1e-3, 7 + r, v, i) == 0
            want.append((v, i))
        torch.cuda.synchronize()
        # the new entry point: outputs allocated here, by the caller, before the calls
        got = [(torch.full((rows, k), float("nan"), device="cuda"), torch.full((rows, k), -7, dtype=torch.int64, device="cuda"))
               for _ in xs]
        for r, x in enumerate(xs):
            assert _call(lib.profk_topk_noalloc_f32, x, k, 1e-3, 7 + r, got[r][0], got[r][1]) == 0
        torch.cuda.synchronize()
        for x, (wv, wi), (gv, gi) in zip(xs, want, got):
            assert torch.equal(wi, gi)                                              # integer work: bit-exact
            assert torch.equal(wv.view(torch.int32), gv.view(torch.int32))          # values bit for bit as well
            ov, oi = o_topk.topk(x.cpu().numpy(), k)                                # and both equal the oracle's full sort
            assert np.array_equal(gi.cpu().numpy(), oi)
            assert np.array_equal(gv.cpu().numpy().view(np.uint32), ov.view(np.uint32))


def test_noalloc_entry_refuses_what_does_not_fit():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    lib = profk.lib()
    torch.cuda.set_device(0)
    x = torch.zeros((8, 1 << 20), device="cuda")
    k = 65536                                            # 8 rows x (2 x 131072 records + bins) is far beyond 16 MiB
    v = torch.zeros((8, k), device="cuda")
    i = torch.zeros((8, k), dtype=torch.int64, device="cuda")
    code = _call(lib.profk_topk_noalloc_f32, x, k, 1e-3, 0, v, i)
    assert code == -5 and b"too large" in lib.profk_strerror(code)
    torch.cuda.synchronize()
    assert int(i.abs().sum()) == 0                       # nothing was launched
