"""Stream order is all a caller relies on: the call's input may be produced on the stream just before the call, by a
kernel that releases its programmatic dependents before it has written anything -- a GEMM epilogue with programmatic
launch feeding the flattened BatchTopK of Section 5, or this library's own last kernel when one call's output is the
next call's input.  The filtering scan of Section 3 reads x; it must be the caller's x."""
import ctypes

import numpy as np
import pytest
import torch

import cuda_helpers
import paper_2608_12573_b200 as profk
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    profk.lib()
    cuda_helpers.lib()
    torch.cuda.set_device(0)


def bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


@pytest.mark.parametrize("n,k", [(1 << 22, 64), (1 << 24, 1000), (3_000_001, 32)])
def test_producer_that_releases_its_dependents_before_it_writes(n, k):
    """Six rounds with no synchronisation in between: a hand-written producer triggers its dependents on entry, idles
    ~100 us (bounded), then copies a fresh snapshot into the call's input buffer, which still holds the previous
    snapshot (the first time: a ramp whose top-k is the end of the buffer)."""
    helpers = cuda_helpers.lib()
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    snaps = [workloads.normal(1, n, seed=900 + j)[0] for j in range(6)]
    dsnaps = [s.cuda() for s in snaps]
    x = torch.arange(n, dtype=torch.float32, device="cuda")               # stale contents
    outs = [(torch.empty((1, k), dtype=torch.float32, device="cuda"), torch.empty((1, k), dtype=torch.int64, device="cuda"))
            for _ in range(6)]
    profk.topk(x, k, eps=1e-3, seed=0)                                     # first use of the shape: attributes, workspace
    torch.cuda.synchronize()
    for j in range(6):
        rc = helpers.profk_test_early_trigger_copy_f32(ctypes.c_void_p(dsnaps[j].data_ptr()), ctypes.c_void_p(x.data_ptr()),
                                                       ctypes.c_int64(n), ctypes.c_int64(200_000), stream)
        assert rc == 0
        profk.topk(x, k, eps=1e-3, seed=j, out=outs[j])
    torch.cuda.synchronize()
    for j in range(6):
        ov, oi = o_topk.topk_row(workloads.as_numpy(snaps[j]), k)
        assert np.array_equal(outs[j][1][0].cpu().numpy(), oi), f"round {j}: indices differ from the oracle"
        assert np.array_equal(bits(outs[j][0][0].cpu().numpy()), bits(ov)), f"round {j}: values differ from the oracle"


@pytest.mark.parametrize("rows,n,k1,k2", [(1, 1 << 24, 1 << 18, 32),       # call 1 ends with the grid-wide large-k refine
                                          (8, 1 << 20, 16384, 64),         # ... with the cluster refine
                                          (32, 1 << 18, 4096, 100)])       # ... with the exact-selection kernel behind the refine
def test_one_calls_output_is_the_next_calls_input(rows, n, k1, k2):
    """Call 2 selects from call 1's values (rows x k1 read as one row), enqueued right behind it.  The library's last
    kernels release their dependents at their top, so call 2's kernels are on the GPU while call 1 still writes."""
    for trial in range(3):
        x = workloads.normal(rows, n, seed=950 + trial)
        xd = x.cuda()
        mid_v = torch.arange(rows * k1, dtype=torch.float32, device="cuda").view(rows, k1)      # stale contents: a ramp
        mid_i = torch.empty((rows, k1), dtype=torch.int64, device="cuda")
        pl1 = profk.plan(n, k1, 1e-3, rows=rows)
        pl2 = profk.plan(rows * k1, k2, 1e-3)
        assert pl2.mode == 0
        big = max((pl1, rows, k1), (pl2, 1, k2), key=lambda t: profk.workspace_bytes(t[1], t[0].capacity, t[2]))
        profk.ensure_workspace(big[1], big[0].capacity, big[2], xd.device)      # one workspace that serves both calls
        torch.cuda.synchronize()
        profk.topk(xd, k1, eps=1e-3, seed=trial, out=(mid_v, mid_i))
        v2, i2 = profk.topk(mid_v.view(-1), k2, eps=1e-3, seed=trial)
        torch.cuda.synchronize()
        ov1, _ = o_topk.topk(workloads.as_numpy(x), k1)
        assert np.array_equal(bits(mid_v.cpu().numpy()), bits(ov1))
        ov2, oi2 = o_topk.topk_row(ov1.reshape(-1), k2)
        assert np.array_equal(i2.cpu().numpy(), oi2) and np.array_equal(bits(v2.cpu().numpy()), bits(ov2)), trial
