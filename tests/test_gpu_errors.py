"""Error behaviour of the C ABI on a GPU: bad arguments and a missing or short workspace are refused with the
documented codes before anything is launched, and the library works normally afterwards."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, workloads

pytestmark = pytest.mark.gpu

EINVAL, EWORKSPACE = -1, -2


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    profk.lib()
    torch.cuda.set_device(0)


def _raw_topk(x, rows, n, k, vals, idx, eps=1e-3, recall=1.0):
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return profk.lib().profk_topk_f32(ctypes.c_void_p(x.data_ptr() if x is not None else None), ctypes.c_int64(rows),
                                      ctypes.c_int64(n), ctypes.c_int64(k), ctypes.c_double(eps), ctypes.c_double(recall),
                                      ctypes.c_uint64(0), st, ctypes.c_void_p(vals.data_ptr()), ctypes.c_void_p(idx.data_ptr()))


def test_bad_arguments_are_refused_and_nothing_is_launched():
    n, k = 1 << 20, 32
    x = torch.randn(n, device="cuda")
    vals = torch.full((k,), 7.0, device="cuda")
    idx = torch.full((k,), -7, dtype=torch.int64, device="cuda")
    profk.topk(x, k)                                             # registers a workspace for this shape
    assert _raw_topk(x, 1, n, n + 1, vals, idx) == EINVAL        # k > N
    assert _raw_topk(x, 1, n, 0, vals, idx) == EINVAL            # k < 1
    assert _raw_topk(x, 0, n, k, vals, idx) == EINVAL            # no rows
    assert _raw_topk(x, 1, 0, k, vals, idx) == EINVAL            # empty row
    assert _raw_topk(None, 1, n, k, vals, idx) == EINVAL         # null input
    assert _raw_topk(x, 1, n, k, vals, idx, eps=0.0) == EINVAL   # eps outside (0, 1)
    assert _raw_topk(x, 1, n, k, vals, idx, recall=1.5) == EINVAL
    torch.cuda.synchronize()
    assert profk.last_launch_count() == 0
    assert torch.all(vals == 7.0) and torch.all(idx == -7)       # outputs untouched
    assert b"invalid" in profk.lib().profk_strerror(EINVAL).lower()


def test_plan_that_does_not_fit_the_call_is_refused():
    x = workloads.normal(1, 200_000, seed=31)[0].cuda()
    with pytest.raises(profk.ProfkError):
        profk.topk(x, 64, plan_override=profk.Plan(m=4096, r=40, capacity=32, k_accept=64, mode=0))      # capacity < k
    with pytest.raises(profk.ProfkError):
        profk.topk(x, 64, plan_override=profk.Plan(m=4096, r=5000, capacity=4096, k_accept=64, mode=0))  # rank beyond the sample
    with pytest.raises(profk.ProfkError):
        profk.topk(x, 64, plan_override=profk.Plan(m=4096, r=40, capacity=4096, k_accept=65, mode=0))    # accepts more than k


def test_missing_or_short_workspace_is_reported_and_recoverable():
    n, k = 300_000, 50
    x = workloads.normal(1, n, seed=32)[0]
    xg = x.cuda()
    v, i = profk.topk(xg, k)                                     # a good call first
    torch.cuda.synchronize()
    vals = torch.empty((k,), device="cuda")
    idx = torch.empty((k,), dtype=torch.int64, device="cuda")
    lib = profk.lib()
    small = torch.empty(4096, dtype=torch.uint8, device="cuda")
    try:
        assert lib.profk_set_workspace(ctypes.c_void_p(small.data_ptr()), ctypes.c_size_t(small.numel())) == 0
        assert _raw_topk(xg, 1, n, k, vals, idx) == EWORKSPACE
        assert lib.profk_set_workspace(ctypes.c_void_p(None), ctypes.c_size_t(0)) == 0
        assert _raw_topk(xg, 1, n, k, vals, idx) == EWORKSPACE
    finally:
        profk._workspaces.clear()                                # make the binding register a fresh one
        profk._workspace_ok.clear()
    v, i = profk.topk(xg, k)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(workloads.as_numpy(x), k)
    assert np.array_equal(i.cpu().numpy(), oi)
    assert np.array_equal(workloads.as_numpy(v).view(np.uint32), ov.view(np.uint32))
