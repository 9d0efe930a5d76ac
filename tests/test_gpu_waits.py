"""Every wait inside the kernels is bounded.  These tests make two of them run out -- without hanging anything: the
barrier's poll limit is a few hundred polls, and nothing here faults -- and check what the caller then sees."""
import ctypes

import numpy as np
import pytest
import torch

import cuda_helpers
import paper_2608_12573_b200 as profk
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, workloads

pytestmark = pytest.mark.gpu

PROFK_ETIMEOUT = -4


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    profk.lib()
    cuda_helpers.lib()
    torch.cuda.set_device(0)


def bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def test_barrier_wait_that_runs_out_is_reported_and_the_next_call_is_exact():
    x = workloads.normal(4, 1 << 18, seed=31)
    xd = x.cuda()
    k = 50
    v, i = profk.topk(xd, k, eps=1e-3, seed=1)                             # registers a workspace
    torch.cuda.synchronize()
    ws = profk._workspaces[torch.cuda.current_device()]
    ctas = 24
    returned = torch.zeros(ctas, dtype=torch.int32, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    # a barrier that expects one CTA more than the grid has, 500 polls: every CTA gives up and returns
    rc = cuda_helpers.lib().profk_test_barrier_timeout(ctypes.c_void_p(ws.data_ptr()), ctypes.c_uint32(ctas), ctypes.c_uint32(ctas + 1),
                                                       ctypes.c_uint32(500), ctypes.c_void_p(returned.data_ptr()), stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert returned.cpu().tolist() == [1] * ctas                           # every CTA came back, each reporting "gave up"
    header = ws[:16].view(torch.int32).cpu().tolist()
    assert header[2] == 1                                                  # WsHeader.error
    arr = (profk._StatsStruct * 4)()
    rc = profk.lib().profk_read_stats(stream, ctypes.c_int64(4), arr)
    assert rc == PROFK_ETIMEOUT and profk.lib().profk_strerror(rc).decode() == "device-side wait timed out"
    assert all(s.status & 0x80000000 for s in arr)
    with pytest.raises(profk.ProfkError):
        profk.read_stats(4)
    # the next ordinary call resets the barrier words and the flag, and is exact
    v, i = profk.topk(xd, k, eps=1e-3, seed=2)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(workloads.as_numpy(x), k)
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(v.cpu().numpy()), bits(ov))
    assert all(s[3] == profk.ROW_OK for s in profk.read_stats(4))
    # ... also one that uses the grid barrier itself (forced overflow in every row of a batch: the grid-wide exact selection)
    xb = workloads.normal(24, 1 << 16, seed=32)
    v, i = profk.topk(xb.cuda(), k, plan_override=profk.Plan(m=2048, r=30, capacity=k, k_accept=k, mode=0), seed=3)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(workloads.as_numpy(xb), k)
    assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(v.cpu().numpy()), bits(ov))
    assert all(s[3] == profk.ROW_OVERFLOW for s in profk.read_stats(24))


def test_filter_gives_up_on_its_prefetched_tiles_and_reads_them_again():
    """With zero polls allowed, every CTA of the single-row scan abandons the tiles it copied into shared memory
    during the wait for the threshold and reads them with plain loads; the result is the same."""
    x = workloads.normal(1, 1 << 24, seed=33)[0]
    xd = x.cuda()
    ov, oi = o_topk.topk_row(workloads.as_numpy(x), 256)
    try:
        for polls in (0, 1, -1):
            assert profk.lib().profk_debug_set_prefetch_wait_polls(ctypes.c_int64(polls)) == 0
            for seed in (0, 1):
                v, i = profk.topk(xd, 256, eps=1e-4, seed=seed)
                torch.cuda.synchronize()
                assert np.array_equal(i.cpu().numpy(), oi) and np.array_equal(bits(v.cpu().numpy()), bits(ov)), (polls, seed)
                assert profk.read_stats(1)[0][3] == profk.ROW_OK
    finally:
        profk.lib().profk_debug_set_prefetch_wait_polls(ctypes.c_int64(-1))
