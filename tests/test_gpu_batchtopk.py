"""Flattened BatchTopK (Section 5, "Application"): the kept set in its three forms -- unordered (value, index) pairs, a
bit mask, a dense array -- against the oracle's kept set, bit for bit; compared as a set where the order is free."""
import numpy as np
import pytest
import torch

import paper_2608_12573_b200 as profk
from oracle import topk as o_topk
from paper_2608_12573_b200 import _build, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    _build.build()
    profk.lib()
    torch.cuda.set_device(0)


def bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def check_forms(xn, k, out, mask_want=None):
    """All forms present in `out` against the oracle's kept set of the flattened host array xn."""
    flat = xn.reshape(-1)
    if mask_want is None:
        mask_want = o_topk.kept_mask(flat, k)
    if "indices" in out:
        idx = out["indices"].cpu().numpy()
        vals = workloads.as_numpy(out["values"])
        assert np.unique(idx).size == k and idx.min() >= 0 and idx.max() < flat.shape[0]
        assert np.array_equal(np.sort(idx), np.flatnonzero(mask_want)), "kept indices differ from the oracle's set"
        assert np.array_equal(bits(vals), bits(flat[idx])), "a value is not the input's entry at its index"
    if "mask" in out:
        words = out["mask"].cpu().numpy().view(np.uint32)
        assert np.array_equal(words, o_topk.pack_mask(mask_want)), "bit mask differs from the oracle's"
    if "dense" in out:
        dense = workloads.as_numpy(out["dense"]).reshape(-1)
        want = np.zeros_like(flat)
        want[mask_want] = flat[mask_want]
        assert np.array_equal(bits(dense), bits(want)), "dense result differs from the oracle's"


def run(xd, k, **kw):
    out = profk.batchtopk(xd, k, **kw)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n,k", [(1 << 22, 4096), (3_000_001, 20_000), (1 << 24, 131_072), (1 << 20, 1), (1 << 21, 17)])
def test_all_forms_on_relu_activations(dtype, n, k):
    x = workloads.relu_gaussian(n, seed=60 + (k % 7), dtype=dtype)           # many exact zeros, ties among bf16 values
    xn = workloads.as_numpy(x)
    want = o_topk.kept_mask(xn, k)
    xd = x.cuda()
    for seed in (0, 1):
        out = run(xd, k, eps=1e-3, seed=seed, want_pairs=True, want_mask=True, want_dense=True)
        check_forms(xn, k, out, want)
        assert profk.read_stats(1)[0][3] == profk.ROW_OK
    # each form alone, and the in-place dense form
    check_forms(xn, k, run(xd, k, seed=2, want_pairs=True), want)
    check_forms(xn, k, run(xd, k, seed=2, want_pairs=False, want_mask=True), want)
    xc = xd.clone()
    out = run(xc, k, seed=3, want_pairs=False, in_place=True)
    assert out["dense"].data_ptr() == xc.data_ptr()
    check_forms(xn, k, out, want)


def test_a_token_by_latent_matrix_and_an_unaligned_view():
    x = workloads.relu_gaussian(64 * 8192, seed=61, dtype=torch.float32).view(64, 8192)      # 64 tokens x 8192 latents, k = 32 per token
    xn = workloads.as_numpy(x)
    out = run(x.cuda(), 64 * 32, want_pairs=True, want_mask=True, want_dense=True)
    assert out["dense"].shape == (64, 8192)
    check_forms(xn, 64 * 32, out)
    big = workloads.normal(1, 1_000_003 + 8, seed=62)[0].cuda()
    for off in (1, 3):                                                       # input and dense output start off a 16-byte boundary
        v = big[off: off + 1_000_003].clone()
        host = v.cpu().numpy()
        scratch = torch.empty(1_000_003 + 8, device="cuda")
        w = scratch[off: off + 1_000_003]
        w.copy_(v)                                                           # w starts 4 * off bytes after a 16-byte boundary
        assert w.data_ptr() % 16 != 0
        out = run(w, 5000, want_pairs=True, want_mask=True, in_place=True)
        check_forms(host, 5000, out)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_heavy_ties_go_through_the_deeper_levels_of_the_select(dtype):
    """Rows whose K-th value is shared by thousands of entries: the boundary class of the logarithmic level is crowded
    and the linear levels separate its records by index; the kept copies are the lowest-indexed ones."""
    n, k = 1 << 22, 50_000
    cases = {"constant": torch.full((n,), 1.5), "few values": workloads.few_values(n, seed=63, distinct=16),
             "relu, coarse": workloads.relu_gaussian(n, seed=64, dtype=torch.bfloat16).float()}
    for name, x in cases.items():
        x = x.to(dtype)
        xn = workloads.as_numpy(x)
        want = o_topk.kept_mask(xn, k)
        for rule in (profk.TIES_BY_INDEX, profk.TIES_KEEP_ALL):
            pl = profk.plan(n, k, 1e-3)
            pl = profk.Plan(m=pl.m, r=pl.r, capacity=pl.capacity, k_accept=k, mode=pl.mode, tie_rule=rule)
            out = run(x.cuda(), k, plan_override=pl, seed=4, want_pairs=True, want_mask=True, want_dense=True)
            check_forms(xn, k, out, want)
            status = profk.read_stats(1)[0][3]
            assert status == profk.ROW_OK if rule == profk.TIES_BY_INDEX or name == "relu, coarse" else status in (profk.ROW_OK, profk.ROW_OVERFLOW), (name, rule)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_forced_overflow_recall_failure_and_direct_mode(dtype):
    n, k = 2_000_000, 3000
    x = workloads.normal(1, n, seed=65, dtype=dtype)[0]
    xn = workloads.as_numpy(x)
    want = o_topk.kept_mask(xn, k)
    xd = x.cuda()
    for plan, status in ((profk.Plan(m=4096, r=40, capacity=k, k_accept=k, mode=0), profk.ROW_OVERFLOW),
                         (profk.Plan(m=65536, r=1, capacity=20_000, k_accept=k, mode=0), profk.ROW_RECALL),
                         (profk.Plan(m=0, r=0, capacity=k, k_accept=k, mode=1), profk.ROW_DIRECT)):
        out = run(xd, k, plan_override=plan, seed=5, want_pairs=True, want_mask=True, want_dense=True)
        check_forms(xn, k, out, want)
        assert profk.read_stats(1)[0][3] == status
    xc = xd.clone()                                                          # in place with the exact selection re-reading the input
    out = run(xc, k, plan_override=profk.Plan(m=4096, r=40, capacity=k, k_accept=k, mode=0), seed=6, want_pairs=True, in_place=True)
    check_forms(xn, k, out, want)


def test_special_values_and_k_equal_n():
    x = workloads.normal(1, 1 << 20, seed=66)[0]
    x[::1000] = float("nan")
    x[1::1000] = -float("nan")
    x[2::1000] = float("inf")
    x[3::5000] = -0.0
    x[4::5000] = 0.0
    xn = workloads.as_numpy(x)
    for k in (100, 3000, 1 << 19):
        check_forms(xn, k, run(x.cuda(), k, want_pairs=True, want_mask=True, want_dense=True))
    small = workloads.normal(1, 5000, seed=67)[0]
    check_forms(workloads.as_numpy(small), 5000, run(small.cuda(), 5000, want_pairs=True, want_mask=True, want_dense=True))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_the_papers_sae_shape(dtype):
    """N = 4096 x 12288 = 50,331,648 activations, K = 4096 x 32 = 131,072 (Section 5, "Application")."""
    n, k = 50_331_648, 131_072
    x = workloads.relu_gaussian(n, seed=3, dtype=dtype)
    xn = workloads.as_numpy(x)
    want = o_topk.kept_mask(xn, k)
    xd = x.cuda().view(4096, 12288)
    for seed in (0, 1):
        out = run(xd, k, eps=1e-3, seed=seed, want_pairs=True, want_mask=True, want_dense=True)
        check_forms(xn, k, out, want)
    assert profk.read_stats(1)[0][3] == profk.ROW_OK
    assert profk.last_launch_count() == 4                                    # gather, threshold, filter, select + emit


def test_config4_flattened_2p29_bf16():
    n, k = 1 << 29, 32 * 4096
    x = workloads.relu_gaussian(n, seed=3)
    xn = workloads.as_numpy(x)
    keys = o_topk.order_key(xn)
    xd = x.cuda()
    del x
    out = run(xd, k, eps=1e-3, seed=0, want_pairs=True, want_mask=True, want_dense=False)
    idx = out["indices"].cpu().numpy()
    vals = workloads.as_numpy(out["values"])
    # the pairs, put in the order of the definition, must pass the oracle's O(N) checker of a claimed top-k ...
    order = np.lexsort((idx, ~o_topk.order_key(vals)))
    assert o_topk.verify_topk(xn, k, vals[order], idx[order], keys=keys) == []
    # ... and the mask must be the same set
    mask = np.zeros(n, dtype=bool)
    mask[idx] = True
    assert np.array_equal(out["mask"].cpu().numpy().view(np.uint32), o_topk.pack_mask(mask))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_a_selection_so_dense_that_the_filters_candidate_list_overflows(dtype):
    """A quarter of the row is kept: every CTA of the deferring filter notes more candidates than its list holds, the
    rest leave through the inline slow path without being counted in the bins, and the kernel behind the filter is told to
    count for itself.  Both entry points stay exact."""
    n, k = 1 << 24, 1 << 22
    pl = profk.plan(n, k, 1e-3)
    assert pl.mode == 0 and pl.capacity > 444 * 6144          # more candidates than all lists together
    x = workloads.normal(1, n, seed=63, dtype=dtype)[0]
    xn = workloads.as_numpy(x)
    xd = x.cuda()
    check_forms(xn, k, run(xd, k, seed=1, want_pairs=True, want_mask=True, want_dense=True))
    assert profk.read_stats(1)[0][3] == profk.ROW_OK
    v, i = profk.topk(xd, k, seed=2)
    torch.cuda.synchronize()
    ov, oi = o_topk.topk(xn[None, :], k)
    assert np.array_equal(i.cpu().numpy(), oi[0])
    assert np.array_equal(bits(workloads.as_numpy(v)), bits(ov[0]))
    assert profk.read_stats(1)[0][3] == profk.ROW_OK
