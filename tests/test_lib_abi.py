"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, validates arguments, and its host plan equals the oracle's plan."""
import ctypes
import os
import re

import pytest

import paper_2608_12573_b200 as profk
from oracle import plan as oracle_plan
from paper_2608_12573_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build()
    return profk.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "profk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(profk_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in profk.h but not exported"
    assert set(names) == set(profk.EXPORTS)


SHAPES = [(2 ** 20, 64, 1e-3, 1.0), (2 ** 26, 16, 1e-2, 1.0), (2 ** 26, 16, 1e-4, 1.0), (2 ** 26, 256, 1e-2, 1.0),
          (2 ** 26, 256, 1e-4, 1.0), (2 ** 26, 4096, 1e-2, 1.0), (2 ** 26, 4096, 1e-4, 1.0), (2 ** 26, 4096, 1e-2, 0.95),
          (2 ** 26, 16, 1e-2, 0.95), (2 ** 20, 32, 1e-3, 1.0), (2 ** 29, 131072, 1e-3, 1.0), (2 ** 30, 1, 1e-3, 1.0),
          (2 ** 30, 64, 1e-3, 1.0), (2 ** 30, 1024, 1e-3, 1.0), (2 ** 30, 65536, 1e-3, 1.0), (10 ** 9, 100, 1e-3, 1.0),
          (50331648, 131072, 1e-3, 1.0), (1_000_003, 77, 1e-3, 1.0), (50000, 10, 1e-3, 1.0), (2 ** 20, 2 ** 19, 1e-3, 1.0),
          (100, 100, 1e-3, 1.0), (1, 1, 0.5, 1.0), (3_000_001, 2999, 0.2, 0.5), (2 ** 24, 5, 1e-6, 1.0)]


@pytest.mark.parametrize("N,k,eps,recall", SHAPES)
@pytest.mark.parametrize("tuning", ["paper", "library", "library, batch"])
def test_host_plan_equals_oracle_plan(lib, N, k, eps, recall, tuning):
    if tuning == "paper":        # Section 4's S_min = 32768, S_max = 2^17, cost ratio 1: the oracle's defaults
        got = profk.plan(N, k, eps, recall, **profk.PAPER_TUNING)
        want = oracle_plan.plan_guarded(N, k, eps, recall)
    else:                        # the library's own tuning inputs (a floor that follows short rows, a cost ratio that grows
        rows = 1 if tuning == "library" else 5      # with long ones), handed to the oracle as tuning inputs
        s_min = min(32768, max(1024, N // 512))
        ratio = min(max(N / 2 ** 22, 1.0), 16.0 if rows <= 4 else 4.0)
        s_max = 131072
        assert profk.default_tuning(N, rows=rows) == dict(s_min=s_min, s_max=s_max, cost_ratio=ratio)
        got = profk.plan(N, k, eps, recall, rows=rows)
        want = oracle_plan.plan_guarded(N, k, eps, recall, s_min=s_min, s_max=s_max, cost_ratio=ratio)
    assert (got.m, got.r, got.capacity, got.k_accept, got.mode) == (want.m, want.r, want.capacity, want.k_accept, want.mode)
    assert (got.r_tight, got.r_loose) == (want.r_tight, want.r_loose)
    assert got.z == pytest.approx(want.z, rel=1e-12)
    assert got.alpha == want.alpha
    assert got.p_recall_fail == pytest.approx(want.p_recall_fail, rel=1e-6, abs=1e-300)
    assert got.p_overflow == pytest.approx(want.p_overflow, rel=1e-6, abs=1e-300)


def test_plan_with_tuning_inputs(lib):
    got = profk.plan(2 ** 20, 32, 1e-3, 1.0, s_min=2048, s_max=4096)
    want = oracle_plan.plan_guarded(2 ** 20, 32, 1e-3, 1.0, s_min=2048, s_max=4096)
    assert (got.m, got.r, got.capacity) == (want.m, want.r, want.capacity)
    got = profk.plan(2 ** 28, 1024, 1e-3, 1.0, cost_ratio=4.0, s_max=262144)
    want = oracle_plan.plan_guarded(2 ** 28, 1024, 1e-3, 1.0, cost_ratio=4.0, s_max=262144)
    assert (got.m, got.r, got.capacity) == (want.m, want.r, want.capacity)


def test_argument_validation_without_a_device(lib):
    out = profk._PlanStruct()
    bad = [(0, 1, 1e-3, 1.0), (10, 0, 1e-3, 1.0), (10, 11, 1e-3, 1.0), (10, 5, 0.0, 1.0), (10, 5, 1.0, 1.0),
           (10, 5, 1e-3, 0.0), (10, 5, 1e-3, 1.5), (2 ** 32, 5, 1e-3, 1.0)]
    for N, k, eps, recall in bad:
        assert lib.profk_plan(ctypes.c_int64(N), ctypes.c_int64(k), ctypes.c_double(eps), ctypes.c_double(recall),
                              ctypes.byref(out)) == -1
    assert lib.profk_plan(ctypes.c_int64(10), ctypes.c_int64(5), ctypes.c_double(1e-3), ctypes.c_double(1.0), None) == -1
    n = ctypes.c_size_t()
    assert lib.profk_workspace_bytes(ctypes.c_int64(0), ctypes.c_int64(10), ctypes.c_int64(5), ctypes.byref(n)) == -1
    assert lib.profk_workspace_bytes(ctypes.c_int64(1), ctypes.c_int64(4), ctypes.c_int64(5), ctypes.byref(n)) == -1
    assert lib.profk_workspace_bytes(ctypes.c_int64(4), ctypes.c_int64(700), ctypes.c_int64(64), ctypes.byref(n)) == 0
    assert n.value >= 4 * 700 * 8
    assert lib.profk_strerror(-2).decode() == "workspace missing or too small"
    with pytest.raises(profk.ProfkError):
        profk.plan(10, 11)
