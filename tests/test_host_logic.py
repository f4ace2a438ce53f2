"""CPU-only checks of the CUDA library's host side: it loads, exports what the header declares,
validates arguments, and its band plan is sound (no compute calls: there is no GPU here)."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import binding, build as build_mod, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spdy_dp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spdy_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.library()
    names = declared_functions()
    assert len(names) >= 10
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/spdy_dp.h but not exported"
    assert sorted(binding.EXPORTS) == names
    assert lib.spdy_version() >= 1000
    assert lib.spdy_strerror(0) == b"success" and lib.spdy_strerror(-3)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.library()


def test_plan_rejects_bad_arguments():
    lib = binding.library()
    t = np.ones((3, 4), np.int32)
    h = ctypes.c_void_p()
    ptr = t.ctypes.data_as(ctypes.c_void_p)
    assert lib.spdy_plan_create(None, ptr, 3, 4, 10, -1, None) == -1
    assert lib.spdy_plan_create(ctypes.byref(h), None, 3, 4, 10, -1, None) == -1
    assert lib.spdy_plan_create(ctypes.byref(h), ptr, 0, 4, 10, -1, None) == -1
    assert lib.spdy_plan_create(ctypes.byref(h), ptr, 3, 0, 10, -1, None) == -1
    assert lib.spdy_plan_create(ctypes.byref(h), ptr, 3, 4, -1, -1, None) == -1
    big = np.ones((1, 256), np.int32)
    assert lib.spdy_plan_create(ctypes.byref(h), big.ctypes.data_as(ctypes.c_void_p), 1, 256, 10, -1, None) == -1
    neg = t.copy()
    neg[1, 2] = -1
    assert lib.spdy_plan_create(ctypes.byref(h), neg.ctypes.data_as(ctypes.c_void_p), 3, 4, 10, -1, None) == -1
    with pytest.raises(binding.SpdyError):
        binding.Plan(t, 10, device=-1, threads=100)
    with pytest.raises(binding.SpdyError):
        binding.Plan(t, 10, device=-1, table_format=7)
    # a host-only plan cannot solve
    p = binding.Plan(t, 10, device=-1)
    assert lib.spdy_solve_batch(p._h, 1, 1, 1, 1, 1, 1, 0, None) == -1
    assert lib.spdy_workspace_bytes(None, 5) == 0 and p.workspace_bytes(0) == 0


def python_bands(times, B):
    L, K = times.shape
    usable = times <= B
    mn = np.array([times[l][usable[l]].min() if usable[l].any() else 0 for l in range(L)], np.int64)
    mx = np.array([times[l][usable[l]].max() if usable[l].any() else 0 for l in range(L)], np.int64)
    feasible = all(usable[l].any() for l in range(L)) and mn.sum() <= B
    lo = np.cumsum(mn)
    hi = np.minimum(np.minimum(B, np.cumsum(mx)), B - (mn.sum() - np.cumsum(mn)))
    return feasible, lo, hi - lo + 1


@pytest.mark.parametrize("cfg", [0, 1, 2, 3])
def test_bands_of_the_named_configs(cfg):
    wl = W.make_workload(cfg, N=1)
    plan = binding.Plan(wl.times, wl.B, device=-1)
    feasible, lo, width = python_bands(wl.times, wl.B)
    plo, pwidth = plan.bands()
    info = plan.info
    assert info["feasible"] == 1 and feasible
    assert np.array_equal(plo, lo) and np.array_equal(pwidth, width)
    assert info["max_width"] == width.max() and info["band_cells"] == width.sum()
    assert info["nominal_updates"] == wl.L * wl.K * wl.B
    assert 0 < info["distinct_updates"] <= info["useful_updates"] <= info["nominal_updates"] + wl.L * wl.K
    assert info["distinct_updates"] <= info["issued_updates"]
    # the byte table merges the same groups (for candidates where that is exact) in a second table set
    arg = binding.Plan(wl.times, wl.B, device=-1, table_format=binding.SPDY_TABLE_ARG_U8).info
    assert arg["useful_updates"] == info["useful_updates"]
    assert arg["distinct_updates"] == info["distinct_updates"] <= arg["issued_updates"]
    assert arg["launches_per_wave"] == (5 if arg["distinct_updates"] < arg["useful_updates"] else 2)
    assert info["launches_per_wave"] == 2
    # merged work recomputed from the timing table: one shift per distinct usable time of a layer
    lo_prev, w_prev, distinct = 0, 1, 0
    for l in range(wl.L):
        usable = np.unique(wl.times[l][wl.times[l] <= wl.B])
        for tau in usable:
            a = int(tau - usable.min())
            b = min(int(width[l]) - 1, w_prev - 1 + a)
            distinct += max(0, b - a + 1)
        w_prev = int(width[l])
    assert distinct == info["distinct_updates"]
    assert info["smem_bytes"] <= 232448
    assert info["table_bytes_per_candidate"] % 256 == 0


@pytest.mark.parametrize("seed", range(40))
def test_cells_outside_the_band_never_matter(seed):
    """Every finite cell of the full-width rows outside the plan's band must be unable to finish
    within the budget, and the band must hold every cell of the optimal path."""
    wl = W.tiny_random_instance(500 + seed, max_L=5, max_K=4, max_B=48)
    plan = binding.Plan(wl.times, wl.B, device=-1)
    lo, width = plan.bands()
    feasible, _, _ = python_bands(wl.times, wl.B)
    assert plan.info["feasible"] == int(feasible)
    p, c, t = oracle.solve_batch(wl.errors[:1], wl.times, wl.B)
    if not feasible:
        assert t[0] == -1
        return
    usable_min = np.array([wl.times[l][wl.times[l] <= wl.B].min() for l in range(wl.L)])
    for l in range(wl.L):
        row = oracle.last_row(wl.errors[0][: l + 1], wl.times[: l + 1], wl.B)
        rest = int(usable_min[l + 1:].sum())
        for tt in np.flatnonzero(np.isfinite(row)):
            inside = lo[l] <= tt < lo[l] + width[l]
            assert inside or tt + rest > wl.B
    if t[0] >= 0:
        tt = 0
        for l in range(wl.L):
            tt += int(wl.times[l][p[0][l]])
            assert lo[l] <= tt < lo[l] + width[l]


def test_infeasible_and_degenerate_plans():
    t = np.array([[5, 6], [7, 9]], np.int32)
    assert binding.Plan(t, 11, device=-1).info["feasible"] == 0
    assert binding.Plan(t, 12, device=-1).info["feasible"] == 1
    one = np.array([[0]], np.int32)
    info = binding.Plan(one, 0, device=-1).info
    assert info["feasible"] == 1 and info["max_width"] == 1
    over = np.array([[50, 60]], np.int32)  # every choice above the budget
    assert binding.Plan(over, 10, device=-1).info["feasible"] == 0


def test_wide_rows_leave_shared_memory():
    wl = W.make_workload(4, N=1, B=100000)
    info = binding.Plan(wl.times, wl.B, device=-1).info
    assert info["rows_in_global"] == 1 and info["cluster"] == 1 and info["threads"] == 1024
    info = binding.Plan(wl.times, wl.B, device=-1, threads=512).info
    assert info["cluster"] in (2, 4, 8) and info["smem_bytes"] <= 232448 and info["rows_in_global"] == 0
    for c in (4, 8):
        info = binding.Plan(wl.times, wl.B, device=-1, cluster=c).info
        assert info["cluster"] == c and info["smem_bytes"] <= 232448
    with pytest.raises(binding.SpdyError) as e:  # one CTA cannot hold it
        binding.Plan(wl.times, wl.B, device=-1, cluster=1)
    assert e.value.status == -3
    with pytest.raises(binding.SpdyError):
        binding.Plan(wl.times, wl.B, device=-1, cluster=3)
    small = W.make_workload(2, N=1)
    for c in (2, 4, 8):
        info = binding.Plan(small.times, small.B, device=-1, cluster=c).info
        assert info["cluster"] == c and info["distinct_updates"] <= info["issued_updates"]


def test_option_validation_of_the_newer_fields():
    t = np.ones((3, 4), np.int32)
    with pytest.raises(binding.SpdyError):
        binding.Plan(t, 10, device=-1, rows_in_global=2)
    with pytest.raises(binding.SpdyError):
        binding.Plan(t, 10, device=-1, rows_in_global=1, cluster=2)
    info = binding.Plan(t, 10, device=-1, rows_in_global=1).info
    assert info["rows_in_global"] == 1 and info["threads"] == 1024 and info["table_bytes_per_candidate"] % 256 == 0
    # equal times everywhere: the byte table gets its merged table set, the row table merges always
    arg = binding.Plan(t, 10, device=-1, table_format=binding.SPDY_TABLE_ARG_U8).info
    row = binding.Plan(t, 10, device=-1).info
    assert arg["launches_per_wave"] == 5 and row["launches_per_wave"] == 2
    assert arg["distinct_updates"] == row["distinct_updates"] < row["useful_updates"]
    distinct = np.arange(12, dtype=np.int32).reshape(3, 4)  # no two choices of a layer share a time
    assert binding.Plan(distinct, 20, device=-1, table_format=binding.SPDY_TABLE_ARG_U8).info["launches_per_wave"] == 2
