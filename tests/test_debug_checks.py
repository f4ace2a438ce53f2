"""The debug build of the library (same sources, -DSPDY_DEBUG_CHECKS): every row-buffer and table access of
the forward kernels tests its index first and records a bad one in the plan's status word instead of
performing it, and the new row's buffer is poisoned before each layer so that a read of a cell nobody wrote
shows.  On correct plans the word must stay zero and the outputs must equal the oracle's: this is the check
that the +inf guard cells, which stand in for per-cell bounds checks in the release build, are wide enough."""
import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import binding, build as build_mod, workloads as W

pytestmark = pytest.mark.gpu
FORMATS = [binding.SPDY_TABLE_ARG_U8, binding.SPDY_TABLE_ROW_F32]


@pytest.fixture(scope="module", autouse=True)
def debug_library():
    build_mod.build(debug=True)
    lib = binding.select_library("debug")
    assert lib.spdy_debug_checks_enabled() == 1
    yield
    binding._lib = None
    assert binding.library().spdy_debug_checks_enabled() == 0


def solve_checked(wl, fmt, **kw):
    import torch

    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, **kw)
    p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda())
    torch.cuda.synchronize()
    word = plan.status_word()
    plan.close()
    assert word == 0, f"status word {word:#x}: an index check inside the forward kernel fired ({kw})"
    return p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()


def same(got, ref):
    assert np.array_equal(got[2], ref[2]) and got[1].tobytes() == ref[1].tobytes() and np.array_equal(got[0], ref[0])


SHAPES = [dict(), dict(kernel=binding.SPDY_KERNEL_WARP), dict(kernel=binding.SPDY_KERNEL_CTA), dict(threads=256),
          dict(threads=1024), dict(rows_in_global=1), dict(cluster=2), dict(cluster=8), dict(schedule=1),
          dict(schedule=3), dict(schedule=4 << 8)]


@pytest.mark.parametrize("fmt", FORMATS)
def test_index_checks_stay_silent_on_tiny_shapes(fmt):
    for seed in range(40):
        for exact in (False, True):
            wl = W.tiny_random_instance(seed + (10_000 if exact else 0), exact=exact, N=4)
            ref = oracle.solve_batch(wl.errors, wl.times, wl.B)
            for kw in SHAPES[:7] if seed % 2 else SHAPES[3:]:
                same(solve_checked(wl, fmt, **kw), ref)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("cfg,B,n", [(0, None, 1), (1, None, 6), (2, None, 6), (4, 1000, 9), (4, 2500, 6)])
def test_index_checks_stay_silent_on_the_named_shapes(cfg, B, n, fmt):
    wl = W.make_workload(cfg, N=n, B=B)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=4)
    for kw in SHAPES:
        try:
            same(solve_checked(wl, fmt, **kw), ref)
        except binding.SpdyError as e:
            assert e.status == -3, (kw, e)  # a launch shape this problem cannot take


def test_wide_rows_and_small_batches_in_the_debug_build():
    wl = W.make_workload(4, N=2, B=100000)  # rows in global memory by default
    same(solve_checked(wl, binding.SPDY_TABLE_ROW_F32), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=2))
    wl = W.make_workload(3, N=2)  # one CTA of 512 threads, 212 KB of rows
    same(solve_checked(wl, binding.SPDY_TABLE_ARG_U8), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=2))


def test_the_debug_build_holds_the_default_cell_updates_only():
    wl = W.make_workload(0)
    with pytest.raises(binding.SpdyError) as e:
        binding.Plan(wl.times, wl.B, device=0, forward_mode=3)
    assert e.value.status == -3
