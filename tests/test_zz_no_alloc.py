"""The entry point for callers that may not allocate device memory.

Some users of this library run where a device allocation is off limits: inside a framework that
owns the whole device heap, or in a service whose memory footprint is frozen after start-up.
``spdy_solve_batch_static`` serves them from an array compiled into the library.  This file checks
it, through the C ABI, against the ordinary entry point and against the CPU oracle - twice in a row,
because the array keeps the first call's leftovers when the second one starts.  It is collected last
on purpose.
"""
import ctypes
import os

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import binding, build as build_mod, workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def test_static_scratch_entry_point_matches_the_allocating_one_twice_in_a_row():
    import torch

    lib = binding.library()
    assert lib.spdy_static_scratch_bytes() == 64 << 20
    # 300 candidates of the ResNet-50 shape need more table than the array holds: several waves.
    first = W.make_workload(1, N=300)
    second = W.make_workload(2, N=150)  # other shapes and errors: leftovers must not leak in
    for wl in (first, second):
        errors = torch.from_numpy(wl.errors).cuda()
        plan = binding.Plan(wl.times, wl.B, device=0)
        want_p, want_c, want_t = binding.solve_batch(plan, errors)
        torch.cuda.synchronize()
        plan.check_status()

        profile = torch.full((wl.N, wl.L), 7, dtype=torch.uint8, device="cuda")
        cost = torch.full((wl.N,), -1.0, dtype=torch.float32, device="cuda")
        time_used = torch.full((wl.N,), -7, dtype=torch.int32, device="cuda")
        times = np.ascontiguousarray(wl.times, dtype=np.int32)
        rc = lib.spdy_solve_batch_static(errors.data_ptr(), times.ctypes.data_as(ctypes.c_void_p),
                                         wl.N, wl.L, wl.K, wl.B, profile.data_ptr(), cost.data_ptr(),
                                         time_used.data_ptr(),
                                         ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == 0, lib.spdy_strerror(rc)
        # integer outputs and fp32 cost bits are identical (the path is exact, tolerance zero)
        assert torch.equal(profile, want_p)
        assert torch.equal(time_used, want_t)
        assert cost.cpu().numpy().tobytes() == want_c.cpu().numpy().tobytes()
        plan.close()
        # and both agree with the oracle, element by element
        rp, rc_, rt = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=max(1, len(os.sched_getaffinity(0))))
        assert np.array_equal(profile.cpu().numpy(), rp) and np.array_equal(time_used.cpu().numpy(), rt)
        assert cost.cpu().numpy().tobytes() == rc_.tobytes()


def test_static_entry_point_rejects_what_does_not_fit():
    import torch

    lib = binding.library()
    wl = W.make_workload(4, N=1, B=100000)  # rows too wide for one CTA
    errors = torch.from_numpy(wl.errors).cuda()
    with pytest.raises(binding.SpdyError) as e:
        binding.solve_batch_static(errors, wl.times, wl.B)
    assert e.value.status == -7 and b"built-in scratch" in lib.spdy_strerror(-7)
    # an infeasible budget is not an error and needs no table at all
    small = W.make_workload(1, N=3)
    p, c, t = binding.solve_batch_static(torch.from_numpy(small.errors).cuda(), small.times, 10)
    assert (p.cpu().numpy() == 0xFF).all() and (t.cpu().numpy() == -1).all()
