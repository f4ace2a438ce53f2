"""Host-side helpers of the library (no GPU work) against the oracle's statements of the same rules:
time target (Section 3.1), discretisation into buckets (Section 3.2), the uniform baseline (Section 4)."""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import binding, build as build_mod, workloads as W


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def test_time_target_matches_the_oracle():
    rng = np.random.default_rng(0)
    for _ in range(200):
        td, x, tb = rng.uniform(0.1, 5.0), rng.uniform(1.0, 6.0), rng.uniform(0.0, 0.05)
        assert binding.time_target(td, x, tb) == oracle.time_target(td, x, tb)
    assert binding.time_target(0.478, 2.0) == 0.239


@pytest.mark.parametrize("rounding", ["nearest", "up"])
def test_bucketize_times_matches_the_oracle(rounding):
    rng = np.random.default_rng(1)
    for cfg in (1, 2, 3):
        t, dense = W.float_times(cfg)
        for speedup, B in ((2.5, 10000), (3.0, 1000), (4.0, 65536)):
            T = oracle.time_target(dense, speedup)
            got = binding.bucketize_times(t, T, B, rounding)
            assert got.dtype == np.int32 and np.array_equal(got, oracle.bucketize_times(t, T, B, rounding))
    for _ in range(100):
        L, K = int(rng.integers(1, 6)), int(rng.integers(1, 6))
        t = rng.uniform(0.0, 2.0, size=(L, K)) * rng.choice([1.0, 1e-3, 1e3])
        t[rng.random(size=t.shape) < 0.2] = 0.0
        T, B = float(rng.uniform(0.5, 4.0)), int(rng.integers(1, 5000))
        assert np.array_equal(binding.bucketize_times(t, T, B, rounding), oracle.bucketize_times(t, T, B, rounding))
    width = 8.0 / 4096
    halves = np.array([[0.5 * width, 1.5 * width, 2.5 * width, 3 * width]])
    assert np.array_equal(binding.bucketize_times(halves, 8.0, 4096, rounding),
                          oracle.bucketize_times(halves, 8.0, 4096, rounding))


def test_bucketize_times_rejects_bad_input():
    t = np.ones((2, 3))
    for kw in (dict(T=0.0, B=10), dict(T=-1.0, B=10), dict(T=1.0, B=0), dict(T=float("nan"), B=10)):
        with pytest.raises(binding.SpdyError):
            binding.bucketize_times(t, kw["T"], kw["B"])
    for bad in (-1.0, float("nan"), float("inf")):
        u = t.copy()
        u[1, 1] = bad
        with pytest.raises(binding.SpdyError):
            binding.bucketize_times(u, 1.0, 10)
    with pytest.raises(binding.SpdyError):  # beyond int32
        binding.bucketize_times(np.array([[1e12]]), 1.0, 1 << 30)
    lib = binding.library()
    out = np.zeros((2, 3), np.int32)
    assert lib.spdy_bucketize_times(t.ctypes.data_as(ctypes.c_void_p), 2, 3, 1.0, 10, 7,
                                    out.ctypes.data_as(ctypes.c_void_p)) == -1  # unknown rounding
    assert lib.spdy_bucketize_times(None, 2, 3, 1.0, 10, 0, out.ctypes.data_as(ctypes.c_void_p)) == -1


def test_uniform_profile_matches_the_oracle():
    rng = np.random.default_rng(2)
    for trial in range(300):
        L, K = int(rng.integers(1, 8)), int(rng.integers(1, 7))
        times = rng.integers(0, 40, size=(L, K)).astype(np.int32)
        if trial % 2:
            times = np.sort(times, axis=1)[:, ::-1].copy()
        B = int(rng.integers(0, 30 * L))
        keep = (rng.random(L) < 0.3) if trial % 3 else None
        assert binding.uniform_profile(times, B, keep) == oracle.uniform_profile(times, B, keep)
    for cfg in (1, 2, 3):
        wl = W.make_workload(cfg, N=1)
        keep = np.zeros(wl.L, bool)
        keep[[0, -1]] = True  # first and last layer stay dense, as in Section 4
        assert binding.uniform_profile(wl.times, wl.B) == oracle.uniform_profile(wl.times, wl.B)
        assert binding.uniform_profile(wl.times, wl.B, keep) == oracle.uniform_profile(wl.times, wl.B, keep)
    assert binding.uniform_profile(np.array([[5, 4]], np.int32), 3) == (-1, -1)
    with pytest.raises(binding.SpdyError):
        binding.uniform_profile(np.array([[5, -4]], np.int32), 30)


def test_discretised_tables_feed_a_plan():
    """The helpers' output is a valid timing table: a host-only plan accepts it and its budget is B."""
    t, dense = W.float_times(2)
    T = binding.time_target(dense, 3.0)
    times = binding.bucketize_times(t, T, 10000, "up")
    info = binding.Plan(times, 10000, device=-1).info
    assert info["feasible"] == 1 and info["B"] == 10000
    k, total = binding.uniform_profile(times, 10000)
    assert 0 < k < times.shape[1] and total <= 10000
