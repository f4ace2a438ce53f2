"""The pins must be sharp: plant plausible mistakes in a *copy* of the oracle's source (CPU only)
and check that the pin battery rejects every one of them while accepting the original."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import workloads as W
from helpers import brute_force, check_solution, knapsack_01

SRC = os.path.join(os.path.dirname(oracle.lib_path()), "spdy_ref.c")

MUTANTS = {
    "highest_index_wins": ("if (v < cur[t]) {\n                    cur[t] = v;\n                    P[t]",
                           "if (v <= cur[t]) {\n                    cur[t] = v;\n                    P[t]"),
    "dropped_error_term": ("const float v = prev[t - tau] + e; /* Eq. 2", "const float v = prev[t - tau]; /* Eq. 2"),
    "range_starts_one_late": ("for (int32_t t = tau; t <= B; ++t) {\n                const float v = prev[t - tau] + e; /* Eq. 2",
                              "for (int32_t t = tau + 1; t <= B; ++t) {\n                const float v = prev[t - tau] + e; /* Eq. 2"),
    "shift_sign_flipped": ("const float v = prev[t - tau] + e; /* Eq. 2", "const float v = prev[B - t + tau > B ? 0 : B - t + tau] + e; /* Eq. 2"),
    "highest_t_wins": ("if (prev[t] < best) {\n            best = prev[t];\n            t_best = t;",
                       "if (prev[t] <= best) {\n            best = prev[t];\n            t_best = t;"),
    "errors_transposed": ("const float e = errors[(size_t)l * K + k];\n            for (int32_t t = tau; t <= B; ++t) {\n                const float v = prev[t - tau] + e; /* Eq. 2",
                          "const float e = errors[(size_t)k * L + l];\n            for (int32_t t = tau; t <= B; ++t) {\n                const float v = prev[t - tau] + e; /* Eq. 2"),
    "max_instead_of_min": ("if (v < cur[t]) {\n                    cur[t] = v;\n                    P[t]",
                           "if (v > cur[t] || cur[t] == INFINITY) {\n                    cur[t] = v;\n                    P[t]"),
    "row_not_reset": ("            cur[t] = INFINITY;\n            P[t] = 0xFF;", "            P[t] = 0xFF;"),
}


def _compile(tmp_path, name, text):
    c = tmp_path / f"{name}.c"
    so = tmp_path / f"lib{name}.so"
    c.write_text(text)
    subprocess.run(["gcc", "-O2", "-fno-fast-math", "-ffp-contract=off", "-std=c11", "-shared",
                    "-fPIC", "-o", str(so), str(c), "-lm"], check=True)
    lib = ctypes.CDLL(str(so))
    f32p, i32p, u8p = (ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32),
                       ctypes.POINTER(ctypes.c_uint8))
    lib.spdy_ref_solve_range.restype = ctypes.c_int
    lib.spdy_ref_solve_range.argtypes = [f32p, i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                         ctypes.c_int64, ctypes.c_int64, u8p, f32p, i32p]

    def solve1(errors_one, times, B):
        e = np.ascontiguousarray(errors_one, dtype=np.float32)
        t = np.ascontiguousarray(times, dtype=np.int32)
        L, K = t.shape
        p = np.empty(L, np.uint8)
        c_ = np.empty(1, np.float32)
        tu = np.empty(1, np.int32)
        rc = lib.spdy_ref_solve_range(e.ctypes.data_as(f32p), t.ctypes.data_as(i32p), L, K, int(B),
                                      0, 1, p.ctypes.data_as(u8p), c_.ctypes.data_as(f32p),
                                      tu.ctypes.data_as(i32p))
        assert rc == 0, f"solver returned {rc}"
        return p, c_[0], int(tu[0])

    return solve1


def pin_battery(solve1):
    """A condensed run of the pins in test_oracle_pins.py; raises AssertionError on a miss."""
    for seed in range(3):
        wl = W.make_workload(0, seed_shift=seed)
        p, c, t = solve1(wl.errors[0], wl.times, wl.B)
        bc, bt, bp = brute_force(wl.errors[0], wl.times, wl.B)
        assert c.tobytes() == bc.tobytes() and t == bt and np.array_equal(p, bp)
    for seed in range(60):
        for exact in (False, True):
            wl = W.tiny_random_instance(seed + (10_000 if exact else 0), exact=exact)
            p, c, t = solve1(wl.errors[0], wl.times, wl.B)
            bc, bt, bp = brute_force(wl.errors[0], wl.times, wl.B)
            assert c.tobytes() == bc.tobytes() and (t < 0) == (bt < 0)
            check_solution(wl.errors[0], wl.times, wl.B, p, c, t)
            if exact:
                assert t == bt and (bp is None or np.array_equal(p, bp))
    times = np.array([[0, 3], [0, 2], [4, 1]], dtype=np.int32)
    errors = np.array([[1.0, 0.0], [1.0, 0.0], [0.0, 8.0]], dtype=np.float32)
    p, c, t = solve1(errors, times, 4)
    assert list(p) == [0, 0, 0] and c == np.float32(2.0) and t == 4
    rng = np.random.default_rng(3)
    w = rng.integers(1, 60, size=20)
    v = rng.integers(1, 1000, size=20)
    times = np.stack([w, np.zeros_like(w)], axis=1).astype(np.int32)
    errors = np.stack([np.zeros(20), v.astype(np.float64)], axis=1).astype(np.float32)
    p, c, t = solve1(errors, times, 300)
    assert int(v.sum()) - int(c) == knapsack_01(list(map(int, w)), list(map(int, v)), 300)


def test_unmodified_source_passes_the_battery(tmp_path):
    pin_battery(_compile(tmp_path, "orig", open(SRC).read()))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(tmp_path, name):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, "mutation site not found; update the mutant table"
    # The main solver comes first in the file; mutate only that occurrence.
    solve1 = _compile(tmp_path, name, text.replace(old, new, 1))
    with pytest.raises(AssertionError):
        pin_battery(solve1)
