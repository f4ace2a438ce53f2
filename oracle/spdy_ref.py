"""ctypes front end of ``spdy_ref.c`` (the CPU oracle; test infrastructure, not product code).

``solve_batch`` fans candidates out over host threads, one oracle instance per thread over a
disjoint candidate range; each instance is the plain single-threaded solver.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spdy_ref.c")
_LIB = os.path.join(_HERE, "libspdy_ref.so")
_CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-std=c11", "-shared", "-fPIC"]
_lock = threading.Lock()
_lib = None


def lib_path() -> str:
    return _LIB


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than the source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.run(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"], check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        f32p, i32p, u8p = (ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32),
                           ctypes.POINTER(ctypes.c_uint8))
        lib.spdy_ref_solve_range.restype = ctypes.c_int
        lib.spdy_ref_solve_range.argtypes = [f32p, i32p, ctypes.c_int32, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                             u8p, f32p, i32p]
        lib.spdy_ref_last_row.restype = ctypes.c_int
        lib.spdy_ref_last_row.argtypes = [f32p, i32p, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_int32, f32p]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def solve_batch(errors: np.ndarray, times: np.ndarray, B: int, threads: int = 1):
    """errors [N][L][K] fp32, times [L][K] int32, budget B -> (profile [N][L] u8, cost [N] f32,
    time_used [N] i32).  ``threads`` host threads each run the single-threaded solver on their
    own slice of the candidates."""
    lib = _load()
    errors = np.ascontiguousarray(errors, dtype=np.float32)
    times = np.ascontiguousarray(times, dtype=np.int32)
    if errors.ndim != 3 or times.ndim != 2 or errors.shape[1:] != times.shape:
        raise ValueError("errors must be [N][L][K] and times [L][K]")
    N, L, K = errors.shape
    profile = np.empty((N, L), dtype=np.uint8)
    cost = np.empty(N, dtype=np.float32)
    time_used = np.empty(N, dtype=np.int32)
    if N == 0:
        return profile, cost, time_used

    def run(first: int, count: int) -> int:
        return lib.spdy_ref_solve_range(_ptr(errors, ctypes.c_float), _ptr(times, ctypes.c_int32),
                                        L, K, int(B), first, count, _ptr(profile, ctypes.c_uint8),
                                        _ptr(cost, ctypes.c_float), _ptr(time_used, ctypes.c_int32))

    threads = max(1, min(int(threads), N))
    if threads == 1:
        codes = [run(0, N)]
    else:
        bounds = np.linspace(0, N, threads + 1).astype(np.int64)
        with ThreadPoolExecutor(max_workers=threads) as pool:
            codes = list(pool.map(lambda i: run(int(bounds[i]), int(bounds[i + 1] - bounds[i])),
                                  range(threads)))
    for rc in codes:
        if rc != 0:
            raise RuntimeError(f"spdy_ref_solve_range failed with code {rc}")
    return profile, cost, time_used


def last_row(errors_one: np.ndarray, times: np.ndarray, B: int) -> np.ndarray:
    """E_L^t for t = 0..B of a single candidate (errors_one is [L][K])."""
    lib = _load()
    errors_one = np.ascontiguousarray(errors_one, dtype=np.float32)
    times = np.ascontiguousarray(times, dtype=np.int32)
    L, K = times.shape
    row = np.empty(int(B) + 1, dtype=np.float32)
    rc = lib.spdy_ref_last_row(_ptr(errors_one, ctypes.c_float), _ptr(times, ctypes.c_int32),
                               L, K, int(B), _ptr(row, ctypes.c_float))
    if rc != 0:
        raise RuntimeError(f"spdy_ref_last_row failed with code {rc}")
    return row
