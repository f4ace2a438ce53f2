"""Thin ctypes binding of ``include/spdy_dp.h``: argument marshalling only.

Every step of the path (forward dynamic program, final minimum, walk back) runs in the CUDA
library; PyTorch supplies device buffers and the stream.  There is no CPU fallback: if the
library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libspdy_dp.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libspdy_dp_debug.so")  # same sources with index checks in the kernels
HOST_LIB_PATH = os.path.join(_PKG, "libspdy_plan_host.so")  # spdy_plan.cpp alone: plans and host helpers

SPDY_KERNEL_AUTO, SPDY_KERNEL_CTA, SPDY_KERNEL_WARP = 0, 1, 2

SPDY_TABLE_DEFAULT, SPDY_TABLE_ARG_U8, SPDY_TABLE_ROW_F32 = 0, 1, 2

EXPORTS = (
    "spdy_plan_create", "spdy_plan_destroy", "spdy_plan_get_info", "spdy_plan_get_bands",
    "spdy_workspace_bytes", "spdy_solve_batch", "spdy_solve_batch_host", "spdy_solve_batch_simple",
    "spdy_plan_check_status", "spdy_plan_enable_timing", "spdy_plan_last_timing",
    "spdy_solve_batch_static", "spdy_static_scratch_bytes", "spdy_strerror", "spdy_last_cuda_error", "spdy_version",
    "spdy_solve_batch_coeffs", "spdy_solve_batch_coeffs_host", "spdy_quadratic_errors",
    "spdy_time_target", "spdy_bucketize_times", "spdy_uniform_profile", "spdy_probe_peaks",
    "spdy_plan_get_tables", "spdy_plan_verify", "spdy_plan_status_word", "spdy_debug_checks_enabled",
    "spdy_plan_shape_for_batch", "spdy_search",
)
# What the host-only library holds (everything that needs no CUDA).
HOST_EXPORTS = (
    "spdy_plan_create", "spdy_plan_destroy", "spdy_plan_get_info", "spdy_plan_get_bands", "spdy_workspace_bytes",
    "spdy_plan_get_tables", "spdy_plan_verify", "spdy_plan_shape_for_batch", "spdy_search", "spdy_time_target", "spdy_bucketize_times", "spdy_uniform_profile",
    "spdy_strerror", "spdy_version",
)


class SpdyOptions(ctypes.Structure):
    _fields_ = [("table_format", ctypes.c_int32), ("threads", ctypes.c_int32),
                ("cluster", ctypes.c_int32), ("forward_mode", ctypes.c_int32),
                ("rows_in_global", ctypes.c_int32), ("kernel", ctypes.c_int32),
                ("schedule", ctypes.c_int32), ("auto_shape", ctypes.c_int32)]


class SpdySearchOptions(ctypes.Structure):
    _fields_ = [("trials", ctypes.c_int32), ("patience", ctypes.c_int32), ("delta", ctypes.c_double),
                ("max_batch", ctypes.c_int64)]


class SpdySearchResult(ctypes.Structure):
    _fields_ = [("loss", ctypes.c_double), ("evals", ctypes.c_int64), ("accepted", ctypes.c_int64),
                ("dp_batches", ctypes.c_int64), ("dp_candidates", ctypes.c_int64),
                ("dp_seconds", ctypes.c_double), ("eval_seconds", ctypes.c_double)]


EVAL_FN = ctypes.CFUNCTYPE(ctypes.c_double, ctypes.POINTER(ctypes.c_uint8), ctypes.c_int32, ctypes.c_void_p)
DRAW_FN = ctypes.CFUNCTYPE(None, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32),
                           ctypes.POINTER(ctypes.c_float), ctypes.c_void_p)
SOLVE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.c_int64,
                            ctypes.POINTER(ctypes.c_uint8), ctypes.c_void_p)


class SpdyPlanTables(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int32), ("K", ctypes.c_int32), ("kernel_kind", ctypes.c_int32),
                ("threads", ctypes.c_int32), ("warps_per_candidate", ctypes.c_int32), ("cluster", ctypes.c_int32),
                ("forward_mode", ctypes.c_int32), ("max_cells_per_lane", ctypes.c_int32),
                ("row_stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("out_stride", ctypes.c_int32),
                ("win_stride", ctypes.c_int32), ("mask_words", ctypes.c_int32), ("n_passes", ctypes.c_int32),
                ("pitch", ctypes.c_int64), ("layers", ctypes.c_void_p), ("slots", ctypes.c_void_p),
                ("passes", ctypes.c_void_p), ("pass_masks", ctypes.c_void_p), ("pass_ptr", ctypes.c_void_p),
                ("slices", ctypes.c_void_p)]


class SpdyPlanInfo(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int32), ("K", ctypes.c_int32), ("B", ctypes.c_int32),
                ("feasible", ctypes.c_int32), ("max_width", ctypes.c_int32),
                ("span", ctypes.c_int32), ("threads", ctypes.c_int32), ("cluster", ctypes.c_int32),
                ("table_format", ctypes.c_int32), ("ctas_per_sm", ctypes.c_int32),
                ("sm_count", ctypes.c_int32), ("rows_in_global", ctypes.c_int32),
                ("smem_bytes", ctypes.c_int64), ("table_bytes_per_candidate", ctypes.c_int64),
                ("band_cells", ctypes.c_int64), ("useful_updates", ctypes.c_int64),
                ("issued_updates", ctypes.c_int64), ("nominal_updates", ctypes.c_int64),
                ("distinct_updates", ctypes.c_int64), ("launches_per_wave", ctypes.c_int32),
                ("kernel", ctypes.c_int32), ("forward_mode", ctypes.c_int32), ("candidates_per_cta", ctypes.c_int32),
                ("alternates", ctypes.c_int32), ("reserved1", ctypes.c_int32)]

    def as_dict(self) -> dict:
        return {name: int(getattr(self, name)) for name, _ in self._fields_}


class SpdyError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = _load()
        text = lib.spdy_strerror(status).decode()
        extra = f" (cudaError {lib.spdy_last_cuda_error()})" if status == -4 and hasattr(lib, "spdy_last_cuda_error") else ""
        super().__init__(f"{where}: {text}{extra} [{status}]")


_lib = None
_loaded = {}


def _configure(lib, host_only: bool = False):
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.spdy_plan_create.restype = ctypes.c_int
    lib.spdy_plan_create.argtypes = [ctypes.POINTER(vp), vp, i32, i32, i32, ctypes.c_int,
                                     ctypes.POINTER(SpdyOptions)]
    lib.spdy_plan_destroy.restype = None
    lib.spdy_plan_destroy.argtypes = [vp]
    lib.spdy_plan_get_info.restype = ctypes.c_int
    lib.spdy_plan_get_info.argtypes = [vp, ctypes.POINTER(SpdyPlanInfo)]
    lib.spdy_plan_get_bands.restype = ctypes.c_int
    lib.spdy_plan_get_bands.argtypes = [vp, vp, vp]
    lib.spdy_plan_get_tables.restype = ctypes.c_int
    lib.spdy_plan_get_tables.argtypes = [vp, i32, ctypes.POINTER(SpdyPlanTables)]
    lib.spdy_plan_verify.restype = ctypes.c_int
    lib.spdy_plan_verify.argtypes = [vp]
    lib.spdy_plan_shape_for_batch.restype = ctypes.c_int32
    lib.spdy_plan_shape_for_batch.argtypes = [vp, i64, ctypes.c_size_t]
    lib.spdy_workspace_bytes.restype = ctypes.c_size_t
    lib.spdy_workspace_bytes.argtypes = [vp, i64]
    lib.spdy_search.restype = ctypes.c_int
    lib.spdy_search.argtypes = [vp, vp, vp, ctypes.POINTER(SpdySearchOptions), DRAW_FN, vp, EVAL_FN, vp, SOLVE_FN, vp,
                                vp, vp, vp, ctypes.POINTER(SpdySearchResult), vp, vp, i64]
    lib.spdy_time_target.restype = ctypes.c_double
    lib.spdy_time_target.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double]
    lib.spdy_bucketize_times.restype = ctypes.c_int
    lib.spdy_bucketize_times.argtypes = [vp, i32, i32, ctypes.c_double, i32, i32, vp]
    lib.spdy_uniform_profile.restype = ctypes.c_int
    lib.spdy_uniform_profile.argtypes = [vp, i32, i32, i32, vp, ctypes.POINTER(i32), ctypes.POINTER(i64)]
    lib.spdy_strerror.restype = ctypes.c_char_p
    lib.spdy_strerror.argtypes = [ctypes.c_int]
    lib.spdy_version.restype = ctypes.c_int
    if host_only:
        return lib
    lib.spdy_solve_batch.restype = ctypes.c_int
    lib.spdy_solve_batch.argtypes = [vp, vp, i64, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.spdy_solve_batch_host.restype = ctypes.c_int
    lib.spdy_solve_batch_host.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    lib.spdy_solve_batch_coeffs.restype = ctypes.c_int
    lib.spdy_solve_batch_coeffs.argtypes = [vp, vp, i64, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.spdy_solve_batch_coeffs_host.restype = ctypes.c_int
    lib.spdy_solve_batch_coeffs_host.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    lib.spdy_quadratic_errors.restype = ctypes.c_int
    lib.spdy_quadratic_errors.argtypes = [vp, i64, i32, i32, vp, vp]
    lib.spdy_probe_peaks.restype = ctypes.c_int
    lib.spdy_probe_peaks.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.spdy_solve_batch_simple.restype = ctypes.c_int
    lib.spdy_solve_batch_simple.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.spdy_plan_check_status.restype = ctypes.c_int
    lib.spdy_plan_check_status.argtypes = [vp, vp]
    lib.spdy_plan_status_word.restype = ctypes.c_int
    lib.spdy_plan_status_word.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.spdy_debug_checks_enabled.restype = ctypes.c_int
    lib.spdy_plan_enable_timing.restype = ctypes.c_int
    lib.spdy_plan_enable_timing.argtypes = [vp, ctypes.c_int]
    lib.spdy_plan_last_timing.restype = ctypes.c_int
    lib.spdy_plan_last_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_float),
                                          ctypes.POINTER(ctypes.c_float)]
    lib.spdy_solve_batch_static.restype = ctypes.c_int
    lib.spdy_solve_batch_static.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.spdy_static_scratch_bytes.restype = ctypes.c_size_t
    lib.spdy_last_cuda_error.restype = ctypes.c_int
    return lib


def open_library(path: str, host_only: bool = False):
    """Load and type one build of the library (cached per path); raises if the file is missing."""
    if path not in _loaded:
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with "
                               "`python -m paper_2201_13096_b200.build` (needs nvcc); "
                               "there is no fallback implementation")
        _loaded[path] = _configure(ctypes.CDLL(path), host_only)
    return _loaded[path]


def select_library(which: str = "release"):
    """Make every call of this module go to one build of the library: "release" (libspdy_dp.so, the
    default), "debug" (libspdy_dp_debug.so, index checks inside the kernels) or "host"
    (libspdy_plan_host.so: plans and host helpers only, no device).  Returns the library.  Plans made
    with one build must not be handed to another."""
    global _lib
    path = {"release": LIB_PATH, "debug": DEBUG_LIB_PATH, "host": HOST_LIB_PATH}[which]
    _lib = open_library(path, host_only=(which == "host"))
    return _lib


def _load():
    global _lib
    if _lib is None:
        _lib = open_library(LIB_PATH)
    return _lib


def library():
    """The loaded ``ctypes.CDLL`` (raises if the library has not been built)."""
    return _load()


def _check(status: int, where: str):
    if status != 0:
        raise SpdyError(status, where)


def _stream_handle(stream) -> Optional[int]:
    import torch

    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class Plan:
    """``spdy_plan``: everything that depends only on ``times`` and ``B``."""

    def __init__(self, times, B: int, device: int = 0, table_format: int = SPDY_TABLE_DEFAULT,
                 threads: int = 0, cluster: int = 0, forward_mode: int = 0, rows_in_global: int = 0,
                 kernel: int = SPDY_KERNEL_AUTO, schedule: int = 0, auto_shape: int = 0):
        lib = _load()
        t = np.ascontiguousarray(np.asarray(times), dtype=np.int32)
        if t.ndim != 2:
            raise ValueError("times must be [L][K]")
        self.L, self.K, self.B, self.device = int(t.shape[0]), int(t.shape[1]), int(B), int(device)
        opts = SpdyOptions(table_format=table_format, threads=threads, cluster=cluster,
                           forward_mode=forward_mode, rows_in_global=rows_in_global, kernel=kernel,
                           schedule=schedule, auto_shape=auto_shape)
        self._lib = lib  # the build this plan belongs to
        handle = ctypes.c_void_p()
        _check(lib.spdy_plan_create(ctypes.byref(handle), t.ctypes.data_as(ctypes.c_void_p),
                                    self.L, self.K, self.B, self.device, ctypes.byref(opts)),
               "spdy_plan_create")
        self._h = handle
        self._ws = None

    def close(self):
        if getattr(self, "_h", None):
            self._lib.spdy_plan_destroy(self._h)
            self._h = None
        self._ws = None

    __del__ = close

    @property
    def info(self) -> dict:
        out = SpdyPlanInfo()
        _check(_load().spdy_plan_get_info(self._h, ctypes.byref(out)), "spdy_plan_get_info")
        return out.as_dict()

    def bands(self):
        lo = np.empty(self.L, np.int32)
        width = np.empty(self.L, np.int32)
        _check(_load().spdy_plan_get_bands(self._h, lo.ctypes.data_as(ctypes.c_void_p),
                                           width.ctypes.data_as(ctypes.c_void_p)),
               "spdy_plan_get_bands")
        return lo, width

    def workspace_bytes(self, N: int) -> int:
        return int(_load().spdy_workspace_bytes(self._h, int(N)))

    def verify(self):
        """``spdy_plan_verify``: the host-side proof that every access of the kernels stays in bounds."""
        _check(_load().spdy_plan_verify(self._h), "spdy_plan_verify")

    def tables(self, which: int = 0) -> dict:
        """``spdy_plan_get_tables`` as NumPy copies: ``which`` 0 = main launch shape, -1 = the byte table's
        merged set, i >= 1 = the i-th launch shape for small batches."""
        t = SpdyPlanTables()
        _check(_load().spdy_plan_get_tables(self._h, int(which), ctypes.byref(t)), "spdy_plan_get_tables")

        def arr(ptr, ctype, shape):
            n = int(np.prod(shape))
            if not ptr or n == 0:
                return np.zeros(shape, dtype=np.dtype(ctype))
            return np.ctypeslib.as_array(ctypes.cast(ptr, ctypes.POINTER(ctype)), shape=(n,)).reshape(shape).copy()

        out = {name: int(getattr(t, name)) for name, ct in SpdyPlanTables._fields_ if ct is not ctypes.c_void_p}
        W = max(1, out["warps_per_candidate"])
        out["layers"] = arr(t.layers, ctypes.c_int32, (out["L"], 8))
        out["slots"] = arr(t.slots, ctypes.c_int32, (out["L"], out["K"], 2))
        out["passes"] = arr(t.passes, ctypes.c_int32, (out["n_passes"], 2))
        out["pass_masks"] = arr(t.pass_masks, ctypes.c_uint64, (out["n_passes"], out["mask_words"]))
        out["pass_ptr"] = arr(t.pass_ptr, ctypes.c_int32, (out["L"] * W + 1,)) if t.pass_ptr else None
        out["slices"] = arr(t.slices, ctypes.c_int32, (out["L"], out["cluster"], 8)) if t.slices else None
        return out

    def shape_for_batch(self, N: int, workspace_bytes: Optional[int] = None) -> dict:
        """The launch shape ``spdy_solve_batch`` would use for N candidates (``spdy_plan_shape_for_batch``):
        kernel kind, threads per CTA, CTAs per candidate, and the table-set index."""
        ws = self.workspace_bytes(N) if workspace_bytes is None else int(workspace_bytes)
        which = int(_load().spdy_plan_shape_for_batch(self._h, int(N), ws))
        t = SpdyPlanTables()
        _check(_load().spdy_plan_get_tables(self._h, which, ctypes.byref(t)), "spdy_plan_get_tables")
        return {"which": which, "kernel_kind": int(t.kernel_kind), "threads": int(t.threads), "cluster": int(t.cluster)}

    def status_word(self, stream=None) -> int:
        """``spdy_plan_status_word``: read and clear the self-check word (0 = nothing flagged)."""
        word = ctypes.c_int32()
        _check(_load().spdy_plan_status_word(self._h, _stream_handle(stream), ctypes.byref(word)),
               "spdy_plan_status_word")
        return int(word.value)

    def enable_timing(self, on: bool = True):
        _check(_load().spdy_plan_enable_timing(self._h, int(on)), "spdy_plan_enable_timing")

    def last_timing(self):
        """(forward_ms, walkback_ms) of the last solve; waits for it."""
        f, w = ctypes.c_float(), ctypes.c_float()
        _check(_load().spdy_plan_last_timing(self._h, ctypes.byref(f), ctypes.byref(w)),
               "spdy_plan_last_timing")
        return float(f.value), float(w.value)

    def check_status(self, stream=None):
        _check(_load().spdy_plan_check_status(self._h, _stream_handle(stream)),
               "spdy_plan_check_status")


def solve_batch(plan: Plan, errors, profile=None, cost=None, time_used=None, workspace=None,
                stream=None):
    """``spdy_solve_batch`` on device tensors.  ``errors`` is a contiguous CUDA fp32 tensor
    [N][L][K]; outputs and workspace are allocated with torch when not given.  Asynchronous on
    ``stream`` (default: torch's current stream).  Returns (profile u8 [N][L], cost f32 [N],
    time_used i32 [N])."""
    import torch

    if not (errors.is_cuda and errors.dtype == torch.float32 and errors.is_contiguous()):
        raise ValueError("errors must be a contiguous CUDA float32 tensor")
    if errors.dim() != 3 or errors.shape[1] != plan.L or errors.shape[2] != plan.K:
        raise ValueError("errors must be [N][L][K] matching the plan")
    N = int(errors.shape[0])
    dev = errors.device
    if profile is None:
        profile = torch.empty((N, plan.L), dtype=torch.uint8, device=dev)
    if cost is None:
        cost = torch.empty(N, dtype=torch.float32, device=dev)
    if time_used is None:
        time_used = torch.empty(N, dtype=torch.int32, device=dev)
    if workspace is None:
        need = plan.workspace_bytes(N)
        if plan._ws is None or plan._ws.numel() < need or plan._ws.device != dev:
            plan._ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        workspace = plan._ws
    _check(_load().spdy_solve_batch(plan._h, errors.data_ptr(), N, profile.data_ptr(),
                                    cost.data_ptr(), time_used.data_ptr(), workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(),
                                    _stream_handle(stream)), "spdy_solve_batch")
    return profile, cost, time_used


def solve_batch_host(plan: Plan, errors: np.ndarray, profile=None, cost=None, time_used=None,
                     stream=None):
    """``spdy_solve_batch_host``: NumPy (or pinned torch CPU) buffers in and out, copies included."""
    def addr(x):
        return x.ctypes.data if isinstance(x, np.ndarray) else x.data_ptr()

    N = int(errors.shape[0])
    if profile is None:
        profile = np.empty((N, plan.L), np.uint8)
    if cost is None:
        cost = np.empty(N, np.float32)
    if time_used is None:
        time_used = np.empty(N, np.int32)
    _check(_load().spdy_solve_batch_host(plan._h, addr(errors), N, addr(profile), addr(cost),
                                         addr(time_used), _stream_handle(stream)),
           "spdy_solve_batch_host")
    return profile, cost, time_used


def solve_batch_simple(errors, times, B: int, stream=None):
    """``spdy_solve_batch_simple``: the one-shot call (errors, times on the device, budget) ->
    (profile, cost, time_used); synchronous."""
    import torch

    N, L, K = (int(x) for x in errors.shape)
    dev = errors.device
    profile = torch.empty((N, L), dtype=torch.uint8, device=dev)
    cost = torch.empty(N, dtype=torch.float32, device=dev)
    time_used = torch.empty(N, dtype=torch.int32, device=dev)
    _check(_load().spdy_solve_batch_simple(errors.data_ptr(), times.data_ptr(), N, L, K, int(B),
                                           profile.data_ptr(), cost.data_ptr(),
                                           time_used.data_ptr(), _stream_handle(stream)),
           "spdy_solve_batch_simple")
    return profile, cost, time_used


def solve_batch_static(errors, times, B: int, profile=None, cost=None, time_used=None, stream=None):
    """``spdy_solve_batch_static``: the whole path without any device allocation by the library.
    For callers that may not allocate on the device (a framework owns the heap, or the memory
    budget is fixed at start-up): the library works inside an array compiled into it.  ``errors``
    is a CUDA fp32 tensor [N][L][K], ``times`` a host int32 array [L][K]; pass the three output
    tensors to keep this wrapper from allocating them with torch.  Synchronous.  Calls must not
    overlap on one device, and the first call per device must come before any stream capture."""
    import torch

    t = np.ascontiguousarray(np.asarray(times), dtype=np.int32)
    N, L, K = (int(x) for x in errors.shape)
    if t.shape != (L, K):
        raise ValueError("times must be [L][K] matching errors")
    dev = errors.device
    if profile is None:
        profile = torch.empty((N, L), dtype=torch.uint8, device=dev)
    if cost is None:
        cost = torch.empty(N, dtype=torch.float32, device=dev)
    if time_used is None:
        time_used = torch.empty(N, dtype=torch.int32, device=dev)
    _check(_load().spdy_solve_batch_static(errors.data_ptr(), t.ctypes.data_as(ctypes.c_void_p), N, L,
                                           K, int(B), profile.data_ptr(), cost.data_ptr(),
                                           time_used.data_ptr(), _stream_handle(stream)),
           "spdy_solve_batch_static")
    return profile, cost, time_used


def solve_batch_coeffs(plan: Plan, coeffs, profile=None, cost=None, time_used=None, workspace=None,
                       stream=None):
    """``spdy_solve_batch_coeffs``: like ``solve_batch`` with Eq. 4's sensitivity coefficients
    (contiguous CUDA fp32 tensor [N][L]) in place of an error table."""
    import torch

    if not (coeffs.is_cuda and coeffs.dtype == torch.float32 and coeffs.is_contiguous()):
        raise ValueError("coeffs must be a contiguous CUDA float32 tensor")
    if coeffs.dim() != 2 or coeffs.shape[1] != plan.L:
        raise ValueError("coeffs must be [N][L] matching the plan")
    N = int(coeffs.shape[0])
    dev = coeffs.device
    if profile is None:
        profile = torch.empty((N, plan.L), dtype=torch.uint8, device=dev)
    if cost is None:
        cost = torch.empty(N, dtype=torch.float32, device=dev)
    if time_used is None:
        time_used = torch.empty(N, dtype=torch.int32, device=dev)
    if workspace is None:
        need = plan.workspace_bytes(N)
        if plan._ws is None or plan._ws.numel() < need or plan._ws.device != dev:
            plan._ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        workspace = plan._ws
    _check(_load().spdy_solve_batch_coeffs(plan._h, coeffs.data_ptr(), N, profile.data_ptr(),
                                           cost.data_ptr(), time_used.data_ptr(), workspace.data_ptr(),
                                           workspace.numel() * workspace.element_size(),
                                           _stream_handle(stream)), "spdy_solve_batch_coeffs")
    return profile, cost, time_used


def solve_batch_coeffs_host(plan: Plan, coeffs, profile=None, cost=None, time_used=None, stream=None):
    """``spdy_solve_batch_coeffs_host``: coefficients [N][L] and outputs in host memory (NumPy or
    pinned torch CPU tensors), copies included."""
    def addr(x):
        return x.ctypes.data if isinstance(x, np.ndarray) else x.data_ptr()

    if isinstance(coeffs, np.ndarray):
        coeffs = np.ascontiguousarray(coeffs, dtype=np.float32)
    N = int(coeffs.shape[0])
    if profile is None:
        profile = np.empty((N, plan.L), np.uint8)
    if cost is None:
        cost = np.empty(N, np.float32)
    if time_used is None:
        time_used = np.empty(N, np.int32)
    _check(_load().spdy_solve_batch_coeffs_host(plan._h, addr(coeffs), N, addr(profile), addr(cost),
                                                addr(time_used), _stream_handle(stream)),
           "spdy_solve_batch_coeffs_host")
    return profile, cost, time_used


def quadratic_errors(coeffs, K: int, stream=None):
    """``spdy_quadratic_errors``: Eq. 4's error table [N][L][K] for coefficients [N][L] (CUDA fp32)."""
    import torch

    N, L = (int(x) for x in coeffs.shape)
    out = torch.empty((N, L, int(K)), dtype=torch.float32, device=coeffs.device)
    _check(_load().spdy_quadratic_errors(coeffs.data_ptr(), N, L, int(K), out.data_ptr(),
                                         _stream_handle(stream)), "spdy_quadratic_errors")
    return out


def time_target(t_dense: float, speedup: float, t_base: float = 0.0) -> float:
    """``spdy_time_target``: T_dense / X - T_base."""
    return float(_load().spdy_time_target(float(t_dense), float(speedup), float(t_base)))


def bucketize_times(times, T: float, B: int, rounding: str = "nearest") -> np.ndarray:
    """``spdy_bucketize_times``: real layer times [L][K] -> int32 buckets of width T / B."""
    t = np.ascontiguousarray(np.asarray(times), dtype=np.float64)
    if t.ndim != 2:
        raise ValueError("times must be [L][K]")
    mode = {"nearest": 0, "up": 1}[rounding]
    out = np.empty(t.shape, np.int32)
    _check(_load().spdy_bucketize_times(t.ctypes.data_as(ctypes.c_void_p), int(t.shape[0]), int(t.shape[1]),
                                        float(T), int(B), mode, out.ctypes.data_as(ctypes.c_void_p)),
           "spdy_bucketize_times")
    return out


def uniform_profile(times, B: int, keep_dense=None):
    """``spdy_uniform_profile``: (lowest common choice index that fits B, its total time) or (-1, -1)."""
    t = np.ascontiguousarray(np.asarray(times), dtype=np.int32)
    keep = None if keep_dense is None else np.ascontiguousarray(np.asarray(keep_dense), dtype=np.uint8)
    k, total = ctypes.c_int32(), ctypes.c_int64()
    _check(_load().spdy_uniform_profile(t.ctypes.data_as(ctypes.c_void_p), int(t.shape[0]), int(t.shape[1]), int(B),
                                        None if keep is None else keep.ctypes.data_as(ctypes.c_void_p),
                                        ctypes.byref(k), ctypes.byref(total)), "spdy_uniform_profile")
    return int(k.value), int(total.value)


def probe_peaks(device: int = 0):
    """``spdy_probe_peaks``: (shared-memory 4-byte reads per second, arithmetic-only cell updates per second)."""
    lds, alu = ctypes.c_double(), ctypes.c_double()
    _check(_load().spdy_probe_peaks(int(device), ctypes.byref(lds), ctypes.byref(alu)), "spdy_probe_peaks")
    return float(lds.value), float(alu.value)
