"""SPDY's search for sensitivity coefficients (Section 3.3; Appendix B, Algorithm 4) with the dynamic
programs of many trials solved in one GPU batch: a thin binding of ``spdy_search``.

Algorithm 4 is sequential: every trial mutates the current best vector c* and replaces it when the
mutated vector's profile evaluates better.  What a trial resamples (which entries, which values) does
not depend on c*, though, so the library forms the proposals of all remaining trials of a neighbourhood
size from the current c* at once and solves their dynamic programs as one batch
(``spdy_solve_batch_coeffs_host``: Eq. 4's errors are formed inside the kernels).  The profiles are then
evaluated one by one in trial order, stopping at the first improvement; the proposals behind it were
built from a c* that is now stale and are rebuilt in the next batch.  Trial for trial this takes the
same decisions as the sequential algorithm and calls the (expensive) evaluation exactly as often; only
dynamic programs are solved speculatively.  The loop itself runs in the library (``csrc/spdy_search.cpp``);
this module only marshals arguments and callbacks.

The evaluation - the calibration loss of the model stitched together for a profile, Section 3.4 - is
the caller's: ``eval_fn(profile) -> float``, lower is better, +inf for an infeasible profile (bytes
0xFF).  The random numbers are the caller's too (``c0``, ``phase1``, ``draws``), see ``workloads``.
"""
from __future__ import annotations

import ctypes
import math
from typing import Callable, Optional

import numpy as np

__all__ = ["search", "gpu_solver"]


def gpu_solver(times, B: int, device: int = 0, **plan_options):
    """``solver(coeffs [N][L] fp32) -> profiles [N][L] uint8`` on the CUDA library (host buffers in and
    out).  One plan serves every batch of a search: ``times`` and ``B`` never change during it."""
    from . import binding

    plan = binding.Plan(times, B, device=device, **plan_options)

    def solver(coeffs: np.ndarray) -> np.ndarray:
        profile, _, _ = binding.solve_batch_coeffs_host(plan, np.ascontiguousarray(coeffs, dtype=np.float32))
        plan.check_status()
        return profile

    solver.plan = plan
    return solver


def search(times, B: int, c0, phase1, draws: Callable[[int, int], tuple],
           eval_fn: Callable[[np.ndarray], float], trials: int = 100, delta: float = 0.1,
           patience: Optional[int] = None, solver: Optional[Callable[[np.ndarray], np.ndarray]] = None,
           device: int = 0, max_batch: int = 65536) -> dict:
    """Algorithm 4 with batched dynamic programs (``spdy_search``).

    ``c0`` [L]: the first sampled vector; ``phase1`` [trials][L]: the samples of the first loop;
    ``draws(d, j)`` -> (indices [d], values [d]) resampled by trial j of neighbourhood size d.
    ``patience=None`` runs ``trials`` trials per size as Algorithm 4 prints it; an integer stops a
    size after that many trials in a row without improvement, as the text of Section 3.3 says.
    ``solver``: None = the CUDA library on ``device`` (there is no CPU implementation here); the result of
    ``gpu_solver`` = the CUDA library on that solver's plan; any other callable ``coeffs [n][L] ->
    profiles [n][L]`` is handed to the library's loop as its solver callback (tests pass the oracle).

    Returns a dict: ``c`` [L] fp32, ``profile`` [L] uint8, ``loss``, ``evals`` (calls of ``eval_fn``),
    ``accepted`` (list of (d, j), d = 0 for the first loop), ``dp_batches``, ``dp_candidates``, and the wall
    time spent in the solver and in ``eval_fn`` (``dp_seconds``, ``eval_seconds``).
    """
    from . import binding

    lib = binding.library()
    times = np.ascontiguousarray(np.asarray(times), dtype=np.int32)
    L = int(times.shape[0])
    c0 = np.ascontiguousarray(np.asarray(c0), dtype=np.float32)
    phase1 = np.ascontiguousarray(np.asarray(phase1, dtype=np.float32)[:trials]).reshape(-1, L)
    trials_run = int(phase1.shape[0]) if patience is None else int(trials)
    if patience is not None and phase1.shape[0] < trials:
        raise ValueError("phase1 must hold `trials` vectors")
    plan = getattr(solver, "plan", None)
    callback_solver = solver if plan is None else None
    if plan is None:
        plan = binding.Plan(times, B, device=-1 if callback_solver is not None else device)
    failure = []

    def draw_cb(d, trial, idx_ptr, val_ptr, _user):
        try:
            idx, val = draws(int(d), int(trial))
            for q in range(int(d)):
                idx_ptr[q] = int(idx[q])
                val_ptr[q] = float(val[q])
        except BaseException as exc:  # surfaces after the call: exceptions cannot cross the C frames
            failure.append(exc)
            for q in range(int(d)):
                idx_ptr[q], val_ptr[q] = q % max(L, 1), 0.0

    def eval_cb(profile_ptr, n, _user):
        try:
            return float(eval_fn(np.ctypeslib.as_array(profile_ptr, shape=(int(n),)).copy()))
        except BaseException as exc:
            failure.append(exc)
            return math.inf

    def solve_cb(coeffs_ptr, n, profile_ptr, _user):
        try:
            coeffs = np.ctypeslib.as_array(coeffs_ptr, shape=(int(n), L)).copy()
            out = np.ascontiguousarray(np.asarray(callback_solver(coeffs)), dtype=np.uint8).reshape(int(n), L)
            np.ctypeslib.as_array(profile_ptr, shape=(int(n), L))[...] = out
            return 0
        except BaseException as exc:
            failure.append(exc)
            return -6

    opts = binding.SpdySearchOptions(trials=trials_run, patience=0 if patience is None else int(patience),
                                     delta=float(delta), max_batch=int(max_batch))
    result = binding.SpdySearchResult()
    c_out = np.empty(L, np.float32)
    profile_out = np.empty(L, np.uint8)
    # room for the accepted trials: Algorithm 4 runs at most trials * (1 + ceil(delta L)) of them; with the
    # text's stop rule there is no bound, and a list that overflows is cut (``accepted_count`` has them all)
    capacity = max(65536, 1 + trials_run * (1 + int(math.ceil(delta * L))))
    acc_d, acc_j = np.empty(capacity, np.int32), np.empty(capacity, np.int32)
    vp = ctypes.c_void_p
    rc = lib.spdy_search(plan._h, c0.ctypes.data_as(vp), phase1.ctypes.data_as(vp), ctypes.byref(opts),
                         binding.DRAW_FN(draw_cb), None, binding.EVAL_FN(eval_cb), None,
                         binding.SOLVE_FN(solve_cb) if callback_solver is not None else binding.SOLVE_FN(0), None,
                         None, c_out.ctypes.data_as(vp), profile_out.ctypes.data_as(vp), ctypes.byref(result),
                         acc_d.ctypes.data_as(vp), acc_j.ctypes.data_as(vp), capacity)
    if failure:
        raise failure[0]
    binding._check(rc, "spdy_search")
    n_acc = min(int(result.accepted), capacity)
    return {"c": c_out, "profile": profile_out, "loss": float(result.loss),
            "accepted": [(int(acc_d[i]), int(acc_j[i])) for i in range(n_acc)], "accepted_count": int(result.accepted),
            "evals": int(result.evals), "dp_batches": int(result.dp_batches),
            "dp_candidates": int(result.dp_candidates), "dp_seconds": float(result.dp_seconds),
            "eval_seconds": float(result.eval_seconds)}
