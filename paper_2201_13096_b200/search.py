"""SPDY's search for sensitivity coefficients (Section 3.3; Appendix B, Algorithm 4) with the dynamic
programs of many trials solved in one GPU batch.

Algorithm 4 is sequential: every trial mutates the current best vector c* and replaces it when the
mutated vector's profile evaluates better.  What a trial resamples (which entries, which values) does
not depend on c*, though, so the proposals of all remaining trials of a neighbourhood size can be
formed from the current c* at once and their dynamic programs solved as one batch
(``spdy_solve_batch_coeffs``: Eq. 4's errors are formed inside the kernels).  The profiles are then
evaluated one by one in trial order, stopping at the first improvement; the proposals behind it were
built from a c* that is now stale and are rebuilt in the next batch.  Trial for trial this takes the
same decisions as the sequential algorithm and calls the (expensive) evaluation exactly as often; only
dynamic programs are solved speculatively.

The evaluation - the calibration loss of the model stitched together for a profile, Section 3.4 - is
the caller's: ``eval_fn(profile) -> float``, lower is better, +inf for an infeasible profile (bytes
0xFF).  The random numbers are the caller's too (``c0``, ``phase1``, ``draws``), see ``workloads``.
"""
from __future__ import annotations

import math
import time
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
    """Algorithm 4 with batched dynamic programs.

    ``c0`` [L]: the first sampled vector; ``phase1`` [trials][L]: the samples of the first loop;
    ``draws(d, j)`` -> (indices [d], values [d]) resampled by trial j of neighbourhood size d.
    ``patience=None`` runs ``trials`` trials per size as Algorithm 4 prints it; an integer stops a
    size after that many trials in a row without improvement, as the text of Section 3.3 says.
    ``solver`` defaults to the CUDA library on ``device``; there is no CPU implementation here.

    Returns a dict: ``c`` [L] fp32, ``profile`` [L] uint8, ``loss``, ``evals`` (calls of ``eval_fn``),
    ``accepted`` (list of (d, j), d = 0 for the first loop), ``dp_batches``, ``dp_candidates``, and the wall
    time spent in the solver and in ``eval_fn`` (``dp_seconds``, ``eval_seconds``).
    """
    times = np.ascontiguousarray(np.asarray(times), dtype=np.int32)
    L = int(times.shape[0])
    if solver is None:
        solver = gpu_solver(times, B, device=device)
    stats = {"evals": 0, "dp_batches": 0, "dp_candidates": 0, "dp_seconds": 0.0, "eval_seconds": 0.0}

    def solve(coeffs: np.ndarray) -> np.ndarray:
        out = []
        t0 = time.perf_counter()
        for lo in range(0, len(coeffs), max_batch):
            out.append(np.asarray(solver(coeffs[lo:lo + max_batch])))
            stats["dp_batches"] += 1
        stats["dp_candidates"] += len(coeffs)
        stats["dp_seconds"] += time.perf_counter() - t0
        return np.concatenate(out, axis=0)

    def evaluate(profile: np.ndarray) -> float:
        stats["evals"] += 1
        t0 = time.perf_counter()
        value = float(eval_fn(profile))
        stats["eval_seconds"] += time.perf_counter() - t0
        return value

    c_star = np.array(c0, dtype=np.float32)
    phase1 = np.asarray(phase1, dtype=np.float32)[:trials]
    profiles = solve(np.concatenate([c_star[None, :], phase1], axis=0))
    best, prof_star = evaluate(profiles[0]), profiles[0]
    accepted = []
    for j in range(len(phase1)):
        v = evaluate(profiles[1 + j])
        if v < best:
            c_star, best, prof_star = phase1[j].copy(), v, profiles[1 + j]
            accepted.append((0, j))

    for d in range(int(math.ceil(delta * L)), 0, -1):
        j = 0
        since_improved = 0
        while True:
            remaining = (trials - j) if patience is None else (patience - since_improved)
            if remaining <= 0:
                break
            count = min(remaining, max_batch)
            proposals = np.repeat(c_star[None, :], count, axis=0)
            for i in range(count):
                idx, val = draws(d, j + i)
                proposals[i, np.asarray(idx)] = np.asarray(val, dtype=np.float32)
            profiles = solve(proposals)
            improved_at = -1
            for i in range(count):
                v = evaluate(profiles[i])
                if v < best:
                    c_star, best, prof_star = proposals[i].copy(), v, profiles[i]
                    accepted.append((d, j + i))
                    improved_at = i
                    break
            if improved_at >= 0:
                j += improved_at + 1
                since_improved = 0
            else:
                j += count
                since_improved += count
    return {"c": c_star, "profile": np.asarray(prof_star, dtype=np.uint8), "loss": best,
            "accepted": accepted, **stats}
