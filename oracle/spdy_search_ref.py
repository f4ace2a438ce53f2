"""CPU oracle of what surrounds the dynamic program in SPDY's search.  TEST INFRASTRUCTURE ONLY:
tests, the smoke check and the benchmark's CPU-baseline leg may import it, product code may not.

Plain NumPy / Python, written from the paper's statements, one function per statement:

* ``quadratic_errors``  - the error model of Section 3.3, Eq. 4;
* ``time_target``       - the execution-time target for a speedup target (Section 3.1);
* ``bucketize_times``   - time discretisation into B buckets of width T / B (Section 3.2);
* ``uniform_profile``   - the "uniform" baseline profile of Section 4 (minimal sparsity that meets the
  time target with one sparsity for all layers);
* ``search``            - the search for sensitivity coefficients of Section 3.3 / Appendix A,
  Algorithm 4, sequential, one dynamic program per evaluation.

Readings adopted where the paper leaves room (mirrored by the CUDA library so that results can be
compared bit for bit):
* Eq. 4 is evaluated as e = fl32(c * q_i) with q_i = fl32((i / (|S| - 1))^2) formed in fp64 and
  rounded once; |S| = 1 gives q_0 = 0.  The paper states no precision.
* Discretisation: a time t becomes t * B / T buckets (fp64, in this order of operations), rounded
  to the nearest integer, halves away from zero ("nearest"), or up ("up", which keeps the
  guarantee sum of real times <= T whenever the bucket sum is <= B).  The paper says only
  "buckets of width T / B".
* Algorithm 4 runs a fixed number of trials per neighbourhood size d, while the text of
  Section 3.3 stops a size after 100 trials without improvement; ``patience=None`` follows
  Algorithm 4, an integer follows the text.
* The random numbers the search draws are inputs (``phase1`` and ``draws``), so that two
  implementations can be fed the same ones.
"""
from __future__ import annotations

import math
from typing import Callable, Optional, Sequence

import numpy as np

from .spdy_ref import solve_batch


def quadratic_errors(c: np.ndarray, K: int) -> np.ndarray:
    """Eq. 4: e[n][l][i] = c[n][l] * (i / (K - 1))^2 for i = 0..K-1, as one fp32 multiply of c with
    the fp32-rounded square.  c is [N][L]; returns [N][L][K] fp32."""
    c = np.asarray(c, dtype=np.float32)
    if c.ndim != 2 or K < 1:
        raise ValueError("c must be [N][L] and K >= 1")
    if K == 1:
        q = np.zeros(1, dtype=np.float32)
    else:
        q = ((np.arange(K, dtype=np.float64) / np.float64(K - 1)) ** 2).astype(np.float32)
    return (c[:, :, None] * q[None, None, :]).astype(np.float32)


def time_target(t_dense: float, speedup: float, t_base: float = 0.0) -> float:
    """Section 3.1: the execution-time target of a speedup target X is T_dense / X - T_base."""
    if not speedup > 0:
        raise ValueError("speedup must be positive")
    return float(np.float64(t_dense) / np.float64(speedup) - np.float64(t_base))


def bucketize_times(times: np.ndarray, T: float, B: int, rounding: str = "nearest") -> np.ndarray:
    """Section 3.2: buckets of width T / B, so that the budget T becomes B.  times [L][K] fp64 -> int32."""
    times = np.asarray(times, dtype=np.float64)
    if not (T > 0 and B >= 1) or (times < 0).any() or not np.isfinite(times).all():
        raise ValueError("need T > 0, B >= 1 and finite non-negative times")
    v = times * np.float64(B) / np.float64(T)
    if rounding == "nearest":
        out = np.floor(v + 0.5)
    elif rounding == "up":
        out = np.ceil(v)
    else:
        raise ValueError("rounding must be 'nearest' or 'up'")
    if (out > 2**31 - 1).any():
        raise ValueError("a time does not fit int32 buckets")
    return out.astype(np.int32)


def uniform_profile(times: np.ndarray, B: int, keep_dense: Optional[Sequence[bool]] = None):
    """Section 4, baseline "uniform": the lowest choice index k (choices ordered by increasing
    sparsity) such that giving every layer choice k - except layers flagged in ``keep_dense``, which
    stay at choice 0 - fits the budget.  Returns (k, total time), or (-1, -1) if no k fits."""
    times = np.asarray(times, dtype=np.int64)
    L, K = times.shape
    keep = np.zeros(L, dtype=bool) if keep_dense is None else np.asarray(keep_dense, dtype=bool)
    for k in range(K):
        total = 0
        for l in range(L):
            total += int(times[l][0 if keep[l] else k])
        if total <= B:
            return k, total
    return -1, -1


def search(times: np.ndarray, B: int, c0: np.ndarray, phase1: np.ndarray,
           draws: Callable[[int, int], tuple], eval_fn: Callable[[np.ndarray], float],
           trials: int = 100, delta: float = 0.1, patience: Optional[int] = None):
    """Algorithm 4 (Appendix A), sequentially.

    ``c0`` [L] is the first sampled coefficient vector, ``phase1`` [trials][L] the further uniform
    samples of the first loop, ``draws(d, j)`` returns the (indices [d], values [d]) that trial j
    of neighbourhood size d resamples.  ``eval_fn(profile)`` stands for the calibration loss of the
    stitched model of a profile (lower is better; an infeasible profile, all 0xFF, must score
    +inf).  eval(c) = eval_fn(profile of the dynamic program run on Eq. 4's errors for c).

    Returns a dict with the final ``c``, its ``profile`` and ``loss``, the number of ``evals`` and the
    list ``accepted`` of (d, j) trials that replaced c* (d = 0 for the first loop).
    """
    times = np.ascontiguousarray(times, dtype=np.int32)
    L, K = times.shape
    evals = 0

    def ev(c):
        nonlocal evals
        evals += 1
        errors = quadratic_errors(np.asarray(c, np.float32)[None, :], K)
        profile, _, _ = solve_batch(errors, times, B)
        return float(eval_fn(profile[0])), profile[0]

    c_star = np.array(c0, dtype=np.float32)
    best, prof_star = ev(c_star)
    accepted = []
    for j in range(trials):
        c = np.array(phase1[j], dtype=np.float32)
        v, prof = ev(c)
        if v < best:
            c_star, best, prof_star = c, v, prof
            accepted.append((0, j))
    for d in range(int(math.ceil(delta * L)), 0, -1):
        j = 0
        since_improved = 0
        while (j < trials) if patience is None else (since_improved < patience):
            c = c_star.copy()
            idx, val = draws(d, j)
            c[np.asarray(idx)] = np.asarray(val, dtype=np.float32)
            v, prof = ev(c)
            if v < best:
                c_star, best, prof_star = c, v, prof
                accepted.append((d, j))
                since_improved = 0
            else:
                since_improved += 1
            j += 1
    return {"c": c_star, "profile": prof_star, "loss": best, "evals": evals, "accepted": accepted}
