"""Checks written straight from the problem statement, independent of both solvers."""
from __future__ import annotations

import itertools

import numpy as np


def brute_force(errors_one: np.ndarray, times: np.ndarray, B: int):
    """Enumerate all K^L profiles (Eq. 1).  Returns (cost, time_used, profile) under the rule:
    minimum left-to-right fp32 sum, then minimum total time, then lexicographically smallest
    (k_L, ..., k_1); or (inf, -1, None) if no profile fits the budget with finite error."""
    L, K = times.shape
    grids = np.indices((K,) * L).reshape(L, -1)  # grids[l][p] = choice of layer l in profile p
    total_t = np.zeros(grids.shape[1], dtype=np.int64)
    acc = np.zeros(grids.shape[1], dtype=np.float32)
    for l in range(L):
        total_t += times[l][grids[l]].astype(np.int64)
        acc = (acc + errors_one[l][grids[l]].astype(np.float32)).astype(np.float32)
    ok = (total_t <= B) & np.isfinite(acc)
    if not ok.any():
        return np.float32(np.inf), -1, None
    cost = acc[ok].min()
    cand = np.flatnonzero(ok & (acc == cost))
    tmin = total_t[cand].min()
    cand = cand[total_t[cand] == tmin]
    keys = [tuple(int(grids[l][p]) for l in reversed(range(L))) for p in cand]
    best = cand[min(range(len(cand)), key=lambda i: keys[i])]
    return np.float32(cost), int(tmin), grids[:, best].astype(np.uint8)


def check_solution(errors_one, times, B, profile, cost, time_used):
    """Invariants every returned solution must satisfy (Eq. 1's constraint; exact-time rows)."""
    L, K = times.shape
    if time_used < 0:
        assert np.isinf(cost) and cost > 0
        assert (profile == 0xFF).all()
        return
    assert (profile < K).all()
    tt = int(sum(int(times[l][profile[l]]) for l in range(L)))
    assert tt == time_used <= B
    acc = np.float32(0.0)
    for l in range(L):
        acc = np.float32(acc + errors_one[l][profile[l]])
    assert acc.tobytes() == np.float32(cost).tobytes(), (acc, cost)


def knapsack_01(weights, values, capacity: int) -> int:
    """Textbook 0/1 knapsack (integer weights/values): best total value within capacity."""
    best = [0] * (capacity + 1)
    for w, v in zip(weights, values):
        for c in range(capacity, w - 1, -1):
            best[c] = max(best[c], best[c - w] + v)
    return best[capacity]


def profiles_iter(L, K):
    return itertools.product(range(K), repeat=L)
