"""Pins of the oracle's search-side functions (Eq. 4 errors, time target, discretisation, the uniform
baseline, Algorithm 4) against exact rational arithmetic, closed forms, brute force and invariants."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import workloads as W


def round_to_f32(x: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) fp32 value of an exact rational."""
    guess = np.float32(float(x))
    cands = {guess, np.nextafter(guess, np.float32(np.inf)), np.nextafter(guess, np.float32(-np.inf))}
    best = None
    for c in cands:
        if not np.isfinite(c):
            continue
        err = abs(Fraction(float(c)) - x)
        even = (int(np.float32(c).view(np.uint32)) & 1) == 0
        key = (err, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, np.float32(c))
    return best[1]


@pytest.mark.parametrize("K", [2, 3, 5, 7, 42, 64])
def test_eq4_errors_are_the_correctly_rounded_product(K):
    rng = np.random.default_rng(K)
    c = rng.uniform(0.0, 1.0, size=(3, 4)).astype(np.float32)
    c[0, 0], c[0, 1], c[1, 0] = 0.0, 1.0, np.float32(1e-30)
    e = oracle.quadratic_errors(c, K)
    assert e.shape == (3, 4, K) and e.dtype == np.float32
    for n in range(3):
        for l in range(4):
            for i in range(K):
                q = round_to_f32(Fraction(i, K - 1) ** 2)
                want = round_to_f32(Fraction(float(c[n, l])) * Fraction(float(q)))
                assert e[n, l, i].tobytes() == want.tobytes(), (n, l, i)


def test_eq4_closed_forms():
    c = np.array([[0.3, 0.7, 1.0, 0.0]], np.float32)
    e5 = oracle.quadratic_errors(c, 5)  # (i/4)^2 = 0, 1/16, 1/4, 9/16, 1: all exact in fp32
    for i, (num, den) in enumerate([(0, 1), (1, 16), (1, 4), (9, 16), (1, 1)]):
        exact = np.array([round_to_f32(Fraction(float(x)) * Fraction(num, den)) for x in c[0]], np.float32)
        assert e5[0, :, i].tobytes() == exact.tobytes()
    for K in (2, 3, 42):
        e = oracle.quadratic_errors(c, K)
        assert (e[:, :, 0] == 0).all() and e[:, :, K - 1].tobytes() == c.tobytes()
        assert (np.diff(e, axis=2) >= 0).all()  # non-decreasing in the sparsity index for c >= 0
    assert (oracle.quadratic_errors(c, 1) == 0).all()
    assert oracle.quadratic_errors(np.array([[0.5]], np.float32), 3)[0, 0, 1] == np.float32(0.125)


def test_time_target_closed_forms():
    assert oracle.time_target(2.0, 1.0) == 2.0
    assert oracle.time_target(0.478, 2.0, 0.0) == 0.239
    assert oracle.time_target(3.0, 2.0, 1.5) == 0.0
    assert oracle.time_target(1.0, 4.0, 0.125) == 0.125
    with pytest.raises(ValueError):
        oracle.time_target(1.0, 0.0)


def test_discretisation_bounds_and_exact_cases():
    rng = np.random.default_rng(3)
    T, B = 8.0, 1 << 12  # bucket width 2^-9: multiples are exact
    width = T / B
    exact = rng.integers(0, 3000, size=(5, 6)) * width
    for mode in ("nearest", "up"):
        assert np.array_equal(oracle.bucketize_times(exact, T, B, mode), np.rint(exact / width).astype(np.int32))
    assert oracle.bucketize_times(np.array([[T]]), T, B)[0, 0] == B  # the budget T becomes B
    t = rng.uniform(0.0, 3.0, size=(7, 9))
    near = oracle.bucketize_times(t, T, B, "nearest").astype(np.float64)
    up = oracle.bucketize_times(t, T, B, "up").astype(np.float64)
    assert (np.abs(near * width - t) <= width / 2 * (1 + 1e-12)).all()
    assert (up * width >= t * (1 - 1e-15)).all() and (up * width < t + width).all()
    assert (up >= near - 0).all() and (up - near <= 1).all()
    half = np.array([[0.5 * width, 1.5 * width, 2.5 * width]])
    assert oracle.bucketize_times(half, T, B, "nearest").tolist() == [[1, 2, 3]]  # halves away from zero
    # "up" keeps the guarantee: a profile within B buckets is within T seconds
    for _ in range(50):
        pick = rng.integers(0, 9, size=7)
        if up[np.arange(7), pick].sum() <= B:
            assert t[np.arange(7), pick].sum() <= T * (1 + 1e-12)
    for bad in (dict(T=0.0, B=10), dict(T=1.0, B=0)):
        with pytest.raises(ValueError):
            oracle.bucketize_times(t, **bad)
    with pytest.raises(ValueError):
        oracle.bucketize_times(-t, T, B)


def test_uniform_profile_is_the_first_feasible_common_choice():
    rng = np.random.default_rng(4)
    for trial in range(200):
        L, K = int(rng.integers(1, 7)), int(rng.integers(1, 6))
        times = np.sort(rng.integers(0, 30, size=(L, K)), axis=1)[:, ::-1].astype(np.int32)  # faster when sparser
        if trial % 3 == 0:
            times = rng.integers(0, 30, size=(L, K)).astype(np.int32)  # not monotone either
        B = int(rng.integers(0, 25 * L))
        keep = rng.random(L) < 0.3
        k, total = oracle.uniform_profile(times, B, keep)
        totals = [int(sum(times[l][0 if keep[l] else kk] for l in range(L))) for kk in range(K)]
        feasible = [kk for kk in range(K) if totals[kk] <= B]
        if not feasible:
            assert (k, total) == (-1, -1)
        else:
            assert k == feasible[0] and total == totals[k]
    wl = W.make_workload(2, N=1)
    k, total = oracle.uniform_profile(wl.times, wl.B)
    assert 0 < k < wl.K and total <= wl.B < int(wl.times[:, k - 1].sum())


def _replay(c0, phase1, draws, accepted):
    c = np.array(c0, np.float32)
    for d, j in accepted:
        if d == 0:
            c = np.array(phase1[j], np.float32)
        else:
            idx, val = draws(d, j)
            c = c.copy()
            c[idx] = val
    return c


def _small_search_problem(seed):
    wl = W.make_workload(0, seed_shift=seed)  # L 8, K 4, B <= 256: one solve takes microseconds
    loss = W.synthetic_calibration_loss(seed, wl.L, wl.K, s_max=0.9)
    return wl, loss, W.sensitivity_samples(seed, wl.L, 1)[0], W.sensitivity_samples(seed + 100, wl.L, 12), \
        W.mutation_draws(seed, wl.L)


@pytest.mark.parametrize("seed", range(6))
def test_algorithm4_bookkeeping_and_invariants(seed):
    wl, loss, c0, phase1, draws = _small_search_problem(seed)
    r = oracle.search(wl.times, wl.B, c0, phase1, draws, loss, trials=12, delta=0.3)
    dmax = math.ceil(0.3 * wl.L)
    assert r["evals"] == 1 + 12 + 12 * dmax
    # the result is reproduced by replaying the accepted trials from the recorded random draws
    assert _replay(c0, phase1, draws, r["accepted"]).tobytes() == r["c"].tobytes()
    # it is consistent: profile = dynamic program on Eq. 4's errors of c, loss = eval of that profile
    p, _, _ = oracle.solve_batch(oracle.quadratic_errors(r["c"][None], wl.K), wl.times, wl.B)
    assert np.array_equal(p[0], r["profile"]) and loss(p[0]) == r["loss"]
    # never worse than the start or any first-loop sample; accepted trials are in order
    for c in [c0, *phase1]:
        pc, _, _ = oracle.solve_batch(oracle.quadratic_errors(np.asarray(c)[None], wl.K), wl.times, wl.B)
        assert r["loss"] <= loss(pc[0])
    order = [(-(d if d else 10**6), j) for d, j in r["accepted"]]
    assert order == sorted(order)
    # losses along the accepted chain strictly decrease
    chain, prev = [], None
    c = np.array(c0, np.float32)
    pc, _, _ = oracle.solve_batch(oracle.quadratic_errors(c[None], wl.K), wl.times, wl.B)
    prev = loss(pc[0])
    for k in range(len(r["accepted"])):
        c = _replay(c0, phase1, draws, r["accepted"][: k + 1])
        pc, _, _ = oracle.solve_batch(oracle.quadratic_errors(c[None], wl.K), wl.times, wl.B)
        assert loss(pc[0]) < prev
        prev = loss(pc[0])
    assert prev == r["loss"]


def test_algorithm4_special_cases():
    wl, loss, c0, phase1, draws = _small_search_problem(11)
    # a constant loss never improves (strict "<"): the first sample survives
    r = oracle.search(wl.times, wl.B, c0, phase1, draws, lambda p: 1.0, trials=12, delta=0.3)
    assert r["accepted"] == [] and r["c"].tobytes() == c0.tobytes() and r["loss"] == 1.0
    # a loss that falls with every call accepts every trial
    calls = []

    def falling(p):
        calls.append(1)
        return -float(len(calls))

    r = oracle.search(wl.times, wl.B, c0, phase1, draws, falling, trials=5, delta=0.2)
    dmax = math.ceil(0.2 * wl.L)
    assert len(r["accepted"]) == 5 + 5 * dmax and r["evals"] == len(calls)
    # the text's stop rule: a neighbourhood size ends after `patience` trials without improvement
    r = oracle.search(wl.times, wl.B, c0, phase1, draws, lambda p: 1.0, trials=12, delta=0.3, patience=4)
    assert r["evals"] == 1 + 12 + 4 * math.ceil(0.3 * wl.L)
    rp = oracle.search(wl.times, wl.B, c0, phase1, draws, loss, trials=12, delta=0.3, patience=3)
    assert _replay(c0, phase1, draws, rp["accepted"]).tobytes() == rp["c"].tobytes()
    # an infeasible budget: every profile is 0xFF, the loss is +inf, nothing is accepted
    r = oracle.search(wl.times, int(wl.times.min(axis=1).sum()) - 1, c0, phase1, draws, loss, trials=3)
    assert r["loss"] == float("inf") and r["accepted"] == [] and (r["profile"] == 0xFF).all()
