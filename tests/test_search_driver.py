"""The batched search driver against the oracle's sequential Algorithm 4 on the same random draws:
same accepted trials, same final coefficients, profile and loss, and the same number of evaluations."""
import math

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import search as S, workloads as W


def oracle_solver(times, B):
    K = times.shape[1]
    return lambda c: oracle.solve_batch(oracle.quadratic_errors(c, K), times, B)[0]


def same_result(got, ref):
    assert got["accepted"] == ref["accepted"]
    assert got["c"].tobytes() == ref["c"].tobytes()
    assert np.array_equal(got["profile"], ref["profile"]) and got["loss"] == ref["loss"]
    assert got["evals"] == ref["evals"]


def problem(seed, trials):
    wl = W.make_workload(0, seed_shift=seed)
    return (wl, W.synthetic_calibration_loss(seed, wl.L, wl.K, s_max=0.9), W.sensitivity_samples(seed, wl.L, 1)[0],
            W.sensitivity_samples(seed + 100, wl.L, trials), W.mutation_draws(seed, wl.L))


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("patience", [None, 3])
def test_host_logic_of_the_batched_search(seed, patience):
    """CPU: the driver's batching, with the dynamic program supplied by the test, equals the
    sequential algorithm."""
    wl, loss, c0, phase1, draws = problem(seed, 12)
    ref = oracle.search(wl.times, wl.B, c0, phase1, draws, loss, trials=12, delta=0.3, patience=patience)
    got = S.search(wl.times, wl.B, c0, phase1, draws, loss, trials=12, delta=0.3, patience=patience,
                   solver=oracle_solver(wl.times, wl.B))
    same_result(got, ref)
    if patience is None:
        # one batch for the first loop; per size one batch per accepted trial, plus a last one unless
        # the size's final trial itself was accepted
        want = 1
        for d in range(math.ceil(0.3 * wl.L), 0, -1):
            js = [j for dd, j in ref["accepted"] if dd == d]
            want += len(js) + (0 if js and js[-1] == 11 else 1)
        assert got["dp_batches"] == want
    small = S.search(wl.times, wl.B, c0, phase1, draws, loss, trials=12, delta=0.3, patience=patience,
                     solver=oracle_solver(wl.times, wl.B), max_batch=2)
    same_result(small, ref)


def test_search_entry_point_checks_its_arguments_and_passes_failures_on():
    import ctypes

    from paper_2201_13096_b200 import binding

    wl, loss, c0, phase1, draws = problem(3, 4)
    solver = oracle_solver(wl.times, wl.B)
    with pytest.raises(ZeroDivisionError):  # an exception inside a callback comes back out of the call
        S.search(wl.times, wl.B, c0, phase1, draws, lambda p: 1 / 0, trials=4, solver=solver)
    with pytest.raises(ValueError):  # so does the failure of a solver callback (here: profiles of the wrong shape)
        S.search(wl.times, wl.B, c0, phase1, draws, loss, trials=4, solver=lambda c: np.zeros((1, 1)))
    lib = binding.library()
    plan = binding.Plan(wl.times, wl.B, device=-1)
    res = binding.SpdySearchResult()
    opts = binding.SpdySearchOptions(trials=4, patience=0, delta=0.3, max_batch=0)
    out_c, out_p = np.empty(wl.L, np.float32), np.empty(wl.L, np.uint8)
    vp = ctypes.c_void_p
    args = [plan._h, c0.ctypes.data_as(vp), phase1.ctypes.data_as(vp), ctypes.byref(opts), binding.DRAW_FN(lambda *a: None),
            None, binding.EVAL_FN(lambda *a: 0.0), None, binding.SOLVE_FN(0), None, None, out_c.ctypes.data_as(vp),
            out_p.ctypes.data_as(vp), ctypes.byref(res), None, None, 0]
    assert lib.spdy_search(*args) == -8  # no solver given and the plan has no device
    bad = list(args)
    bad[0] = None
    assert lib.spdy_search(*bad) == -1
    opts.delta = 1.5
    assert lib.spdy_search(*args) == -1


def test_special_cases_of_the_batched_search():
    wl, loss, c0, phase1, draws = problem(21, 6)
    solver = oracle_solver(wl.times, wl.B)
    flat = S.search(wl.times, wl.B, c0, phase1, draws, lambda p: 1.0, trials=6, delta=0.3, solver=solver)
    assert flat["accepted"] == [] and flat["c"].tobytes() == c0.tobytes()
    assert flat["dp_batches"] == 1 + math.ceil(0.3 * wl.L)  # nothing accepted: one batch per size
    calls = []

    def falling(p):
        calls.append(1)
        return -float(len(calls))

    ref = oracle.search(wl.times, wl.B, c0, phase1, draws, falling, trials=6, delta=0.3)
    calls.clear()
    got = S.search(wl.times, wl.B, c0, phase1, draws, falling, trials=6, delta=0.3, solver=solver)
    same_result(got, ref)  # every trial accepted: every batch is cut after its first proposal
    bad_B = int(wl.times.min(axis=1).sum()) - 1
    inf = S.search(wl.times, bad_B, c0, phase1, draws, loss, trials=3, solver=oracle_solver(wl.times, bad_B))
    assert inf["loss"] == float("inf") and (inf["profile"] == 0xFF).all()


@pytest.mark.gpu
@pytest.mark.parametrize("cfg,trials", [(0, 20), (1, 8), (2, 8)])
def test_search_on_the_gpu_matches_the_sequential_oracle(cfg, trials):
    """GPU: the dynamic programs run in the CUDA library (coefficient input through the C ABI)."""
    wl = W.make_workload(cfg, N=1)
    loss = W.synthetic_calibration_loss(cfg, wl.L, wl.K, s_max=0.9 if cfg == 0 else 0.99)
    c0 = W.sensitivity_samples(cfg, wl.L, 1)[0]
    phase1 = W.sensitivity_samples(cfg + 100, wl.L, trials)
    draws = W.mutation_draws(cfg, wl.L)
    delta = 0.3 if cfg == 0 else 0.05
    ref = oracle.search(wl.times, wl.B, c0, phase1, draws, loss, trials=trials, delta=delta)
    got = S.search(wl.times, wl.B, c0, phase1, draws, loss, trials=trials, delta=delta, device=0)
    same_result(got, ref)
    assert got["dp_candidates"] >= got["evals"]
