"""Pins for the CPU oracle: things fixed by the paper's problem statement (Eq. 1-3, Algorithm 1)
and by mathematics, none of which re-use the oracle's own code."""
import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import workloads as W
from helpers import brute_force, check_solution, knapsack_01


def solve1(errors_one, times, B):
    p, c, t = oracle.solve_batch(errors_one[None], times, B)
    return p[0], c[0], int(t[0])


# ---- exhaustive enumeration (Eq. 1) -------------------------------------------------------

@pytest.mark.parametrize("seed", range(12))
def test_config0_matches_enumeration_of_all_4_pow_8_profiles(seed):
    wl = W.make_workload(0, seed_shift=seed)
    assert wl.times.shape == (8, 4) and wl.B <= 256
    p, c, t = solve1(wl.errors[0], wl.times, wl.B)
    bc, bt, bp = brute_force(wl.errors[0], wl.times, wl.B)
    assert c.tobytes() == bc.tobytes()  # fp32 cost is bit-exact (fl(x+e) is monotone in x)
    check_solution(wl.errors[0], wl.times, wl.B, p, c, t)
    # With generic real-valued errors the optimum is unique, so the profile is pinned too.
    assert t == bt and np.array_equal(p, bp)


@pytest.mark.parametrize("seed", range(300))
def test_random_tiny_instances_cost_and_feasibility(seed):
    wl = W.tiny_random_instance(seed)
    p, c, t = solve1(wl.errors[0], wl.times, wl.B)
    bc, bt, _ = brute_force(wl.errors[0], wl.times, wl.B)
    assert c.tobytes() == bc.tobytes()
    assert (t < 0) == (bt < 0)
    check_solution(wl.errors[0], wl.times, wl.B, p, c, t)


@pytest.mark.parametrize("seed", range(300))
def test_tie_breaks_on_exactly_representable_errors(seed):
    """Errors in {0, 1/4, ..., 1}: all sums exact, many equal-cost optima.  The canonical answer
    is min cost, then min total time, then lowest choice index from the last layer backwards
    (strict '<' over ascending choices in Algorithm 1; lowest t in the final argmin)."""
    wl = W.tiny_random_instance(10_000 + seed, exact=True)
    p, c, t = solve1(wl.errors[0], wl.times, wl.B)
    bc, bt, bp = brute_force(wl.errors[0], wl.times, wl.B)
    assert c.tobytes() == bc.tobytes() and t == bt
    if bp is None:
        assert (p == 0xFF).all()
    else:
        assert np.array_equal(p, bp)


def test_all_equal_errors_pick_lowest_indices():
    L, K, B = 5, 4, 40
    times = np.tile(np.array([4, 4, 2, 2], dtype=np.int32), (L, 1))
    errors = np.full((L, K), 0.5, dtype=np.float32)
    p, c, t = solve1(errors, times, B)
    bc, bt, bp = brute_force(errors, times, B)
    assert c == np.float32(2.5) and t == bt == 10 and np.array_equal(p, bp)
    assert (p == 2).all()  # min time first, then the lower of the two equal-time choices


# ---- closed forms --------------------------------------------------------------------------

@pytest.mark.parametrize("cfg", [0, 1, 2])
def test_budget_at_least_dense_time_gives_all_dense_zero_error(cfg):
    wl = W.make_workload(cfg, N=2)
    dense = int(wl.times[:, 0].sum())
    for B in (dense, dense + 17):
        p, c, t = oracle.solve_batch(wl.errors, wl.times, B)
        assert (p == 0).all() and (t == dense).all()
        assert all(x.tobytes() == np.float32(0.0).tobytes() for x in c)  # +0.0 exactly


@pytest.mark.parametrize("cfg", [0, 1, 2])
def test_budget_below_minimum_total_time_is_infeasible(cfg):
    wl = W.make_workload(cfg, N=2)
    tmin = int(wl.times.min(axis=1).sum())
    p, c, t = oracle.solve_batch(wl.errors, wl.times, tmin - 1)
    assert (p == 0xFF).all() and (t == -1).all() and np.isposinf(c).all()
    p, c, t = oracle.solve_batch(wl.errors, wl.times, tmin)  # exactly reachable: the all-min profile
    assert (t == tmin).all()
    assert np.array_equal(p[0], wl.times.argmin(axis=1).astype(np.uint8))


def test_single_choice_forces_the_profile():
    rng = np.random.default_rng(5)
    L = 9
    times = rng.integers(0, 6, size=(L, 1)).astype(np.int32)
    errors = rng.lognormal(size=(L, 1)).astype(np.float32)
    B = int(times.sum())
    p, c, t = solve1(errors, times, B)
    acc = np.float32(0)
    for l in range(L):
        acc = np.float32(acc + errors[l, 0])
    assert (p == 0).all() and t == B and c.tobytes() == acc.tobytes()
    p, c, t = solve1(errors, times, B - 1) if B > 0 else (None, np.float32(np.inf), -1)
    assert t == -1


def test_single_layer_picks_cheapest_choice_that_fits():
    times = np.array([[9, 7, 5, 5, 3, 11]], dtype=np.int32)
    errors = np.array([[0.0, 0.25, 0.5, 0.5, 2.0, -1.0]], dtype=np.float32)
    expect = {2: (-1, None), 3: (3, 4), 4: (3, 4), 5: (5, 2), 6: (5, 2), 7: (7, 1), 8: (7, 1),
              9: (9, 0), 10: (9, 0), 11: (11, 5), 50: (11, 5)}
    for B, (tt, k) in expect.items():
        p, c, t = solve1(errors, times, B)
        assert t == tt
        if k is not None:
            assert p[0] == k and c == errors[0, k]


def test_zero_time_prefix_is_allowed_as_in_eq_2():
    """A layer may take zero buckets: the recurrence reads E_{l-1}^{0} (Eq. 2 has no lower cut)."""
    times = np.array([[0, 3], [0, 2], [4, 1]], dtype=np.int32)
    errors = np.array([[1.0, 0.0], [1.0, 0.0], [0.0, 8.0]], dtype=np.float32)
    p, c, t = solve1(errors, times, 4)
    assert list(p) == [0, 0, 0] and c == np.float32(2.0) and t == 4
    p, c, t = solve1(errors, times, 0)
    assert t == -1
    p, c, t = solve1(errors, times, 1)
    assert list(p) == [0, 0, 1] and c == np.float32(10.0) and t == 1


# ---- textbook special case -----------------------------------------------------------------

@pytest.mark.parametrize("seed", range(25))
def test_two_choices_reduce_to_01_knapsack(seed):
    """K = 2 with (time, error) = (w, 0) 'keep' and (0, v) 'drop': minimising the dropped value
    within the budget is 0/1 knapsack; sum(v) - cost must be the knapsack optimum."""
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, 40))
    w = rng.integers(1, 60, size=L)
    v = rng.integers(1, 1000, size=L)
    cap = int(rng.integers(0, w.sum() + 5))
    times = np.stack([w, np.zeros_like(w)], axis=1).astype(np.int32)
    errors = np.stack([np.zeros(L), v.astype(np.float64)], axis=1).astype(np.float32)
    p, c, t = solve1(errors, times, cap)
    assert t >= 0
    assert int(v.sum()) - int(c) == knapsack_01(list(map(int, w)), list(map(int, v)), cap)
    check_solution(errors, times, cap, p, c, t)


# ---- invariants on the paper-sized shapes ---------------------------------------------------

@pytest.mark.parametrize("cfg", [1, 2])
def test_full_shape_solutions_are_self_consistent(cfg):
    wl = W.make_workload(cfg, N=4)
    p, c, t = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=4)
    for n in range(wl.N):
        check_solution(wl.errors[n], wl.times, wl.B, p[n], c[n], int(t[n]))
        assert t[n] <= wl.B


def test_cost_is_non_increasing_in_budget():
    wl = W.make_workload(2, N=1)
    row = oracle.last_row(wl.errors[0], wl.times, wl.B)  # E_L^t, t = 0..B
    prefix_min = np.minimum.accumulate(row)
    tmin = int(wl.times.min(axis=1).sum())
    assert np.isinf(row[:tmin]).all() and np.isfinite(row[tmin])
    for B in (tmin, tmin + 1, 5000, 7777, wl.B):
        _, c, t = solve1(wl.errors[0], wl.times, B)
        assert c.tobytes() == prefix_min[B].tobytes()
        assert t == int(np.flatnonzero(row[: B + 1] == prefix_min[B])[0])
    costs = [solve1(wl.errors[0], wl.times, B)[1] for B in range(tmin, tmin + 400, 7)]
    assert all(a >= b for a, b in zip(costs, costs[1:]))


def test_threads_do_not_change_results():
    wl = W.make_workload(1, N=12)
    a = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=1)
    b = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=5)
    for x, y in zip(a, b):
        assert x.tobytes() == y.tobytes()


def test_sparsity_grid_matches_the_papers_setup():
    """Section 4 'Setup': dense, then 41 levels from 0.4 to 0.99, each pruning about 10% more of
    the remaining weights."""
    s = W.sparsity_levels(42, 0.99)
    assert s[0] == 0.0 and abs(s[1] - 0.4) < 1e-12 and abs(s[-1] - 0.99) < 1e-12
    step = 1.0 - (1.0 - s[2:]) / (1.0 - s[1:-1])
    assert np.allclose(step, step[0]) and 0.09 < step[0] < 0.11
