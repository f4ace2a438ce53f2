"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact profiles, fp32 costs
and time_used on the same seeded inputs."""
import os

import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import binding, build as build_mod, workloads as W

pytestmark = pytest.mark.gpu

FORMATS = [binding.SPDY_TABLE_ARG_U8, binding.SPDY_TABLE_ROW_F32]
CORES = max(1, len(os.sched_getaffinity(0)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def gpu_solve(wl, fmt=0, **kw):
    import torch

    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, **kw)
    errors = torch.from_numpy(wl.errors).cuda()
    p, c, t = binding.solve_batch(plan, errors)
    torch.cuda.synchronize()
    plan.check_status()
    out = p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()
    plan.close()
    return out


def assert_same(gpu, ref):
    gp, gc, gt = gpu
    rp, rc, rt = ref
    assert np.array_equal(gt, rt), "time_used differs"
    assert gc.tobytes() == rc.tobytes(), "cost bits differ"
    assert np.array_equal(gp, rp), "profiles differ"


@pytest.mark.parametrize("fmt", FORMATS)
def test_config0_many_seeds(fmt):
    for seed in range(25):
        wl = W.make_workload(0, seed_shift=seed)
        assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B))


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("cfg,N", [(1, 96), (2, 96), (3, 6)])
def test_named_configs_element_by_element(cfg, N, fmt):
    wl = W.make_workload(cfg, N=N)
    assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))


@pytest.mark.parametrize("fmt", FORMATS)
def test_sweep_budgets_of_config4(fmt):
    for B, N in ((1000, 64), (10000, 16)):
        wl = W.make_workload(4, N=N, B=B)
        assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))


@pytest.mark.parametrize("fmt", FORMATS)
def test_adversarial_tiny_instances(fmt):
    """Ties, zero times, times above the budget, +inf and negative errors, infeasible budgets."""
    for seed in range(120):
        for exact in (False, True):
            wl = W.tiny_random_instance(seed + (10_000 if exact else 0), exact=exact, N=5)
            assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B))


@pytest.mark.parametrize("fmt", FORMATS)
def test_tie_heavy_wide_instance(fmt):
    """Errors from {0, 1/4, 1/2, 1} and repeated / zero times on rows several spans wide."""
    rng = np.random.default_rng(77)
    L, K, B, N = 12, 9, 3000, 24
    times = rng.integers(0, 400, size=(L, K)).astype(np.int32)
    times[:, 3] = times[:, 2]
    times[4, :] = 0
    errors = rng.choice(np.array([0, 0.25, 0.5, 1.0], np.float32), size=(N, L, K)).astype(np.float32)
    wl = W.Workload("ties", times, errors, B)
    assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))


@pytest.mark.parametrize("fmt", FORMATS)
def test_paper_shaped_errors_of_eq4(fmt):
    wl2 = W.make_workload(2, N=1)
    errors = W.paper_shaped_errors(wl2.L, wl2.K, 48, seed=9)
    wl = W.Workload("eq4", wl2.times, errors, wl2.B)
    assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))


@pytest.mark.parametrize("fmt", FORMATS)
def test_degenerate_shapes(fmt):
    import torch

    cases = [
        W.Workload("K1", np.array([[2], [0], [5]], np.int32), np.array([[[1.5], [2.5], [-0.25]]], np.float32), 7),
        W.Workload("L1", np.array([[9, 7, 5, 5, 3, 11]], np.int32),
                   np.array([[[0.0, 0.25, 0.5, 0.5, 2.0, -1.0]]], np.float32), 6),
        W.Workload("B0", np.array([[0, 1], [0, 0]], np.int32), np.array([[[3.0, 1.0], [2.0, 2.0]]], np.float32), 0),
        W.Workload("B0-infeasible", np.array([[1, 1]], np.int32), np.array([[[3.0, 1.0]]], np.float32), 0),
        W.Workload("over", np.array([[50, 4], [60, 70]], np.int32), np.array([[[0.0, 1.0], [0.0, 1.0]]], np.float32), 10),
        W.Workload("all-inf-layer", np.array([[1, 2], [1, 2]], np.int32),
                   np.array([[[1.0, 2.0], [np.inf, np.inf]], [[1.0, 2.0], [3.0, np.inf]]], np.float32), 4),
        W.Workload("neg-zero", np.array([[1, 2], [1, 2]], np.int32),
                   np.array([[[-0.0, 2.0], [-0.0, 1.0]]], np.float32), 4),
    ]
    for wl in cases:
        assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B))
    # K = 255 (the largest choice count) and N = 0
    rng = np.random.default_rng(1)
    wl = W.Workload("K255", rng.integers(1, 40, size=(4, 255)).astype(np.int32),
                    rng.lognormal(size=(3, 4, 255)).astype(np.float32), 90)
    assert_same(gpu_solve(wl, fmt), oracle.solve_batch(wl.errors, wl.times, wl.B))
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    p, c, t = binding.solve_batch(plan, torch.empty((0, 4, 255), device="cuda"))
    assert p.shape == (0, 4) and c.numel() == 0


@pytest.mark.parametrize("fmt", FORMATS)
def test_small_workspace_runs_in_waves(fmt):
    import torch

    wl = W.make_workload(1, N=23)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    ws = torch.empty(plan.workspace_bytes(5), dtype=torch.uint8, device="cuda")
    p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda(), workspace=ws)
    torch.cuda.synchronize()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()),
                oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))
    # (a plan with one launch shape: spdy_workspace_bytes of the default plan covers its largest shape)
    single = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, auto_shape=1)
    tiny = torch.empty(single.workspace_bytes(1) - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.SpdyError) as e:
        binding.solve_batch(single, torch.from_numpy(wl.errors).cuda(), workspace=tiny)
    assert e.value.status == -2
    single.close()
    with pytest.raises(binding.SpdyError) as e:  # misaligned workspace
        binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda(), workspace=ws[8:])
    assert e.value.status == -1


@pytest.mark.parametrize("threads", [128, 256, 512, 1024])
@pytest.mark.parametrize("mode", [1, 2, 3, 4, 5])
def test_every_launch_shape_and_cell_update_variant_gives_the_same_answer(threads, mode):
    wl = W.make_workload(2, N=8)
    fmt = 1 if mode in (1, 2, 5) else 2
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    assert_same(gpu_solve(wl, fmt, threads=threads, forward_mode=mode), ref)
    tiny = W.tiny_random_instance(10_007, exact=True, N=5)
    assert_same(gpu_solve(tiny, fmt, threads=threads, forward_mode=mode),
                oracle.solve_batch(tiny.errors, tiny.times, tiny.B))


def test_host_buffer_and_one_shot_entry_points():
    import torch

    wl = W.make_workload(1, N=40)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    plan = binding.Plan(wl.times, wl.B, device=0)
    assert_same(binding.solve_batch_host(plan, wl.errors), ref)
    assert_same(binding.solve_batch_host(plan, wl.errors[:7]), tuple(x[:7] for x in ref))
    pinned = torch.from_numpy(wl.errors).pin_memory()
    assert_same(binding.solve_batch_host(plan, pinned), ref)
    p, c, t = binding.solve_batch_simple(torch.from_numpy(wl.errors).cuda(), torch.from_numpy(wl.times).cuda(), wl.B)
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
    # a plan-level infeasible budget goes through the fill kernel
    B_bad = int(wl.times.min(axis=1).sum()) - 1
    p, c, t = binding.solve_batch_simple(torch.from_numpy(wl.errors).cuda(), torch.from_numpy(wl.times).cuda(), B_bad)
    assert (p.cpu().numpy() == 0xFF).all() and (t.cpu().numpy() == -1).all() and np.isposinf(c.cpu().numpy()).all()


_ORACLE_CACHE = {}


def oracle_on(wl, key, sample=None):
    """Oracle outputs for the candidates `sample` (all when None) of a named workload, computed once per
    test session: the table formats and launch options under test share them."""
    if key not in _ORACLE_CACHE:
        errors = wl.errors if sample is None else wl.errors[sample]
        _ORACLE_CACHE[key] = oracle.solve_batch(errors, wl.times, wl.B, threads=CORES)
    return _ORACLE_CACHE[key]


def check_full_size(wl, key, sample_size=None, fmt=0, workspace_bytes=None, **plan_kw):
    """A batch at its full size, in the launch shape the plan picks by default: every candidate against the
    oracle (`sample_size` None), or - where the oracle would take minutes - a seeded sample of that size
    against the oracle and, on every candidate, the invariants that hold at any size."""
    import torch

    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, **plan_kw)
    ws = None
    if workspace_bytes is not None:
        per = plan.workspace_bytes(1)
        ws = torch.empty(max(per, workspace_bytes // per * per), dtype=torch.uint8, device="cuda")
    p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda(), workspace=ws)
    torch.cuda.synchronize()
    plan.check_status()
    p, c, t = p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()
    del ws
    plan.close()
    if sample_size is None:
        assert_same((p, c, t), oracle_on(wl, key))
        return
    assert (t >= 0).all() and (t <= wl.B).all() and (p < wl.K).all()
    idx = p.astype(np.int64)
    assert np.array_equal(wl.times[np.arange(wl.L)[None, :], idx].sum(axis=1), t)
    e_sel = np.take_along_axis(wl.errors, idx[:, :, None], axis=2)[:, :, 0]
    acc = np.zeros(wl.N, np.float32)
    for l in range(wl.L):
        acc = (acc + e_sel[:, l]).astype(np.float32)
    assert acc.tobytes() == c.tobytes()
    sample = np.sort(np.random.default_rng(0).choice(wl.N, size=min(sample_size, wl.N), replace=False))
    assert_same((p[sample], c[sample], t[sample]), oracle_on(wl, (key, sample_size), sample))


@pytest.mark.parametrize("fmt", FORMATS)
def test_full_size_resnet50_batch_every_candidate(fmt):
    """Config 1 at its full N = 1024, every candidate against the oracle."""
    check_full_size(W.make_workload(1), "cfg1", fmt=fmt)


@pytest.mark.parametrize("fmt", FORMATS)
def test_full_size_bert_base_batch_every_candidate_in_the_benchmark_configuration(fmt):
    """Config 2, N = 4096, as the benchmark times it (default plan, one wave): every candidate's profile,
    cost bits and time_used against the oracle."""
    wl = W.make_workload(2)
    assert wl.N == 4096
    check_full_size(wl, "cfg2", fmt=fmt)


@pytest.mark.parametrize("fmt", FORMATS)
def test_full_size_bert_large_batch_every_candidate(fmt):
    """Config 3 at its full N = 1024 (B = 65536, K = 64), every candidate against the oracle."""
    check_full_size(W.make_workload(3), "cfg3", fmt=fmt)


@pytest.mark.parametrize("fmt", FORMATS)
def test_full_size_sweep_points(fmt):
    """Config 4's largest points.  N = 65536 runs in waves inside a 12 GB workspace and is compared with the
    oracle on 4096 seeded candidates; B = 1000 on all 4096; B = 100000 (rows in global memory) on 256 of
    1024.  The sampled points also get the any-size invariants on every candidate."""
    check_full_size(W.make_workload(4, N=65536), "N65536", 4096, fmt=fmt, workspace_bytes=12 << 30)
    check_full_size(W.make_workload(4, N=4096, B=1000), "B1000", fmt=fmt)
    check_full_size(W.make_workload(4, N=1024, B=100000), "B100000", 256, fmt=fmt)


def test_sweep_points_with_few_candidates_every_candidate():
    """Config 4's small batches (N = 1, 16, 256), every candidate, both table formats."""
    for n in (1, 16, 256):
        wl = W.make_workload(4, N=n)
        ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
        for fmt in FORMATS:
            assert_same(gpu_solve(wl, fmt), ref)


@pytest.mark.parametrize("cluster", [2, 4, 8])
@pytest.mark.parametrize("mode", [1, 3, 4, 5])
def test_cluster_split_of_one_candidate_gives_the_same_answer(cluster, mode):
    """A candidate cut over a thread-block cluster (slices of every row, windows gathered through
    distributed shared memory) must match the oracle like the single-CTA kernel.  (The predicated-move
    update, mode 2, has no cluster build.)"""
    fmt = 1 if mode in (1, 5) else 2
    wl = W.make_workload(2, N=6)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    assert_same(gpu_solve(wl, fmt, cluster=cluster, forward_mode=mode), ref)
    for seed in (10_003, 10_007, 21, 33):  # rows narrower than the cluster: empty slices
        tiny = W.tiny_random_instance(seed, exact=seed >= 10_000, N=3)
        assert_same(gpu_solve(tiny, fmt, cluster=cluster, forward_mode=mode),
                    oracle.solve_batch(tiny.errors, tiny.times, tiny.B))


@pytest.mark.parametrize("fmt", FORMATS)
def test_budget_100000_does_not_fit_one_cta(fmt):
    """B = 100000: a band-limited row is about 210 KB, so two rows cannot live in one CTA's shared
    memory.  By default the rows then go to global memory; on request a cluster shares them."""
    wl = W.make_workload(4, N=5, B=100000)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    assert plan.info["rows_in_global"] == 1 and plan.info["cluster"] == 1
    plan.close()
    assert_same(gpu_solve(wl, fmt), ref)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, cluster=4)
    assert plan.info["cluster"] == 4 and plan.info["rows_in_global"] == 0
    plan.close()
    assert_same(gpu_solve(wl, fmt, cluster=4), ref)
    assert_same(gpu_solve(wl, fmt, threads=512), ref)  # a pinned CTA size selects the cluster path


def test_cluster_with_ties_and_wide_rows():
    rng = np.random.default_rng(78)
    L, K, B, N = 10, 7, 5000, 12
    times = rng.integers(0, 900, size=(L, K)).astype(np.int32)
    times[3, :] = 0
    errors = rng.choice(np.array([0, 0.25, 0.5, 1.0], np.float32), size=(N, L, K)).astype(np.float32)
    wl = W.Workload("ties-cluster", times, errors, B)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    for cluster in (2, 4, 8):
        for fmt in FORMATS:
            assert_same(gpu_solve(wl, fmt, cluster=cluster), ref)


def coeff_cases():
    rng = np.random.default_rng(5)
    for cfg, N in ((1, 48), (2, 48), (3, 4)):
        wl = W.make_workload(cfg, N=1)
        yield wl.times, wl.B, rng.uniform(0.0, 1.0, size=(N, wl.L)).astype(np.float32)
    wl = W.make_workload(4, N=1, B=1000)
    yield wl.times, wl.B, rng.uniform(0.0, 1.0, size=(40, wl.L)).astype(np.float32)
    wl = W.make_workload(2, N=1)
    c = rng.normal(size=(16, wl.L)).astype(np.float32)  # signed coefficients are accepted too
    c[0], c[1] = 0.0, 1.0
    yield wl.times, wl.B, c


def test_eq4_error_table_element_by_element():
    import torch

    rng = np.random.default_rng(6)
    for K in (1, 2, 3, 5, 42, 64, 255):
        c = rng.uniform(0.0, 1.0, size=(37, 11)).astype(np.float32)
        c[0, :4] = [0.0, 1.0, 1e-30, -0.75]
        got = binding.quadratic_errors(torch.from_numpy(c).cuda(), K).cpu().numpy()
        assert got.tobytes() == oracle.quadratic_errors(c, K).tobytes()


@pytest.mark.parametrize("fmt", FORMATS)
def test_coefficient_input_matches_the_oracle_on_eq4_errors(fmt):
    """spdy_solve_batch_coeffs forms Eq. 4's errors inside the kernels; the oracle forms the table
    first and runs the same dynamic program."""
    import torch

    for times, B, c in coeff_cases():
        ref = oracle.solve_batch(oracle.quadratic_errors(c, times.shape[1]), times, B, threads=CORES)
        plan = binding.Plan(times, B, device=0, table_format=fmt)
        p, cost, t = binding.solve_batch_coeffs(plan, torch.from_numpy(c).cuda())
        torch.cuda.synchronize()
        plan.check_status()
        assert_same((p.cpu().numpy(), cost.cpu().numpy(), t.cpu().numpy()), ref)
        # the table route through the library gives the same bits
        e = binding.quadratic_errors(torch.from_numpy(c).cuda(), times.shape[1])
        p2, c2, t2 = binding.solve_batch(plan, e)
        torch.cuda.synchronize()
        assert_same((p2.cpu().numpy(), c2.cpu().numpy(), t2.cpu().numpy()), ref)
        plan.close()


def test_coefficient_input_host_buffers_cluster_and_tiny_shapes():
    import torch

    times, B, c = next(coeff_cases())
    ref = oracle.solve_batch(oracle.quadratic_errors(c, times.shape[1]), times, B, threads=CORES)
    plan = binding.Plan(times, B, device=0)
    assert_same(binding.solve_batch_coeffs_host(plan, c), ref)
    assert_same(binding.solve_batch_coeffs_host(plan, torch.from_numpy(c).pin_memory()), ref)
    plan.close()
    for cluster in (2, 8):
        plan = binding.Plan(times, B, device=0, cluster=cluster)
        p, cost, t = binding.solve_batch_coeffs(plan, torch.from_numpy(c[:6]).cuda())
        torch.cuda.synchronize()
        assert_same((p.cpu().numpy(), cost.cpu().numpy(), t.cpu().numpy()), tuple(x[:6] for x in ref))
        plan.close()
    rng = np.random.default_rng(8)
    for seed in range(60):  # ties, zero and repeated times, K = 1, infeasible budgets
        wl = W.tiny_random_instance(seed, N=1)
        c = rng.choice(np.array([0.0, 0.25, 0.5, 1.0], np.float32), size=(5, wl.L)).astype(np.float32)
        ref = oracle.solve_batch(oracle.quadratic_errors(c, wl.K), wl.times, wl.B)
        plan = binding.Plan(wl.times, wl.B, device=0)
        p, cost, t = binding.solve_batch_coeffs(plan, torch.from_numpy(c).cuda())
        torch.cuda.synchronize()
        assert_same((p.cpu().numpy(), cost.cpu().numpy(), t.cpu().numpy()), ref)
        plan.close()
    with pytest.raises(ValueError):
        binding.solve_batch_coeffs(binding.Plan(times, B, device=0), torch.zeros((2, 3), device="cuda"))


@pytest.mark.parametrize("fmt", FORMATS)
def test_rows_in_global_memory_give_the_same_answer(fmt):
    """The wide-band fallback (row buffers in the workspace instead of shared memory), forced on
    shapes the oracle finishes quickly."""
    import torch

    wl = W.make_workload(2, N=7)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    assert_same(gpu_solve(wl, fmt, rows_in_global=1), ref)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, rows_in_global=1)
    assert plan.info["rows_in_global"] == 1 and plan.info["threads"] == 1024
    ws = torch.empty(plan.workspace_bytes(3), dtype=torch.uint8, device="cuda")  # 7 candidates in 3 waves
    p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda(), workspace=ws)
    torch.cuda.synchronize()
    plan.check_status()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
    plan.close()
    for seed in range(40):
        for exact in (False, True):
            tiny = W.tiny_random_instance(seed + (10_000 if exact else 0), exact=exact, N=4)
            assert_same(gpu_solve(tiny, fmt, rows_in_global=1), oracle.solve_batch(tiny.errors, tiny.times, tiny.B))
    with pytest.raises(binding.SpdyError):
        binding.Plan(wl.times, wl.B, device=0, rows_in_global=1, cluster=2)


def test_budget_400000_falls_back_to_rows_in_global_memory():
    """B = 400000: a band of about 210 000 cells does not fit a cluster of eight CTAs either."""
    wl = W.make_workload(4, N=2, B=400000)
    plan = binding.Plan(wl.times, wl.B, device=0)
    assert plan.info["rows_in_global"] == 1 and plan.info["cluster"] == 1
    plan.close()
    assert_same(gpu_solve(wl), oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))


def test_host_buffer_path_uploads_in_chunks():
    """Batches larger than one wave go up in several chunks on a second stream; results must not
    depend on that, call after call, for error tables and for coefficients."""
    import torch

    wl = W.make_workload(1, N=2500)
    plan = binding.Plan(wl.times, wl.B, device=0)
    p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda())
    torch.cuda.synchronize()
    dev = (p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy())
    pinned = torch.from_numpy(wl.errors).pin_memory()
    for errors in (wl.errors, pinned, wl.errors[:700], wl.errors):
        n = len(errors)
        assert_same(binding.solve_batch_host(plan, errors), tuple(x[:n] for x in dev))
    assert_same(dev, oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES))
    coeffs = W.sensitivity_samples(3, wl.L, 2500)
    pc, cc, tc = binding.solve_batch_coeffs(plan, torch.from_numpy(coeffs).cuda())
    torch.cuda.synchronize()
    assert_same(binding.solve_batch_coeffs_host(plan, coeffs), (pc.cpu().numpy(), cc.cpu().numpy(), tc.cpu().numpy()))
    plan.enable_timing(True)  # timing covers all chunks of a host-buffer call
    binding.solve_batch_host(plan, pinned)
    fwd_host, _ = plan.last_timing()
    binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda())
    fwd_dev, _ = plan.last_timing()
    assert 0.5 * fwd_dev < fwd_host < 3.0 * fwd_dev
    plan.close()


def test_peak_probes_are_in_range():
    """The shared-memory probe must land just under 32 reads per clock per SM, the arithmetic probe
    well above it (otherwise the roofline's binding unit would be misjudged)."""
    import torch

    lds, alu = binding.probe_peaks(0)
    props = torch.cuda.get_device_properties(0)
    per_clk_sm = lds / (props.multi_processor_count * 1.965e9)
    assert 20.0 < per_clk_sm <= 33.0
    assert alu > 1.5 * lds


@pytest.mark.parametrize("fmt", FORMATS)
def test_nan_inputs_are_contained(fmt):
    """NaN errors are outside the value domain: the candidate that holds them may come back flagged
    (self-check word) or as infeasible, but its neighbours in the batch must be unaffected.  Every
    table access of the walk back is range-checked, so nothing can go out of bounds."""
    import torch

    wl = W.make_workload(1, N=12)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    bad = wl.errors.copy()
    bad[5, :, :] = np.nan
    bad[9, 3, 7] = np.nan
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    p, c, t = binding.solve_batch(plan, torch.from_numpy(bad).cuda())
    torch.cuda.synchronize()
    try:
        plan.check_status()
    except binding.SpdyError as e:
        assert e.status == -6
    plan.check_status()  # the word was cleared by the read above
    good = [n for n in range(12) if n not in (5, 9)]
    assert_same((p.cpu().numpy()[good], c.cpu().numpy()[good], t.cpu().numpy()[good]), tuple(x[good] for x in ref))
    assert t.cpu().numpy()[5] == -1 and (p.cpu().numpy()[5] == 0xFF).all()
    plan.close()


def test_byte_table_merges_equal_time_choices_only_where_exact():
    """With the uint8 table, candidates whose errors rise with the choice index inside every group of
    equal-time choices run on merged slots, the others on one slot per choice - in one batch."""
    import torch

    wl = W.make_workload(4, N=40, B=1000)  # many equal times after rounding
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=binding.SPDY_TABLE_ARG_U8)
    info = plan.info
    assert info["launches_per_wave"] == 5 and info["distinct_updates"] < info["useful_updates"]
    errors = wl.errors.copy()
    rng = np.random.default_rng(12)
    for n in range(0, 40, 3):  # every third candidate: errors in random order, some equal
        errors[n] = rng.permuted(errors[n], axis=1)
        errors[n, :, 5] = errors[n, :, 6]
    for n in range(1, 40, 7):  # flat errors: every choice ties
        errors[n] = np.float32(0.5)
    ref = oracle.solve_batch(errors, wl.times, wl.B, threads=CORES)
    p, c, t = binding.solve_batch(plan, torch.from_numpy(errors).cuda())
    torch.cuda.synchronize()
    plan.check_status()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
    ws = torch.empty(plan.workspace_bytes(7), dtype=torch.uint8, device="cuda")  # several waves
    p, c, t = binding.solve_batch(plan, torch.from_numpy(errors).cuda(), workspace=ws)
    torch.cuda.synchronize()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
    plan.close()
    # coefficients of either sign: negative ones make Eq. 4's errors fall with the index
    coeffs = rng.normal(size=(30, wl.L)).astype(np.float32)
    ref = oracle.solve_batch(oracle.quadratic_errors(coeffs, wl.K), wl.times, wl.B, threads=CORES)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=binding.SPDY_TABLE_ARG_U8)
    p, c, t = binding.solve_batch_coeffs(plan, torch.from_numpy(coeffs).cuda())
    torch.cuda.synchronize()
    plan.check_status()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
    plan.close()


def test_random_shapes_formats_and_launch_options():
    """Seeded fuzz over shapes (K up to 255: several mask words; times above the budget, zeros, repeats),
    both table formats and the launch options, against the oracle."""
    rng = np.random.default_rng(2024)
    for trial in range(200):
        L = int(rng.integers(1, 13)) if trial % 4 else int(rng.integers(13, 41))
        K = int(rng.choice([1, 2, 3, 17, 64, 65, 130, 255]))
        B = int(rng.choice([0, 7, 300, 1500, 4000])) if trial % 4 else int(rng.choice([3000, 9000, 20000, 70000]))
        scale = max(1, int(B * rng.choice([0.05, 0.3, 1.2]) / max(L, 1)) + 1)
        times = rng.integers(0, 2 * scale + 1, size=(L, K)).astype(np.int32)
        if rng.random() < 0.5:  # sorted like real timing tables: sparser is faster, with repeats
            times = np.sort(times, axis=1)[:, ::-1].copy()
        if rng.random() < 0.3:
            times[rng.integers(L), :] = 0
        kind = trial % 3
        if kind == 0:
            errors = rng.lognormal(0.0, 1.0, size=(3, L, K)).astype(np.float32)
        elif kind == 1:
            errors = rng.choice(np.array([0, 0.25, 0.5, 1.0], np.float32), size=(3, L, K)).astype(np.float32)
        else:
            errors = np.sort(rng.lognormal(0.0, 1.0, size=(3, L, K)).astype(np.float32), axis=2)
            errors[1] = -errors[1]
        wl = W.Workload(f"fuzz-{trial}", times, errors, B)
        ref = oracle.solve_batch(wl.errors, wl.times, wl.B)
        options = [dict(), dict(cluster=int(rng.choice([2, 4, 8]))), dict(rows_in_global=1),
                   dict(threads=int(rng.choice([256, 512, 1024]))), dict(kernel=binding.SPDY_KERNEL_WARP),
                   dict(kernel=binding.SPDY_KERNEL_CTA, schedule=int(rng.integers(1, 4))), dict(schedule=int(rng.integers(1, 9)) << 8)]
        for fmt in FORMATS:
            kw = options[int(rng.integers(len(options)))]
            try:
                got = gpu_solve(wl, fmt, **kw)
            except binding.SpdyError as e:  # a warp per candidate stages at most 64 shift slots per layer
                assert e.status == -3 and kw.get("kernel") == binding.SPDY_KERNEL_WARP, (trial, fmt, kw)
                continue
            assert_same(got, ref), (trial, fmt, kw)


@pytest.mark.parametrize("fmt", FORMATS)
def test_two_live_plans_of_one_kernel_variant(fmt):
    """A wide plan (more than 48 KB of dynamic shared memory per CTA) must keep working after a narrower
    plan of the same table format and CTA size has been created, and after a call of the static entry
    point: the shared-memory limit is a property of the kernel on the device, not of a plan."""
    import torch

    wide = W.make_workload(1, N=12)
    narrow = W.make_workload(4, N=12, B=2500)
    ref_wide = oracle.solve_batch(wide.errors, wide.times, wide.B, threads=CORES)
    ref_narrow = oracle.solve_batch(narrow.errors, narrow.times, narrow.B, threads=CORES)
    for between in (False, True):
        a = binding.Plan(wide.times, wide.B, device=0, table_format=fmt, threads=128)
        b = binding.Plan(narrow.times, narrow.B, device=0, table_format=fmt, threads=128)
        assert a.info["smem_bytes"] > 48 * 1024 > b.info["smem_bytes"]
        if between:
            binding.solve_batch_static(torch.from_numpy(narrow.errors).cuda(), narrow.times, narrow.B)
        for plan, wl, ref in ((a, wide, ref_wide), (b, narrow, ref_narrow), (a, wide, ref_wide)):
            p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda())
            torch.cuda.synchronize()
            plan.check_status()
            assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
        a.close()
        b.close()


def test_plan_level_infeasible_budget_fills_every_candidate():
    """The marker outputs of an infeasible plan reach every candidate, also of a batch with more
    candidates than 65535 blocks of 256 threads."""
    import torch

    times = np.array([[5, 6], [7, 9]], np.int32)
    N = 65535 * 256 + 999
    plan = binding.Plan(times, 11, device=0)
    assert plan.info["feasible"] == 0
    p, c, t = binding.solve_batch(plan, torch.empty((N, 2, 2), device="cuda"))
    torch.cuda.synchronize()
    assert (p == 0xFF).all().item() and (t == -1).all().item() and torch.isposinf(c).all().item()
    plan.close()


@pytest.mark.parametrize("fmt", FORMATS)
def test_one_warp_per_candidate_gives_the_same_answer(fmt):
    """The kernel for narrow rows (a warp owns a candidate; four candidates per CTA, no block barrier): chosen
    by itself at B = 1000, forced on wider and on tiny shapes, batch sizes that leave warps of the last CTA idle."""
    import torch

    wl = W.make_workload(4, N=203, B=1000)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    assert plan.info["kernel"] == binding.SPDY_KERNEL_WARP and plan.info["candidates_per_cta"] == 4
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    for n in (203, 1, 2, 5):
        p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors[:n]).cuda())
        torch.cuda.synchronize()
        plan.check_status()
        assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), tuple(x[:n] for x in ref))
    ws = torch.empty(plan.workspace_bytes(10), dtype=torch.uint8, device="cuda")  # waves of 10 candidates
    p, c, t = binding.solve_batch(plan, torch.from_numpy(wl.errors).cuda(), workspace=ws)
    torch.cuda.synchronize()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
    assert_same(binding.solve_batch_host(plan, wl.errors), ref)
    plan.close()
    for cfg, B, n in ((4, 2500, 9), (4, 5000, 5)):  # several passes per layer in one warp
        wide = W.make_workload(cfg, N=n, B=B)
        assert_same(gpu_solve(wide, fmt, kernel=binding.SPDY_KERNEL_WARP),
                    oracle.solve_batch(wide.errors, wide.times, wide.B, threads=CORES))
    for seed in range(60):
        for exact in (False, True):
            tiny = W.tiny_random_instance(seed + (10_000 if exact else 0), exact=exact, N=6)
            assert_same(gpu_solve(tiny, fmt, kernel=binding.SPDY_KERNEL_WARP),
                        oracle.solve_batch(tiny.errors, tiny.times, tiny.B))
    wl2 = W.make_workload(2, N=1)
    c = np.random.default_rng(3).uniform(0, 1, size=(37, wl.L)).astype(np.float32)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    p, cost, t = binding.solve_batch_coeffs(plan, torch.from_numpy(c).cuda())
    torch.cuda.synchronize()
    assert_same((p.cpu().numpy(), cost.cpu().numpy(), t.cpu().numpy()),
                oracle.solve_batch(oracle.quadratic_errors(c, wl.K), wl.times, wl.B, threads=CORES))
    plan.close()
    del wl2


@pytest.mark.parametrize("fmt", FORMATS)
def test_pass_schedules_give_the_same_answer(fmt):
    """The plan's choice, passes of one length, levelled passes, cost-sized passes, capped pass lengths."""
    wl = W.make_workload(2, N=6)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    for schedule in (0, 1, 2, 3, 5 << 8, 3 | (3 << 8), 2 | (16 << 8)):
        for threads in (128, 512):
            assert_same(gpu_solve(wl, fmt, schedule=schedule, threads=threads), ref)


@pytest.mark.parametrize("fmt", FORMATS)
def test_small_batches_pick_their_launch_shape_by_themselves(fmt):
    """With the launch shape left open, batches that cannot fill the device run as clusters or larger CTAs;
    the answer does not depend on it, nor on the workspace being too small for that choice."""
    import torch

    wl = W.make_workload(2, N=300)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)
    plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
    assert plan.info["alternates"] >= 4
    errors = torch.from_numpy(wl.errors).cuda()
    for n in (1, 3, 18, 19, 37, 38, 74, 75, 148, 149, 295, 296, 300):
        p, c, t = binding.solve_batch(plan, errors[:n])
        torch.cuda.synchronize()
        plan.check_status()
        assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), tuple(x[:n] for x in ref))
    pinned = binding.Plan(wl.times, wl.B, device=0, table_format=fmt, auto_shape=1)
    tight = torch.empty(pinned.workspace_bytes(2), dtype=torch.uint8, device="cuda")
    p, c, t = binding.solve_batch(plan, errors[:7], workspace=tight)  # waves of the main shape
    torch.cuda.synchronize()
    assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), tuple(x[:7] for x in ref))
    assert_same(binding.solve_batch_host(plan, wl.errors[:20]), tuple(x[:20] for x in ref))
    assert_same(binding.solve_batch_host(plan, wl.errors[:160]), tuple(x[:160] for x in ref))
    plan.close()
    pinned.close()


def test_plans_solved_from_two_host_threads_at_once():
    """The library keeps no global state: two host threads, each with its own plan, stream and buffers, solve
    different problems at the same time, again and again, and both stay bit-exact."""
    import threading

    import torch

    jobs = []
    for cfg, n, fmt in ((2, 40, binding.SPDY_TABLE_ROW_F32), (1, 60, binding.SPDY_TABLE_ARG_U8)):
        wl = W.make_workload(cfg, N=n)
        jobs.append((wl, fmt, oracle.solve_batch(wl.errors, wl.times, wl.B, threads=CORES)))
    failures = []

    def worker(wl, fmt, ref):
        try:
            stream = torch.cuda.Stream()
            plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
            errors = torch.from_numpy(wl.errors).cuda()
            torch.cuda.synchronize()
            for _ in range(12):
                p, c, t = binding.solve_batch(plan, errors, stream=stream)
                stream.synchronize()
                plan.check_status(stream)
                assert_same((p.cpu().numpy(), c.cpu().numpy(), t.cpu().numpy()), ref)
                assert_same(binding.solve_batch_host(plan, wl.errors, stream=stream), ref)
            plan.close()
        except BaseException as exc:  # reported by the main thread
            failures.append(exc)

    threads = [threading.Thread(target=worker, args=job) for job in jobs]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not failures, failures
