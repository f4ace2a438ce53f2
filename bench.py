#!/usr/bin/env python
"""Benchmark of the batched SPDY dynamic program.

One "step" = one pass of the whole path (forward dynamic program, final minimum over the budget
axis, walk back) over one batch of synthetic candidates.  The default workload is the
BERT-base-shaped search (L 72, K 42, B 10000, N 4096 candidates per GPU).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

prints one JSON line on rank 0.  `--impl reference` times the CPU oracle on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

SM_COUNT_NOMINAL = 148
SM_MAX_MHZ_NOMINAL = 1965.0
CELLS_PER_CLK_PER_SM = 32.0  # one 4-byte shared-memory read per cell update, 32 banks x 4 B per clock

# DRAM bytes (read + write) of the forward kernel from an ncu capture of one wave of the BERT-base shape:
# kept, with the capture command and the library version it is valid for, in this file.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "forward_kernel_bert_base_dram_traffic.txt")


def load_ncu_traffic(path: str = TRAFFIC_FILE) -> dict:
    """`key = value` lines of the traffic record ('#' starts a comment); {} if the file is missing."""
    out = {}
    try:
        for raw in open(path):
            text = raw.split("#", 1)[0].strip()
            if "=" in text:
                key, value = (x.strip() for x in text.split("=", 1))
                out[key] = value
    except OSError:
        pass
    return out


def ncu_traffic_per_launch(record: dict, library_version: int, workload_name: str, budget: int, cluster: int,
                           table_name: str, candidates_per_launch: float):
    """(bytes per launch or None, note).  None - said loudly - when the record was taken with another
    library version (the kernel has changed since) or covers another workload."""
    if not record:
        return None, "no ncu traffic record under profiles/"
    if int(record.get("library_version", -1)) != int(library_version):
        return None, (f"ncu traffic record is for library version {record.get('library_version')}, this is "
                      f"{library_version}: the kernel changed since the counters were taken; re-capture")
    if (not workload_name.startswith(record.get("workload_prefix", "?")) or int(record.get("budget", -1)) != int(budget)
            or cluster != 1 or f"{table_name}_bytes" not in record):
        return None, "the ncu traffic record covers another workload or launch shape"
    per_candidate = float(record[f"{table_name}_bytes"]) / float(record["candidates_captured"])
    return per_candidate * candidates_per_launch, (f"ncu dram read+write of one launch over {record['candidates_captured']} "
                                                   "candidates, scaled by the candidates of this launch "
                                                   "(profiles/forward_kernel_bert_base_dram_traffic.txt)")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload config 1..4 (default 2: BERT-base shape)")
    ap.add_argument("--n", type=int, default=None, help="candidates per GPU (default: the config's)")
    ap.add_argument("--budget", type=int, default=None, help="override B (config 4 sweep)")
    ap.add_argument("--table", default="default", choices=["default", "arg", "row"])
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--mode", type=int, default=0, help="forward kernel variant (see spdy_options.forward_mode)")
    ap.add_argument("--cluster", type=int, default=0, help="CTAs per candidate (0 = plan's choice)")
    ap.add_argument("--rows-in-global", type=int, default=0, help="1: row buffers in the workspace (wide-band fallback)")
    ap.add_argument("--kernel", type=int, default=0, help="1: one CTA per candidate, 2: one warp per candidate (0 = plan's choice)")
    ap.add_argument("--schedule", type=int, default=0, help="pass schedule (see spdy_options.schedule)")
    ap.add_argument("--auto-shape", type=int, default=0, help="1: never switch launch shape for small batches")
    ap.add_argument("--search", type=int, default=0, metavar="TRIALS",
                    help="also run Algorithm 4 with this many trials per loop on the workload's timing table "
                         "(synthetic loss) and report where the time goes, under the key 'search'")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of one line: every named shape and sweep point (N in 1..65536, B in 10^3..10^5), "
                         "each with its oracle sample and a bit-exact check; prints one JSON line per point and a "
                         "markdown table on stderr")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU work budget of the oracle legs")
    return ap.parse_args()


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period: float = 0.01):
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.error = None

    def _run(self):
        try:
            import pynvml

            pynvml.nvmlInit()
            uuid = None
            try:
                import torch

                uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            except Exception:
                pass
            h = None
            if uuid:
                for cand in (f"GPU-{uuid}", uuid):
                    try:
                        h = pynvml.nvmlDeviceGetHandleByUUID(cand.encode() if isinstance(cand, str) else cand)
                        break
                    except Exception:
                        h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            names = {
                pynvml.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                pynvml.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                pynvml.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                pynvml.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
                pynvml.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake",
            }
            while not self._stop.is_set():
                self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                mask = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
                time.sleep(self.period)
        except Exception as exc:  # NVML missing: report it, never fail the bench
            self.error = repr(exc)

    def __enter__(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=2.0)

    def summary(self) -> dict:
        out = {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.error:
            out["error"] = self.error
        return out


def oracle_baseline(wl, cpu_seconds: float, gpu_outputs=None):
    """The oracle as it stands on the host cores, on a bounded prefix of the same candidates.  Returns
    (cpu_baseline, parity): with `gpu_outputs` = (profile, cost, time_used) as NumPy arrays, the oracle's
    results for that prefix are compared with them bit for bit."""
    import oracle

    cores = host_cores()
    t0 = time.perf_counter()
    oracle.solve_batch(wl.errors[:1], wl.times, wl.B, threads=1)
    t_one = max(time.perf_counter() - t0, 1e-6)
    n = int(min(wl.N, max(cores, cpu_seconds * cores / t_one)))
    threads = min(cores, n)
    t0 = time.perf_counter()
    ref = oracle.solve_batch(wl.errors[:n], wl.times, wl.B, threads=threads)
    dt = time.perf_counter() - t0
    parity = None
    if gpu_outputs is not None:
        p, c, t = gpu_outputs
        exact = bool(np.array_equal(p[:n], ref[0]) and c[:n].tobytes() == ref[1].tobytes()
                     and np.array_equal(t[:n], ref[2]))
        parity = {"compared": n, "of": wl.N, "bit_exact": exact,
                  "what": "profile, fp32 cost bits and time_used of the timed launch configuration against the oracle"}
    base = {"value": n / dt, "unit": "candidates/s", "cores": threads, "kind": "oracle",
            "sample": f"first {n} of {wl.N} candidates of {wl.name}, one single-threaded solver per core",
            "single_core_ms_per_candidate": 1e3 * t_one, "seconds": dt}
    return base, parity


def run_reference(args):
    """CPU oracle as the reference arm; rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2201_13096_b200 import workloads as W
    import oracle

    cores = host_cores()
    wl = W.make_workload(args.config, N=args.n, B=args.budget)
    t0 = time.perf_counter()
    oracle.solve_batch(wl.errors[:1], wl.times, wl.B, threads=1)
    t_one = max(time.perf_counter() - t0, 1e-6)
    total_steps = args.steps + args.warmup
    per_step_s = min(20.0, 150.0 / max(total_steps, 1))
    n = int(min(wl.N, max(cores, per_step_s * cores / t_one)))
    threads = min(cores, n)
    for _ in range(args.warmup):
        oracle.solve_batch(wl.errors[:n], wl.times, wl.B, threads=threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.solve_batch(wl.errors[:n], wl.times, wl.B, threads=threads)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = f"each step solves the first {n} of {wl.N} candidates of {wl.name}"
    line = {
        "impl": "reference", "metric": "candidate_profiles_per_s", "value": value, "unit": "candidates/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "L": wl.L, "K": wl.K, "B": wl.B, "candidates_per_step": n},
        "nominal_cell_updates_per_s": value * wl.L * wl.K * wl.B,
        "cpu_baseline": {"value": value, "unit": "candidates/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "candidates/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2201_13096_b200 import binding, sharding, workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the solver has no CPU path")
    if args.gpus > 1 and not sharding.under_launcher():
        # Started plainly with --gpus N: start the N ranks here, one process per GPU; rank 0 prints the line.
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus} asked for, {torch.cuda.device_count()} CUDA devices visible")
        raise SystemExit(sharding.spawn_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    # Candidates are independent problems: every rank solves its own shard of one long candidate
    # stream against the same timing table; no data-path collective.
    probe = W.make_workload(args.config, N=1, B=args.budget)
    n_per_rank = args.n if args.n is not None else {1: 1024, 2: 4096, 3: 1024, 4: 4096}[args.config]
    start, count = sharding.shard_range(world * n_per_rank, rank, world)
    wl = W.make_workload(args.config, N=count, B=args.budget, start=start)
    assert np.array_equal(probe.times, wl.times)
    fmt = {"default": 0, "arg": 1, "row": 2}[args.table]
    if args.mode:
        fmt = 1 if args.mode in (1, 2, 5) else 2
    plan = binding.Plan(wl.times, wl.B, device=local_rank, table_format=fmt, threads=args.threads,
                        forward_mode=args.mode, cluster=args.cluster, rows_in_global=args.rows_in_global,
                        kernel=args.kernel, schedule=args.schedule, auto_shape=args.auto_shape)
    info = plan.info
    plan.enable_timing(True)

    errors = torch.from_numpy(wl.errors).to(dev)
    profile = torch.empty((wl.N, wl.L), dtype=torch.uint8, device=dev)
    cost = torch.empty(wl.N, dtype=torch.float32, device=dev)
    time_used = torch.empty(wl.N, dtype=torch.int32, device=dev)
    ws_bytes = min(plan.workspace_bytes(wl.N), 48 << 30)
    workspace = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
    waves = -(-plan.workspace_bytes(wl.N) // max(ws_bytes, 1)) if info["feasible"] else 1
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)  # > 126 MB L2
    stream = torch.cuda.current_stream()

    def step():
        binding.solve_batch(plan, errors, profile, cost, time_used, workspace, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 0)):
        flush.fill_(1)
        step()
    barrier()
    plan.check_status()

    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    fwd_ms, back_ms = [], []
    with ClockSampler(local_rank) as clocks:
        barrier()
        for i in range(args.steps):
            flush.fill_(i & 0xFF)  # evict L2 between timed steps (outside the event pair)
            starts[i].record(stream)
            step()
            stops[i].record(stream)
            f, b = plan.last_timing()  # waits for this step
            fwd_ms.append(f)
            back_ms.append(b)
        barrier()
    step_ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    total_ms = float(sum(step_ms))
    total_ms = sharding.max_over_ranks(total_ms, dev)
    plan.check_status()

    # End to end through the host-buffer entry point: pinned host inputs, copies inside the timing.
    e2e = None
    if not args.no_e2e:
        h_err = torch.from_numpy(wl.errors).pin_memory()
        h_prof = torch.empty((wl.N, wl.L), dtype=torch.uint8).pin_memory()
        h_cost = torch.empty(wl.N, dtype=torch.float32).pin_memory()
        h_time = torch.empty(wl.N, dtype=torch.int32).pin_memory()
        for _ in range(2):
            binding.solve_batch_host(plan, h_err, h_prof, h_cost, h_time, stream)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            binding.solve_batch_host(plan, h_err, h_prof, h_cost, h_time, stream)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e_s = sharding.max_over_ranks(e2e_s, dev)
        same = (torch.equal(h_prof, profile.cpu()) and torch.equal(h_time, time_used.cpu())
                and h_cost.numpy().tobytes() == cost.cpu().numpy().tobytes())
        if not same:
            raise SystemExit("host-buffer path disagrees with the device-buffer path")
        e2e = {"value": sharding.whole_job_rate(wl.N * args.steps, world, e2e_s), "unit": "candidates/s",
               "h2d_bytes_per_step": int(h_err.numel() * 4),
               "d2h_bytes_per_step": int(wl.N * (wl.L + 8)), "ms_per_step": 1e3 * e2e_s / args.steps}

    # The same end-to-end step with Eq. 4's coefficients as input (what one search step submits):
    # K times fewer bytes go to the device.  Extra figure; the headline `e2e` above takes error tables.
    e2e_coeffs = None
    if not args.no_e2e:
        h_c = torch.from_numpy(W.sensitivity_samples(7000 + rank, wl.L, wl.N)).pin_memory()
        for _ in range(2):
            binding.solve_batch_coeffs_host(plan, h_c, h_prof, h_cost, h_time, stream)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            binding.solve_batch_coeffs_host(plan, h_c, h_prof, h_cost, h_time, stream)
        torch.cuda.synchronize()
        c_s = sharding.max_over_ranks(time.perf_counter() - t0, dev)
        plan.check_status()
        e2e_coeffs = {"value": sharding.whole_job_rate(wl.N * args.steps, world, c_s), "unit": "candidates/s",
                      "h2d_bytes_per_step": int(h_c.numel() * 4), "d2h_bytes_per_step": int(wl.N * (wl.L + 8)),
                      "ms_per_step": 1e3 * c_s / args.steps,
                      "input": "Eq. 4 coefficients [N][L], uniform in [0,1] (spdy_solve_batch_coeffs_host)"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    cand_per_s = sharding.whole_job_rate(wl.N, world, ms_per_step * 1e-3)
    fwd = float(np.mean(fwd_ms))
    back = float(np.mean(back_ms))
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    try:
        probe = binding.probe_peaks(local_rank)
    except binding.SpdyError:
        probe = (0.0, 0.0)
    sm_max = float(peaks.get("sm_max_mhz", SM_MAX_MHZ_NOMINAL))
    peak_cells = info["sm_count"] * sm_max * 1e6 * CELLS_PER_CLK_PER_SM
    # Work the forward pass has to do per launch: one update per (cell, distinct shift) pair.
    useful = info["distinct_updates"] * wl.N  # (uint8 table: valid because the synthetic errors rise with the choice index)
    achieved = useful / waves / (fwd / waves * 1e-3) if fwd > 0 else 0.0
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    cellb = 4 if info["table_format"] == 2 else 1
    hbm_bytes = wl.N * (info["band_cells"] * cellb + wl.L * wl.K * 4)
    table_name = {1: "arg_u8", 2: "row_f32"}[info["table_format"]]
    shape = plan.shape_for_batch(wl.N, workspace.numel())  # small batches run on a launch shape of their own
    kernel_name = {0: "one CTA per candidate", 1: "one CTA per candidate, rows in global memory",
                   2: "one cluster per candidate", 3: "one warp per candidate"}[shape["kernel_kind"]]
    traffic, traffic_note = ncu_traffic_per_launch(load_ncu_traffic(), binding.library().spdy_version(), wl.name, wl.B,
                                                   shape["cluster"] if shape["kernel_kind"] in (0, 2) else 0, table_name,
                                                   wl.N / waves)
    if traffic is None:
        print(f"bench.py: roofline.traffic = null: {traffic_note}", file=sys.stderr, flush=True)
    line = {
        "metric": "candidate_profiles_per_s", "value": cand_per_s, "unit": "candidates/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "L": wl.L, "K": wl.K, "B": wl.B, "candidates_per_gpu": wl.N,
                   "l2": "256 MiB buffer rewritten between timed steps (L2 flush); the walk-back table "
                         f"written per step is {info['table_bytes_per_candidate'] * wl.N / 1e6:.0f} MB",
                   "timing": "sum of per-step CUDA-event pairs on the launch stream, max over ranks",
                   "table_format": table_name,
                   "kernel": kernel_name, "threads": shape["threads"], "cluster": shape["cluster"],
                   "ctas_per_sm": info["ctas_per_sm"], "span": info["span"], "waves": int(waves)},
        "nominal_cell_updates_per_s": cand_per_s * info["nominal_updates"],
        "useful_cell_updates_per_s": cand_per_s * info["useful_updates"],
        "distinct_cell_updates_per_s": cand_per_s * info["distinct_updates"],
        "roofline": {
            "bound": "alu", "kernel": "spdy_forward_kernel" if shape["kernel_kind"] < 2 else ("spdy_forward_cluster_kernel" if shape["kernel_kind"] == 2 else "spdy_forward_warp_kernel"),
            "achieved": achieved / 1e9, "peak": peak_cells / 1e9, "unit": "Gcell-updates/s",
            "frac": achieved / peak_cells, "traffic": traffic,
            "traffic_unit": "bytes per launch", "traffic_source": traffic_note,
            "binding_unit": "shared-memory data path of the SM (32 banks x 4 B per clock): this kernel needs one 4-byte "
                            "read of the previous row per cell update, so the ceiling is a property of the design "
                            "(a design that re-used a read for several updates would sit under the arithmetic "
                            "ceiling instead); no tensor cores, HBM far from binding (roofline_hbm)",
            "peak_is": f"{info['sm_count']} SMs x {sm_max:.0f} MHz x 32 four-byte shared-memory reads per clock "
                       "(one read per cell update); of nominal unit counts, max clock of measured",
            "frac_of_arithmetic_peak": (achieved / probe[1]) if probe[1] else None,
            "peak_measured": probe[0] / 1e9, "frac_of_measured": (achieved / probe[0]) if probe[0] else None,
            "arithmetic_peak_measured": probe[1] / 1e9,
            "peak_measured_is": "spdy_probe_peaks on this device in this run: lane-consecutive 4-byte shared-memory "
                                "reads per second (the binding ceiling), and cell updates per second of the "
                                "arithmetic alone on registers",
            "kernel_ms": fwd, "walkback_ms": back,
            "distinct_updates_per_launch": useful / waves, "issued_updates_per_launch": info["issued_updates"] * wl.N / waves,
        },
        "roofline_hbm": {"bound": "hbm", "achieved": hbm_bytes / (fwd * 1e-3) / 1e9 if fwd > 0 else 0.0,
                         "peak": hbm_peak, "unit": "GB/s",
                         "frac": (hbm_bytes / (fwd * 1e-3) / 1e9 / hbm_peak) if fwd > 0 else 0.0,
                         "note": "secondary: table writes + error reads of the forward kernel, of measured copy bandwidth"},
        "gpu_launches": int(info["launches_per_wave"] * waves * args.steps),
        "clocks": clocks.summary(),
    }
    # The table format the problem statement names (one byte per cell, the argmin itself) beside the default:
    # a short second timing pass on the same inputs, device-resident, events as above.
    if info["table_format"] == 2 and not args.mode and info["feasible"]:
        plan8 = binding.Plan(wl.times, wl.B, device=local_rank, table_format=1, threads=args.threads,
                             cluster=args.cluster, rows_in_global=args.rows_in_global, kernel=args.kernel,
                             schedule=args.schedule, auto_shape=args.auto_shape)
        info8 = plan8.info
        plan8.enable_timing(True)
        ws8_bytes = min(plan8.workspace_bytes(wl.N), 48 << 30)
        ws8 = workspace[:ws8_bytes] if ws8_bytes <= workspace.numel() else torch.empty(ws8_bytes, dtype=torch.uint8, device=dev)
        waves8 = -(-plan8.workspace_bytes(wl.N) // max(ws8_bytes, 1))
        p8, c8, t8 = (torch.empty_like(x) for x in (profile, cost, time_used))
        f8, s8 = [], []
        for i in range(3 + 5):
            flush.fill_(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            binding.solve_batch(plan8, errors, p8, c8, t8, ws8, stream)
            b.record(stream)
            fw, _ = plan8.last_timing()
            if i >= 3:
                f8.append(fw)
                s8.append(a.elapsed_time(b))
        plan8.check_status()
        if not (torch.equal(p8, profile) and torch.equal(t8, time_used) and torch.equal(c8.view(torch.int32), cost.view(torch.int32))):
            raise SystemExit("the uint8-table path disagrees with the fp32-table path")
        ach8 = info8["distinct_updates"] * wl.N / (float(np.mean(f8)) * 1e-3)
        line["roofline_arg_u8"] = {"table_format": "arg_u8", "kernel_ms": float(np.mean(f8)), "ms_per_step": float(np.mean(s8)),
                                   "achieved": ach8 / 1e9, "peak": peak_cells / 1e9, "unit": "Gcell-updates/s",
                                   "frac": ach8 / peak_cells, "workspace_bytes": int(plan8.workspace_bytes(wl.N)),
                                   "workspace_bytes_row_f32": int(plan.workspace_bytes(wl.N)), "waves": int(waves8),
                                   "launches_per_step": int(info8["launches_per_wave"] * waves8),
                                   "note": "5 timed steps after 3 warm-ups; outputs identical to the fp32-table path; "
                                           "bound by instruction issue, see profiles/forward_kernel_bert_base_one_wave.md"}
        plan8.close()
    if e2e:
        line["e2e"] = e2e
    if e2e_coeffs:
        line["e2e_coeffs"] = e2e_coeffs
    if args.search > 0:
        from paper_2201_13096_b200 import search as S

        solver = S.gpu_solver(wl.times, wl.B, device=local_rank)
        loss = W.synthetic_calibration_loss(args.config, wl.L, wl.K)
        t0 = time.perf_counter()
        res = S.search(wl.times, wl.B, W.sensitivity_samples(args.config, wl.L, 1)[0],
                       W.sensitivity_samples(args.config + 100, wl.L, args.search),
                       W.mutation_draws(args.config, wl.L), loss, trials=args.search, solver=solver)
        wall = time.perf_counter() - t0
        line["search"] = {"trials_per_loop": args.search, "neighbourhood_sizes": int(np.ceil(0.1 * wl.L)),
                          "evals": res["evals"], "accepted": len(res["accepted"]), "loss": res["loss"],
                          "dp_batches": res["dp_batches"], "dp_candidates": res["dp_candidates"],
                          "dp_ms": 1e3 * res["dp_seconds"], "eval_ms": 1e3 * res["eval_seconds"], "wall_ms": 1e3 * wall,
                          "note": "synthetic loss (microseconds per call); with a real stitched-model evaluation "
                                  "the evaluations dominate, as the paper reports"}
    parity = None
    if not args.no_cpu_baseline and world == 1:
        gpu_out = (profile.cpu().numpy(), cost.cpu().numpy(), time_used.cpu().numpy())
        line["cpu_baseline"], parity = oracle_baseline(wl, args.cpu_seconds, gpu_out)
        line["parity"] = parity
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    if parity is not None and not parity["bit_exact"]:
        raise SystemExit("the timed launch configuration disagrees with the oracle")


SWEEP_POINTS = [  # (config, N, B override)
    (4, 1, None), (4, 16, None), (4, 256, None), (4, 4096, None), (4, 65536, None),
    (4, 4096, 1000), (4, 4096, 100000), (1, None, None), (2, None, None), (3, None, None),
]


def run_sweep(args):
    """Every named shape and sweep point on one GPU: device-resident timing, and the oracle on the same
    candidates (all of them up to N = 4096, a seeded sample beyond), timed and compared bit for bit with
    the GPU's outputs."""
    import torch

    import oracle
    from paper_2201_13096_b200 import binding, workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the solver has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cores = host_cores()
    lds_peak, _ = binding.probe_peaks(0)
    fmt = {"default": 0, "arg": 1, "row": 2}[args.table]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rows = []
    for cfg, n, budget in SWEEP_POINTS:
        wl = W.make_workload(cfg, N=n, B=budget)
        plan = binding.Plan(wl.times, wl.B, device=0, table_format=fmt)
        info = plan.info
        plan.enable_timing(True)
        errors = torch.from_numpy(wl.errors).to(dev)
        ws = torch.empty(max(256, min(plan.workspace_bytes(wl.N), 48 << 30)), dtype=torch.uint8, device=dev)
        out = None
        fwd, back, total = [], [], []
        for it in range(3 + 5):
            flush.fill_(it)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            out = binding.solve_batch(plan, errors, workspace=ws)
            b.record()
            f, w = plan.last_timing()
            if it >= 3:
                fwd.append(f)
                back.append(w)
                total.append(a.elapsed_time(b))
        plan.check_status()
        ms, f_ms = float(np.mean(total)), float(np.mean(fwd))
        # oracle: single-core time of one candidate, then a bounded sample on all cores, compared
        t0 = time.perf_counter()
        oracle.solve_batch(wl.errors[:1], wl.times, wl.B, threads=1)
        one = time.perf_counter() - t0
        # every candidate up to N = 4096; a seeded sample of 4096 at N = 65536 and of 256 at B = 10^5, where
        # the whole batch would take the oracle minutes (its time there is extrapolated linearly in N)
        k = wl.N if (wl.N <= 4096 and wl.B < 100000) else (256 if wl.B >= 100000 else 4096)
        k = int(min(wl.N, k))
        sample = np.sort(np.random.default_rng(1).choice(wl.N, size=k, replace=False))
        t0 = time.perf_counter()
        ref = oracle.solve_batch(wl.errors[sample], wl.times, wl.B, threads=min(cores, k))
        dt = time.perf_counter() - t0
        p, c, t = (x.cpu().numpy() for x in out)
        exact = bool(np.array_equal(p[sample], ref[0]) and c[sample].tobytes() == ref[1].tobytes()
                     and np.array_equal(t[sample], ref[2]))
        cellb = 4 if info["table_format"] == 2 else 1
        hbm_bytes = wl.N * (info["band_cells"] * cellb + wl.L * wl.K * 4)
        shape = plan.shape_for_batch(wl.N, ws.numel())  # small batches run on a launch shape of their own
        row = {"workload": wl.name, "N": wl.N, "L": wl.L, "K": wl.K, "B": wl.B,
               "table_format": {1: "arg_u8", 2: "row_f32"}[info["table_format"]],
               "threads": shape["threads"], "cluster": shape["cluster"], "rows_in_global": info["rows_in_global"],
               "warp_per_candidate": int(shape["kernel_kind"] == 3),
               "gpu_ms": ms, "forward_ms": f_ms, "walkback_ms": float(np.mean(back)),
               "candidates_per_s": wl.N / (ms * 1e-3),
               "nominal_cell_updates_per_s": wl.N * info["nominal_updates"] / (ms * 1e-3),
               "executed_cell_updates_per_s": wl.N * info["distinct_updates"] / (f_ms * 1e-3),
               "roofline_frac_of_measured_lds": wl.N * info["distinct_updates"] / (f_ms * 1e-3) / lds_peak,
               "table_and_errors_gb_per_s": hbm_bytes / (f_ms * 1e-3) / 1e9,
               "oracle_ms_per_candidate_one_core": 1e3 * one,
               "oracle_candidates_per_s_all_cores": k / dt, "oracle_cores": min(cores, k), "oracle_sample": k,
               "bit_exact_on_sample": exact}
        rows.append(row)
        print(json.dumps(row), flush=True)
        plan.close()
        del errors, ws
        torch.cuda.empty_cache()
    head = ("| workload | table | CTA | GPU ms | candidates/s | nominal upd/s | executed upd/s | frac | table+errors GB/s "
            "| oracle ms (1 core) | oracle cand/s (cores) | bit-exact (candidates compared) |")
    print(head, file=sys.stderr)
    print("|" + "---|" * 12, file=sys.stderr)
    for r in rows:
        shape = (f'{r["threads"]} thr' + (f' x{r["cluster"]}' if r["cluster"] > 1 else "")
                 + (", rows in global" if r["rows_in_global"] else "") + (", warp per candidate" if r["warp_per_candidate"] else ""))
        print(f'| {r["workload"]} | {r["table_format"]} | {shape} | {r["gpu_ms"]:.3f} | {r["candidates_per_s"]:.4g} | '
              f'{r["nominal_cell_updates_per_s"]:.3g} | {r["executed_cell_updates_per_s"]:.3g} | '
              f'{r["roofline_frac_of_measured_lds"]:.3f} | {r["table_and_errors_gb_per_s"]:.0f} | '
              f'{r["oracle_ms_per_candidate_one_core"]:.2f} | {r["oracle_candidates_per_s_all_cores"]:.4g} ({r["oracle_cores"]}) | '
              f'{"yes" if r["bit_exact_on_sample"] else "NO"} ({r["oracle_sample"]}) |', file=sys.stderr)
    if not all(r["bit_exact_on_sample"] for r in rows):
        raise SystemExit("a sweep point disagrees with the oracle")


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
