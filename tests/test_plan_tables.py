"""The host side of a plan, tested without nvcc and without a GPU: the tables that steer the kernels (live
bands, shift slots, warp passes, guard cells, table layout) are read back through the C ABI of the
host-only library and checked two ways, both written here from the definitions and independent of the C++:

* margins - for every layer, pass and slot the lowest and highest previous-row cell a lane reads
  (Algorithm 1's shifted read D[l-1, t - t_l^s]) lies inside the cells known to hold the row or +inf, every
  cell of a row is written exactly once, and rows and tables fit their buffers;
* replay - a NumPy replay of the forward pass that follows the plan's passes literally (same buffers, same
  guard cells, unwritten cells poisoned) reproduces the oracle's cost and time_used.
"""
import numpy as np
import pytest

import oracle
from paper_2201_13096_b200 import binding, build as build_mod, workloads as W

U8, F32 = binding.SPDY_TABLE_ARG_U8, binding.SPDY_TABLE_ROW_F32


@pytest.fixture(scope="module", autouse=True)
def host_library():
    build_mod.build_host()
    binding.select_library("host")
    yield
    binding._lib = None  # back to the default build for the modules that follow


def pass_fields(row):
    start, kr = int(row[0]), int(np.uint32(row[1]))
    return start, kr & 0xFF, (kr >> 8) & 0xFF, (kr >> 16) & 1, kr >> 24


def mask_bits(masks, n_slots):
    """[passes][n_slots] 0/1 from the packed 64-bit words."""
    words = np.ascontiguousarray(masks, dtype="<u8")
    bits = np.unpackbits(words.view(np.uint8).reshape(words.shape[0], -1), axis=1, bitorder="little")
    return bits[:, :n_slots].astype(bool)


def check_margins(t):
    """Independent re-derivation of what spdy_plan_verify proves (vectorised over the passes of a layer)."""
    L, K, pad, stride = t["L"], t["K"], t["pad"], t["row_stride"]
    layers, slots, passes = t["layers"], t["slots"].astype(np.int64), t["passes"]
    width, rowoff, extent, nslots, fill = layers[:, 0], layers[:, 1].astype(np.int64), layers[:, 4], layers[:, 5], layers[:, 6]
    start_all = passes[:, 0].astype(np.int64)
    kr = passes[:, 1].astype(np.uint32)
    u_lo_all, u_hi_all = (kr & 0xFF).astype(int), ((kr >> 8) & 0xFF).astype(int)
    dense_all, cpl_all = ((kr >> 16) & 1).astype(bool), (kr >> 24).astype(np.int64)
    bits_all = mask_bits(t["pass_masks"], K) if t["n_passes"] else np.zeros((0, K), bool)
    for l in range(L):
        end = rowoff[l] + (width[l] if t["kernel_kind"] == 2 else extent[l])
        assert end <= (rowoff[l + 1] if l + 1 < L else t["pitch"]), "table rows overlap"
        assert extent[l] >= width[l] >= 1 and extent[l] % 32 == 0

    def check_passes(l, idx, cells, read_lo, read_hi):
        """Passes `idx` of layer l, each `cells` long: mask == overlap, and every read inside [read_lo, read_hi)."""
        n = int(nslots[l])
        a, b = slots[l, :n, 0][None, :], slots[l, :n, 1][None, :]
        start = start_all[idx][:, None]
        cells = np.broadcast_to(np.asarray(cells, np.int64).reshape(-1, 1), start.shape)
        over = (b >= a) & (start + cells > a) & (start <= b)
        assert np.array_equal(over, bits_all[idx][:, :n]), "a pass's slot mask differs from the slots that overlap it"
        assert not bits_all[idx][:, n:].any()
        lo = np.where(over, start - a, read_lo)
        hi = np.where(over, start + cells - 1 - a, read_lo)
        assert (lo >= read_lo).all() and (hi < read_hi).all(), f"layer {l}: a read leaves the cells that hold the row or +inf"
        u = np.arange(n)[None, :]
        inside = (u >= u_lo_all[idx][:, None]) & (u < u_hi_all[idx][:, None])
        assert (inside | ~over).all()
        assert (~(dense_all[idx][:, None] & inside) | over).all()

    def covered_once(starts, lengths, upto):
        seen = np.zeros(upto + 1, int)
        np.add.at(seen, starts, 1)
        np.add.at(seen, np.minimum(starts + lengths, upto), -1)
        assert (np.cumsum(seen)[:upto] == 1).all(), "every cell of a row is written exactly once"

    if t["kernel_kind"] == 2:
        C, sl = t["cluster"], t["slices"].astype(np.int64)
        for l in range(L):
            starts, lengths = [], []
            for r in range(C):
                lo, hi, cpl, nsp, first, q0, win_len, prev_slice = (int(x) for x in sl[l, r])
                assert 0 <= lo <= hi <= width[l] and hi - lo <= t["out_stride"] and win_len <= t["win_stride"]
                if nsp == 0:
                    assert lo == hi
                    continue
                idx = np.arange(first, first + nsp)
                assert np.array_equal(start_all[idx], lo + np.arange(nsp) * 32 * cpl)
                check_passes(l, idx, 32 * cpl, q0, q0 + win_len)
                starts.append(start_all[idx])
                lengths.append(np.minimum(start_all[idx] + 32 * cpl, hi) - start_all[idx])
            covered_once(np.concatenate(starts), np.concatenate(lengths), int(width[l]))
        return
    Wc, ptr = t["warps_per_candidate"], t["pass_ptr"]
    assert len(ptr) == L * Wc + 1 and ptr[-1] == t["n_passes"] and (np.diff(ptr) >= 0).all()
    for l in range(L):
        assert fill[l] >= 0 and extent[l] + fill[l] <= stride - pad, "row and its +inf tail must fit the buffer"
        idx = np.arange(ptr[l * Wc], ptr[(l + 1) * Wc])
        cells = 32 * cpl_all[idx]
        assert (cpl_all[idx] >= 1).all() and (cpl_all[idx] <= t["max_cells_per_lane"]).all()
        assert (start_all[idx] % 32 == 0).all() and (start_all[idx] + cells <= extent[l]).all()
        check_passes(l, idx, cells, -pad, stride - pad if l == 0 else extent[l - 1] + fill[l - 1])
        covered_once(start_all[idx], cells, int(extent[l]))


def slot_errors(times, errors_one, B, l, t, merged):
    """Error each shift slot of layer l carries: the smallest error among the usable choices at that shift
    (row-value table and the byte table's merged set), or the choice's own (byte table, slot u = choice u)."""
    n = int(t["layers"][l, 5])
    mn = int(t["layers"][l, 3])
    out = np.full(n, np.inf, np.float32)
    for u in range(n):
        a, b = (int(x) for x in t["slots"][l, u])
        if b < a:
            continue
        if merged:
            ks = [k for k in range(times.shape[1]) if times[l, k] <= B and times[l, k] - mn == a]
            out[u] = min(errors_one[l, k] for k in ks)
        else:
            out[u] = errors_one[l, u]
    return out


def replay(t, times, errors_one, B, merged):
    """The forward pass exactly as the plan's passes prescribe it (values only), for one candidate."""
    L, pad, stride = t["L"], t["pad"], t["row_stride"]
    layers, slots, passes, masks, ptr = t["layers"], t["slots"], t["passes"], t["pass_masks"], t["pass_ptr"]
    Wc = t["warps_per_candidate"]
    buf = np.full((2, stride), np.inf, np.float32)
    buf[0, pad] = 0.0
    for l in range(L):
        prev, cur = buf[l & 1], buf[(l + 1) & 1]
        extent = int(layers[l, 4])
        cur[pad:pad + extent] = np.nan  # unwritten
        e = slot_errors(times, errors_one, B, l, t, merged)
        for p in range(ptr[l * Wc], ptr[(l + 1) * Wc]):
            start, u_lo, u_hi, dense, cpl = pass_fields(passes[p])
            cells = start + np.arange(32 * cpl)
            best = np.full(32 * cpl, np.inf, np.float32)
            for u in range(int(layers[l, 5])):
                if (int(masks[p][u >> 6]) >> (u & 63)) & 1:
                    src = prev[pad + cells - int(slots[l, u, 0])]
                    assert not np.isnan(src).any(), "read of a cell nobody wrote"
                    best = np.minimum(best, (src + e[u]).astype(np.float32))
            cur[pad + cells] = best
        cur[pad + extent:pad + extent + int(layers[l, 6])] = np.inf
        cur[pad + extent + int(layers[l, 6]):] = np.nan  # beyond the refilled tail nothing may be read
    last = buf[L & 1][pad:pad + int(layers[L - 1, 0])]
    if not np.isfinite(last).any():
        return np.float32(np.inf), -1
    tt = int(np.argmin(last))  # first minimum = lowest t
    return last[tt], int(layers[L - 1, 2]) + tt


SHAPES = [dict(), dict(table_format=U8), dict(schedule=1), dict(schedule=2), dict(schedule=3), dict(table_format=U8, schedule=2), dict(threads=256), dict(threads=512), dict(threads=1024),
          dict(rows_in_global=1), dict(kernel=binding.SPDY_KERNEL_WARP), dict(kernel=binding.SPDY_KERNEL_CTA),
          dict(table_format=U8, kernel=binding.SPDY_KERNEL_WARP), dict(schedule=3 | (6 << 8)), dict(schedule=5 << 8),
          dict(cluster=2), dict(cluster=4), dict(cluster=8), dict(table_format=U8, cluster=4)]


def plans_of(times, B, **kw):
    """A plan and every table set it carries: (label, tables, merged?)."""
    try:
        plan = binding.Plan(times, B, device=-1, **kw)
    except binding.SpdyError as e:
        assert e.status == -3, (kw, e)  # a shape this problem cannot take (unsupported), never anything else
        return None, []
    sets = []
    info = plan.info
    if info["feasible"]:
        fmt_row = info["table_format"] == F32
        sets.append(("main", plan.tables(0), fmt_row))
        if info["launches_per_wave"] == 5:
            sets.append(("merged", plan.tables(-1), True))
        for i in range(info["alternates"]):
            sets.append((f"alt{i + 1}", plan.tables(i + 1), fmt_row))
    return plan, sets


@pytest.mark.parametrize("cfg,B", [(0, None), (1, None), (2, None), (3, None), (4, 1000), (4, 2500), (4, 100000)])
def test_margins_of_the_named_shapes_in_every_launch_shape(cfg, B):
    wl = W.make_workload(cfg, N=1, B=B)
    checked = 0
    for kw in SHAPES:
        plan, sets = plans_of(wl.times, wl.B, **kw)
        if plan is None:
            continue
        plan.verify()
        for label, t, _ in sets:
            check_margins(t)
            checked += 1
    assert checked >= 8


def test_margins_and_replay_on_fuzzed_shapes():
    """The shapes of the GPU fuzz test (K up to 255: several mask words; zero, repeated and over-budget times)."""
    rng = np.random.default_rng(2024)
    for trial in range(60):
        L = int(rng.integers(1, 13))
        K = int(rng.choice([1, 2, 3, 17, 64, 65, 130, 255]))
        B = int(rng.choice([0, 7, 300, 1500, 4000]))
        scale = max(1, int(B * rng.choice([0.05, 0.3, 1.2]) / max(L, 1)) + 1)
        times = rng.integers(0, 2 * scale + 1, size=(L, K)).astype(np.int32)
        if rng.random() < 0.5:
            times = np.sort(times, axis=1)[:, ::-1].copy()
        if rng.random() < 0.3:
            times[rng.integers(L), :] = 0
        errors = rng.lognormal(0.0, 1.0, size=(1, L, K)).astype(np.float32)
        ref = oracle.solve_batch(errors, times, B)
        for kw in (dict(), dict(table_format=U8), dict(kernel=binding.SPDY_KERNEL_WARP), dict(schedule=1), dict(schedule=3),
                   dict(cluster=int(rng.choice([2, 4, 8]))), dict(rows_in_global=1)):
            plan, sets = plans_of(times, B, **kw)
            if plan is None:
                continue
            plan.verify()
            for label, t, merged in sets:
                check_margins(t)
                if t["kernel_kind"] != 2 and (merged or label != "merged"):
                    if label == "merged" and not np.all(np.diff(errors[0], axis=1) >= 0):
                        continue  # the merged byte-table set is only run for candidates it is exact for
                    cost, tu = replay(t, times, errors[0], B, merged)
                    assert np.float32(cost).tobytes() == ref[1][0].tobytes() and tu == ref[2][0], (trial, kw, label)


@pytest.mark.parametrize("cfg,B,kw", [(2, None, dict()), (2, None, dict(table_format=U8)), (1, None, dict()),
                                      (4, 1000, dict()), (4, 1000, dict(kernel=binding.SPDY_KERNEL_CTA)),
                                      (4, 2500, dict(threads=256)), (2, None, dict(schedule=1)), (2, None, dict(schedule=3))])
def test_replay_of_the_named_shapes_matches_the_oracle(cfg, B, kw):
    wl = W.make_workload(cfg, N=2, B=B)
    ref = oracle.solve_batch(wl.errors, wl.times, wl.B)
    plan, sets = plans_of(wl.times, wl.B, **kw)
    for label, t, merged in sets:
        if t["kernel_kind"] == 2:
            continue
        for n in range(wl.N):
            cost, tu = replay(t, wl.times, wl.errors[n], wl.B, merged)
            assert np.float32(cost).tobytes() == ref[1][n].tobytes() and tu == ref[2][n], (label, n)


def test_pass_schedules_trade_wasted_updates_against_passes():
    """A pass is all-or-nothing per slot.  Passes of one length waste most updates on partly overlapping
    slots, levelled passes (the default with the fp32 table) fewer with as many passes, cost-sized passes
    fewest with half as many passes again; the work that has to be done is the same."""
    wl = W.make_workload(2, N=1)
    plans = {s: binding.Plan(wl.times, wl.B, device=-1, auto_shape=1, schedule=s) for s in (0, 1, 2, 3)}
    info = {s: p.info for s, p in plans.items()}
    passes = {s: p.tables(0)["n_passes"] for s, p in plans.items()}
    assert len({i["distinct_updates"] for i in info.values()}) == 1
    d = info[1]["distinct_updates"]
    assert d <= info[3]["issued_updates"] < info[2]["issued_updates"] < info[1]["issued_updates"] < 1.06 * d
    assert info[0]["issued_updates"] == info[2]["issued_updates"] < 1.03 * d
    assert passes[2] <= 1.05 * passes[1] and passes[3] > 1.2 * passes[1]
    u8 = {s: binding.Plan(wl.times, wl.B, device=-1, auto_shape=1, table_format=U8, schedule=s).info for s in (0, 1)}
    assert u8[0]["issued_updates"] == u8[1]["issued_updates"]  # the byte table keeps passes of one length
    # the fp32 table's 128-thread build unrolls passes twice as long: half as many passes
    assert passes[1] < 0.6 * binding.Plan(wl.times, wl.B, device=-1, auto_shape=1, table_format=U8, schedule=1).tables(0)["n_passes"]


def test_small_batches_get_their_own_launch_shapes():
    wl = W.make_workload(2, N=1)
    plan = binding.Plan(wl.times, wl.B, device=-1)
    info = plan.info
    assert info["alternates"] >= 4
    kinds = [(plan.tables(i + 1)["kernel_kind"], plan.tables(i + 1)["threads"], plan.tables(i + 1)["cluster"])
             for i in range(info["alternates"])]
    assert {c for k, _, c in kinds if k == 2} == {2, 4, 8}
    assert any(k == 0 and th > info["threads"] for k, th, _ in kinds)
    # the workspace asked for covers whichever shape runs
    one = binding.Plan(wl.times, wl.B, device=-1, auto_shape=1)
    assert plan.workspace_bytes(7) >= one.workspace_bytes(7)
    assert one.info["alternates"] == 0
    for pinned in (dict(threads=128), dict(cluster=2), dict(kernel=binding.SPDY_KERNEL_CTA)):
        assert binding.Plan(wl.times, wl.B, device=-1, **pinned).info["alternates"] == 0


def test_launch_shape_by_batch_size():
    """Which table set a batch runs on: the largest cluster that still gives every CTA an SM, a 512-thread CTA
    while every candidate can have an SM to itself, the main shape from there on - and the main shape whenever
    the workspace is too small for the shape picked."""
    wl = W.make_workload(2, N=1)
    plan = binding.Plan(wl.times, wl.B, device=-1)
    shape = {n: plan.shape_for_batch(n) for n in (1, 18, 19, 37, 38, 74, 75, 148, 149, 295, 296, 4096)}
    assert [shape[n]["cluster"] for n in (1, 18, 19, 37, 38, 74)] == [8, 8, 4, 4, 2, 2]
    assert all(shape[n]["kernel_kind"] == 2 for n in (1, 18, 19, 37, 38, 74))
    assert shape[75]["kernel_kind"] == 0 and shape[75]["threads"] == 512 and shape[148]["threads"] == 512
    for n in (149, 295, 296, 4096):
        assert shape[n]["which"] == 0 and shape[n]["threads"] == plan.info["threads"]
    tight = binding.Plan(wl.times, wl.B, device=-1, auto_shape=1).workspace_bytes(2)
    assert plan.shape_for_batch(7, tight)["which"] == 0
    assert binding.library().spdy_plan_shape_for_batch(None, 5, 0) == -1


def test_narrow_rows_take_the_warp_kernel():
    wl = W.make_workload(4, N=1, B=1000)
    info = binding.Plan(wl.times, wl.B, device=-1).info
    assert info["kernel"] == binding.SPDY_KERNEL_WARP and info["candidates_per_cta"] == 4
    wide = W.make_workload(2, N=1)
    assert binding.Plan(wide.times, wide.B, device=-1).info["kernel"] == binding.SPDY_KERNEL_CTA
    with pytest.raises(binding.SpdyError) as e:  # more than 64 shift slots per layer: two per lane do not suffice
        rng = np.random.default_rng(0)
        binding.Plan(rng.permuted(np.tile(np.arange(1, 101, dtype=np.int32), (3, 1)), axis=1), 400, device=-1,
                     kernel=binding.SPDY_KERNEL_WARP)
    assert e.value.status == -3


def test_host_library_has_no_device_code():
    lib = binding.library()
    for name in binding.HOST_EXPORTS:
        assert hasattr(lib, name)
    assert not hasattr(lib, "spdy_solve_batch")
    t = np.ones((2, 3), np.int32)
    with pytest.raises(binding.SpdyError) as e:
        binding.Plan(t, 5, device=0)
    assert e.value.status == -8 and b"host side only" in lib.spdy_strerror(-8)
    assert binding.time_target(0.478, 2.0) == pytest.approx(0.239)
