// Host side of the batched SPDY dynamic program: plans (live bands, shift slots, warp passes, table
// layout, launch shape), the exhaustive check of their index arithmetic, and the host helpers of
// Sections 3.1, 3.2 and 4.  Plain C++: builds with the host compiler alone.
//
// Section 3.2 (Eq. 2-3) and Appendix A (Algorithm 1) define the dynamic program these tables describe.
#include "spdy_plan.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <utility>

namespace spdy {

namespace {

const DeviceHooks *g_hooks = nullptr;

// Eq. 4's squares (i / (K - 1))^2, formed in fp64 and rounded once to fp32; K = 1 gives 0.
void fill_qtab(spdy_plan *p)
{
    p->qtab.assign(p->K, 0.0f);
    for (int i = 0; i < p->K && p->K > 1; ++i) {
        const double r = static_cast<double>(i) / static_cast<double>(p->K - 1);
        p->qtab[i] = static_cast<float>(r * r);
    }
}

// Live band of every row and the range of every (layer, choice) pair.
//   lo_l = sum_{j<=l} mn_j,  hi_l = min(B, sum_{j<=l} mx_j, B - sum_{j>l} mn_j)
// with mn/mx the smallest/largest usable (<= B) time of a layer.  A cell below lo_l is
// unreachable, a cell above hi_l is unreachable or cannot be completed within B; a cell inside
// the band depends only on cells inside the previous band.
int build_bands(spdy_plan *p)
{
    const int L = p->L, K = p->K;
    const int64_t B = p->B;
    std::vector<int64_t> mn(L), mx(L);
    p->feasible = true;
    for (int l = 0; l < L; ++l) {
        int64_t lo = -1, hi = -1;
        for (int k = 0; k < K; ++k) {
            const int64_t tau = p->times[static_cast<size_t>(l) * K + k];
            if (tau < 0) return SPDY_ERR_INVALID_ARG;
            if (tau > B) continue;
            lo = (lo < 0 || tau < lo) ? tau : lo;
            hi = tau > hi ? tau : hi;
        }
        if (lo < 0) p->feasible = false;
        mn[l] = lo < 0 ? 0 : lo;
        mx[l] = hi < 0 ? 0 : hi;
    }
    int64_t total_mn = 0;
    for (int l = 0; l < L; ++l) total_mn += mn[l];
    if (total_mn > B) p->feasible = false;

    p->layers.assign(L, LayerDesc{0, 0, 0, 0, 0, 0, 0, 0});
    p->taps.assign(static_cast<size_t>(L) * K, TapRange{0, -1});
    p->band_cells = p->useful_updates = 0;
    p->max_width = 0;
    if (!p->feasible) return SPDY_OK;

    int64_t sum_mn = 0, sum_mx = 0, prev_width = 1;
    for (int l = 0; l < L; ++l) {
        sum_mn += mn[l];
        sum_mx += mx[l];
        const int64_t lo = sum_mn;
        const int64_t hi = std::min<int64_t>(std::min<int64_t>(B, sum_mx), B - (total_mn - sum_mn));
        const int64_t width = hi - lo + 1;
        p->layers[l].width = static_cast<int32_t>(width);
        p->layers[l].lo = static_cast<int32_t>(lo);
        p->layers[l].mn = static_cast<int32_t>(mn[l]);
        p->band_cells += width;
        p->max_width = std::max<int32_t>(p->max_width, static_cast<int32_t>(width));
        for (int k = 0; k < K; ++k) {
            const int64_t tau = p->times[static_cast<size_t>(l) * K + k];
            if (tau > B) continue;
            const int64_t a = tau - mn[l];
            const int64_t b = std::min<int64_t>(width - 1, prev_width - 1 + a);
            if (b < a) continue;
            p->taps[static_cast<size_t>(l) * K + k] = TapRange{static_cast<int32_t>(a), static_cast<int32_t>(b)};
            p->useful_updates += b - a + 1;
        }
        prev_width = width;
    }
    return SPDY_OK;
}

// Shift slots of every layer (see TapRange).
// merge: 0 = slot u is choice u; 1 = groups of equal time in ascending time order (row-value
// table); 2 = groups of equal time in the order of their lowest member (byte table, second plan).
void build_slots(spdy_plan *p, int merge)
{
    const int L = p->L, K = p->K;
    p->slots.assign(static_cast<size_t>(L) * K, TapRange{0, -1});
    p->slot_ptr.assign(static_cast<size_t>(L) * (K + 1), 0);
    p->slot_member.assign(static_cast<size_t>(L) * K, 0);
    p->distinct_updates = 0;
    std::vector<int> order(K);
    for (int l = 0; l < L; ++l) {
        const TapRange *taps = &p->taps[static_cast<size_t>(l) * K];
        TapRange *slots = &p->slots[static_cast<size_t>(l) * K];
        uint8_t *ptr = &p->slot_ptr[static_cast<size_t>(l) * (K + 1)];
        uint8_t *member = &p->slot_member[static_cast<size_t>(l) * K];
        int nslots = 0, nmembers = 0;
        if (!merge) {
            for (int k = 0; k < K; ++k) {
                slots[k] = taps[k];
                ptr[k] = static_cast<uint8_t>(k);
                member[k] = static_cast<uint8_t>(k);
            }
            nslots = nmembers = K;
        } else {
            int usable = 0;
            for (int k = 0; k < K; ++k)
                if (taps[k].b >= taps[k].a) order[usable++] = k;
            std::stable_sort(order.begin(), order.begin() + usable,
                             [&](int x, int y) { return taps[x].a < taps[y].a; });
            if (merge == 2) {
                // groups (runs of equal shift in `order`, members ascending) re-ordered by first member
                std::vector<std::pair<int, int>> runs;  // [begin, end) in `order`
                for (int i = 0; i < usable;) {
                    int j = i + 1;
                    while (j < usable && taps[order[j]].a == taps[order[i]].a) ++j;
                    runs.emplace_back(i, j);
                    i = j;
                }
                std::sort(runs.begin(), runs.end(),
                          [&](const std::pair<int, int> &x, const std::pair<int, int> &y) { return order[x.first] < order[y.first]; });
                std::vector<int> reordered;
                for (const auto &r : runs)
                    for (int i = r.first; i < r.second; ++i) reordered.push_back(order[i]);
                std::copy(reordered.begin(), reordered.end(), order.begin());
            }
            for (int i = 0; i < usable; ++i) {
                const int k = order[i];
                if (nslots == 0 || slots[nslots - 1].a != taps[k].a) {
                    ptr[nslots] = static_cast<uint8_t>(nmembers);
                    slots[nslots++] = taps[k];  // equal times have equal ranges
                }
                member[nmembers++] = static_cast<uint8_t>(k);
            }
        }
        for (int u = nslots; u <= K; ++u) ptr[u] = static_cast<uint8_t>(nmembers);
        p->layers[l].nslots = nslots;
        for (int u = 0; u < nslots; ++u)
            if (slots[u].b >= slots[u].a) p->distinct_updates += slots[u].b - slots[u].a + 1;
    }
}

// A 1024-thread CTA leaves 64 registers per thread: not enough for 24 cells per lane.  With the rows in
// global memory the addresses are 64-bit, which costs a few more registers still.
int cells_per_lane_cap(int kind, int threads, int mode)
{
    if (kind == KERNEL_CTA_GLOBAL) return threads >= 1024 ? global_rows_cap_1024(mode) : kRmax;
    if (kind == KERNEL_WARP) return long_pass_cap(mode);
    if (threads == 128 || threads == 512) return long_pass_cap(mode);  // 128 registers per thread available
    return threads >= 1024 ? cells_per_lane_1024(mode) : kRmax;
}

// The kernel builds differ in the largest pass they unroll; a plan picks the smallest that holds its passes.
int rcap_for(int kind, int threads, int mode, int max_cpl)
{
    if (kind == KERNEL_CTA_GLOBAL) return cells_per_lane_cap(kind, threads, mode);
    if (kind == KERNEL_WARP) return max_cpl <= warp_short_cap(mode) ? warp_short_cap(mode) : long_pass_cap(mode);
    return max_cpl <= 8 ? 8 : cells_per_lane_cap(kind, threads, mode);
}

// CTA size of the rows-in-global-memory kernel when the caller leaves it open.
constexpr int kGlobalRowsThreads = 1024;

// Room left under the per-CTA shared-memory limit for the kernels' small static arrays (reductions).
constexpr int64_t kStaticSmemReserve = 1024;

// One pass over blocks [i, j) of 32 cells each and the slots that overlap it.
struct PassPlan {
    int i, j;
    int u_lo, u_hi, count;
    double cost;
};

// Passes of one layer.  `ba`/`bb`: first and last 32-cell block each slot touches.  A pass is all-or-nothing
// per slot: a slot that overlaps it only partly costs the whole pass.
// SCHED_UNIFORM: passes of one length, chosen so that the rounds of W passes are equally full, dealt
// round-robin: every warp runs the same unrolled body.
// SCHED_LEVELLED: as many passes as that, but cut where their costs (in shared-memory wavefronts) are
// level: a pass over the ramp at either end of a band, where few slots overlap, is longer or shorter than
// one in the middle so that all cost the same, which both trims the partly overlapping work (4.5 % -> 2.6 %
// of the issued updates at the BERT-base shape) and keeps the warps level at the layer's barrier.
// SCHED_SIZED: pass boundaries by dynamic programming over the blocks, minimising the summed cost (short
// passes where slots begin and end, long ones in between), then dealt to the warps longest first onto the
// least loaded warp, the pass length cap shrinking until the warps are level within a few per cent.  It
// wastes least (1.6 %) and measures slowest: it makes half as many passes again, and every pass pays for its
// own slot reads and set-up.  One warp per candidate has nobody to level with and takes it as its LEVELLED.
constexpr int SCHED_UNIFORM = 1, SCHED_LEVELLED = 2, SCHED_SIZED = 3;

void plan_layer_passes(const std::vector<int> &ba, const std::vector<int> &bb, int nb, int W, int R, int schedule,
                       std::vector<std::vector<PassPlan>> &per_warp, double *total_cost, double *makespan,
                       int *blocks_covered)
{
    *blocks_covered = nb;
    *total_cost = *makespan = 0.0;
    per_warp.assign(W, {});
    if (nb == 0) return;  // a layer of an infeasible plan
    const int ns = static_cast<int>(ba.size());
    std::vector<int> started(nb + 2, 0), ended(nb + 2, 0);  // started[j]: slots with ba < j; ended[i]: slots with bb < i
    for (int u = 0; u < ns; ++u) {
        if (bb[u] < ba[u]) continue;
        started[std::min(ba[u] + 1, nb + 1)] += 1;
        ended[std::min(bb[u] + 1, nb + 1)] += 1;
    }
    for (int j = 1; j <= nb + 1; ++j) {
        started[j] += started[j - 1];
        ended[j] += ended[j - 1];
    }
    auto overlapping = [&](int i, int j) { return started[std::min(j, nb + 1)] - ended[std::min(i, nb + 1)]; };
    // Cost of a pass in wavefronts of the shared-memory data path, the unit the kernel is bound by: one per
    // slot and 32 cells, the 16-byte slot-pair reads (measured: about three wavefronts per pair), the stores
    // of the new row, and the pass's own descriptor and set-up.
    auto pass_cost = [&](int i, int j) {
        const int n = overlapping(i, j);
        return static_cast<double>(n) * ((j - i) + 1.5) + 1.3 * (j - i) + 6.0;
    };
    auto finish = [&](std::vector<PassPlan> &passes) {
        for (PassPlan &pp : passes) {
            pp.u_lo = pp.u_hi = pp.count = 0;
            for (int u = 0; u < ns; ++u)
                if (bb[u] >= ba[u] && ba[u] < pp.j && bb[u] >= pp.i) {
                    if (pp.count == 0) pp.u_lo = u;
                    pp.u_hi = u + 1;
                    ++pp.count;
                }
            pp.cost = pass_cost(pp.i, pp.j);
        }
    };
    auto deal = [&](const std::vector<PassPlan> &passes, bool round_robin) {
        per_warp.assign(W, {});
        std::vector<double> load(W, 0.0);
        if (round_robin) {
            for (size_t i = 0; i < passes.size(); ++i) {
                per_warp[i % W].push_back(passes[i]);
                load[i % W] += passes[i].cost;
            }
        } else {
            std::vector<int> order(passes.size());
            for (size_t i = 0; i < order.size(); ++i) order[i] = static_cast<int>(i);
            std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return passes[x].cost > passes[y].cost; });
            for (int idx : order) {
                const int w = static_cast<int>(std::min_element(load.begin(), load.end()) - load.begin());
                per_warp[w].push_back(passes[idx]);
                load[w] += passes[idx].cost;
            }
            for (auto &list : per_warp)
                std::sort(list.begin(), list.end(), [](const PassPlan &x, const PassPlan &y) { return x.i < y.i; });
        }
        *total_cost = 0.0;
        for (double v : load) *total_cost += v;
        *makespan = *std::max_element(load.begin(), load.end());
    };

    std::vector<PassPlan> passes;
    if (schedule == SCHED_UNIFORM) {
        const int64_t per_round = static_cast<int64_t>(W) * R;
        const int64_t rounds = std::max<int64_t>(1, (nb + per_round - 1) / per_round);
        int64_t cpl = (nb + W * rounds - 1) / (W * rounds);
        cpl = std::min<int64_t>(R, std::max<int64_t>(1, cpl));
        for (int i = 0; i < nb; i += static_cast<int>(cpl)) passes.push_back(PassPlan{i, static_cast<int>(i + cpl), 0, 0, 0, 0.0});
        *blocks_covered = passes.back().j;  // the last pass may run past the band; those cells hold +inf
        finish(passes);
        deal(passes, true);
        return;
    }
    if (schedule == SCHED_LEVELLED && W > 1) {
        // Levelled partition: for one, two or three more rounds than the row needs, cut the blocks into
        // W * rounds contiguous passes whose largest cost is as small as possible (binary search on that
        // bottleneck; a pass is extended while it stays under it), deal them round-robin, and keep the
        // partition with the smallest load on the busiest warp - the uniform schedule included.
        const int r0 = std::max(1, (nb + W * R - 1) / (W * R));
        std::vector<PassPlan> best_passes;
        double best_span = 1e300;
        auto cut = [&](double bound, std::vector<PassPlan> *out) {
            int count = 0;
            for (int i = 0; i < nb;) {
                int j = i + 1;
                while (j < nb && j - i < R && pass_cost(i, j + 1) <= bound) ++j;
                if (out) out->push_back(PassPlan{i, j, 0, 0, 0, 0.0});
                ++count;
                i = j;
            }
            return count;
        };
        for (int rounds = r0; rounds <= r0 + 2; ++rounds) {
            const int P = std::min(nb, W * rounds);
            double lo = 0.0, hi = pass_cost(0, std::min(nb, R)) * 2.0 + 1.0;
            for (int i = 0; i < nb; ++i) lo = std::max(lo, pass_cost(i, i + 1));
            if (cut(hi, nullptr) > P) continue;
            for (int it = 0; it < 24 && hi - lo > 0.25; ++it) {
                const double mid = 0.5 * (lo + hi);
                if (cut(mid, nullptr) <= P) hi = mid;
                else lo = mid;
            }
            std::vector<PassPlan> trial;
            cut(hi, &trial);
            finish(trial);
            deal(trial, true);
            if (*makespan < best_span) {
                best_span = *makespan;
                best_passes = trial;
            }
        }
        {
            const int64_t rounds = r0;
            int64_t cpl = (nb + W * rounds - 1) / (W * rounds);
            cpl = std::min<int64_t>(R, std::max<int64_t>(1, cpl));
            std::vector<PassPlan> trial;
            for (int i = 0; i < nb; i += static_cast<int>(cpl)) trial.push_back(PassPlan{i, static_cast<int>(std::min<int64_t>(nb, i + cpl)), 0, 0, 0, 0.0});
            finish(trial);
            deal(trial, true);
            if (*makespan <= best_span) {
                best_span = *makespan;
                best_passes = trial;
            }
        }
        deal(best_passes, true);
        return;
    }
    std::vector<double> best(nb + 1);
    std::vector<int> from(nb + 1);
    for (int cap = R; cap >= 1; cap = (cap > 4 ? cap - 2 : cap - 1)) {
        best[0] = 0.0;
        for (int j = 1; j <= nb; ++j) {
            best[j] = 1e300;
            for (int i = std::max(0, j - cap); i < j; ++i) {
                const double c = best[i] + pass_cost(i, j);
                if (c < best[j]) {
                    best[j] = c;
                    from[j] = i;
                }
            }
        }
        passes.clear();
        for (int j = nb; j > 0; j = from[j]) passes.push_back(PassPlan{from[j], j, 0, 0, 0, 0.0});
        std::reverse(passes.begin(), passes.end());
        finish(passes);
        deal(passes, false);
        // Level within 4 %, or passes already as short as is sensible.
        if (W == 1 || *makespan * W <= 1.04 * *total_cost || cap <= 4) break;
    }
}

// Pass shapes for `W` warps sharing a candidate (threads / 32 for a CTA per candidate, 1 for a warp per
// candidate), row offsets, table pitch, guard width and issued work.
int layout_table(spdy_plan *p, int kind, int threads, double *efficiency)
{
    const int W = kind == KERNEL_WARP ? 1 : threads / 32;
    int R = cells_per_lane_cap(kind, threads, p->mode);
    if (p->pass_cap > 0) R = std::min(R, p->pass_cap);
    const int mw = mask_words(p);
    const int K = p->K;
    p->passes.clear();
    p->pass_masks.clear();
    p->pass_ptr.assign(static_cast<size_t>(p->L) * W + 1, 0);
    int64_t off = 0, max_extent = 32, max_cpl = 1;
    int64_t need_left = 0;
    std::vector<int64_t> need_right(static_cast<size_t>(p->L) + 1, 0);  // cells beyond row l-1's extent that layer l reads
    double sum_span = 0.0;
    p->issued_updates = 0;
    std::vector<int> ba, bb;
    std::vector<std::vector<PassPlan>> per_warp;
    int64_t prev_extent = 0;
    for (int l = 0; l < p->L; ++l) {
        LayerDesc &ld = p->layers[l];
        if (off > 0xffffffffLL) return SPDY_ERR_UNSUPPORTED;
        ld.rowoff = static_cast<uint32_t>(off);
        const int nb = static_cast<int>((static_cast<int64_t>(ld.width) + 31) / 32);
        const TapRange *slots = &p->slots[static_cast<size_t>(l) * K];
        ba.assign(ld.nslots, 0);
        bb.assign(ld.nslots, -1);
        for (int u = 0; u < ld.nslots; ++u)
            if (slots[u].b >= slots[u].a) {
                ba[u] = slots[u].a / 32;
                bb[u] = slots[u].b / 32;
            }
        double total = 0.0, span = 0.0;
        int covered = nb;
        plan_layer_passes(ba, bb, nb, W, R, p->schedule, per_warp, &total, &span, &covered);
        sum_span += span * W;
        ld.extent = 32 * covered;
        max_extent = std::max<int64_t>(max_extent, ld.extent);
        off += round_up(ld.extent, 128);
        for (int w = 0; w < W; ++w) {
            p->pass_ptr[static_cast<size_t>(l) * W + w] = static_cast<int32_t>(p->passes.size());
            for (const PassPlan &pp : per_warp[w]) {
                const int cpl = pp.j - pp.i;
                const int64_t start = 32LL * pp.i, cells = 32LL * cpl;
                max_cpl = std::max<int64_t>(max_cpl, cpl);
                uint64_t words[4] = {0, 0, 0, 0};
                int count = 0, u_lo = 0, u_hi = 0;
                for (int u = 0; u < ld.nslots; ++u) {
                    const TapRange tr = slots[u];
                    if (tr.b >= tr.a && start + cells > tr.a && start <= tr.b) {
                        words[u >> 6] |= 1ULL << (u & 63);
                        if (count == 0) u_lo = u;
                        u_hi = u + 1;
                        ++count;
                        p->issued_updates += cells;
                        // Lowest and highest previous-row cell a lane of this pass reads through this slot.
                        need_left = std::max<int64_t>(need_left, tr.a - start);
                        if (l > 0) need_right[l] = std::max<int64_t>(need_right[l], (start + cells - 1 - tr.a) - (prev_extent - 1));
                    }
                }
                const uint32_t dense = (count == u_hi - u_lo) ? 1u : 0u;
                p->passes.push_back(PassDesc{static_cast<int32_t>(start),
                                             static_cast<uint32_t>(u_lo) | static_cast<uint32_t>(u_hi) << 8 | dense << 16 |
                                                 static_cast<uint32_t>(cpl) << 24});
                for (int wd = 0; wd < mw; ++wd) p->pass_masks.push_back(words[wd]);
            }
        }
        prev_extent = ld.extent;
    }
    p->pass_ptr[static_cast<size_t>(p->L) * W] = static_cast<int32_t>(p->passes.size());
    p->pitch = off;
    // Guard cells of +inf on either side of a row: reads of a pass that only partly overlaps a slot's range
    // land there.  Below cell 0 the guard is `pad` cells wide (the furthest any pass of the plan reaches) and is
    // written once; behind a row it is refilled after every layer and only as wide as the NEXT layer reaches
    // beyond this row's extent (`fill`): bands grow fast while rows are narrow and hardly at all where they
    // are widest, so the buffer is sized by the largest extent + fill, not by the largest of each.  Layer 1
    // reads the virtual row 0, whose buffer is +inf everywhere but at t = 0.
    p->pad = static_cast<int32_t>(std::max<int64_t>(32, round_up(need_left, 32)));
    int64_t max_row = max_extent;
    for (int l = 0; l < p->L; ++l) {
        const int64_t fill = l + 1 < p->L ? round_up(std::max<int64_t>(0, need_right[l + 1]), 32) : 0;
        p->layers[l].fill = static_cast<int32_t>(fill);
        max_row = std::max<int64_t>(max_row, p->layers[l].extent + fill);
    }
    p->row_stride = static_cast<int32_t>(round_up(max_row, 32) + p->pad);
    p->warps_per_cand = W;
    p->rcap = rcap_for(kind, threads, p->mode, static_cast<int>(max_cpl));
    const int64_t tap_bytes = 2LL * ((K + 1) & ~1) * 8;
    if (kind == KERNEL_CTA_GLOBAL) p->smem_bytes = tap_bytes;
    else if (kind == KERNEL_WARP) p->smem_bytes = (threads / 32) * (2LL * p->row_stride * 4 + tap_bytes);
    else p->smem_bytes = 2LL * p->row_stride * 4 + tap_bytes;
    // Needed cell updates per data-path wavefront the busiest warps take: falls with partly overlapping slots,
    // with the passes' own slot reads (short passes pay more of them) and with warps that wait for others.
    if (efficiency) *efficiency = sum_span > 0.0 ? (static_cast<double>(p->distinct_updates) / 32.0) / sum_span : 0.0;
    return SPDY_OK;
}

// Pass shapes when C CTAs share a candidate: every row is cut into C slices of equal length (a
// multiple of 32 cells); see the cluster kernel for the data flow.
int layout_cluster(spdy_plan *p, int threads, int C)
{
    const int nwarps = threads / 32;
    const int mw = mask_words(p);
    p->passes.clear();
    p->pass_masks.clear();
    p->pass_ptr.clear();
    p->slices.assign(static_cast<size_t>(p->L) * C, SliceDesc{});
    p->issued_updates = 0;
    int64_t off = 0, max_slice = 32, max_win = 32, prev_slice = 1;
    for (int l = 0; l < p->L; ++l) {
        LayerDesc &ld = p->layers[l];
        if (off > 0xffffffffLL) return SPDY_ERR_UNSUPPORTED;
        ld.rowoff = static_cast<uint32_t>(off);
        const int64_t width = ld.width;
        ld.extent = static_cast<int32_t>(round_up(width, 32));
        off += round_up(width, 128);
        const int64_t slice = round_up((width + C - 1) / C, 32);
        max_slice = std::max(max_slice, slice);
        int64_t amax = 0;
        for (int k = 0; k < ld.nslots; ++k) {
            const TapRange tr = p->slots[static_cast<size_t>(l) * p->K + k];
            if (tr.b >= tr.a) amax = std::max<int64_t>(amax, tr.a);
        }
        for (int r = 0; r < C; ++r) {
            SliceDesc &sd = p->slices[static_cast<size_t>(l) * C + r];
            const int64_t lo = std::min<int64_t>(width, r * slice);
            const int64_t hi = std::min<int64_t>(width, (r + 1) * slice);
            const int64_t ws = hi - lo;
            int64_t cpl = 1, nspans = 0;
            if (ws > 0) {
                const int64_t cap = cluster_cells_per_lane(threads);
                const int64_t per_round = 32LL * nwarps * cap;
                const int64_t rounds = (ws + per_round - 1) / per_round;
                cpl = (ws + 32LL * nwarps * rounds - 1) / (32LL * nwarps * rounds);
                cpl = std::min<int64_t>(cap, std::max<int64_t>(1, cpl));
                nspans = (ws + 32 * cpl - 1) / (32 * cpl);
            }
            const int64_t span = 32 * cpl;
            sd.slice_lo = static_cast<int32_t>(lo);
            sd.slice_hi = static_cast<int32_t>(hi);
            sd.cpl = static_cast<int32_t>(cpl);
            sd.nspans = static_cast<int32_t>(nspans);
            sd.mask_off = static_cast<int32_t>(p->passes.size());
            sd.q0 = static_cast<int32_t>(lo - amax);
            sd.win_len = static_cast<int32_t>(nspans > 0 ? amax + nspans * span : 0);
            sd.prev_slice = static_cast<int32_t>(prev_slice);
            max_win = std::max<int64_t>(max_win, sd.win_len);
            for (int64_t sp = 0; sp < nspans; ++sp) {
                const int64_t s0 = lo + sp * span;
                uint64_t words[4] = {0, 0, 0, 0};
                int k_lo = 0, k_hi = 0, count = 0;
                for (int k = 0; k < ld.nslots; ++k) {
                    const TapRange tr = p->slots[static_cast<size_t>(l) * p->K + k];
                    if (tr.b >= tr.a && s0 + span > tr.a && s0 <= tr.b) {
                        words[k >> 6] |= 1ULL << (k & 63);
                        p->issued_updates += span;
                        if (count == 0) k_lo = k;
                        k_hi = k + 1;
                        ++count;
                    }
                }
                for (int w = 0; w < mw; ++w) p->pass_masks.push_back(words[w]);
                const uint32_t dense = (count == k_hi - k_lo) ? 1u : 0u;
                p->passes.push_back(PassDesc{static_cast<int32_t>(s0),
                                             static_cast<uint32_t>(k_lo) | static_cast<uint32_t>(k_hi) << 8 | dense << 16 |
                                                 static_cast<uint32_t>(cpl) << 24});
            }
        }
        prev_slice = slice;
    }
    p->pitch = off;
    p->out_stride = static_cast<int32_t>(round_up(max_slice, 32));
    p->win_stride = static_cast<int32_t>(round_up(max_win, 32));
    p->row_stride = 0;
    p->pad = 0;
    p->warps_per_cand = nwarps;
    p->rcap = cluster_cells_per_lane(threads);
    p->smem_bytes = (2LL * p->out_stride + p->win_stride) * 4 + 2LL * ((p->K + 1) & ~1) * 8;
    return SPDY_OK;
}

int choose_cluster_shape(spdy_plan *p, const spdy_options *opts)
{
    const int requested = (opts && opts->cluster > 1) ? opts->cluster : 0;
    const int sizes[] = {2, 4, 8};
    for (int C : sizes) {
        if (requested && C != requested) continue;
        for (int threads : {512, 256}) {
            if (opts && opts->threads && opts->threads != threads) continue;
            if (threads < p->K) continue;
            int rc = layout_cluster(p, threads, C);
            if (rc != SPDY_OK) return rc;
            if (p->smem_bytes > p->limits.smem_per_block - kStaticSmemReserve) continue;
            // Narrow slices do not fill 16 warps; prefer the smaller CTA then.
            if (threads == 512 && !(opts && opts->threads) && p->out_stride < 32 * 16 * 4) continue;
            p->kind = KERNEL_CLUSTER;
            p->cluster = C;
            p->threads = threads;
            p->ctas_per_sm = 1;
            return SPDY_OK;
        }
    }
    return SPDY_ERR_UNSUPPORTED;  // no cluster size (or not the one asked for) holds these rows
}

// Wide-band fallback: one CTA of 1024 threads per candidate, row buffers in the workspace.
int choose_global_row_shape(spdy_plan *p, int threads)
{
    if (threads < p->K) return SPDY_ERR_UNSUPPORTED;
    p->mode = p->table_format == SPDY_TABLE_ARG_U8 ? MODE_ARG_PAIR : MODE_ROW2;  // the builds this shape has
    p->cluster = 1;
    p->slices.clear();
    int rc = layout_table(p, KERNEL_CTA_GLOBAL, threads, nullptr);
    if (rc != SPDY_OK) return rc;
    p->kind = KERNEL_CTA_GLOBAL;
    p->threads = threads;
    p->ctas_per_sm = 1;
    return SPDY_OK;
}

// Resident CTAs per SM a launch shape allows by shared memory and thread count (the device part of the
// library replaces this estimate with the occupancy the driver reports).
int resident_ctas(const spdy_plan *p, int threads, int64_t smem_bytes)
{
    const int64_t by_smem = std::max<int64_t>(1, p->limits.smem_per_sm / (smem_bytes + 1024));
    return static_cast<int>(std::min<int64_t>(std::min<int64_t>(by_smem, 2048 / threads), 32));
}

// One warp per candidate pays off when a row is a pass or two wide: a layer then needs no block barrier
// and its fixed costs (slot staging, descriptors) are spread over the whole row instead of a quarter of it.
bool warp_kernel_fits(const spdy_plan *p)
{
    int max_slots = 0;
    for (const LayerDesc &ld : p->layers) max_slots = std::max(max_slots, ld.nslots);
    return mode_is_row(p->mode) ? (max_slots <= 64 && p->mode == MODE_ROW2)
                                : (max_slots <= 64 && p->mode == MODE_ARG_PAIR);
}

// The warp kernel's two builds unroll passes of up to 8 cells per lane in 64 registers (8 CTAs of 128
// threads per SM) or up to long_pass_cap() in 128 registers (4 CTAs).  Measured over budgets of 750 to 3000
// buckets: while shared memory lets seven or more CTAs share an SM the short passes with twice the resident
// warps win (B = 1000: 0.53 against 0.62 ms); from there on one long pass per layer does (B = 1500: 0.73
// against 0.99 ms).
int choose_warp_shape(spdy_plan *p)
{
    const int threads = 128;
    const int asked_cap = p->pass_cap;
    int rc = layout_table(p, KERNEL_WARP, threads, nullptr);
    if (rc != SPDY_OK) return rc;
    if (asked_cap == 0 && p->rcap > warp_short_cap(p->mode) && resident_ctas(p, threads, p->smem_bytes) >= 7) {
        p->pass_cap = warp_short_cap(p->mode);
        rc = layout_table(p, KERNEL_WARP, threads, nullptr);
        p->pass_cap = asked_cap;
        if (rc != SPDY_OK) return rc;
    }
    if (p->smem_bytes > p->limits.smem_per_block - kStaticSmemReserve) return SPDY_ERR_UNSUPPORTED;
    p->kind = KERNEL_WARP;
    p->threads = threads;
    p->cluster = 1;
    p->ctas_per_sm = resident_ctas(p, threads, p->smem_bytes);
    return SPDY_OK;
}

int choose_launch_shape(spdy_plan *p, const spdy_options *opts)
{
    p->table_format = (opts && opts->table_format) ? opts->table_format : SPDY_TABLE_ROW_F32;
    if (p->table_format != SPDY_TABLE_ARG_U8 && p->table_format != SPDY_TABLE_ROW_F32)
        return SPDY_ERR_INVALID_ARG;
    p->mode = p->table_format == SPDY_TABLE_ARG_U8 ? MODE_ARG_PAIR : MODE_ROW2;
    if (opts && opts->forward_mode) {
        p->mode = opts->forward_mode;
        if (!(mode_is_row(p->mode) || mode_is_arg(p->mode))) return SPDY_ERR_INVALID_ARG;
        if (mode_is_row(p->mode) != (p->table_format == SPDY_TABLE_ROW_F32)) return SPDY_ERR_INVALID_ARG;
    }
    p->schedule = opts ? (opts->schedule & 0xFF) : 0;
    p->pass_cap = opts ? ((opts->schedule >> 8) & 0xFF) : 0;
    if (p->schedule < 0 || p->schedule > SCHED_SIZED || (opts && (opts->schedule >> 16) != 0) || p->pass_cap > kRmaxLong)
        return SPDY_ERR_INVALID_ARG;
    // Left open: levelled passes where the shared-memory data path binds (row-value table); passes of one
    // length where instruction issue binds (byte table: one unrolled body per layer measured 3 % faster).
    if (p->schedule == 0) p->schedule = mode_is_row(p->mode) ? SCHED_LEVELLED : SCHED_UNIFORM;
    build_slots(p, mode_is_row(p->mode) ? 1 : (p->merge_first ? 2 : 0));
    p->cluster = 1;
    p->kind = KERNEL_CTA;
    if (opts && opts->cluster != 0 && opts->cluster != 1 && opts->cluster != 2 && opts->cluster != 4 &&
        opts->cluster != 8)
        return SPDY_ERR_INVALID_ARG;
    if (opts && opts->rows_in_global != 0 && opts->rows_in_global != 1) return SPDY_ERR_INVALID_ARG;
    const int want_kernel = opts ? opts->kernel : SPDY_KERNEL_AUTO;
    if (want_kernel != SPDY_KERNEL_AUTO && want_kernel != SPDY_KERNEL_CTA && want_kernel != SPDY_KERNEL_WARP)
        return SPDY_ERR_INVALID_ARG;
    if (opts && opts->rows_in_global) {
        if (opts->cluster > 1 || want_kernel == SPDY_KERNEL_WARP) return SPDY_ERR_INVALID_ARG;
        if (opts->threads && opts->threads != 512 && opts->threads != 1024) return SPDY_ERR_INVALID_ARG;
        return choose_global_row_shape(p, opts->threads ? opts->threads : kGlobalRowsThreads);
    }
    if (opts && opts->cluster > 1) {
        if (want_kernel == SPDY_KERNEL_WARP) return SPDY_ERR_INVALID_ARG;
        return choose_cluster_shape(p, opts);
    }
    if (want_kernel == SPDY_KERNEL_WARP) {
        if (!warp_kernel_fits(p) || (opts->threads && opts->threads != 128)) return SPDY_ERR_UNSUPPORTED;
        return choose_warp_shape(p);
    }

    // Candidate CTA sizes; keep the one whose rounds are fullest, preferring more resident warps.
    const int sizes[] = {128, 256, 512, 1024};
    int best_threads = 0;
    double best_score = -1.0;
    // (scored with passes of one length, which cost a tenth of the levelled partition to lay out and rank the
    // CTA sizes the same way; the chosen size is laid out for good below)
    const int wanted_schedule = p->schedule;
    for (int threads : sizes) {
        if (opts && opts->threads && opts->threads != threads) continue;
        if (threads < p->K) continue;  // one thread per choice stages the next layer
        double eff = 0.0;
        p->schedule = SCHED_UNIFORM;
        int rc = layout_table(p, KERNEL_CTA, threads, &eff);
        p->schedule = wanted_schedule;
        if (rc != SPDY_OK) return rc;
        if (p->smem_bytes > p->limits.smem_per_block - kStaticSmemReserve) continue;
        const double warps = static_cast<double>(resident_ctas(p, threads, p->smem_bytes) * threads / 32);
        // Below about 16 resident warps an SM cannot cover shared-memory latency.
        const double score = eff * std::min(1.0, warps / 16.0) + 1e-3 * std::min(warps, 32.0) / 32.0;
        if (score > best_score) {
            best_score = score;
            best_threads = threads;
        }
    }
    if (best_threads == 0) {
        // No single CTA can hold two rows of this width in shared memory (the caller may have
        // insisted on that).
        if (opts && opts->cluster == 1) return SPDY_ERR_UNSUPPORTED;
        // Rows in global memory, read through L1, measured faster than a cluster for such widths
        // (B = 10^5: 1.6x, B = 2*10^5: 1.9x) and have no width limit.  A cluster is still used when the
        // caller asks for one (cluster > 1, handled above) or pins a launch shape the fallback lacks.
        if (opts && ((opts->threads && opts->threads != kGlobalRowsThreads) || opts->forward_mode))
            return choose_cluster_shape(p, opts);
        return choose_global_row_shape(p, kGlobalRowsThreads);
    }
    // Narrow rows: a warp per candidate, unless the caller pinned a CTA shape.
    if (want_kernel == SPDY_KERNEL_AUTO && !(opts && opts->threads) && warp_kernel_fits(p) &&
        p->max_width <= kWarpKernelMaxWidth) {
        spdy_plan trial = *p;  // plain members and vectors only at this point
        if (choose_warp_shape(&trial) == SPDY_OK && trial.ctas_per_sm * 4 >= 12) {
            *p = std::move(trial);
            return SPDY_OK;
        }
    }
    int rc = layout_table(p, KERNEL_CTA, best_threads, nullptr);
    if (rc != SPDY_OK) return rc;
    p->kind = KERNEL_CTA;
    p->threads = best_threads;
    p->ctas_per_sm = resident_ctas(p, best_threads, p->smem_bytes);
    return SPDY_OK;
}

}  // namespace

int64_t table_bytes_one(const spdy_plan *p) { return std::max<int64_t>(256, round_up(p->pitch * cell_bytes(p), 256)); }
int64_t row_bytes_one(const spdy_plan *p)
{
    if (p->kind != KERNEL_CTA_GLOBAL) return 0;
    const int64_t stride = std::max(p->row_stride, p->merged ? p->merged->row_stride : 0);  // both table sets fit
    return round_up(2LL * stride * 4, 256);
}
int64_t flag_bytes_one(const spdy_plan *p) { return p->merged ? 256 : 0; }

void register_device_hooks(const DeviceHooks *hooks) { g_hooks = hooks; }
const DeviceHooks *device_hooks() { return g_hooks; }

int create_host_plan(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B, int device,
                     const spdy_options *opts, const DeviceLimits &limits, bool merge_first)
{
    if (!out) return SPDY_ERR_INVALID_ARG;
    *out = nullptr;
    if (!times_host || L < 1 || K < 1 || K > 255 || B < 0 || device < -1) return SPDY_ERR_INVALID_ARG;
    if (opts) {
        if (opts->threads != 0 && (opts->threads % 32 != 0 || opts->threads < 32 || opts->threads > 1024))
            return SPDY_ERR_INVALID_ARG;
        if (opts->auto_shape != 0 && opts->auto_shape != 1) return SPDY_ERR_INVALID_ARG;
    }
    spdy_plan *p = new (std::nothrow) spdy_plan();
    if (!p) return SPDY_ERR_NO_MEMORY;
    p->L = L;
    p->K = K;
    p->B = B;
    p->device = device;
    p->limits = limits;
    p->merge_first = merge_first;
    int rc = SPDY_OK;
    try {
        p->times.assign(times_host, times_host + static_cast<size_t>(L) * K);
        fill_qtab(p);
        rc = build_bands(p);
        if (rc == SPDY_OK) rc = choose_launch_shape(p, opts);
        if (rc == SPDY_OK && p->feasible) rc = verify_plan(p);
    } catch (const std::bad_alloc &) {
        rc = SPDY_ERR_NO_MEMORY;
    }
    if (rc != SPDY_OK) {
        delete p;
        return rc;
    }
    *out = p;
    return SPDY_OK;
}

void destroy_host_plan(spdy_plan *p) { delete p; }

int verify_plan(const spdy_plan *p)
{
    if (!p->feasible) return SPDY_OK;
    const int L = p->L, K = p->K, mw = mask_words(p);
    auto slot_in_pass = [&](size_t pass, int u) { return (p->pass_masks[pass * mw + (u >> 6)] >> (u & 63)) & 1ULL; };
    int64_t table_end = 0;
    for (int l = 0; l < L; ++l) {
        const LayerDesc &ld = p->layers[l];
        if (ld.width < 1 || ld.extent < ld.width || ld.extent % 32 != 0 || ld.nslots < 0 || ld.nslots > K) return SPDY_ERR_INTERNAL;
        if (static_cast<int64_t>(ld.rowoff) < table_end) return SPDY_ERR_INTERNAL;  // rows of the table do not overlap
        table_end = static_cast<int64_t>(ld.rowoff) + (p->kind == KERNEL_CLUSTER ? ld.width : ld.extent);
        if (table_end > p->pitch) return SPDY_ERR_INTERNAL;
    }
    if (p->kind == KERNEL_CLUSTER) {
        const int C = p->cluster;
        for (int l = 0; l < L; ++l) {
            const LayerDesc &ld = p->layers[l];
            std::vector<int> covered(ld.width, 0);
            for (int r = 0; r < C; ++r) {
                const SliceDesc &sd = p->slices[static_cast<size_t>(l) * C + r];
                if (sd.slice_lo < 0 || sd.slice_hi < sd.slice_lo || sd.slice_hi > ld.width) return SPDY_ERR_INTERNAL;
                if (sd.slice_hi - sd.slice_lo > p->out_stride || sd.win_len > p->win_stride || sd.prev_slice < 1) return SPDY_ERR_INTERNAL;
                if (sd.prev_slice > p->out_stride && l > 0) return SPDY_ERR_INTERNAL;
                if (sd.cpl < 1 || sd.cpl > kRmax) return SPDY_ERR_INTERNAL;
                for (int sp = 0; sp < sd.nspans; ++sp) {
                    const size_t pi = static_cast<size_t>(sd.mask_off) + sp;
                    if (pi >= p->passes.size()) return SPDY_ERR_INTERNAL;
                    const int64_t s = p->passes[pi].start, cells = 32LL * sd.cpl;
                    if (s != sd.slice_lo + sp * cells) return SPDY_ERR_INTERNAL;
                    for (int64_t c = s; c < std::min<int64_t>(s + cells, sd.slice_hi); ++c) covered[c] += 1;
                    for (int u = 0; u < ld.nslots; ++u) {
                        const TapRange tr = p->slots[static_cast<size_t>(l) * K + u];
                        const bool overlaps = tr.b >= tr.a && s + cells > tr.a && s <= tr.b;
                        if (overlaps != static_cast<bool>(slot_in_pass(pi, u))) return SPDY_ERR_INTERNAL;
                        if (!overlaps) continue;
                        // window cells read: [s - a, s + cells - 1 - a] must lie inside [q0, q0 + win_len)
                        if (s - tr.a < sd.q0 || s + cells - 1 - tr.a >= sd.q0 + static_cast<int64_t>(sd.win_len)) return SPDY_ERR_INTERNAL;
                    }
                }
            }
            for (int c = 0; c < ld.width; ++c)
                if (covered[c] != 1) return SPDY_ERR_INTERNAL;
        }
        return SPDY_OK;
    }
    const int W = p->warps_per_cand;
    if (p->pass_ptr.size() != static_cast<size_t>(L) * W + 1) return SPDY_ERR_INTERNAL;
    const int64_t buffer_lo = -static_cast<int64_t>(p->pad), buffer_hi = static_cast<int64_t>(p->row_stride) - p->pad;
    int64_t prev_extent = 0;
    for (int l = 0; l < L; ++l) {
        const LayerDesc &ld = p->layers[l];
        if (ld.fill < 0 || static_cast<int64_t>(ld.extent) + ld.fill > buffer_hi) return SPDY_ERR_INTERNAL;  // row and its +inf tail fit
        // Cells of the previous row's buffer known to hold the row or +inf when this layer runs.
        const int64_t ok_lo = buffer_lo, ok_hi = l == 0 ? buffer_hi : prev_extent + p->layers[l - 1].fill;
        std::vector<int> covered(ld.extent, 0);
        for (int w = 0; w < W; ++w) {
            const int32_t p0 = p->pass_ptr[static_cast<size_t>(l) * W + w], p1 = p->pass_ptr[static_cast<size_t>(l) * W + w + 1];
            if (p0 > p1 || p1 > static_cast<int32_t>(p->passes.size())) return SPDY_ERR_INTERNAL;
            for (int32_t pi = p0; pi < p1; ++pi) {
                const PassDesc pd = p->passes[pi];
                const int cpl = pass_cpl(pd);
                if (cpl < 1 || cpl > p->rcap) return SPDY_ERR_INTERNAL;
                const int64_t s = pd.start, cells = 32LL * cpl;
                if (s < 0 || s % 32 != 0 || s + cells > ld.extent) return SPDY_ERR_INTERNAL;
                for (int64_t c = s; c < s + cells; ++c) covered[c] += 1;
                const int u_lo = pd.krange & 0xFF, u_hi = (pd.krange >> 8) & 0xFF;
                const bool dense = (pd.krange >> 16) & 1;
                for (int u = 0; u < ld.nslots; ++u) {
                    const TapRange tr = p->slots[static_cast<size_t>(l) * K + u];
                    const bool overlaps = tr.b >= tr.a && s + cells > tr.a && s <= tr.b;
                    if (overlaps != static_cast<bool>(slot_in_pass(pi, u))) return SPDY_ERR_INTERNAL;
                    if (overlaps && (u < u_lo || u >= u_hi)) return SPDY_ERR_INTERNAL;
                    if (dense && !overlaps && u >= u_lo && u < u_hi) return SPDY_ERR_INTERNAL;
                    if (!overlaps) continue;
                    if (s - tr.a < ok_lo || s + cells - 1 - tr.a >= ok_hi) return SPDY_ERR_INTERNAL;
                }
            }
        }
        for (int c = 0; c < ld.extent; ++c)
            if (covered[c] != 1) return SPDY_ERR_INTERNAL;  // every cell of the row written exactly once
        // every cell a slot contributes to is inside the row, and its source inside the previous row
        for (int u = 0; u < ld.nslots; ++u) {
            const TapRange tr = p->slots[static_cast<size_t>(l) * K + u];
            if (tr.b < tr.a) continue;
            const int64_t pw = l == 0 ? 1 : p->layers[l - 1].width;
            if (tr.a < 0 || tr.b >= ld.width || tr.b - tr.a >= pw) return SPDY_ERR_INTERNAL;
        }
        prev_extent = ld.extent;
    }
    return SPDY_OK;
}

TableLayout table_layout(const spdy_plan *p)
{
    const size_t n = static_cast<size_t>(p->L) * p->K;
    TableLayout t;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off += static_cast<size_t>(round_up(static_cast<int64_t>(bytes) + 16, 256));
        return at;
    };
    t.times = take(n * sizeof(int32_t));
    t.layers = take(p->L * sizeof(LayerDesc));
    t.slots = take(n * sizeof(TapRange));
    t.slot_ptr = take(static_cast<size_t>(p->L) * (p->K + 1));
    t.slot_member = take(n);
    t.masks = take(p->pass_masks.size() * sizeof(uint64_t));
    t.passes = take(p->passes.size() * sizeof(PassDesc));
    t.pass_ptr = take(p->pass_ptr.size() * sizeof(int32_t));
    t.status = take(256);
    t.slices = take(p->slices.size() * sizeof(SliceDesc));
    t.qtab = take(p->qtab.size() * sizeof(float));
    t.total = off;
    return t;
}

// Host image of the table block (the status word starts at zero).
void pack_tables(const spdy_plan *p, const TableLayout &t, std::vector<unsigned char> &host)
{
    host.assign(t.total, 0);
    auto put = [&](size_t at, const void *src, size_t bytes) {
        if (bytes) std::memcpy(host.data() + at, src, bytes);
    };
    put(t.times, p->times.data(), p->times.size() * sizeof(int32_t));
    put(t.layers, p->layers.data(), p->layers.size() * sizeof(LayerDesc));
    put(t.slots, p->slots.data(), p->slots.size() * sizeof(TapRange));
    put(t.slot_ptr, p->slot_ptr.data(), p->slot_ptr.size());
    put(t.slot_member, p->slot_member.data(), p->slot_member.size());
    put(t.masks, p->pass_masks.data(), p->pass_masks.size() * sizeof(uint64_t));
    put(t.passes, p->passes.data(), p->passes.size() * sizeof(PassDesc));
    put(t.pass_ptr, p->pass_ptr.data(), p->pass_ptr.size() * sizeof(int32_t));
    put(t.slices, p->slices.data(), p->slices.size() * sizeof(SliceDesc));
    put(t.qtab, p->qtab.data(), p->qtab.size() * sizeof(float));
}

namespace {

size_t workspace_one(const spdy_plan *p)
{
    return static_cast<size_t>(table_bytes_one(p) + row_bytes_one(p) + flag_bytes_one(p));
}

}  // namespace

const spdy_plan *pick_for_batch(const spdy_plan *p, int64_t N, size_t workspace_bytes)
{
    if (p->alternates.empty() || !p->feasible) return p;
    // Candidates the main shape keeps resident at once; a batch of at least half of that fills the device.
    const int64_t per_cta = p->kind == KERNEL_WARP ? p->threads / 32 : 1;
    const int64_t resident = static_cast<int64_t>(p->limits.sm_count) * std::max(1, p->ctas_per_sm) * per_cta;
    if (2 * N >= resident) return p;
    const spdy_plan *best = p;
    for (const spdy_plan *alt : p->alternates) {
        if (workspace_one(alt) * static_cast<size_t>(N) > workspace_bytes) continue;
        if (alt->kind == KERNEL_CLUSTER) {
            // A cluster per candidate while all clusters still find an SM per CTA; the largest such cluster.
            if (N * alt->cluster > p->limits.sm_count) continue;
            if (best->kind != KERNEL_CLUSTER || alt->cluster > best->cluster) best = alt;
        } else if (best->kind != KERNEL_CLUSTER) {
            // A larger CTA per candidate when every candidate can have an SM to itself (measured: with two
            // or more candidates per SM the main shape's longer passes per warp win again).
            if (N <= p->limits.sm_count && alt->threads > best->threads) best = alt;
        }
    }
    return best;
}

}  // namespace spdy

using namespace spdy;

namespace {

void destroy_tree(spdy_plan *plan)
{
    if (!plan) return;
    if (plan->merged) destroy_tree(plan->merged);
    plan->merged = nullptr;
    for (spdy_plan *alt : plan->alternates) destroy_tree(alt);
    plan->alternates.clear();
    if (plan->dev && device_hooks()) device_hooks()->release(plan);
    destroy_host_plan(plan);
}

int create_one(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B, int device,
               const spdy_options *opts, const DeviceLimits &limits, bool merge_first)
{
    int rc = create_host_plan(out, times_host, L, K, B, device, opts, limits, merge_first);
    if (rc != SPDY_OK) return rc;
    if (device >= 0) {
        rc = device_hooks()->attach(*out);
        if (rc != SPDY_OK) {
            destroy_tree(*out);
            *out = nullptr;
        }
    }
    return rc;
}

// A plan with its second table set (byte table) and, for a main plan whose launch shape the caller left
// open, the launch shapes for batches too small to fill the device.
int create_with_children(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B, int device,
                         const spdy_options *opts, const DeviceLimits &limits, bool as_alternate)
{
    int rc = create_one(out, times_host, L, K, B, device, opts, limits, false);
    if (rc != SPDY_OK) return rc;
    spdy_plan *p = *out;
    p->is_alternate = as_alternate;
    // Byte table, one CTA (or warp) per candidate: add the second plan with merged equal-time choices when
    // merging removes any work.  It shares the rows and the table layout of the first.
    if (p->table_format == SPDY_TABLE_ARG_U8 && p->cluster == 1 && p->feasible) {
        spdy_options o = {};
        if (opts) o = *opts;
        o.table_format = SPDY_TABLE_ARG_U8;
        o.threads = p->kind == KERNEL_WARP ? 0 : p->threads;
        o.cluster = 1;
        o.forward_mode = p->mode;
        o.rows_in_global = p->kind == KERNEL_CTA_GLOBAL ? 1 : 0;
        o.kernel = p->kind == KERNEL_WARP ? SPDY_KERNEL_WARP : (p->kind == KERNEL_CTA ? SPDY_KERNEL_CTA : SPDY_KERNEL_AUTO);
        spdy_plan *m = nullptr;
        if (create_one(&m, times_host, L, K, B, device, &o, limits, true) == SPDY_OK) {
            bool same_table = m->pitch == p->pitch && m->kind == p->kind && m->threads == p->threads;
            for (int l = 0; same_table && l < L; ++l) same_table = m->layers[l].rowoff == p->layers[l].rowoff;
            if (same_table && m->distinct_updates < p->distinct_updates) p->merged = m;
            else destroy_tree(m);
        }
    }
    const bool shape_open = !opts || (opts->threads == 0 && opts->cluster == 0 && opts->rows_in_global == 0 &&
                                      opts->kernel == SPDY_KERNEL_AUTO && opts->auto_shape == 0);
    if (!as_alternate && shape_open && p->feasible && p->kind == KERNEL_CTA) {
        spdy_options o = {};
        if (opts) o = *opts;
        o.table_format = p->table_format;
        o.auto_shape = 1;
        for (int threads : {256, 512}) {
            if (threads <= p->threads || threads < K) continue;
            o.threads = threads;
            o.cluster = 0;
            o.kernel = SPDY_KERNEL_CTA;
            spdy_plan *alt = nullptr;
            if (create_with_children(&alt, times_host, L, K, B, device, &o, limits, true) == SPDY_OK) {
                if (alt->kind == KERNEL_CTA) p->alternates.push_back(alt);
                else destroy_tree(alt);
            }
        }
        for (int C : {2, 4, 8}) {
            o.threads = 0;
            o.cluster = C;
            o.kernel = SPDY_KERNEL_AUTO;
            spdy_plan *alt = nullptr;
            if (create_with_children(&alt, times_host, L, K, B, device, &o, limits, true) == SPDY_OK)
                p->alternates.push_back(alt);
        }
    }
    return SPDY_OK;
}

size_t per_candidate_bytes(const spdy_plan *p)
{
    size_t one = static_cast<size_t>(table_bytes_one(p) + row_bytes_one(p) + flag_bytes_one(p));
    for (const spdy_plan *alt : p->alternates) one = std::max(one, per_candidate_bytes(alt));
    return one;
}

}  // namespace

extern "C" {

int spdy_version(void) { return kLibraryVersion; }

const char *spdy_strerror(int status)
{
    switch (status) {
        case SPDY_OK: return "success";
        case SPDY_ERR_INVALID_ARG: return "invalid argument";
        case SPDY_ERR_WORKSPACE_TOO_SMALL: return "workspace too small for one candidate";
        case SPDY_ERR_UNSUPPORTED: return "problem shape not supported on this device";
        case SPDY_ERR_CUDA: return "CUDA runtime call failed";
        case SPDY_ERR_NO_MEMORY: return "out of memory";
        case SPDY_ERR_INTERNAL: return "internal self-check failed";
        case SPDY_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of spdy_solve_batch_static";
        case SPDY_ERR_NO_DEVICE_CODE: return "this build of the library holds the host side only";
        default: return "unknown status";
    }
}

int spdy_plan_create(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B,
                     int device, const spdy_options *opts)
{
    if (out) *out = nullptr;
    DeviceLimits limits;
    if (device >= 0) {
        if (!device_hooks()) return SPDY_ERR_NO_DEVICE_CODE;
        int rc = device_hooks()->limits(device, &limits);
        if (rc != SPDY_OK) return rc;
    }
    return create_with_children(out, times_host, L, K, B, device, opts, limits, false);
}

void spdy_plan_destroy(spdy_plan *plan) { destroy_tree(plan); }

int spdy_plan_get_info(const spdy_plan *plan, spdy_plan_info *info)
{
    if (!plan || !info) return SPDY_ERR_INVALID_ARG;
    std::memset(info, 0, sizeof(*info));
    info->L = plan->L;
    info->K = plan->K;
    info->B = plan->B;
    info->feasible = plan->feasible ? 1 : 0;
    info->max_width = plan->max_width;
    info->span = 32 * plan->rcap;
    info->threads = plan->threads;
    info->cluster = plan->cluster;
    info->table_format = plan->table_format;
    info->ctas_per_sm = plan->ctas_per_sm;
    info->sm_count = plan->limits.sm_count;
    info->rows_in_global = plan->kind == KERNEL_CTA_GLOBAL ? 1 : 0;
    info->smem_bytes = plan->smem_bytes;
    info->table_bytes_per_candidate = static_cast<int64_t>(spdy_workspace_bytes(plan, 1));
    info->band_cells = plan->band_cells;
    info->useful_updates = plan->useful_updates;
    info->issued_updates = plan->issued_updates;
    info->distinct_updates = plan->merged ? plan->merged->distinct_updates : plan->distinct_updates;
    if (plan->merged) info->issued_updates = plan->merged->issued_updates;
    info->launches_per_wave = plan->merged ? 5 : 2;
    info->nominal_updates = static_cast<int64_t>(plan->L) * plan->K * plan->B;
    info->kernel = plan->kind == KERNEL_WARP ? SPDY_KERNEL_WARP : SPDY_KERNEL_CTA;
    info->forward_mode = plan->mode;
    info->candidates_per_cta = plan->kind == KERNEL_WARP ? plan->threads / 32 : 1;
    info->alternates = static_cast<int32_t>(plan->alternates.size());
    return SPDY_OK;
}

int spdy_plan_get_bands(const spdy_plan *plan, int32_t *lo_host, int32_t *width_host)
{
    if (!plan) return SPDY_ERR_INVALID_ARG;
    for (int l = 0; l < plan->L; ++l) {
        if (lo_host) lo_host[l] = plan->layers[l].lo;
        if (width_host) width_host[l] = plan->layers[l].width;
    }
    return SPDY_OK;
}

size_t spdy_workspace_bytes(const spdy_plan *plan, int64_t N)
{
    if (!plan || N <= 0) return 0;
    return per_candidate_bytes(plan) * static_cast<size_t>(N);
}

int spdy_plan_get_tables(const spdy_plan *plan, int32_t which, spdy_plan_tables *out)
{
    if (!plan || !out || which < -1) return SPDY_ERR_INVALID_ARG;
    const spdy_plan *p = plan;
    if (which == -1) p = plan->merged;
    else if (which > 0) p = which <= static_cast<int32_t>(plan->alternates.size()) ? plan->alternates[which - 1] : nullptr;
    if (!p) return SPDY_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    out->L = p->L;
    out->K = p->K;
    out->kernel_kind = p->kind;
    out->threads = p->threads;
    out->warps_per_candidate = p->warps_per_cand;
    out->cluster = p->cluster;
    out->forward_mode = p->mode;
    out->max_cells_per_lane = p->rcap;
    out->row_stride = p->row_stride;
    out->pad = p->pad;
    out->out_stride = p->out_stride;
    out->win_stride = p->win_stride;
    out->mask_words = mask_words(p);
    out->n_passes = static_cast<int32_t>(p->passes.size());
    out->pitch = p->pitch;
    out->layers = reinterpret_cast<const int32_t *>(p->layers.data());
    out->slots = reinterpret_cast<const int32_t *>(p->slots.data());
    out->passes = reinterpret_cast<const int32_t *>(p->passes.data());
    out->pass_masks = p->pass_masks.data();
    out->pass_ptr = p->pass_ptr.empty() ? nullptr : p->pass_ptr.data();
    out->slices = p->slices.empty() ? nullptr : reinterpret_cast<const int32_t *>(p->slices.data());
    return SPDY_OK;
}

int32_t spdy_plan_shape_for_batch(const spdy_plan *plan, int64_t N, size_t workspace_bytes)
{
    if (!plan) return -1;
    const spdy_plan *shape = pick_for_batch(plan, N, workspace_bytes);
    for (size_t i = 0; i < plan->alternates.size(); ++i)
        if (plan->alternates[i] == shape) return static_cast<int32_t>(i + 1);
    return 0;
}

int spdy_plan_verify(const spdy_plan *plan)
{
    if (!plan) return SPDY_ERR_INVALID_ARG;
    int rc = verify_plan(plan);
    if (rc == SPDY_OK && plan->merged) rc = verify_plan(plan->merged);
    for (const spdy_plan *alt : plan->alternates)
        if (rc == SPDY_OK) rc = spdy_plan_verify(alt);
    return rc;
}

double spdy_time_target(double t_dense, double speedup, double t_base)
{
    return t_dense / speedup - t_base;
}

int spdy_bucketize_times(const double *times_host, int32_t L, int32_t K, double T, int32_t B, int32_t rounding,
                         int32_t *out_host)
{
    if (!times_host || !out_host || L < 1 || K < 1 || B < 1 || !(T > 0.0) || !std::isfinite(T)) return SPDY_ERR_INVALID_ARG;
    if (rounding != SPDY_ROUND_NEAREST && rounding != SPDY_ROUND_UP) return SPDY_ERR_INVALID_ARG;
    const size_t n = static_cast<size_t>(L) * K;
    for (size_t i = 0; i < n; ++i) {
        const double t = times_host[i];
        if (!(t >= 0.0) || !std::isfinite(t)) return SPDY_ERR_INVALID_ARG;
        const double v = t * static_cast<double>(B) / T;
        const double r = rounding == SPDY_ROUND_UP ? std::ceil(v) : std::floor(v + 0.5);
        if (r > 2147483647.0) return SPDY_ERR_INVALID_ARG;
    }
    for (size_t i = 0; i < n; ++i) {
        const double v = times_host[i] * static_cast<double>(B) / T;
        out_host[i] = static_cast<int32_t>(rounding == SPDY_ROUND_UP ? std::ceil(v) : std::floor(v + 0.5));
    }
    return SPDY_OK;
}

int spdy_uniform_profile(const int32_t *times_host, int32_t L, int32_t K, int32_t B, const uint8_t *keep_dense_host,
                         int32_t *choice_out, int64_t *total_out)
{
    if (!times_host || !choice_out || L < 1 || K < 1 || B < 0) return SPDY_ERR_INVALID_ARG;
    *choice_out = -1;
    if (total_out) *total_out = -1;
    for (size_t i = 0; i < static_cast<size_t>(L) * K; ++i)
        if (times_host[i] < 0) return SPDY_ERR_INVALID_ARG;
    for (int k = 0; k < K; ++k) {
        int64_t total = 0;
        for (int l = 0; l < L; ++l) {
            const int use = (keep_dense_host && keep_dense_host[l]) ? 0 : k;
            total += times_host[static_cast<size_t>(l) * K + use];
        }
        if (total <= B) {
            *choice_out = k;
            if (total_out) *total_out = total;
            break;
        }
    }
    return SPDY_OK;
}

}  // extern "C"
