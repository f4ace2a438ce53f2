// Batched SPDY dynamic program for B200 (sm_100a): host plan, kernels and the C ABI.
//
// One candidate = one min-plus dynamic program over L layers (Section 3.2, Eq. 2-3) followed by
// the final minimum over the budget axis and the walk back through the choice table (Appendix A,
// Algorithm 1).  The forward kernel keeps two band-limited DP rows in shared memory and streams
// one table row per layer to global memory; a second kernel walks the table back.
//
// Bit-exactness contract: every cell value is produced by exactly one fp32 round-to-nearest add
// (previous-row value + error) and compared with strict "<" in ascending choice order, so the
// results equal a plain sequential evaluation of Algorithm 1 with Eq. 2's bucket range.
#include "../../include/spdy_dp.h"

#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

namespace {

thread_local int g_last_cuda_error = 0;

#define SPDY_CUDA_TRY(expr)                                  \
    do {                                                     \
        cudaError_t err__ = (expr);                          \
        if (err__ != cudaSuccess) {                          \
            g_last_cuda_error = static_cast<int>(err__);     \
            return SPDY_ERR_CUDA;                            \
        }                                                    \
    } while (0)

// ----------------------------------------------------------------------------------------------
// Device-side layout
// ----------------------------------------------------------------------------------------------

#ifndef SPDY_RMAX
#define SPDY_RMAX 24
#endif
constexpr int RMAX = SPDY_RMAX;  // most band cells one lane owns in one pass (<= 24)

// How the forward kernel forms a cell and what it stores for the walk back.
enum ForwardMode {
    MODE_ARG = 1,      // compare + two selects per cell, byte table of winning choices
    MODE_ARG_PRED = 2, // compare + two predicated moves per cell, byte table
    MODE_ROW = 3,      // value-only minimum, fp32 table of row values
    MODE_ROW2 = 4      // value-only, two choices per step: packed f32x2 adds and 3-input minimum
};

// Row l (1-based; stored at index l-1) lives on the band [lo, lo + width).  A band cell is
// addressed by t_rel = t - lo.  Within a layer every warp pass covers 32*cpl consecutive cells
// ("span"); `rowoff` is where the row starts inside one candidate's table, in cells.
struct LayerDesc {
    int32_t width;
    uint32_t rowoff;
    int32_t lo;
    int32_t mn;      // smallest usable time of the layer: lo_l = lo_{l-1} + mn
    int32_t cpl;     // cells per lane per pass, 1..RMAX
    int32_t nspans;  // passes needed to cover the band: ceil(width / (32*cpl))
    int32_t mask_off;  // index of the layer's first pass in the pass-mask table
    int32_t nslots;    // shift slots of the layer (see TapRange)
};

// One (layer, choice) pair in band coordinates: the choice contributes to cells t_rel in [a, b]
// and reads the previous row at t_rel - a.  An unusable choice has b < a.
//
// The kernels walk "shift slots" rather than choices.  With a byte table (the winning choice is
// stored) slot u of a layer is choice u.  With a row-value table only the minimum matters, and
// since x -> fl32(x + e) is non-decreasing in e, the choices of a layer that share one time
// collapse exactly into one slot carrying the smallest of their errors:
//   min_k fl32(D[t - tau] + e_k) == fl32(D[t - tau] + min_k e_k)   over the k with times[l][k] == tau.
// Slots are then the distinct usable times in ascending order; slot_ptr/slot_member list the
// choices behind each slot.  (D never holds -0, so which zero the minimum picks does not matter.)
struct TapRange {
    int32_t a;
    int32_t b;
};

struct FwdArgs {
    const float *errors;      // [N][L][K], or null when the errors follow from coefficients
    const float *coeffs;      // [N][L] sensitivity coefficients (Eq. 4), used when errors is null
    const float *qtab;        // [K]: fp32((i / (K - 1))^2)
    const TapRange *slots;    // [L][K], the first layers[l].nslots of a layer are valid
    const uint8_t *slot_ptr;     // [L][K+1]: members of slot u are slot_member[slot_ptr[u] .. slot_ptr[u+1])
    const uint8_t *slot_member;  // [L][K]: choice indices grouped by slot
    const LayerDesc *layers;  // [L]
    const unsigned long long *span_masks;  // per pass: one bit per slot that overlaps it
    const unsigned *span_kranges;          // per pass: u_lo | u_hi << 8 | dense << 16
    void *table;              // wave-local walk-back table
    float *cost;              // [N]
    int32_t *time_used;       // [N]
    int64_t pitch;            // table cells per candidate
    int64_t n_first;          // first candidate of this wave
    int32_t L, K;
    int32_t row_stride;       // floats per shared-memory row buffer
    int32_t pad;              // +inf guard cells on either side of a row: 32 * the largest cells-per-lane
    float *grows;             // row buffers in global memory (GROWS kernels), else null
    const uint8_t *cand_flags; // per candidate of the wave, or null: run only candidates whose flag == which
    int32_t which;
};

__device__ __forceinline__ float pos_inf() { return __int_as_float(0x7f800000); }

// Error of choice k of layer l of candidate n: read from the table, or Eq. 4's c * (k / (K-1))^2 as
// one fp32 multiply of the coefficient with the pre-rounded square.
__device__ __forceinline__ float choice_error(const float *errors, const float *coeffs, const float *qtab,
                                              const int64_t n, const int l, const int k, const int L, const int K)
{
    if (errors) return errors[(n * L + l) * K + k];
    return __fmul_rn(coeffs[n * L + l], qtab[k]);
}

// (shift, error bits) of slot u of layer l for one candidate: the smallest error among the
// slot's choices (a single choice unless equal times were merged).
__device__ __forceinline__ int2 stage_slot(const FwdArgs &args, const int64_t n, const int l, const int u)
{
    const int K = args.K, L = args.L;
    const uint8_t *ptr = args.slot_ptr + static_cast<size_t>(l) * (K + 1);
    const uint8_t *member = args.slot_member + static_cast<size_t>(l) * K;
    const int j0 = ptr[u], j1 = ptr[u + 1];
    float e = choice_error(args.errors, args.coeffs, args.qtab, n, l, member[j0], L, K);
    for (int j = j0 + 1; j < j1; ++j)
        e = fminf(e, choice_error(args.errors, args.coeffs, args.qtab, n, l, member[j], L, K));
    return make_int2(args.slots[static_cast<size_t>(l) * K + u].a, __float_as_int(e));
}

// Two independent round-to-nearest fp32 adds in one instruction: (x, y) += (e, e).
__device__ __forceinline__ void add2_rn(float &x, float &y, unsigned long long e2)
{
    unsigned long long p, r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "f"(x), "f"(y));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(p), "l"(e2));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(x), "=f"(y) : "l"(r));
}

__device__ __forceinline__ unsigned long long splat2(float e)
{
    unsigned long long p;
    asm("mov.b64 %0, {%1, %1};" : "=l"(p) : "f"(e));
    return p;
}

__device__ __forceinline__ float min3(float a, float b, float c)
{
    float m;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
    return m;
}

// Cell updates of one choice (or two) on the RR cells a lane owns; `sa`/`sb` point at the lane's
// first source cell of the previous row, consecutive owned cells are 32 floats apart.
template <int RR>
__device__ __forceinline__ void update_min1(float (&best)[RR], const float *sa, const float ea)
{
#pragma unroll
    for (int j = 0; j < RR; ++j) best[j] = fminf(best[j], __fadd_rn(sa[j * 32], ea));
}

template <int RR>
__device__ __forceinline__ void update_min2(float (&best)[RR], const float *sa, const float ea,
                                            const float *sb, const float eb)
{
    const unsigned long long ea2 = splat2(ea), eb2 = splat2(eb);
#pragma unroll
    for (int j = 0; j + 1 < RR; j += 2) {
        float a0 = sa[j * 32], a1 = sa[(j + 1) * 32];
        float b0 = sb[j * 32], b1 = sb[(j + 1) * 32];
        add2_rn(a0, a1, ea2);
        add2_rn(b0, b1, eb2);
        best[j] = min3(best[j], a0, b0);
        best[j + 1] = min3(best[j + 1], a1, b1);
    }
    if (RR & 1) {
        const float a0 = __fadd_rn(sa[(RR - 1) * 32], ea);
        const float b0 = __fadd_rn(sb[(RR - 1) * 32], eb);
        best[RR - 1] = min3(best[RR - 1], a0, b0);
    }
}

template <int RR>
__device__ __forceinline__ void update_arg(float (&best)[RR], int (&idx)[RR], const float *src,
                                           const float e, const int k)
{
#pragma unroll
    for (int j = 0; j < RR; ++j) {
        const float v = __fadd_rn(src[j * 32], e);
        const bool better = v < best[j];  // strict: the lowest k keeps a tie
        best[j] = better ? v : best[j];
        idx[j] = better ? k : idx[j];
    }
}

// Same update with the two selects written as predicated fp32 arithmetic that acts as an exact
// move, to keep them off the integer/compare pipe: best <- v + (-0.0) (== v for every v) and
// idx <- v * 0 + k (== k: a winning v is finite, so v * 0 is +-0).  The index is carried as a float.
template <int RR>
__device__ __forceinline__ void update_arg_pred(float (&best)[RR], float (&idxf)[RR], const float *src,
                                                const float e, const int k)
{
    const float kf = static_cast<float>(k);
    const unsigned long long e2 = splat2(e);
#define SPDY_PRED_UPDATE(J, V)                        \
    asm("{ .reg .pred p; setp.lt.f32 p, %2, %0;\n\t"  \
        "@p add.rn.f32 %0, %2, 0f80000000;\n\t"       \
        "@p fma.rn.f32 %1, %2, 0f00000000, %3; }"     \
        : "+f"(best[J]), "+f"(idxf[J])                \
        : "f"(V), "f"(kf))
#pragma unroll
    for (int j = 0; j + 1 < RR; j += 2) {
        float v0 = src[j * 32], v1 = src[(j + 1) * 32];
        add2_rn(v0, v1, e2);
        SPDY_PRED_UPDATE(j, v0);
        SPDY_PRED_UPDATE(j + 1, v1);
    }
    if (RR & 1) {
        const float v0 = __fadd_rn(src[(RR - 1) * 32], e);
        SPDY_PRED_UPDATE(RR - 1, v0);
    }
#undef SPDY_PRED_UPDATE
}

// One warp pass: the 32*RR band cells starting at s (lane i owns cells s + i, s + i + 32, ...),
// so every shared-memory access is lane-consecutive (conflict-free) whatever the shift.  Both row
// buffers carry `pad` cells of +inf (the widest pass of the plan) on either side of the band: a pass that only partly overlaps a
// choice's range reads +inf for the cells outside it and needs no per-cell bounds check.  Which
// choices overlap the pass at all is known on the host.  `krange` = k_lo | k_hi << 8 | dense << 16:
// the overlapping choices lie in [k_lo, k_hi); when they are all of that range (dense, the usual
// case: times fall as the choice index rises) the loop runs straight over it, otherwise it walks
// the set bits of `mask` (MW 64-bit words, one bit per choice), in ascending order either way.
//
// `prev`/`cur` point at band cell 0 of the previous/new row; taps[k] = (a_k, bits of e_k): choice
// k reads the previous row at t_rel - a_k.
//
// With MASKED only cells below `limit` are stored (a CTA of a cluster owns a slice of the band and
// must not write its neighbour's cells); without it the caller guarantees room for the whole pass.
//
// `prev` and `cur` carry no __restrict__: with the row buffers in global memory (GROWS) the kernel itself
// rewrites the memory behind `prev` two layers later, so those reads must stay ordinary coherent loads.
template <int RR, int MODE, bool MASKED>
__device__ __forceinline__ void process_span(const float *prev, float *cur,
                                             const int2 *__restrict__ taps, const unsigned krange,
                                             const unsigned long long *__restrict__ mask, const int MW,
                                             const int s, const int lane, void *table_row,
                                             const int limit)
{
    const float INF = pos_inf();
    const float *base = prev + s + lane;
    const int k_lo = krange & 0xFF, k_hi = (krange >> 8) & 0xFF;
    const bool dense = (krange >> 16) & 1;
    float best[RR];
#pragma unroll
    for (int j = 0; j < RR; ++j) best[j] = INF;

    if constexpr (MODE == MODE_ROW2 || MODE == MODE_ROW) {
        // Value-only minimum: the order of the choices does not matter, so overlapping choices
        // are taken two at a time (MODE_ROW2) whatever their indices.
        if (dense) {
            int k = k_lo;
            if (MODE == MODE_ROW2) {
                // An odd first slot goes alone so that every pair below is one aligned 16-byte read.
                if ((k & 1) && k < k_hi) {
                    const int2 ta = taps[k];
                    update_min1<RR>(best, base - ta.x, __int_as_float(ta.y));
                    ++k;
                }
#pragma unroll 1
                for (; k + 1 < k_hi; k += 2) {
                    const int4 t = *reinterpret_cast<const int4 *>(taps + k);
                    update_min2<RR>(best, base - t.x, __int_as_float(t.y), base - t.z, __int_as_float(t.w));
                }
            }
#pragma unroll 1
            for (; k < k_hi; ++k) {
                const int2 ta = taps[k];
                update_min1<RR>(best, base - ta.x, __int_as_float(ta.y));
            }
        } else {
#pragma unroll 1
            for (int w = 0; w < MW; ++w) {
                unsigned long long m = __ldg(mask + w);
#pragma unroll 1
                while (m) {
                    const int2 ta = taps[64 * w + __ffsll(static_cast<long long>(m)) - 1];
                    m &= m - 1;
                    update_min1<RR>(best, base - ta.x, __int_as_float(ta.y));
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (!MASKED || s + j * 32 + lane < limit) cur[s + j * 32 + lane] = best[j];
        float *D = static_cast<float *>(table_row) + s + lane;
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (!MASKED || s + j * 32 + lane < limit) D[j * 32] = best[j];
    } else if constexpr (MODE == MODE_ARG) {
        int idx[RR];
#pragma unroll
        for (int j = 0; j < RR; ++j) idx[j] = 0xFF;
        if (dense) {
#pragma unroll 1
            for (int k = k_lo; k < k_hi; ++k) {
                const int2 tp = taps[k];
                update_arg<RR>(best, idx, base - tp.x, __int_as_float(tp.y), k);
            }
        } else {
#pragma unroll 1
            for (int w = 0; w < MW; ++w) {
                unsigned long long m = __ldg(mask + w);
#pragma unroll 1
                while (m) {
                    const int k = 64 * w + __ffsll(static_cast<long long>(m)) - 1;
                    m &= m - 1;
                    const int2 tp = taps[k];
                    update_arg<RR>(best, idx, base - tp.x, __int_as_float(tp.y), k);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (!MASKED || s + j * 32 + lane < limit) cur[s + j * 32 + lane] = best[j];
        unsigned char *P = static_cast<unsigned char *>(table_row) + s + lane;
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (!MASKED || s + j * 32 + lane < limit) P[j * 32] = static_cast<unsigned char>(idx[j]);
    } else {  // MODE_ARG_PRED
        float idxf[RR];
#pragma unroll
        for (int j = 0; j < RR; ++j) idxf[j] = 255.0f;
        if (dense) {
#pragma unroll 1
            for (int k = k_lo; k < k_hi; ++k) {
                const int2 tp = taps[k];
                update_arg_pred<RR>(best, idxf, base - tp.x, __int_as_float(tp.y), k);
            }
        } else {
#pragma unroll 1
            for (int w = 0; w < MW; ++w) {
                unsigned long long m = __ldg(mask + w);
#pragma unroll 1
                while (m) {
                    const int k = 64 * w + __ffsll(static_cast<long long>(m)) - 1;
                    m &= m - 1;
                    const int2 tp = taps[k];
                    update_arg_pred<RR>(best, idxf, base - tp.x, __int_as_float(tp.y), k);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (!MASKED || s + j * 32 + lane < limit) cur[s + j * 32 + lane] = best[j];
        unsigned char *P = static_cast<unsigned char *>(table_row) + s + lane;
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (!MASKED || s + j * 32 + lane < limit)
                P[j * 32] = static_cast<unsigned char>(static_cast<int>(idxf[j]));
    }
}

// RCAP: the largest cells-per-lane this instantiation can run.  The registers a kernel needs grow
// with the largest unrolled pass, so plans whose rows are narrow (few cells per lane) use the
// RCAP = 8 build, which fits twice as many CTAs per SM.
//
// GROWS: keep the two row buffers in global memory (args.grows, 2 * row_stride floats per candidate of
// the wave) instead of shared memory.  This is the fallback for bands too wide even for a cluster of
// eight CTAs; the code is the same, the reads then go through L1/L2.  Writes of one layer are ordered
// before the reads of the next by the same per-layer __syncthreads().
template <int MODE, int NT, int MINB, int RCAP, bool GROWS>
__global__ void __launch_bounds__(NT, MINB) spdy_forward_kernel(const FwdArgs args)
{
    constexpr bool ROWFMT = (MODE == MODE_ROW || MODE == MODE_ROW2);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *rows;
    int2 *tap_buf;
    if constexpr (GROWS) {
        rows = args.grows + static_cast<size_t>(blockIdx.x) * 2 * static_cast<size_t>(args.row_stride);
        tap_buf = reinterpret_cast<int2 *>(smem_raw);
    } else {
        rows = reinterpret_cast<float *>(smem_raw);
        tap_buf = reinterpret_cast<int2 *>(rows + 2 * static_cast<size_t>(args.row_stride));
    }

    // Two table sets may share a wave (see spdy_monotone_flags_kernel): a CTA whose candidate belongs
    // to the other set leaves at once, before any barrier.
    if (args.cand_flags && args.cand_flags[blockIdx.x] != args.which) return;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    constexpr int NWARPS = NT / 32;
    const int L = args.L, K = args.K;
    const int KS = (K + 1) & ~1;  // slots per staging buffer: even, so that slot pairs are 16-byte aligned
    const int64_t n_local = blockIdx.x;
    const int64_t n = args.n_first + n_local;
    const float INF = pos_inf();

    // Both buffers start as +inf everywhere; D_0 is +0 at t = 0 (Eq. 3 via a virtual row 0).
    for (int i = tid; i < 2 * args.row_stride; i += NT) rows[i] = INF;
    for (int u = tid; u < args.layers[0].nslots; u += NT) tap_buf[u] = stage_slot(args, n, 0, u);
    __syncthreads();
    const int PAD = args.pad;
    if (tid == 0) rows[PAD] = 0.0f;
    __syncthreads();

    for (int l = 0; l < L; ++l) {
        const float *prev = rows + (l & 1) * args.row_stride + PAD;
        float *cur = rows + ((l + 1) & 1) * args.row_stride + PAD;
        const int2 *taps = tap_buf + (l & 1) * KS;
        const LayerDesc ld = args.layers[l];

        // Fetch the next layer's slots early; they are parked in shared memory after the pass.
        // (NT >= K is guaranteed by the host, so one thread per slot suffices.)
        int2 next_tap = make_int2(0, 0);
        const bool have_next = (l + 1 < L) && (tid < args.layers[l + 1].nslots);
        if (have_next) next_tap = stage_slot(args, n, l + 1, tid);

        unsigned char *row_base = static_cast<unsigned char *>(args.table) +
                                  (n_local * args.pitch + ld.rowoff) * (ROWFMT ? 4 : 1);
        const int span_cells = 32 * ld.cpl;
        const int MW = (K + 63) >> 6;
        const unsigned long long *masks = args.span_masks + static_cast<size_t>(ld.mask_off) * MW;
        const unsigned *kranges = args.span_kranges + ld.mask_off;
        switch (ld.cpl) {
#define SPDY_CASE(RR)                                                                          \
    case RR:                                                                                   \
        if constexpr (RR <= RMAX && RR <= RCAP)                                                \
            for (int span = warp; span < ld.nspans; span += NWARPS)                            \
                process_span<RR, MODE, false>(prev, cur, taps, __ldg(kranges + span),          \
                                              masks + span * MW, MW, span * (32 * RR), lane,   \
                                              row_base, 0);                                    \
        break;
            SPDY_CASE(1) SPDY_CASE(2) SPDY_CASE(3) SPDY_CASE(4) SPDY_CASE(5) SPDY_CASE(6)
            SPDY_CASE(7) SPDY_CASE(8) SPDY_CASE(9) SPDY_CASE(10) SPDY_CASE(11) SPDY_CASE(12)
            SPDY_CASE(13) SPDY_CASE(14) SPDY_CASE(15) SPDY_CASE(16) SPDY_CASE(17) SPDY_CASE(18)
            SPDY_CASE(19) SPDY_CASE(20) SPDY_CASE(21) SPDY_CASE(22) SPDY_CASE(23) SPDY_CASE(24)
#undef SPDY_CASE
            default: break;
        }
        // Cells [width, width + PAD) of the new row must read as +inf for the next layer.  The
        // passes above wrote +inf from `width` up to nspans*span (those cells saw only +inf
        // sources); PAD more cells of +inf cover the rest.
        for (int i = tid; i < PAD; i += NT) cur[ld.nspans * span_cells + i] = INF;
        if (have_next) tap_buf[((l + 1) & 1) * KS + tid] = next_tap;
        __syncthreads();
    }

    // min over t <= B of D_L[t], lowest t among equals (the band's upper end never exceeds B).
    const float *last = rows + (L & 1) * args.row_stride + PAD;
    const LayerDesc ld = args.layers[L - 1];
    float bv = INF;
    int bt = 0x7fffffff;
    for (int t = tid; t < ld.width; t += NT) {
        const float v = last[t];
        if (v < bv) {
            bv = v;
            bt = t;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int ot = __shfl_xor_sync(0xffffffffu, bt, off);
        if (ov < bv || (ov == bv && ot < bt)) {
            bv = ov;
            bt = ot;
        }
    }
    __shared__ float red_v[32];
    __shared__ int red_t[32];
    if (lane == 0) {
        red_v[warp] = bv;
        red_t[warp] = bt;
    }
    __syncthreads();
    if (warp == 0) {
        bv = lane < NWARPS ? red_v[lane] : INF;
        bt = lane < NWARPS ? red_t[lane] : 0x7fffffff;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int ot = __shfl_xor_sync(0xffffffffu, bt, off);
            if (ov < bv || (ov == bv && ot < bt)) {
                bv = ov;
                bt = ot;
            }
        }
        if (lane == 0) {
            const bool feasible = bv < INF;
            args.cost[n] = feasible ? bv : INF;
            args.time_used[n] = feasible ? ld.lo + bt : -1;
        }
    }
}

// ----------------------------------------------------------------------------------------------
// Cluster variant: one candidate per thread-block cluster
// ----------------------------------------------------------------------------------------------
//
// When two band-limited rows do not fit one CTA's shared memory (or when there are fewer
// candidates than SMs) the band of every row is cut into C contiguous slices, one per CTA of a
// cluster.  Each CTA keeps its slice of the new row in its own shared memory (`out`, double
// buffered) and, before a layer, gathers the window of the previous row its slice depends on -
// its own slice plus up to max_k a_k cells to the left - from the `out` buffers of its cluster
// peers through distributed shared memory into a private window (`win`).  The cell updates then
// run on local shared memory exactly as in the single-CTA kernel.  One hardware cluster barrier
// per layer orders "slices of row l written" before "windows for row l+1 gathered"; every thread
// of every CTA reaches every barrier (there is no early exit), so the barrier cannot wait forever.

// Per (layer, rank) pass shape.  q0 is the first previous-row cell of the window.
struct SliceDesc {
    int32_t slice_lo;   // first band cell of the slice
    int32_t slice_hi;   // one past the last (slice_lo == slice_hi: empty)
    int32_t cpl;        // cells per lane per pass
    int32_t nspans;     // passes covering the slice
    int32_t mask_off;   // first pass in the pass tables
    int32_t q0;         // first previous-row cell the passes may read
    int32_t win_len;    // cells of the window
    int32_t prev_slice; // slice length of the previous row (cells per rank), >= 1
};

struct ClusterArgs {
    FwdArgs f;
    const SliceDesc *slices;  // [L][C]
    int32_t C;
    int32_t out_stride;  // floats per `out` buffer
    int32_t win_stride;  // floats of `win`
};

template <int MODE, int NT>
__global__ void __launch_bounds__(NT, 1) spdy_forward_cluster_kernel(const ClusterArgs cargs)
{
    namespace cg = cooperative_groups;
    constexpr bool ROWFMT = (MODE == MODE_ROW || MODE == MODE_ROW2);
    constexpr int NWARPS = NT / 32;
    const FwdArgs &args = cargs.f;
    cg::cluster_group cluster = cg::this_cluster();
    const int C = cargs.C;
    const int rank = static_cast<int>(cluster.block_rank());

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *out = reinterpret_cast<float *>(smem_raw);                 // [2][out_stride]
    float *win = out + 2 * static_cast<size_t>(cargs.out_stride);     // [win_stride]
    int2 *tap_buf = reinterpret_cast<int2 *>(win + cargs.win_stride);  // [2][K]
    __shared__ float cl_v[16];
    __shared__ int cl_t[16];

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int L = args.L, K = args.K;
    const int KS = (K + 1) & ~1;
    const int64_t n_local = blockIdx.x / C;
    const int64_t n = args.n_first + n_local;
    const float INF = pos_inf();

    // Virtual row 0: +0 at t = 0, held in rank 0's first `out` buffer.
    for (int i = tid; i < 2 * cargs.out_stride; i += NT) out[i] = INF;
    for (int u = tid; u < args.layers[0].nslots; u += NT) tap_buf[u] = stage_slot(args, n, 0, u);
    __syncthreads();
    if (rank == 0 && tid == 0) out[0] = 0.0f;
    cluster.sync();

    int prev_width = 1;
    for (int l = 0; l < L; ++l) {
        const SliceDesc sd = cargs.slices[l * C + rank];
        const LayerDesc ld = args.layers[l];
        const int2 *taps = tap_buf + (l & 1) * KS;
        float *out_prev = out + (l & 1) * cargs.out_stride;
        float *out_cur = out + ((l + 1) & 1) * cargs.out_stride;

        int2 next_tap = make_int2(0, 0);
        const bool have_next = (l + 1 < L) && (tid < args.layers[l + 1].nslots);
        if (have_next) next_tap = stage_slot(args, n, l + 1, tid);

        // Gather the window [q0, q0 + win_len) of the previous row, peer by peer; cells outside
        // the previous band read as +inf.
        {
            const int q_end = sd.q0 + sd.win_len;
            for (int i = tid; i < sd.win_len; i += NT) {
                const int q = sd.q0 + i;
                if (q < 0 || q >= prev_width) win[i] = INF;
            }
            const int q_lo = max(sd.q0, 0), q_hi = min(q_end, prev_width);
            if (q_hi > q_lo) {
                const int first_rank = q_lo / sd.prev_slice;
                const int last_rank = (q_hi - 1) / sd.prev_slice;
                for (int src = first_rank; src <= last_rank; ++src) {
                    const int seg_lo = max(q_lo, src * sd.prev_slice);
                    const int seg_hi = min(q_hi, (src + 1) * sd.prev_slice);
                    const float *remote = (src == rank) ? out_prev : cluster.map_shared_rank(out_prev, src);
                    const float *from = remote + (seg_lo - src * sd.prev_slice);
                    float *to = win + (seg_lo - sd.q0);
                    for (int i = tid; i < seg_hi - seg_lo; i += NT) to[i] = from[i];
                }
            }
        }
        __syncthreads();

        const float *prev = win - sd.q0;          // prev[q] for q in [q0, q0 + win_len)
        float *cur = out_cur - sd.slice_lo;       // cur[t_rel] for t_rel in the slice
        unsigned char *row_base = static_cast<unsigned char *>(args.table) +
                                  (n_local * args.pitch + ld.rowoff) * (ROWFMT ? 4 : 1);
        const int MW = (K + 63) >> 6;
        const unsigned long long *masks = args.span_masks + static_cast<size_t>(sd.mask_off) * MW;
        const unsigned *kranges = args.span_kranges + sd.mask_off;
        switch (sd.cpl) {
#define SPDY_CASE(RR)                                                                             \
    case RR:                                                                                      \
        if constexpr (RR <= RMAX)                                                                 \
            for (int span = warp; span < sd.nspans; span += NWARPS)                               \
                process_span<RR, MODE, true>(prev, cur, taps, __ldg(kranges + span),              \
                                             masks + span * MW, MW, sd.slice_lo + span * (32 * RR), \
                                             lane, row_base, sd.slice_hi);                        \
        break;
            SPDY_CASE(1) SPDY_CASE(2) SPDY_CASE(3) SPDY_CASE(4) SPDY_CASE(5) SPDY_CASE(6)
            SPDY_CASE(7) SPDY_CASE(8) SPDY_CASE(9) SPDY_CASE(10) SPDY_CASE(11) SPDY_CASE(12)
            SPDY_CASE(13) SPDY_CASE(14) SPDY_CASE(15) SPDY_CASE(16) SPDY_CASE(17) SPDY_CASE(18)
            SPDY_CASE(19) SPDY_CASE(20) SPDY_CASE(21) SPDY_CASE(22) SPDY_CASE(23) SPDY_CASE(24)
#undef SPDY_CASE
            default: break;
        }
        if (have_next) tap_buf[((l + 1) & 1) * KS + tid] = next_tap;
        prev_width = ld.width;
        cluster.sync();  // slices of row l+1 complete everywhere; row l no longer needed
    }

    // Local minimum over the slice of the last row, then across the cluster through rank 0.
    const SliceDesc sd = cargs.slices[(L - 1) * C + rank];
    const LayerDesc ld = args.layers[L - 1];
    const float *last = out + (L & 1) * cargs.out_stride;
    float bv = INF;
    int bt = 0x7fffffff;
    for (int t = sd.slice_lo + tid; t < sd.slice_hi; t += NT) {
        const float v = last[t - sd.slice_lo];
        if (v < bv) {
            bv = v;
            bt = t;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int ot = __shfl_xor_sync(0xffffffffu, bt, off);
        if (ov < bv || (ov == bv && ot < bt)) {
            bv = ov;
            bt = ot;
        }
    }
    __shared__ float red_v[32];
    __shared__ int red_t[32];
    if (lane == 0) {
        red_v[warp] = bv;
        red_t[warp] = bt;
    }
    __syncthreads();
    if (warp == 0) {
        bv = lane < NWARPS ? red_v[lane] : INF;
        bt = lane < NWARPS ? red_t[lane] : 0x7fffffff;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int ot = __shfl_xor_sync(0xffffffffu, bt, off);
            if (ov < bv || (ov == bv && ot < bt)) {
                bv = ov;
                bt = ot;
            }
        }
        if (lane == 0) {
            float *dst_v = cluster.map_shared_rank(cl_v, 0);
            int *dst_t = cluster.map_shared_rank(cl_t, 0);
            dst_v[rank] = bv;
            dst_t[rank] = bt;
        }
    }
    cluster.sync();
    if (rank == 0 && tid == 0) {
        bv = cl_v[0];
        bt = cl_t[0];
        for (int r = 1; r < C; ++r) {
            if (cl_v[r] < bv || (cl_v[r] == bv && cl_t[r] < bt)) {
                bv = cl_v[r];
                bt = cl_t[r];
            }
        }
        const bool feasible = bv < INF;
        args.cost[n] = feasible ? bv : INF;
        args.time_used[n] = feasible ? ld.lo + bt : -1;
    }
}

struct BackArgs {
    const float *errors;      // [N][L][K], or null (see FwdArgs)
    const float *coeffs;      // [N][L]
    const float *qtab;        // [K]
    const int32_t *times;     // [L][K]
    const LayerDesc *layers;  // [L]
    const void *table;
    const float *cost;
    const int32_t *time_used;
    uint8_t *profile;         // [N][L]
    int32_t *status;          // device word, set non-zero if a self-check fails
    int64_t pitch;
    int64_t n_first;
    int64_t n_count;
    int32_t L, K;
    const uint8_t *cand_flags; // as in FwdArgs
    int32_t which;
    const uint8_t *slot_ptr;    // byte table of slot indices: translate through these lists (else null)
    const uint8_t *slot_member;
};

// Walk back through the byte table (end of Algorithm 1): one thread per candidate.
__global__ void spdy_backtrack_arg_kernel(const BackArgs args)
{
    const int64_t n_local = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (n_local >= args.n_count) return;
    if (args.cand_flags && args.cand_flags[n_local] != args.which) return;
    const int64_t n = args.n_first + n_local;
    const int L = args.L, K = args.K;
    uint8_t *prof = args.profile + n * L;
    int t = args.time_used[n];
    if (t < 0) {
        for (int l = 0; l < L; ++l) prof[l] = 0xFF;
        return;
    }
    const unsigned char *P = static_cast<const unsigned char *>(args.table) + n_local * args.pitch;
    bool ok = true;
    for (int l = L - 1; l >= 0; --l) {
        const LayerDesc ld = args.layers[l];
        const int t_rel = t - ld.lo;
        int k = 0xFF;
        if (ok && t_rel >= 0 && t_rel < ld.width) k = P[ld.rowoff + t_rel];
        // A table of slot indices: the slot's winner is its first (lowest) member.
        if (args.slot_member && k < ld.nslots) k = args.slot_member[l * K + args.slot_ptr[l * (K + 1) + k]];
        else if (args.slot_member) k = 0xFF;
        if (k >= K) {
            ok = false;
            k = 0xFF;
        } else {
            t -= args.times[l * K + k];
        }
        prof[l] = static_cast<uint8_t>(k);
    }
    if (!ok || t != 0) atomicExch(args.status, 1);
}

// Walk back through stored row values: one warp per candidate.  At (l, t) the winning choice is
// the lowest k whose fp32 sum D_{l-1}[t - times[l][k]] + errors[n][l][k] equals D_l[t] bit for
// bit; the forward pass formed D_l[t] as the minimum of exactly these sums.
__global__ void spdy_backtrack_row_kernel(const BackArgs args)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_local = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
    if (n_local >= args.n_count) return;
    const int64_t n = args.n_first + n_local;
    const int L = args.L, K = args.K;
    uint8_t *prof = args.profile + n * L;
    int t = args.time_used[n];
    if (t < 0) {
        for (int l = lane; l < L; l += 32) prof[l] = 0xFF;
        return;
    }
    const float INF = pos_inf();
    const float *D = static_cast<const float *>(args.table) + n_local * args.pitch;
    float target = args.cost[n];
    bool ok = true;
    for (int l = L - 1; l >= 0; --l) {
        const LayerDesc ld = args.layers[l];
        const int t_rel = t - ld.lo;
        int prev_width = 1;
        uint32_t prev_off = 0;
        if (l > 0) {
            const LayerDesc pl = args.layers[l - 1];
            prev_width = pl.width;
            prev_off = pl.rowoff;
        }
        int found_k = 0xFF;
        float found_prev = INF;
        int found_tau = 0;
        for (int k0 = 0; k0 < K && found_k == 0xFF; k0 += 32) {
            const int k = k0 + lane;
            float pv = INF;
            int tau = 0;
            bool match = false;
            if (k < K) {
                tau = args.times[l * K + k];
                const int64_t src = static_cast<int64_t>(t_rel) - (static_cast<int64_t>(tau) - ld.mn);
                if (src >= 0 && src < prev_width) {
                    pv = (l == 0) ? 0.0f : D[prev_off + src];
                    const float v = __fadd_rn(pv, choice_error(args.errors, args.coeffs, args.qtab, n, l, k, L, K));
                    match = (v == target) && (pv < INF);
                }
            }
            const unsigned ballot = __ballot_sync(0xffffffffu, match);
            if (ballot) {
                const int src_lane = __ffs(ballot) - 1;
                found_k = k0 + src_lane;
                found_prev = __shfl_sync(0xffffffffu, pv, src_lane);
                found_tau = __shfl_sync(0xffffffffu, tau, src_lane);
            }
        }
        if (found_k == 0xFF) {
            ok = false;
            if (lane == 0) prof[l] = 0xFF;
        } else {
            if (lane == 0) prof[l] = static_cast<uint8_t>(found_k);
            t -= found_tau;
            target = found_prev;
        }
        if (!ok) {
            for (int ll = l - 1 - lane; ll >= 0; ll -= 32) prof[ll] = 0xFF;
            break;
        }
    }
    if ((!ok || t != 0) && lane == 0) atomicExch(args.status, 1);
}

// With the byte table the winning choice index is stored, so choices of equal time may be merged into
// one slot only where the merge cannot change the winner: when, inside every group of equal-time
// choices, the errors do not fall as the index rises.  Then the group's lowest index attains the
// group's smallest sum at every cell and wins every tie inside the group, and among groups the
// lowest first member wins - exactly the choice a scan over all choices in ascending order keeps.
// This kernel tests that condition per candidate (one warp each): flag 1 = merged tables are exact
// for it, flag 0 = it needs one slot per choice.  slot_ptr / slot_member are the merged lists.
__global__ void spdy_monotone_flags_kernel(const float *errors, const float *coeffs, const float *qtab,
                                           const LayerDesc *layers, const uint8_t *slot_ptr,
                                           const uint8_t *slot_member, uint8_t *flags, int64_t n_first,
                                           int64_t n_count, int32_t L, int32_t K)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_local = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
    if (n_local >= n_count) return;
    const int64_t n = n_first + n_local;
    bool ok = true;
    for (int l = 0; l < L; ++l) {
        const int nslots = layers[l].nslots;
        const uint8_t *ptr = slot_ptr + static_cast<size_t>(l) * (K + 1);
        const uint8_t *member = slot_member + static_cast<size_t>(l) * K;
        for (int u = lane; u < nslots; u += 32) {
            const int j0 = ptr[u], j1 = ptr[u + 1];
            float prev = choice_error(errors, coeffs, qtab, n, l, member[j0], L, K);
            for (int j = j0 + 1; j < j1; ++j) {
                const float e = choice_error(errors, coeffs, qtab, n, l, member[j], L, K);
                ok = ok && (prev <= e);  // false for NaN as well
                prev = e;
            }
        }
    }
    ok = __all_sync(0xffffffffu, ok);
    if (lane == 0) flags[n_local] = ok ? 1 : 0;
}

// ----------------------------------------------------------------------------------------------
// Peak probes: what the forward kernel's two ceilings amount to on the device at hand
// ----------------------------------------------------------------------------------------------
//
// spdy_probe_lds_kernel streams 4-byte shared-memory reads the way the forward kernel issues them
// (lane-consecutive, a different word offset per read) into running minima; spdy_probe_alu_kernel
// runs the arithmetic of one cell update (one packed add per two cells, one 3-input minimum per two
// updates) on registers only.  Each thread reports its result so that nothing is optimised away.
constexpr int PROBE_WORDS = 8192;  // floats of shared memory a probe CTA reads from

__global__ void __launch_bounds__(256) spdy_probe_lds_kernel(float *out, int iters)
{
    __shared__ float buf[PROBE_WORDS + 1024];
    for (int i = threadIdx.x; i < PROBE_WORDS + 1024; i += blockDim.x) buf[i] = static_cast<float>(i & 1023);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = pos_inf();
    int off = warp * 37;
    for (int it = 0; it < iters; ++it) {
        const float *src = buf + (off & (PROBE_WORDS - 1)) + lane;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = fminf(acc[j], src[j * 32]);
        off += 293;  // an odd stride: every read starts at a different bank
    }
    float r = acc[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) r = fminf(r, acc[j]);
    out[blockIdx.x * blockDim.x + threadIdx.x] = r;
}

__global__ void __launch_bounds__(256) spdy_probe_alu_kernel(float *out, int iters, float e0, float e1)
{
    float best[8], a[8], b[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        best[j] = pos_inf();
        a[j] = static_cast<float>(threadIdx.x + j);
        b[j] = static_cast<float>(threadIdx.x * 3 + j);
    }
    const unsigned long long e0s = splat2(e0), e1s = splat2(e1);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            add2_rn(a[j], a[j + 1], e0s);
            add2_rn(b[j], b[j + 1], e1s);
            best[j] = min3(best[j], a[j], b[j]);
            best[j + 1] = min3(best[j + 1], a[j + 1], b[j + 1]);
        }
    }
    float r = best[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) r = fminf(r, best[j]);
    out[blockIdx.x * blockDim.x + threadIdx.x] = r;
}

// Eq. 4 written out as a table: errors[n][l][i] = c[n][l] * (i / (K-1))^2, the same fp32 multiply
// of the coefficient with the pre-rounded square that the solver's coefficient mode performs in place.
__global__ void spdy_quadratic_errors_kernel(const float *coeffs, float *errors, int64_t total, int32_t K)
{
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; j < total; j += stride) {
        const int i = static_cast<int>(j % K);
        float q = 0.0f;
        if (K > 1) {
            const double r = static_cast<double>(i) / static_cast<double>(K - 1);
            q = static_cast<float>(r * r);
        }
        errors[j] = __fmul_rn(coeffs[j / K], q);
    }
}

__global__ void spdy_fill_infeasible_kernel(uint8_t *profile, float *cost, int32_t *time_used,
                                            int64_t N, int32_t L)
{
    const int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    const int64_t total = N * L;
    for (int64_t j = i; j < total; j += stride) profile[j] = 0xFF;
    for (int64_t j = i; j < N; j += stride) {
        cost[j] = pos_inf();
        time_used[j] = -1;
    }
}

// ----------------------------------------------------------------------------------------------
// Kernel table
// ----------------------------------------------------------------------------------------------

using FwdKernel = void (*)(const FwdArgs);

struct FwdVariant {
    int mode;
    int threads;
    int rcap;
    FwdKernel fn;
};

#define SPDY_VARIANT(MODE, NT, MINB, RCAP) \
    FwdVariant { MODE, NT, RCAP, spdy_forward_kernel<MODE, NT, MINB, RCAP, false> }
#define SPDY_VARIANTS(MODE)                                                                        \
    SPDY_VARIANT(MODE, 128, 4, RMAX), SPDY_VARIANT(MODE, 256, 3, RMAX), SPDY_VARIANT(MODE, 512, 1, RMAX), \
    SPDY_VARIANT(MODE, 1024, 1, 16), SPDY_VARIANT(MODE, 128, 6, 8), SPDY_VARIANT(MODE, 256, 3, 8),       \
    SPDY_VARIANT(MODE, 512, 1, 8), SPDY_VARIANT(MODE, 1024, 1, 8)

const FwdVariant kVariants[] = {
    SPDY_VARIANTS(MODE_ARG), SPDY_VARIANTS(MODE_ARG_PRED), SPDY_VARIANTS(MODE_ROW), SPDY_VARIANTS(MODE_ROW2),
};

// Rows in global memory: one CTA of 1024 threads per candidate, the default cell update of each
// table format.
const FwdVariant kGlobalRowVariants[] = {
    FwdVariant{MODE_ARG_PRED, 1024, 16, spdy_forward_kernel<MODE_ARG_PRED, 1024, 1, 16, true>},
    FwdVariant{MODE_ROW2, 1024, 16, spdy_forward_kernel<MODE_ROW2, 1024, 1, 16, true>},
};

using ClusterKernel = void (*)(const ClusterArgs);

struct ClusterVariant {
    int mode;
    int threads;
    ClusterKernel fn;
};

#define SPDY_CVARIANT(MODE, NT) \
    ClusterVariant { MODE, NT, spdy_forward_cluster_kernel<MODE, NT> }

const ClusterVariant kClusterVariants[] = {
    SPDY_CVARIANT(MODE_ARG, 256),  SPDY_CVARIANT(MODE_ARG, 512),  SPDY_CVARIANT(MODE_ARG_PRED, 256),
    SPDY_CVARIANT(MODE_ARG_PRED, 512), SPDY_CVARIANT(MODE_ROW, 256), SPDY_CVARIANT(MODE_ROW, 512),
    SPDY_CVARIANT(MODE_ROW2, 256), SPDY_CVARIANT(MODE_ROW2, 512),
};

const ClusterVariant *find_cluster_variant(int mode, int threads)
{
    for (const ClusterVariant &v : kClusterVariants)
        if (v.mode == mode && v.threads == threads) return &v;
    return nullptr;
}

// A CTA of 1024 threads leaves 64 registers per thread: not enough for 24 cells per lane.
inline int cells_per_lane_cap(int threads) { return threads >= 1024 ? (RMAX < 16 ? RMAX : 16) : RMAX; }

const FwdVariant *find_variant(int mode, int threads, int max_cpl)
{
    const int rcap = max_cpl <= 8 ? 8 : cells_per_lane_cap(threads);
    for (const FwdVariant &v : kVariants)
        if (v.mode == mode && v.threads == threads && v.rcap == rcap) return &v;
    return nullptr;
}

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

}  // namespace

// ----------------------------------------------------------------------------------------------
// Plan
// ----------------------------------------------------------------------------------------------

struct spdy_plan {
    int32_t L = 0, K = 0, B = 0;
    int device = -1;
    bool feasible = false;
    int mode = MODE_ARG;
    int threads = 256;
    int cluster = 1;
    int table_format = SPDY_TABLE_ROW_F32;
    int ctas_per_sm = 0;
    int sm_count = 148;
    int64_t smem_bytes = 0;
    int32_t row_stride = 0, pad = 0;
    bool global_rows = false;  // row buffers live in the workspace, not in shared memory
    // Byte table only: `merged` is a second plan over the same rows and passes whose slots are groups
    // of equal-time choices (ordered by their lowest member); candidates for which that is exact run
    // on it, the others on this plan (see spdy_monotone_flags_kernel).  `merge_first` marks such a
    // second plan.
    bool merge_first = false;
    spdy_plan *merged = nullptr;
    int64_t pitch = 0;  // table cells per candidate
    int64_t band_cells = 0, useful_updates = 0, distinct_updates = 0, issued_updates = 0;
    int32_t max_width = 0;
    std::vector<int32_t> times;
    std::vector<float> qtab;          // [K] squares of Eq. 4
    std::vector<LayerDesc> layers;
    std::vector<TapRange> taps;       // [L][K] by choice
    std::vector<TapRange> slots;      // [L][K] by shift slot (first layers[l].nslots valid)
    std::vector<uint8_t> slot_ptr;    // [L][K+1]
    std::vector<uint8_t> slot_member; // [L][K]
    std::vector<uint64_t> span_masks;
    std::vector<uint32_t> span_kranges;
    const FwdVariant *variant = nullptr;
    // cluster variant (cluster > 1)
    const ClusterVariant *cvariant = nullptr;
    std::vector<SliceDesc> slices;
    int32_t out_stride = 0, win_stride = 0;
    SliceDesc *d_slices = nullptr;
    // device tables (one allocation)
    unsigned char *d_blob = nullptr;
    int32_t *d_times = nullptr;
    LayerDesc *d_layers = nullptr;
    TapRange *d_slots = nullptr;
    uint8_t *d_slot_ptr = nullptr;
    uint8_t *d_slot_member = nullptr;
    unsigned long long *d_masks = nullptr;
    unsigned *d_kranges = nullptr;
    int32_t *d_status = nullptr;
    float *d_qtab = nullptr;
    // optional event timing of the last solve (three events per wave)
    bool timing = false;
    std::vector<cudaEvent_t> events;
    size_t events_used = 0;
    // host-buffer entry points: a second stream and events that let the upload of one chunk of
    // candidates overlap the kernels of the chunk before it
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t entry_event = nullptr;
    std::vector<cudaEvent_t> copy_events;
    // staging for the host-buffer entry point
    unsigned char *d_arena = nullptr;
    size_t arena_bytes = 0;
};

namespace {

// Eq. 4's squares (i / (K - 1))^2, formed in fp64 and rounded once to fp32; K = 1 gives 0.
void fill_qtab(spdy_plan *p)
{
    p->qtab.assign(p->K, 0.0f);
    for (int i = 0; i < p->K && p->K > 1; ++i) {
        const double r = static_cast<double>(i) / static_cast<double>(p->K - 1);
        p->qtab[i] = static_cast<float>(r * r);
    }
}

int64_t cell_bytes(const spdy_plan *p) { return p->table_format == SPDY_TABLE_ROW_F32 ? 4 : 1; }

// Workspace one candidate needs: its walk-back table, and its two row buffers when those live in
// global memory.  Both are multiples of 256 bytes.
int64_t table_bytes_one(const spdy_plan *p) { return std::max<int64_t>(256, round_up(p->pitch * cell_bytes(p), 256)); }
int64_t row_bytes_one(const spdy_plan *p) { return p->global_rows ? round_up(2LL * p->row_stride * 4, 256) : 0; }
// One flag byte per candidate when two table sets share the batch (kept 256-byte granular).
int64_t flag_bytes_one(const spdy_plan *p) { return p->merged ? 256 : 0; }

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

    p->layers.assign(L, LayerDesc{0, 0, 0, 0});
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

// Shift slots of every layer (see TapRange).  With `merge` the usable choices of a layer are
// grouped by time, slots in ascending time order; without it slot u is choice u.
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

// Per-layer pass shape for a CTA of `threads` threads, row offsets, table pitch and issued work.
// A layer of `width` cells is covered in `rounds` rounds of NWARPS warp passes; the cells per lane
// (cpl <= RMAX) are chosen so that the passes of a round are as full as possible, which keeps the
// warps of a CTA level at the per-layer barrier.
int layout_table(spdy_plan *p, int threads, double *efficiency)
{
    const int nwarps = threads / 32;
    const int mw = (p->K + 63) / 64;
    p->span_masks.clear();
    p->span_kranges.clear();
    int64_t off = 0, lanes_cells = 0;
    int64_t max_extent = 0, max_cpl = 1;
    p->issued_updates = 0;
    for (int l = 0; l < p->L; ++l) {
        LayerDesc &ld = p->layers[l];
        if (off > 0xffffffffLL) return SPDY_ERR_UNSUPPORTED;
        ld.rowoff = static_cast<uint32_t>(off);
        const int64_t width = ld.width;
        const int64_t rmax = cells_per_lane_cap(threads);
        const int64_t per_round = 32LL * nwarps * rmax;
        const int64_t rounds = std::max<int64_t>(1, (width + per_round - 1) / per_round);
        int64_t cpl = (width + 32LL * nwarps * rounds - 1) / (32LL * nwarps * rounds);
        cpl = std::min<int64_t>(rmax, std::max<int64_t>(1, cpl));
        const int64_t span = 32 * cpl;
        const int64_t nspans = (width + span - 1) / span;
        ld.cpl = static_cast<int32_t>(cpl);
        ld.nspans = static_cast<int32_t>(nspans);
        max_cpl = std::max(max_cpl, cpl);
        max_extent = std::max(max_extent, nspans * span);
        off += round_up(nspans * span, 128);
        lanes_cells += ((nspans + nwarps - 1) / nwarps) * nwarps * span;
        ld.mask_off = static_cast<int32_t>(p->span_masks.size() / mw);
        for (int64_t sp = 0; sp < nspans; ++sp) {
            const int64_t s = sp * span;
            uint64_t words[4] = {0, 0, 0, 0};
            for (int k = 0; k < ld.nslots; ++k) {
                const TapRange tr = p->slots[static_cast<size_t>(l) * p->K + k];
                if (tr.b >= tr.a && s + span > tr.a && s <= tr.b) {
                    words[k >> 6] |= 1ULL << (k & 63);
                    p->issued_updates += span;
                }
            }
            for (int w = 0; w < mw; ++w) p->span_masks.push_back(words[w]);
            int k_lo = 0, k_hi = 0, count = 0;
            for (int k = 0; k < ld.nslots; ++k) {
                if (words[k >> 6] >> (k & 63) & 1) {
                    if (count == 0) k_lo = k;
                    k_hi = k + 1;
                    ++count;
                }
            }
            const uint32_t dense = (count == k_hi - k_lo) ? 1u : 0u;
            p->span_kranges.push_back(static_cast<uint32_t>(k_lo) | static_cast<uint32_t>(k_hi) << 8 | dense << 16);
        }
    }
    p->pitch = off;
    p->pad = static_cast<int32_t>(32 * max_cpl);
    p->row_stride = static_cast<int32_t>(round_up(max_extent, 32) + 2 * p->pad);
    p->smem_bytes = 2LL * p->row_stride * 4 + 2LL * ((p->K + 1) & ~1) * 8;
    if (efficiency) *efficiency = lanes_cells > 0 ? static_cast<double>(p->band_cells) / lanes_cells : 0.0;
    return SPDY_OK;
}

// Pass shapes when C CTAs share a candidate: every row is cut into C slices of equal length (a
// multiple of 32 cells); see the cluster kernel for the data flow.
int layout_cluster(spdy_plan *p, int threads, int C)
{
    const int nwarps = threads / 32;
    const int mw = (p->K + 63) / 64;
    p->span_masks.clear();
    p->span_kranges.clear();
    p->slices.assign(static_cast<size_t>(p->L) * C, SliceDesc{});
    p->issued_updates = 0;
    int64_t off = 0, max_slice = 32, max_win = 32, prev_slice = 1;
    for (int l = 0; l < p->L; ++l) {
        LayerDesc &ld = p->layers[l];
        if (off > 0xffffffffLL) return SPDY_ERR_UNSUPPORTED;
        ld.rowoff = static_cast<uint32_t>(off);
        ld.cpl = 0;
        ld.nspans = 0;
        ld.mask_off = 0;
        const int64_t width = ld.width;
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
                const int64_t per_round = 32LL * nwarps * RMAX;
                const int64_t rounds = (ws + per_round - 1) / per_round;
                cpl = (ws + 32LL * nwarps * rounds - 1) / (32LL * nwarps * rounds);
                cpl = std::min<int64_t>(RMAX, std::max<int64_t>(1, cpl));
                nspans = (ws + 32 * cpl - 1) / (32 * cpl);
            }
            const int64_t span = 32 * cpl;
            sd.slice_lo = static_cast<int32_t>(lo);
            sd.slice_hi = static_cast<int32_t>(hi);
            sd.cpl = static_cast<int32_t>(cpl);
            sd.nspans = static_cast<int32_t>(nspans);
            sd.mask_off = static_cast<int32_t>(p->span_masks.size() / mw);
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
                for (int w = 0; w < mw; ++w) p->span_masks.push_back(words[w]);
                const uint32_t dense = (count == k_hi - k_lo) ? 1u : 0u;
                p->span_kranges.push_back(static_cast<uint32_t>(k_lo) | static_cast<uint32_t>(k_hi) << 8 | dense << 16);
            }
        }
        prev_slice = slice;
    }
    p->pitch = off;
    p->out_stride = static_cast<int32_t>(round_up(max_slice, 32));
    p->win_stride = static_cast<int32_t>(round_up(max_win, 32));
    p->row_stride = 0;
    p->smem_bytes = (2LL * p->out_stride + p->win_stride) * 4 + 2LL * ((p->K + 1) & ~1) * 8;
    return SPDY_OK;
}

int choose_cluster_shape(spdy_plan *p, const spdy_options *opts, int64_t smem_per_block)
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
            if (p->smem_bytes > smem_per_block) continue;
            // Narrow slices do not fill 16 warps; prefer the smaller CTA then.
            if (threads == 512 && !(opts && opts->threads) && p->out_stride < 32 * 16 * 4) continue;
            p->cluster = C;
            p->threads = threads;
            p->cvariant = find_cluster_variant(p->mode, threads);
            if (!p->cvariant) return SPDY_ERR_INVALID_ARG;
            p->ctas_per_sm = 1;
            if (p->device >= 0) {
                // The limit belongs to the kernel on the device, not to this plan: always the device's
                // opt-in maximum, so that plans of different widths can live side by side.
                cudaFuncAttributes fattr;
                SPDY_CUDA_TRY(cudaFuncGetAttributes(&fattr, p->cvariant->fn));
                SPDY_CUDA_TRY(cudaFuncSetAttribute(p->cvariant->fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   static_cast<int>(smem_per_block - static_cast<int64_t>(fattr.sharedSizeBytes))));
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(static_cast<unsigned>(C), 1, 1);
                cfg.blockDim = dim3(static_cast<unsigned>(threads), 1, 1);
                cfg.dynamicSmemBytes = static_cast<size_t>(p->smem_bytes);
                cudaLaunchAttribute attr;
                attr.id = cudaLaunchAttributeClusterDimension;
                attr.val.clusterDim.x = static_cast<unsigned>(C);
                attr.val.clusterDim.y = 1;
                attr.val.clusterDim.z = 1;
                cfg.attrs = &attr;
                cfg.numAttrs = 1;
                int clusters = 0;
                SPDY_CUDA_TRY(cudaOccupancyMaxActiveClusters(&clusters, p->cvariant->fn, &cfg));
                if (clusters < 1) continue;
                p->ctas_per_sm = std::max(1, clusters * C / std::max(1, p->sm_count));
            }
            return SPDY_OK;
        }
    }
    return requested ? SPDY_ERR_INVALID_ARG : SPDY_ERR_UNSUPPORTED;
}

// Wide-band fallback: one CTA of 1024 threads per candidate, row buffers in the workspace.
int choose_global_row_shape(spdy_plan *p)
{
    const int threads = 1024;
    if (threads < p->K) return SPDY_ERR_UNSUPPORTED;
    p->mode = p->table_format == SPDY_TABLE_ARG_U8 ? MODE_ARG_PRED : MODE_ROW2;
    p->cluster = 1;
    p->cvariant = nullptr;
    p->slices.clear();
    int rc = layout_table(p, threads, nullptr);
    if (rc != SPDY_OK) return rc;
    p->global_rows = true;
    p->smem_bytes = 2LL * ((p->K + 1) & ~1) * 8;
    p->threads = threads;
    p->variant = nullptr;
    for (const FwdVariant &v : kGlobalRowVariants)
        if (v.mode == p->mode) p->variant = &v;
    if (!p->variant) return SPDY_ERR_INVALID_ARG;
    p->ctas_per_sm = 1;
    return SPDY_OK;
}

int choose_launch_shape(spdy_plan *p, const spdy_options *opts)
{
    int64_t smem_per_sm = 233472, smem_per_block = 232448;
    p->sm_count = 148;
    if (p->device >= 0) {
        int v = 0;
        SPDY_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, p->device));
        smem_per_sm = v;
        SPDY_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, p->device));
        smem_per_block = v;
        SPDY_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, p->device));
        p->sm_count = v;
    }
    p->table_format = (opts && opts->table_format) ? opts->table_format : SPDY_TABLE_ROW_F32;
    if (p->table_format != SPDY_TABLE_ARG_U8 && p->table_format != SPDY_TABLE_ROW_F32)
        return SPDY_ERR_INVALID_ARG;
    p->mode = p->table_format == SPDY_TABLE_ARG_U8 ? MODE_ARG_PRED : MODE_ROW2;
    if (opts && opts->forward_mode) {
        p->mode = opts->forward_mode;
        const bool row_mode = p->mode == MODE_ROW || p->mode == MODE_ROW2;
        const bool arg_mode = p->mode == MODE_ARG || p->mode == MODE_ARG_PRED;
        if (!(row_mode || arg_mode)) return SPDY_ERR_INVALID_ARG;
        if (row_mode != (p->table_format == SPDY_TABLE_ROW_F32)) return SPDY_ERR_INVALID_ARG;
    }
    build_slots(p, (p->mode == MODE_ROW || p->mode == MODE_ROW2) ? 1 : (p->merge_first ? 2 : 0));
    p->cluster = 1;
    if (opts && opts->cluster != 0 && opts->cluster != 1 && opts->cluster != 2 && opts->cluster != 4 &&
        opts->cluster != 8)
        return SPDY_ERR_INVALID_ARG;
    p->global_rows = false;
    if (opts && opts->rows_in_global != 0 && opts->rows_in_global != 1) return SPDY_ERR_INVALID_ARG;
    if (opts && opts->rows_in_global) {
        if (opts->cluster > 1) return SPDY_ERR_INVALID_ARG;
        return choose_global_row_shape(p);
    }
    if (opts && opts->cluster > 1) return choose_cluster_shape(p, opts, smem_per_block);

    // Candidate CTA sizes; keep the one whose rounds are fullest, preferring more resident warps.
    const int sizes[] = {128, 256, 512, 1024};
    int best_threads = 0;
    double best_score = -1.0;
    for (int threads : sizes) {
        if (opts && opts->threads && opts->threads != threads) continue;
        if (threads < p->K) continue;  // one thread per choice stages the next layer
        double eff = 0.0;
        int rc = layout_table(p, threads, &eff);
        if (rc != SPDY_OK) return rc;
        if (p->smem_bytes > smem_per_block) continue;
        const int64_t by_smem = std::max<int64_t>(1, smem_per_sm / (p->smem_bytes + 1024));
        const int64_t ctas = std::min<int64_t>(std::min<int64_t>(by_smem, 2048 / threads), 32);
        const double warps = static_cast<double>(ctas * threads / 32);
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
        if (opts && ((opts->threads && opts->threads != 1024) || opts->forward_mode))
            return choose_cluster_shape(p, opts, smem_per_block);
        return choose_global_row_shape(p);
    }
    int rc = layout_table(p, best_threads, nullptr);
    if (rc != SPDY_OK) return rc;
    p->threads = best_threads;
    p->variant = find_variant(p->mode, best_threads, p->pad / 32);
    if (!p->variant) return SPDY_ERR_INVALID_ARG;
    const int64_t by_smem = std::max<int64_t>(1, smem_per_sm / (p->smem_bytes + 1024));
    p->ctas_per_sm = static_cast<int>(std::min<int64_t>(by_smem, 2048 / best_threads));
    if (p->device >= 0) {
        // The limit belongs to the kernel on the device, not to this plan: always the device's opt-in
        // maximum less the kernel's static shared memory (every plan writes the same value), so that plans of different widths can live side by side.
        cudaFuncAttributes fattr;
        SPDY_CUDA_TRY(cudaFuncGetAttributes(&fattr, p->variant->fn));
        SPDY_CUDA_TRY(cudaFuncSetAttribute(p->variant->fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(smem_per_block - static_cast<int64_t>(fattr.sharedSizeBytes))));
        int occ = 0;
        SPDY_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, p->variant->fn, best_threads,
                                                                    static_cast<size_t>(p->smem_bytes)));
        if (occ < 1) return SPDY_ERR_UNSUPPORTED;
        p->ctas_per_sm = occ;
    }
    return SPDY_OK;
}

// Where each device table sits inside one 256-byte aligned block of `total` bytes.
struct TableLayout {
    size_t times = 0, layers = 0, slots = 0, slot_ptr = 0, slot_member = 0, masks = 0, kranges = 0,
           status = 0, slices = 0, qtab = 0, total = 0;
};

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
    t.masks = take(p->span_masks.size() * sizeof(uint64_t));
    t.kranges = take(p->span_kranges.size() * sizeof(uint32_t));
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
    put(t.masks, p->span_masks.data(), p->span_masks.size() * sizeof(uint64_t));
    put(t.kranges, p->span_kranges.data(), p->span_kranges.size() * sizeof(uint32_t));
    put(t.slices, p->slices.data(), p->slices.size() * sizeof(SliceDesc));
    put(t.qtab, p->qtab.data(), p->qtab.size() * sizeof(float));
}

void bind_tables(spdy_plan *p, const TableLayout &t, unsigned char *base)
{
    p->d_times = reinterpret_cast<int32_t *>(base + t.times);
    p->d_layers = reinterpret_cast<LayerDesc *>(base + t.layers);
    p->d_slots = reinterpret_cast<TapRange *>(base + t.slots);
    p->d_slot_ptr = base + t.slot_ptr;
    p->d_slot_member = base + t.slot_member;
    p->d_masks = reinterpret_cast<unsigned long long *>(base + t.masks);
    p->d_kranges = reinterpret_cast<unsigned *>(base + t.kranges);
    p->d_status = reinterpret_cast<int32_t *>(base + t.status);
    p->d_slices = reinterpret_cast<SliceDesc *>(base + t.slices);
    p->d_qtab = reinterpret_cast<float *>(base + t.qtab);
}

int upload_tables(spdy_plan *p)
{
    const TableLayout t = table_layout(p);
    std::vector<unsigned char> host;
    pack_tables(p, t, host);
    cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&p->d_blob), t.total);
    if (err != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(err);
        p->d_blob = nullptr;
        return err == cudaErrorMemoryAllocation ? SPDY_ERR_NO_MEMORY : SPDY_ERR_CUDA;
    }
    SPDY_CUDA_TRY(cudaMemcpy(p->d_blob, host.data(), t.total, cudaMemcpyHostToDevice));
    bind_tables(p, t, p->d_blob);
    return SPDY_OK;
}

struct DeviceGuard {
    int saved = -1;
    bool active = false;
    int enter(int device)
    {
        SPDY_CUDA_TRY(cudaGetDevice(&saved));
        if (saved != device) {
            SPDY_CUDA_TRY(cudaSetDevice(device));
            active = true;
        }
        return SPDY_OK;
    }
    ~DeviceGuard()
    {
        if (active) cudaSetDevice(saved);
    }
};

}  // namespace

extern "C" {

int spdy_version(void) { return 1005; }

int spdy_last_cuda_error(void) { return g_last_cuda_error; }

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
        default: return "unknown status";
    }
}

}  // extern "C"

namespace {

int create_plan(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B, int device,
                const spdy_options *opts, bool merge_first)
{
    if (!out) return SPDY_ERR_INVALID_ARG;
    *out = nullptr;
    if (!times_host || L < 1 || K < 1 || K > 255 || B < 0 || device < -1) return SPDY_ERR_INVALID_ARG;
    if (opts) {
        for (int i = 0; i < 3; ++i)
            if (opts->reserved[i] != 0) return SPDY_ERR_INVALID_ARG;
        if (opts->threads != 0 && (opts->threads % 32 != 0 || opts->threads < 32 || opts->threads > 1024))
            return SPDY_ERR_INVALID_ARG;
    }
    spdy_plan *p = new (std::nothrow) spdy_plan();
    if (!p) return SPDY_ERR_NO_MEMORY;
    p->L = L;
    p->K = K;
    p->B = B;
    p->device = device;
    p->merge_first = merge_first;
    int rc = SPDY_OK;
    try {
        p->times.assign(times_host, times_host + static_cast<size_t>(L) * K);
        fill_qtab(p);
        rc = build_bands(p);
        DeviceGuard guard;
        if (rc == SPDY_OK && device >= 0) rc = guard.enter(device);
        if (rc == SPDY_OK) rc = choose_launch_shape(p, opts);
        if (rc == SPDY_OK && device >= 0) rc = upload_tables(p);
    } catch (const std::bad_alloc &) {
        rc = SPDY_ERR_NO_MEMORY;
    }
    if (rc != SPDY_OK) {
        spdy_plan_destroy(p);
        return rc;
    }
    *out = p;
    return SPDY_OK;
}

}  // namespace

extern "C" {

int spdy_plan_create(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B,
                     int device, const spdy_options *opts)
{
    int rc = create_plan(out, times_host, L, K, B, device, opts, false);
    if (rc != SPDY_OK) return rc;
    spdy_plan *p = *out;
    // Byte table, one CTA per candidate: add the second plan with merged equal-time choices when
    // merging removes any work.  It must lay out rows, passes and table exactly like the first.
    if (p->table_format == SPDY_TABLE_ARG_U8 && p->cluster == 1 && p->feasible) {
        spdy_options o = {};
        if (opts) o = *opts;
        o.table_format = SPDY_TABLE_ARG_U8;
        o.threads = p->threads;
        o.cluster = 1;
        o.forward_mode = p->mode;
        o.rows_in_global = p->global_rows ? 1 : 0;
        spdy_plan *m = nullptr;
        if (create_plan(&m, times_host, L, K, B, device, &o, true) == SPDY_OK) {
            const bool same_shape = m->pitch == p->pitch && m->row_stride == p->row_stride && m->pad == p->pad &&
                                    m->threads == p->threads && m->smem_bytes == p->smem_bytes &&
                                    m->global_rows == p->global_rows && m->variant == p->variant;
            if (same_shape && m->distinct_updates < p->distinct_updates) p->merged = m;
            else spdy_plan_destroy(m);
        }
    }
    return SPDY_OK;
}

void spdy_plan_destroy(spdy_plan *plan)
{
    if (!plan) return;
    if (plan->merged) spdy_plan_destroy(plan->merged);
    plan->merged = nullptr;
    if (plan->d_blob || plan->d_arena) {
        DeviceGuard guard;
        guard.enter(plan->device);
        if (plan->d_blob) cudaFree(plan->d_blob);
        if (plan->d_arena) cudaFree(plan->d_arena);
        for (cudaEvent_t e : plan->events) cudaEventDestroy(e);
        for (cudaEvent_t e : plan->copy_events) cudaEventDestroy(e);
        if (plan->entry_event) cudaEventDestroy(plan->entry_event);
        if (plan->copy_stream) cudaStreamDestroy(plan->copy_stream);
    }
    delete plan;
}

int spdy_plan_get_info(const spdy_plan *plan, spdy_plan_info *info)
{
    if (!plan || !info) return SPDY_ERR_INVALID_ARG;
    std::memset(info, 0, sizeof(*info));
    info->L = plan->L;
    info->K = plan->K;
    info->B = plan->B;
    info->feasible = plan->feasible ? 1 : 0;
    info->max_width = plan->max_width;
    info->span = 32 * RMAX;
    info->threads = plan->threads;
    info->cluster = plan->cluster;
    info->table_format = plan->table_format;
    info->ctas_per_sm = plan->ctas_per_sm;
    info->sm_count = plan->sm_count;
    info->rows_in_global = plan->global_rows ? 1 : 0;
    info->smem_bytes = plan->smem_bytes;
    info->table_bytes_per_candidate = static_cast<int64_t>(spdy_workspace_bytes(plan, 1));
    info->band_cells = plan->band_cells;
    info->useful_updates = plan->useful_updates;
    info->issued_updates = plan->issued_updates;
    info->distinct_updates = plan->merged ? plan->merged->distinct_updates : plan->distinct_updates;
    if (plan->merged) info->issued_updates = plan->merged->issued_updates;
    info->launches_per_wave = plan->merged ? 5 : 2;
    info->nominal_updates = static_cast<int64_t>(plan->L) * plan->K * plan->B;
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
    return static_cast<size_t>(table_bytes_one(plan) + row_bytes_one(plan) + flag_bytes_one(plan)) * static_cast<size_t>(N);
}

}  // extern "C"

namespace {

// The whole path for one batch; exactly one of errors_dev / coeffs_dev is non-null.
// phases: bit 0 = forward pass (and final minimum), bit 1 = walk back; the host-buffer path runs them
// separately so that one walk back serves several forward launches into one table.
int solve_impl(const spdy_plan *plan, const float *errors_dev, const float *coeffs_dev, int64_t N,
               uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev, void *workspace_dev,
               size_t workspace_bytes, void *cuda_stream, bool keep_timing = false, int phases = 3)
{
    if (!plan || plan->device < 0 || N < 0) return SPDY_ERR_INVALID_ARG;
    if (N == 0) return SPDY_OK;
    const float *input = errors_dev ? errors_dev : coeffs_dev;
    if (!input || !profile_dev || !cost_dev || !time_used_dev) return SPDY_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(input) % 4 != 0) return SPDY_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;

    if (!plan->feasible) {
        const int blocks = static_cast<int>(std::min<int64_t>((N + 255) / 256, 65535));
        spdy_fill_infeasible_kernel<<<blocks, 256, 0, stream>>>(profile_dev, cost_dev, time_used_dev, N, plan->L);
        SPDY_CUDA_TRY(cudaGetLastError());
        return SPDY_OK;
    }
    if (!workspace_dev || reinterpret_cast<uintptr_t>(workspace_dev) % 256 != 0) return SPDY_ERR_INVALID_ARG;
    const size_t per = spdy_workspace_bytes(plan, 1);
    const int64_t wave = static_cast<int64_t>(std::min<size_t>(workspace_bytes / per, static_cast<size_t>(N)));
    if (wave < 1) return SPDY_ERR_WORKSPACE_TOO_SMALL;
    // The table pitch handed to the kernels is in cells; every candidate's table is 256-byte aligned.
    const int64_t pitch_cells = table_bytes_one(plan) / cell_bytes(plan);
    // Row buffers in global memory (wide-band fallback) follow the tables of the wave.
    float *grows = plan->global_rows
                       ? reinterpret_cast<float *>(static_cast<unsigned char *>(workspace_dev) + wave * table_bytes_one(plan))
                       : nullptr;

    spdy_plan *mplan = const_cast<spdy_plan *>(plan);  // timing state only
    if (plan->timing && !keep_timing) mplan->events_used = 0;
    for (int64_t first = 0; first < N; first += wave) {
        const int64_t count = std::min<int64_t>(wave, N - first);
        cudaEvent_t *ev = nullptr;
        if (plan->timing) {
            while (mplan->events.size() < mplan->events_used + 3) {
                cudaEvent_t e;
                SPDY_CUDA_TRY(cudaEventCreate(&e));
                mplan->events.push_back(e);
            }
            ev = &mplan->events[mplan->events_used];
            mplan->events_used += 3;
            SPDY_CUDA_TRY(cudaEventRecord(ev[0], stream));
        }
        // With a second (merged) table set every candidate of the wave gets a flag saying which set is
        // exact for it; both sets are then launched over the whole wave and every CTA / walk-back thread
        // runs only if its candidate carries the set's flag (the others leave at once).
        uint8_t *flags = nullptr;
        if (plan->merged) flags = static_cast<unsigned char *>(workspace_dev) + wave * (table_bytes_one(plan) + row_bytes_one(plan));
        if (plan->merged && (phases & 1)) {
            const spdy_plan *m = plan->merged;
            const int bt = 128;
            spdy_monotone_flags_kernel<<<static_cast<unsigned>((count * 32 + bt - 1) / bt), bt, 0, stream>>>(
                errors_dev, coeffs_dev, m->d_qtab, m->d_layers, m->d_slot_ptr, m->d_slot_member, flags, first, count,
                plan->L, plan->K);
            SPDY_CUDA_TRY(cudaGetLastError());
        }
        auto forward = [&](const spdy_plan *tp, int which) -> int {
            FwdArgs fa;
            fa.errors = errors_dev;
            fa.coeffs = coeffs_dev;
            fa.qtab = tp->d_qtab;
            fa.slots = tp->d_slots;
            fa.slot_ptr = tp->d_slot_ptr;
            fa.slot_member = tp->d_slot_member;
            fa.layers = tp->d_layers;
            fa.span_masks = tp->d_masks;
            fa.span_kranges = tp->d_kranges;
            fa.table = workspace_dev;
            fa.cost = cost_dev;
            fa.time_used = time_used_dev;
            fa.pitch = pitch_cells;
            fa.n_first = first;
            fa.L = tp->L;
            fa.K = tp->K;
            fa.row_stride = tp->row_stride;
            fa.pad = tp->pad;
            fa.grows = grows;
            fa.cand_flags = flags;
            fa.which = which;
            // Grid x is limited to 2^31-1 CTAs, far above any wave that fits in memory.
            if (tp->cluster > 1) {
                ClusterArgs ca;
                ca.f = fa;
                ca.slices = tp->d_slices;
                ca.C = tp->cluster;
                ca.out_stride = tp->out_stride;
                ca.win_stride = tp->win_stride;
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(static_cast<unsigned>(count * tp->cluster), 1, 1);
                cfg.blockDim = dim3(static_cast<unsigned>(tp->threads), 1, 1);
                cfg.dynamicSmemBytes = static_cast<size_t>(tp->smem_bytes);
                cfg.stream = stream;
                cudaLaunchAttribute attr;
                attr.id = cudaLaunchAttributeClusterDimension;
                attr.val.clusterDim.x = static_cast<unsigned>(tp->cluster);
                attr.val.clusterDim.y = 1;
                attr.val.clusterDim.z = 1;
                cfg.attrs = &attr;
                cfg.numAttrs = 1;
                SPDY_CUDA_TRY(cudaLaunchKernelEx(&cfg, tp->cvariant->fn, ca));
            } else {
                tp->variant->fn<<<static_cast<unsigned>(count), tp->threads, static_cast<size_t>(tp->smem_bytes), stream>>>(fa);
            }
            SPDY_CUDA_TRY(cudaGetLastError());
            return SPDY_OK;
        };
        auto walk_back = [&](const spdy_plan *tp, int which) -> int {
            BackArgs ba;
            ba.errors = errors_dev;
            ba.coeffs = coeffs_dev;
            ba.qtab = tp->d_qtab;
            ba.times = tp->d_times;
            ba.layers = tp->d_layers;
            ba.table = workspace_dev;
            ba.cost = cost_dev;
            ba.time_used = time_used_dev;
            ba.profile = profile_dev;
            ba.status = plan->d_status;  // one self-check word per public plan
            ba.pitch = pitch_cells;
            ba.n_first = first;
            ba.n_count = count;
            ba.L = tp->L;
            ba.K = tp->K;
            ba.cand_flags = flags;
            ba.which = which;
            ba.slot_ptr = tp->merge_first ? tp->d_slot_ptr : nullptr;
            ba.slot_member = tp->merge_first ? tp->d_slot_member : nullptr;
            if (tp->table_format == SPDY_TABLE_ARG_U8) {
                const int bt = 64;
                spdy_backtrack_arg_kernel<<<static_cast<unsigned>((count + bt - 1) / bt), bt, 0, stream>>>(ba);
            } else {
                const int bt = 128;  // 4 warps = 4 candidates per CTA
                spdy_backtrack_row_kernel<<<static_cast<unsigned>((count * 32 + bt - 1) / bt), bt, 0, stream>>>(ba);
            }
            SPDY_CUDA_TRY(cudaGetLastError());
            return SPDY_OK;
        };
        int lrc = SPDY_OK;
        if (phases & 1) {
            if (plan->merged) lrc = forward(plan->merged, 1);
            if (lrc == SPDY_OK) lrc = forward(plan, 0);
            if (lrc != SPDY_OK) return lrc;
        }
        if (ev) SPDY_CUDA_TRY(cudaEventRecord(ev[1], stream));
        if (phases & 2) {
            if (plan->merged) lrc = walk_back(plan->merged, 1);
            if (lrc == SPDY_OK) lrc = walk_back(plan, 0);
            if (lrc != SPDY_OK) return lrc;
        }
        if (ev) SPDY_CUDA_TRY(cudaEventRecord(ev[2], stream));
    }
    return SPDY_OK;
}

}  // namespace

extern "C" {

int spdy_solve_batch(const spdy_plan *plan, const float *errors_dev, int64_t N,
                     uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev,
                     void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    if (!errors_dev && N > 0) return SPDY_ERR_INVALID_ARG;
    return solve_impl(plan, errors_dev, nullptr, N, profile_dev, cost_dev, time_used_dev, workspace_dev,
                      workspace_bytes, cuda_stream);
}

int spdy_solve_batch_coeffs(const spdy_plan *plan, const float *coeffs_dev, int64_t N,
                            uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev,
                            void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    if (!coeffs_dev && N > 0) return SPDY_ERR_INVALID_ARG;
    return solve_impl(plan, nullptr, coeffs_dev, N, profile_dev, cost_dev, time_used_dev, workspace_dev,
                      workspace_bytes, cuda_stream);
}

int spdy_plan_enable_timing(spdy_plan *plan, int on)
{
    if (!plan || plan->device < 0) return SPDY_ERR_INVALID_ARG;
    plan->timing = on != 0;
    plan->events_used = 0;
    return SPDY_OK;
}

int spdy_plan_last_timing(spdy_plan *plan, float *forward_ms_host, float *walkback_ms_host)
{
    if (!plan || plan->device < 0 || !plan->timing) return SPDY_ERR_INVALID_ARG;
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;
    float fwd = 0.f, back = 0.f;
    for (size_t i = 0; i + 3 <= plan->events_used && i + 3 <= plan->events.size(); i += 3) {
        SPDY_CUDA_TRY(cudaEventSynchronize(plan->events[i + 2]));
        float a = 0.f, b = 0.f;
        SPDY_CUDA_TRY(cudaEventElapsedTime(&a, plan->events[i], plan->events[i + 1]));
        SPDY_CUDA_TRY(cudaEventElapsedTime(&b, plan->events[i + 1], plan->events[i + 2]));
        fwd += a;
        back += b;
    }
    if (forward_ms_host) *forward_ms_host = fwd;
    if (walkback_ms_host) *walkback_ms_host = back;
    return SPDY_OK;
}

int spdy_plan_check_status(spdy_plan *plan, void *cuda_stream)
{
    if (!plan || plan->device < 0) return SPDY_ERR_INVALID_ARG;
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;
    int32_t word = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    SPDY_CUDA_TRY(cudaMemcpyAsync(&word, plan->d_status, sizeof(word), cudaMemcpyDeviceToHost, stream));
    SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
    if (word != 0) {
        SPDY_CUDA_TRY(cudaMemsetAsync(plan->d_status, 0, sizeof(word), stream));
        SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
        return SPDY_ERR_INTERNAL;
    }
    return SPDY_OK;
}

}  // extern "C"

namespace {

// Host-buffer form of the path: the input is an error table ([N][L][K]) or, with `coeffs`, Eq. 4's
// coefficients ([N][L]).
int solve_host_impl(spdy_plan *plan, const float *errors_host, bool coeffs, int64_t N,
                    uint8_t *profile_host, float *cost_host, int32_t *time_used_host, void *cuda_stream)
{
    if (!plan || plan->device < 0 || N < 0) return SPDY_ERR_INVALID_ARG;
    if (N == 0) return SPDY_OK;
    if (!errors_host || !profile_host || !cost_host || !time_used_host) return SPDY_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;

    const size_t err_bytes = static_cast<size_t>(N) * plan->L * (coeffs ? 1 : plan->K) * sizeof(float);
    const size_t off_profile = round_up(err_bytes, 256);
    const size_t off_cost = off_profile + round_up(static_cast<size_t>(N) * plan->L, 256);
    const size_t off_time = off_cost + round_up(static_cast<size_t>(N) * 4, 256);
    const size_t off_ws = off_time + round_up(static_cast<size_t>(N) * 4, 256);
    // Cap the table at 8 GiB; larger batches run as waves.
    const size_t ws_full = plan->feasible ? spdy_workspace_bytes(plan, N) : 0;
    const size_t ws_one = plan->feasible ? spdy_workspace_bytes(plan, 1) : 0;
    const size_t ws_cap = std::max<size_t>(ws_one, static_cast<size_t>(8) << 30);
    const size_t ws_bytes = std::min(ws_full, ws_cap) / std::max<size_t>(ws_one, 1) * ws_one;
    const size_t total = off_ws + ws_bytes;
    if (total > plan->arena_bytes) {
        if (plan->d_arena) {
            SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
            SPDY_CUDA_TRY(cudaFree(plan->d_arena));
            plan->d_arena = nullptr;
            plan->arena_bytes = 0;
        }
        cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&plan->d_arena), total);
        if (err != cudaSuccess) {
            g_last_cuda_error = static_cast<int>(err);
            plan->d_arena = nullptr;
            return err == cudaErrorMemoryAllocation ? SPDY_ERR_NO_MEMORY : SPDY_ERR_CUDA;
        }
        plan->arena_bytes = total;
    }
    unsigned char *base = plan->d_arena;
    float *d_err = reinterpret_cast<float *>(base);
    uint8_t *d_profile = base + off_profile;
    float *d_cost = reinterpret_cast<float *>(base + off_cost);
    int32_t *d_time = reinterpret_cast<int32_t *>(base + off_time);
    // An error table goes up in chunks of growing size (one full wave of CTAs first, then six times
    // the previous chunk) on a second stream, so that every upload but the first hides behind the
    // kernels of the chunk before it; an upload takes about a seventh of the time its candidates take
    // to solve.  Every chunk boundary costs a launch tail (and a walk back, unless one serves all), so
    // chunks are few - one wave, then the rest, measured best at the BERT-base shape - and coefficient
    // input (K times smaller) goes up in one piece.
    // Everything from the first queued copy on runs inside `enqueue`: whatever makes it stop early, the
    // copies already queued still read the caller's host buffer, so every exit below waits for both
    // streams before the error goes back to the caller (who may free or reuse the buffer on seeing it).
    auto enqueue = [&]() -> int {
        const int64_t per_cand = static_cast<int64_t>(plan->L) * (coeffs ? 1 : plan->K);
        std::vector<int64_t> bounds(1, 0);
        {
            int64_t size = std::max<int64_t>(1, static_cast<int64_t>(plan->ctas_per_sm) * plan->sm_count / std::max(1, plan->cluster));
            if (coeffs) size = N;
            while (bounds.back() < N) {
                bounds.push_back(std::min<int64_t>(N, bounds.back() + size));
                size *= 6;
            }
        }
        const size_t chunks = bounds.size() - 1;
        if (chunks > 1) {
            if (!plan->copy_stream) SPDY_CUDA_TRY(cudaStreamCreateWithFlags(&plan->copy_stream, cudaStreamNonBlocking));
            if (!plan->entry_event) SPDY_CUDA_TRY(cudaEventCreateWithFlags(&plan->entry_event, cudaEventDisableTiming));
            while (plan->copy_events.size() < chunks) {
                cudaEvent_t e;
                SPDY_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
                plan->copy_events.push_back(e);
            }
            // Work already queued on the caller's stream may still read the staging buffer.
            SPDY_CUDA_TRY(cudaEventRecord(plan->entry_event, stream));
            SPDY_CUDA_TRY(cudaStreamWaitEvent(plan->copy_stream, plan->entry_event, 0));
            for (size_t c = 0; c < chunks; ++c) {
                const int64_t first = bounds[c], count = bounds[c + 1] - bounds[c];
                SPDY_CUDA_TRY(cudaMemcpyAsync(d_err + first * per_cand, errors_host + first * per_cand,
                                              static_cast<size_t>(count * per_cand) * sizeof(float),
                                              cudaMemcpyHostToDevice, plan->copy_stream));
                SPDY_CUDA_TRY(cudaEventRecord(plan->copy_events[c], plan->copy_stream));
            }
        } else {
            SPDY_CUDA_TRY(cudaMemcpyAsync(d_err, errors_host, err_bytes, cudaMemcpyHostToDevice, stream));
        }
        // When the whole batch's table fits the staging workspace (and nothing but tables lives there),
        // the chunks' forward passes write disjoint parts of it and ONE walk back follows: the walk back
        // is a latency chain of L steps whatever the number of candidates.
        const bool one_walk_back = chunks > 1 && plan->feasible && !plan->merged && !plan->global_rows &&
                                   ws_bytes >= ws_one * static_cast<size_t>(N);
        for (size_t c = 0; c < chunks; ++c) {
            const int64_t first = bounds[c], count = bounds[c + 1] - bounds[c];
            if (chunks > 1) SPDY_CUDA_TRY(cudaStreamWaitEvent(stream, plan->copy_events[c], 0));
            const float *in = d_err + first * per_cand;
            if (one_walk_back)
                rc = solve_impl(plan, coeffs ? nullptr : in, coeffs ? in : nullptr, count, d_profile + first * plan->L,
                                d_cost + first, d_time + first, base + off_ws + static_cast<size_t>(first) * ws_one,
                                static_cast<size_t>(count) * ws_one, stream, c > 0, 1);
            else
                rc = solve_impl(plan, coeffs ? nullptr : in, coeffs ? in : nullptr, count, d_profile + first * plan->L,
                                d_cost + first, d_time + first, base + off_ws, ws_bytes, stream, c > 0);
            if (rc != SPDY_OK) return rc;
        }
        if (one_walk_back) {
            rc = solve_impl(plan, coeffs ? nullptr : d_err, coeffs ? d_err : nullptr, N, d_profile, d_cost, d_time,
                            base + off_ws, ws_bytes, stream, true, 2);
            if (rc != SPDY_OK) return rc;
        }
        SPDY_CUDA_TRY(cudaMemcpyAsync(profile_host, d_profile, static_cast<size_t>(N) * plan->L, cudaMemcpyDeviceToHost, stream));
        SPDY_CUDA_TRY(cudaMemcpyAsync(cost_host, d_cost, static_cast<size_t>(N) * 4, cudaMemcpyDeviceToHost, stream));
        SPDY_CUDA_TRY(cudaMemcpyAsync(time_used_host, d_time, static_cast<size_t>(N) * 4, cudaMemcpyDeviceToHost, stream));
        return SPDY_OK;
    };
    rc = enqueue();
    if (rc != SPDY_OK) {
        if (plan->copy_stream) cudaStreamSynchronize(plan->copy_stream);
        cudaStreamSynchronize(stream);
        return rc;
    }
    SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
    return SPDY_OK;
}

}  // namespace

extern "C" {

int spdy_solve_batch_host(spdy_plan *plan, const float *errors_host, int64_t N,
                          uint8_t *profile_host, float *cost_host, int32_t *time_used_host,
                          void *cuda_stream)
{
    return solve_host_impl(plan, errors_host, false, N, profile_host, cost_host, time_used_host, cuda_stream);
}

int spdy_solve_batch_coeffs_host(spdy_plan *plan, const float *coeffs_host, int64_t N,
                                 uint8_t *profile_host, float *cost_host, int32_t *time_used_host,
                                 void *cuda_stream)
{
    return solve_host_impl(plan, coeffs_host, true, N, profile_host, cost_host, time_used_host, cuda_stream);
}

int spdy_quadratic_errors(const float *coeffs_dev, int64_t N, int32_t L, int32_t K, float *errors_dev,
                          void *cuda_stream)
{
    if (N < 0 || L < 1 || K < 1) return SPDY_ERR_INVALID_ARG;
    if (N == 0) return SPDY_OK;
    if (!coeffs_dev || !errors_dev) return SPDY_ERR_INVALID_ARG;
    const int64_t total = N * L * K;
    const int blocks = static_cast<int>(std::min<int64_t>((total + 255) / 256, 148 * 16));
    spdy_quadratic_errors_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(coeffs_dev, errors_dev, total, K);
    SPDY_CUDA_TRY(cudaGetLastError());
    return SPDY_OK;
}

int spdy_probe_peaks(int device, double *lds_reads_per_s, double *cell_updates_alu_per_s)
{
    if (device < 0) return SPDY_ERR_INVALID_ARG;
    DeviceGuard guard;
    int rc = guard.enter(device);
    if (rc != SPDY_OK) return rc;
    int sms = 0;
    SPDY_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    const int ctas = sms * 8, threads = 256, iters = 20000;
    float *out = nullptr;
    cudaEvent_t ev[2] = {nullptr, nullptr};
    cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&out), static_cast<size_t>(ctas) * threads * sizeof(float));
    if (err != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(err);
        return err == cudaErrorMemoryAllocation ? SPDY_ERR_NO_MEMORY : SPDY_ERR_CUDA;
    }
    auto finish = [&](int code) {
        if (ev[0]) cudaEventDestroy(ev[0]);
        if (ev[1]) cudaEventDestroy(ev[1]);
        cudaFree(out);
        return code;
    };
    if (cudaEventCreate(&ev[0]) != cudaSuccess || cudaEventCreate(&ev[1]) != cudaSuccess) return finish(SPDY_ERR_CUDA);
    double rates[2] = {0.0, 0.0};
    for (int which = 0; which < 2; ++which) {
        float best_ms = 0.0f;
        for (int rep = 0; rep < 4; ++rep) {  // first repetition warms up
            cudaEventRecord(ev[0], nullptr);
            if (which == 0) spdy_probe_lds_kernel<<<ctas, threads>>>(out, iters);
            else spdy_probe_alu_kernel<<<ctas, threads>>>(out, iters, 0.25f, 0.5f);
            cudaEventRecord(ev[1], nullptr);
            err = cudaEventSynchronize(ev[1]);
            if (err == cudaSuccess) err = cudaGetLastError();
            if (err != cudaSuccess) {
                g_last_cuda_error = static_cast<int>(err);
                return finish(SPDY_ERR_CUDA);
            }
            float ms = 0.0f;
            cudaEventElapsedTime(&ms, ev[0], ev[1]);
            if (rep > 0 && (best_ms == 0.0f || ms < best_ms)) best_ms = ms;
        }
        // 8 reads (resp. 16 cell updates: 8 cells x 2 choices) per thread per iteration
        const double per_thread = which == 0 ? 8.0 : 16.0;
        rates[which] = per_thread * iters * static_cast<double>(ctas) * threads / (best_ms * 1e-3);
    }
    if (lds_reads_per_s) *lds_reads_per_s = rates[0];
    if (cell_updates_alu_per_s) *cell_updates_alu_per_s = rates[1];
    return finish(SPDY_OK);
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

int spdy_solve_batch_simple(const float *errors_dev, const int32_t *times_dev, int64_t N,
                            int32_t L, int32_t K, int32_t B, uint8_t *profile_dev, float *cost_dev,
                            int32_t *time_used_dev, void *cuda_stream)
{
    if (!times_dev || L < 1 || K < 1 || K > 255 || B < 0 || N < 0) return SPDY_ERR_INVALID_ARG;
    if (N == 0) return SPDY_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int device = 0;
    SPDY_CUDA_TRY(cudaGetDevice(&device));
    std::vector<int32_t> times;
    try {
        times.resize(static_cast<size_t>(L) * K);
    } catch (const std::bad_alloc &) {
        return SPDY_ERR_NO_MEMORY;
    }
    SPDY_CUDA_TRY(cudaMemcpyAsync(times.data(), times_dev, times.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
    spdy_plan *plan = nullptr;
    int rc = spdy_plan_create(&plan, times.data(), L, K, B, device, nullptr);
    if (rc != SPDY_OK) return rc;
    void *ws = nullptr;
    size_t ws_bytes = 0;
    if (plan->feasible) {
        size_t free_b = 0, total_b = 0;
        cudaError_t err = cudaMemGetInfo(&free_b, &total_b);
        const size_t one = spdy_workspace_bytes(plan, 1);
        const size_t want = spdy_workspace_bytes(plan, N);
        ws_bytes = want;
        if (err == cudaSuccess && want > free_b / 2) ws_bytes = std::max(one, (free_b / 2) / one * one);
        err = cudaMalloc(&ws, ws_bytes);
        if (err != cudaSuccess) {
            g_last_cuda_error = static_cast<int>(err);
            spdy_plan_destroy(plan);
            return err == cudaErrorMemoryAllocation ? SPDY_ERR_NO_MEMORY : SPDY_ERR_CUDA;
        }
    }
    rc = spdy_solve_batch(plan, errors_dev, N, profile_dev, cost_dev, time_used_dev, ws, ws_bytes, stream);
    cudaError_t sync_err = cudaStreamSynchronize(stream);
    if (rc == SPDY_OK && sync_err != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(sync_err);
        rc = SPDY_ERR_CUDA;
    }
    if (rc == SPDY_OK) rc = spdy_plan_check_status(plan, stream);
    if (ws) cudaFree(ws);
    spdy_plan_destroy(plan);
    return rc;
}

// ----------------------------------------------------------------------------------------------
// Entry point that performs no device allocation
// ----------------------------------------------------------------------------------------------

}  // extern "C"

namespace {

// Built-in scratch of spdy_solve_batch_static: the plan's small tables at the front, the
// walk-back table behind them.  Resident on every device that loads this library, until exit.
constexpr size_t kStaticScratchBytes = SPDY_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char *g_static_base[kMaxDevices] = {};

// Device address of g_static_scratch on the current device.  In host code the array's name is
// only a handle, never a pointer a kernel may use; the address comes from the runtime, once per
// device.
int static_scratch_address(int device, unsigned char **out)
{
    if (device < 0 || device >= kMaxDevices) return SPDY_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_base[device]) {
        void *ptr = nullptr;
        SPDY_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return SPDY_ERR_CUDA;
        g_static_base[device] = static_cast<unsigned char *>(ptr);
    }
    *out = g_static_base[device];
    return SPDY_OK;
}

}  // namespace

extern "C" {

size_t spdy_static_scratch_bytes(void) { return kStaticScratchBytes; }

int spdy_solve_batch_static(const float *errors_dev, const int32_t *times_host, int64_t N, int32_t L,
                            int32_t K, int32_t B, uint8_t *profile_dev, float *cost_dev,
                            int32_t *time_used_dev, void *cuda_stream)
{
    if (!times_host || L < 1 || K < 1 || K > 255 || B < 0 || N < 0) return SPDY_ERR_INVALID_ARG;
    if (N == 0) return SPDY_OK;
    if (!errors_dev || !profile_dev || !cost_dev || !time_used_dev) return SPDY_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int device = 0;
    SPDY_CUDA_TRY(cudaGetDevice(&device));
    unsigned char *base = nullptr;
    int rc = static_scratch_address(device, &base);
    if (rc != SPDY_OK) return rc;

    // Host-side plan (bands, pass shapes) with the one-byte table so more candidates fit a wave.
    spdy_plan *p = new (std::nothrow) spdy_plan();
    if (!p) return SPDY_ERR_NO_MEMORY;
    p->L = L;
    p->K = K;
    p->B = B;
    p->device = device;
    spdy_options opts = {};
    opts.table_format = SPDY_TABLE_ARG_U8;
    opts.cluster = 1;  // the cluster variant's wider rows would not leave room for a table anyway
    try {
        p->times.assign(times_host, times_host + static_cast<size_t>(L) * K);
        fill_qtab(p);
        rc = build_bands(p);
        if (rc == SPDY_OK) rc = choose_launch_shape(p, &opts);
    } catch (const std::bad_alloc &) {
        rc = SPDY_ERR_NO_MEMORY;
    }
    if (rc == SPDY_ERR_UNSUPPORTED) rc = SPDY_ERR_STATIC_LIMIT;
    if (rc != SPDY_OK) {
        spdy_plan_destroy(p);
        return rc;
    }

    // The plan tables go to the front of the scratch, the walk-back table behind them.
    const TableLayout tl = table_layout(p);
    const size_t off_table = tl.total;
    const size_t one = p->feasible ? spdy_workspace_bytes(p, 1) : 0;
    if (off_table + one > kStaticScratchBytes) {
        spdy_plan_destroy(p);
        return SPDY_ERR_STATIC_LIMIT;
    }
    std::vector<unsigned char> host;
    try {
        pack_tables(p, tl, host);
    } catch (const std::bad_alloc &) {
        spdy_plan_destroy(p);
        return SPDY_ERR_NO_MEMORY;
    }
    bind_tables(p, tl, base);
    // The array keeps the previous call's contents; the image below overwrites every table and
    // carries a zero self-check word, the only thing that must start at zero.
    cudaError_t err = cudaMemcpyAsync(base, host.data(), tl.total, cudaMemcpyHostToDevice, stream);
    if (err != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(err);
        cudaStreamSynchronize(stream);
        spdy_plan_destroy(p);
        return SPDY_ERR_CUDA;
    }
    const size_t table_bytes = p->feasible ? (kStaticScratchBytes - off_table) / one * one : 0;
    rc = spdy_solve_batch(p, errors_dev, N, profile_dev, cost_dev, time_used_dev, base + off_table,
                          table_bytes, stream);
    int32_t word = 0;
    if (rc == SPDY_OK) {
        err = cudaMemcpyAsync(&word, p->d_status, sizeof(word), cudaMemcpyDeviceToHost, stream);
        if (err != cudaSuccess) {
            g_last_cuda_error = static_cast<int>(err);
            rc = SPDY_ERR_CUDA;
        }
    }
    // The host tables above must outlive the copies, so wait before releasing them.
    err = cudaStreamSynchronize(stream);
    if (rc == SPDY_OK && err != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(err);
        rc = SPDY_ERR_CUDA;
    }
    if (rc == SPDY_OK && word != 0) rc = SPDY_ERR_INTERNAL;
    spdy_plan_destroy(p);  // frees host tables only: this plan owns no device memory
    return rc;
}

}  // extern "C"
