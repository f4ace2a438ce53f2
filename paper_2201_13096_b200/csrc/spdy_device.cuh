// Device code of the batched SPDY dynamic program for B200 (sm_100a): the cell updates, the warp pass,
// and the three forward kernels (one CTA, one thread-block cluster, or one warp per candidate).
//
// One candidate = one min-plus dynamic program over L layers (Section 3.2, Eq. 2-3) followed by the
// final minimum over the budget axis; the walk back of Appendix A, Algorithm 1 runs in a second kernel.
// The forward kernels keep two band-limited DP rows in shared memory (or, for very wide rows, in global
// memory) and stream one table row per layer to global memory.
//
// Bit-exactness contract: every cell value is produced by exactly one fp32 round-to-nearest add
// (previous-row value + error) and compared with strict "<" in ascending choice order, so the
// results equal a plain sequential evaluation of Algorithm 1 with Eq. 2's bucket range.
//
// Built with -DSPDY_DEBUG_CHECKS every row-buffer and table access of the forward kernels tests its index
// first: an access outside its buffer, or a read of a cell that holds neither the previous row nor +inf
// (the new row's buffer is filled with NaN before each layer), sets a bit of the plan's status word and
// is skipped - never a trap, never an early exit past a barrier.
#ifndef SPDY_DEVICE_CUH
#define SPDY_DEVICE_CUH

#include "spdy_plan.h"

#include <cooperative_groups.h>
#include <cuda_runtime.h>

namespace spdy {

// Bits of the status word.
constexpr int STATUS_WALK_BACK = 1;   // a table entry was not a valid choice, or the walk did not end at t = 0
constexpr int STATUS_READ_RANGE = 2;  // debug build: a row read outside the region known to hold the row or +inf
constexpr int STATUS_READ_STALE = 4;  // debug build: a row read returned the NaN that marks an unwritten cell
constexpr int STATUS_WRITE_RANGE = 8; // debug build: a row or table store outside its buffer

struct FwdArgs {
    const float *errors;      // [N][L][K], or null when the errors follow from coefficients
    const float *coeffs;      // [N][L] sensitivity coefficients (Eq. 4), used when errors is null
    const float *qtab;        // [K]: fp32((i / (K - 1))^2)
    const TapRange *slots;    // [L][K], the first layers[l].nslots of a layer are valid
    const uint8_t *slot_ptr;     // [L][K+1]: members of slot u are slot_member[slot_ptr[u] .. slot_ptr[u+1])
    const uint8_t *slot_member;  // [L][K]: choice indices grouped by slot
    const LayerDesc *layers;  // [L]
    const PassDesc *passes;   // warp passes grouped by (layer, warp)
    const unsigned long long *pass_masks;  // per pass: one bit per slot that overlaps it
    const int32_t *pass_ptr;  // [L * W + 1]
    void *table;              // wave-local walk-back table
    float *cost;              // [N]
    int32_t *time_used;       // [N]
    int32_t *status;          // the plan's status word
    int64_t pitch;            // table cells per candidate
    int64_t n_first;          // first candidate of this wave
    int64_t n_count;          // candidates of this wave
    int32_t L, K;
    int32_t row_stride;       // floats per row buffer
    int32_t pad;              // +inf guard cells below cell 0 of a row
    float *grows;             // row buffers in global memory (GROWS kernels), else null
    int64_t grows_stride;     // floats between the row buffers of consecutive candidates
    const uint8_t *cand_flags; // per candidate of the wave, or null: run only candidates whose flag == which
    int32_t which;
};

struct ClusterArgs {
    FwdArgs f;
    const SliceDesc *slices;  // [L][C]
    int32_t C;
    int32_t out_stride;  // floats per `out` buffer
    int32_t win_stride;  // floats of `win`
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

// What a pass may touch, for the debug build's index checks; empty otherwise.
struct AccessWindow {
#ifdef SPDY_DEBUG_CHECKS
    int read_lo, read_hi;    // previous-row cells [read_lo, read_hi) hold the row or +inf
    int write_hi;            // new-row cells [0, write_hi) may be stored
    long long table_hi;      // table cells [0, table_hi) of this row may be stored
    int32_t *status;
#endif
};

// The previous row as one lane sees it through one slot: cell j of the lane is p[32 * j].
struct Src {
    const float *p;
#ifdef SPDY_DEBUG_CHECKS
    int cell;  // index of p[0] relative to band cell 0 of the previous row
#endif
    __device__ __forceinline__ float at(const int j, const AccessWindow &w) const
    {
#ifdef SPDY_DEBUG_CHECKS
        const int c = cell + 32 * j;
        if (c < w.read_lo || c >= w.read_hi) {
            atomicOr(w.status, STATUS_READ_RANGE);
            return pos_inf();
        }
        const float v = p[32 * j];
        if (v != v) atomicOr(w.status, STATUS_READ_STALE);
        return v;
#else
        (void)w;
        return p[32 * j];
#endif
    }
};

__device__ __forceinline__ Src make_src(const float *prev, const int first_cell, const int shift)
{
    Src s;
    s.p = prev + first_cell - shift;
#ifdef SPDY_DEBUG_CHECKS
    s.cell = first_cell - shift;
#endif
    return s;
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

// Cell updates of one slot (or two) on the RR cells a lane owns.
template <int RR>
__device__ __forceinline__ void update_min1(float (&best)[RR], const Src sa, const float ea, const AccessWindow &w)
{
#pragma unroll
    for (int j = 0; j < RR; ++j) best[j] = fminf(best[j], __fadd_rn(sa.at(j, w), ea));
}

template <int RR>
__device__ __forceinline__ void update_min2(float (&best)[RR], const Src sa, const float ea, const Src sb,
                                            const float eb, const AccessWindow &w)
{
    const unsigned long long ea2 = splat2(ea), eb2 = splat2(eb);
#pragma unroll
    for (int j = 0; j + 1 < RR; j += 2) {
        float a0 = sa.at(j, w), a1 = sa.at(j + 1, w);
        float b0 = sb.at(j, w), b1 = sb.at(j + 1, w);
        add2_rn(a0, a1, ea2);
        add2_rn(b0, b1, eb2);
        best[j] = min3(best[j], a0, b0);
        best[j + 1] = min3(best[j + 1], a1, b1);
    }
    if (RR & 1) {
        const float a0 = __fadd_rn(sa.at(RR - 1, w), ea);
        const float b0 = __fadd_rn(sb.at(RR - 1, w), eb);
        best[RR - 1] = min3(best[RR - 1], a0, b0);
    }
}

template <int RR>
__device__ __forceinline__ void update_arg(float (&best)[RR], int (&idx)[RR], const Src src, const float e,
                                           const int k, const AccessWindow &w)
{
#pragma unroll
    for (int j = 0; j < RR; ++j) {
        const float v = __fadd_rn(src.at(j, w), e);
        const bool better = v < best[j];  // strict: the lowest k keeps a tie
        best[j] = better ? v : best[j];
        idx[j] = better ? k : idx[j];
    }
}

// Two slots k0 < k1 = k0 + 1 per step, the winner between the two left open: m = min(best, v0, v1); the cell
// changes hands only if m < best (strict: a tie with the old value keeps the old, lower index), and then the
// cell remembers the pair, not the slot: code = 2 * k0 + 1.  Which of the pair it was is settled once per
// pass, after all slots (resolve_pair_codes).  Per update that is half a minimum, half a compare and half
// a select on top of load and add - against a compare and two selects for the plain scan.  (A NaN sum never
// attains the minimum, as in the scan.)
template <int RR>
__device__ __forceinline__ void update_arg_pair(float (&best)[RR], int (&code)[RR], const Src sa, const float ea,
                                                const Src sb, const float eb, const int pair_code,
                                                const AccessWindow &w)
{
    const unsigned long long ea2 = splat2(ea), eb2 = splat2(eb);
#define SPDY_PAIR_UPDATE(J, V0, V1)                         \
    {                                                       \
        const float m = min3(best[J], V0, V1);              \
        code[J] = (m < best[J]) ? pair_code : code[J];      \
        best[J] = m;                                        \
    }
#pragma unroll
    for (int j = 0; j + 1 < RR; j += 2) {
        float a0 = sa.at(j, w), a1 = sa.at(j + 1, w);
        float b0 = sb.at(j, w), b1 = sb.at(j + 1, w);
        add2_rn(a0, a1, ea2);
        add2_rn(b0, b1, eb2);
        SPDY_PAIR_UPDATE(j, a0, b0);
        SPDY_PAIR_UPDATE(j + 1, a1, b1);
    }
    if (RR & 1) {
        const float a0 = __fadd_rn(sa.at(RR - 1, w), ea);
        const float b0 = __fadd_rn(sb.at(RR - 1, w), eb);
        SPDY_PAIR_UPDATE(RR - 1, a0, b0);
    }
#undef SPDY_PAIR_UPDATE
}

// The same step from one array of running minima into another.  In place, the 3-input minimum has to land in a
// fresh register - the compare still needs the old value - and the loop-carried array takes it back with a
// move per cell and pair; taken two pairs at a time, from `in` to `out` and back, the move disappears.
template <int RR>
__device__ __forceinline__ void update_arg_pair_to(const float (&in)[RR], float (&out)[RR], int (&code)[RR], const Src sa,
                                                   const float ea, const Src sb, const float eb, const int pair_code,
                                                   const AccessWindow &w)
{
    const unsigned long long ea2 = splat2(ea), eb2 = splat2(eb);
#pragma unroll
    for (int j = 0; j + 1 < RR; j += 2) {
        float a0 = sa.at(j, w), a1 = sa.at(j + 1, w);
        float b0 = sb.at(j, w), b1 = sb.at(j + 1, w);
        add2_rn(a0, a1, ea2);
        add2_rn(b0, b1, eb2);
        out[j] = min3(in[j], a0, b0);
        code[j] = (out[j] < in[j]) ? pair_code : code[j];
        out[j + 1] = min3(in[j + 1], a1, b1);
        code[j + 1] = (out[j + 1] < in[j + 1]) ? pair_code : code[j + 1];
    }
    if (RR & 1) {
        const float a0 = __fadd_rn(sa.at(RR - 1, w), ea);
        const float b0 = __fadd_rn(sb.at(RR - 1, w), eb);
        out[RR - 1] = min3(in[RR - 1], a0, b0);
        code[RR - 1] = (out[RR - 1] < in[RR - 1]) ? pair_code : code[RR - 1];
    }
}

// Codes of update_arg_pair -> slot indices, once per pass.  A cell whose code names a pair (odd) won with
// m = min(v0, v1) of that pair and nothing after it was smaller, so best still holds that m: the winner is
// k0 if v0 - the same fp32 add of the same operands, hence the same bits - equals best, else k1 (a tie
// between the two goes to the lower index, as in the scan).  An even code 2 * k names slot k itself (slots
// taken singly); the initial code names no slot (0xFF).
template <int RR>
__device__ __forceinline__ void resolve_pair_codes(const float (&best)[RR], int (&code)[RR], const float *prev,
                                                   const int2 *taps, const int first, const int k_any,
                                                   const AccessWindow &w)
{
#pragma unroll
    for (int j = 0; j < RR; ++j) {
        const int c = code[j];
        const bool pair = c & 1;
        const int k0 = c >> 1;
        const int2 tp = taps[pair ? k0 : k_any];  // k_any: some slot of this pass, so that every lane reads in range
        const float v0 = __fadd_rn(make_src(prev, first, tp.x).at(j, w), __int_as_float(tp.y));
        code[j] = (pair && !(v0 == best[j])) ? k0 + 1 : k0;
    }
}

// Same update as update_arg with the two selects written as predicated fp32 arithmetic that acts as an exact
// move, to keep them off the integer/compare pipe: best <- v + (-0.0) (== v for every v) and
// idx <- v * 0 + k (== k: a winning v is finite, so v * 0 is +-0).  The index is carried as a float.
template <int RR>
__device__ __forceinline__ void update_arg_pred(float (&best)[RR], float (&idxf)[RR], const Src src,
                                                const float e, const int k, const AccessWindow &w)
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
        float v0 = src.at(j, w), v1 = src.at(j + 1, w);
        add2_rn(v0, v1, e2);
        SPDY_PRED_UPDATE(j, v0);
        SPDY_PRED_UPDATE(j + 1, v1);
    }
    if (RR & 1) {
        const float v0 = __fadd_rn(src.at(RR - 1, w), e);
        SPDY_PRED_UPDATE(RR - 1, v0);
    }
#undef SPDY_PRED_UPDATE
}

// One warp pass: the 32*RR band cells starting at s (lane i owns cells s + i, s + i + 32, ...),
// so every row access is lane-consecutive (conflict-free in shared memory) whatever the shift.  Both row
// buffers carry guard cells of +inf on either side of the band: a pass that only partly overlaps a
// slot's range reads +inf for the cells outside it and needs no per-cell bounds check (the host proves the
// guard wide enough for every pass of a plan when the plan is built).  Which slots overlap the pass at all
// is known on the host.  `krange` = u_lo | u_hi << 8 | dense << 16: the overlapping slots lie in
// [u_lo, u_hi); when they are all of that range (dense, the usual case: times fall as the choice index
// rises) the loop runs straight over it, otherwise it walks the set bits of `mask` (MW 64-bit words,
// one bit per slot), in ascending order either way.
//
// `prev`/`cur` point at band cell 0 of the previous/new row; taps[u] = (a_u, bits of e_u): slot
// u reads the previous row at t_rel - a_u.
//
// `prev` and `cur` carry no __restrict__: with the row buffers in global memory the kernel itself rewrites the
// memory behind `prev` two layers later, so those reads must stay ordinary coherent loads.
//
// With MASKED only cells below `limit` are stored (a CTA of a cluster owns a slice of the band and
// must not write its neighbour's cells); without it the caller guarantees room for the whole pass.
//
// With STORE_TABLE false (row-value table only) the pass leaves the table alone: the caller copies the whole
// row from shared memory to the table with one bulk copy per layer.
// ROOMY: the build has 128 registers per thread (see update_arg_pair_to).
template <int RR, int MODE, bool MASKED, bool STORE_TABLE = true, bool ROOMY = false>
__device__ __forceinline__ void process_span(const float *prev, float *cur, const int2 *__restrict__ taps,
                                             const unsigned krange, const unsigned long long *__restrict__ mask,
                                             const int MW, const int s, const int lane, void *table_row,
                                             const int limit, const AccessWindow &w)
{
    const float INF = pos_inf();
    const int first = s + lane;
    const int k_lo = krange & 0xFF, k_hi = (krange >> 8) & 0xFF;
    const bool dense = (krange >> 16) & 1;
    float best[RR];
#pragma unroll
    for (int j = 0; j < RR; ++j) best[j] = INF;

    auto store_allowed = [&](const int j) -> bool {
        if (MASKED && !(s + j * 32 + lane < limit)) return false;
#ifdef SPDY_DEBUG_CHECKS
        if (s + j * 32 + lane >= w.write_hi || static_cast<long long>(s) + j * 32 + lane >= w.table_hi) {
            atomicOr(w.status, STATUS_WRITE_RANGE);
            return false;
        }
#endif
        return true;
    };

    if constexpr (MODE == MODE_ROW2 || MODE == MODE_ROW) {
        // Value-only minimum: the order of the slots does not matter, so overlapping slots
        // are taken two at a time (MODE_ROW2) whatever their indices.
        if (dense) {
            int k = k_lo;
            if (MODE == MODE_ROW2) {
                // An odd first slot goes alone so that every pair below is one aligned 16-byte read.
                if ((k & 1) && k < k_hi) {
                    const int2 ta = taps[k];
                    update_min1<RR>(best, make_src(prev, first, ta.x), __int_as_float(ta.y), w);
                    ++k;
                }
#pragma unroll 1
                for (; k + 1 < k_hi; k += 2) {
                    const int4 t = *reinterpret_cast<const int4 *>(taps + k);
                    update_min2<RR>(best, make_src(prev, first, t.x), __int_as_float(t.y), make_src(prev, first, t.z),
                                    __int_as_float(t.w), w);
                }
            }
#pragma unroll 1
            for (; k < k_hi; ++k) {
                const int2 ta = taps[k];
                update_min1<RR>(best, make_src(prev, first, ta.x), __int_as_float(ta.y), w);
            }
        } else {
#pragma unroll 1
            for (int wd = 0; wd < MW; ++wd) {
                unsigned long long m = __ldg(mask + wd);
#pragma unroll 1
                while (m) {
                    const int2 ta = taps[64 * wd + __ffsll(static_cast<long long>(m)) - 1];
                    m &= m - 1;
                    update_min1<RR>(best, make_src(prev, first, ta.x), __int_as_float(ta.y), w);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) cur[s + j * 32 + lane] = best[j];
        if constexpr (STORE_TABLE) {
            float *D = static_cast<float *>(table_row) + s + lane;
#pragma unroll
            for (int j = 0; j < RR; ++j)
                if (store_allowed(j)) D[j * 32] = best[j];
        }
    } else if constexpr (MODE == MODE_ARG) {
        int idx[RR];
#pragma unroll
        for (int j = 0; j < RR; ++j) idx[j] = 0xFF;
        if (dense) {
#pragma unroll 1
            for (int k = k_lo; k < k_hi; ++k) {
                const int2 tp = taps[k];
                update_arg<RR>(best, idx, make_src(prev, first, tp.x), __int_as_float(tp.y), k, w);
            }
        } else {
#pragma unroll 1
            for (int wd = 0; wd < MW; ++wd) {
                unsigned long long m = __ldg(mask + wd);
#pragma unroll 1
                while (m) {
                    const int k = 64 * wd + __ffsll(static_cast<long long>(m)) - 1;
                    m &= m - 1;
                    const int2 tp = taps[k];
                    update_arg<RR>(best, idx, make_src(prev, first, tp.x), __int_as_float(tp.y), k, w);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) cur[s + j * 32 + lane] = best[j];
        unsigned char *P = static_cast<unsigned char *>(table_row) + s + lane;
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) P[j * 32] = static_cast<unsigned char>(idx[j]);
    } else if constexpr (MODE == MODE_ARG_PAIR) {
        // code: 2 * k for "slot k", 2 * k0 + 1 for "slot k0 or k0 + 1" (settled below), 2 * 0xFF for none.
        int code[RR];
#pragma unroll
        for (int j = 0; j < RR; ++j) code[j] = 2 * 0xFF;
        if (dense) {
            int k = k_lo;
            // An odd first slot goes alone so that every pair below is one aligned 16-byte read.
            if ((k & 1) && k < k_hi) {
                const int2 tp = taps[k];
                update_arg<RR>(best, code, make_src(prev, first, tp.x), __int_as_float(tp.y), 2 * k, w);
                ++k;
            }
            // Two pairs per trip, the running minima alternating between `best` and `other` (see
            // update_arg_pair_to) - for passes of up to 20 cells per lane: beyond, the third register array no
            // longer fits the 128 registers of a thread.
            if constexpr (ROOMY && RR <= 20) {
                float other[RR];
#pragma unroll 1
                for (; k + 3 < k_hi; k += 4) {
                    const int4 t = *reinterpret_cast<const int4 *>(taps + k);
                    const int4 t2 = *reinterpret_cast<const int4 *>(taps + k + 2);
                    update_arg_pair_to<RR>(best, other, code, make_src(prev, first, t.x), __int_as_float(t.y),
                                           make_src(prev, first, t.z), __int_as_float(t.w), 2 * k + 1, w);
                    update_arg_pair_to<RR>(other, best, code, make_src(prev, first, t2.x), __int_as_float(t2.y),
                                           make_src(prev, first, t2.z), __int_as_float(t2.w), 2 * k + 5, w);
                }
            }
#pragma unroll 1
            for (; k + 1 < k_hi; k += 2) {
                const int4 t = *reinterpret_cast<const int4 *>(taps + k);
                update_arg_pair<RR>(best, code, make_src(prev, first, t.x), __int_as_float(t.y),
                                    make_src(prev, first, t.z), __int_as_float(t.w), 2 * k + 1, w);
            }
            if (k < k_hi) {
                const int2 tp = taps[k];
                update_arg<RR>(best, code, make_src(prev, first, tp.x), __int_as_float(tp.y), 2 * k, w);
            }
            if (k_lo < k_hi) resolve_pair_codes<RR>(best, code, prev, taps, first, k_lo, w);
        } else {
#pragma unroll 1
            for (int wd = 0; wd < MW; ++wd) {
                unsigned long long m = __ldg(mask + wd);
#pragma unroll 1
                while (m) {
                    const int k = 64 * wd + __ffsll(static_cast<long long>(m)) - 1;
                    m &= m - 1;
                    const int2 tp = taps[k];
                    update_arg<RR>(best, code, make_src(prev, first, tp.x), __int_as_float(tp.y), 2 * k, w);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) cur[s + j * 32 + lane] = best[j];
        unsigned char *P = static_cast<unsigned char *>(table_row) + s + lane;
        // (dense passes hold slot indices after resolve_pair_codes, the others still 2 * k)
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) P[j * 32] = static_cast<unsigned char>(dense && k_lo < k_hi ? code[j] : code[j] >> 1);
    } else {  // MODE_ARG_PRED
        float idxf[RR];
#pragma unroll
        for (int j = 0; j < RR; ++j) idxf[j] = 255.0f;
        if (dense) {
#pragma unroll 1
            for (int k = k_lo; k < k_hi; ++k) {
                const int2 tp = taps[k];
                update_arg_pred<RR>(best, idxf, make_src(prev, first, tp.x), __int_as_float(tp.y), k, w);
            }
        } else {
#pragma unroll 1
            for (int wd = 0; wd < MW; ++wd) {
                unsigned long long m = __ldg(mask + wd);
#pragma unroll 1
                while (m) {
                    const int k = 64 * wd + __ffsll(static_cast<long long>(m)) - 1;
                    m &= m - 1;
                    const int2 tp = taps[k];
                    update_arg_pred<RR>(best, idxf, make_src(prev, first, tp.x), __int_as_float(tp.y), k, w);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) cur[s + j * 32 + lane] = best[j];
        unsigned char *P = static_cast<unsigned char *>(table_row) + s + lane;
#pragma unroll
        for (int j = 0; j < RR; ++j)
            if (store_allowed(j)) P[j * 32] = static_cast<unsigned char>(static_cast<int>(idxf[j]));
    }
}

// Runs the pass `pd` with the unrolled body for its cells-per-lane count (1..RCAP).
template <int MODE, int RCAP, bool MASKED, bool STORE_TABLE = true, bool ROOMY = false>
__device__ __forceinline__ void run_pass(const int cpl, const float *prev, float *cur, const int2 *taps,
                                         const unsigned krange, const unsigned long long *mask, const int MW,
                                         const int s, const int lane, void *table_row, const int limit,
                                         const AccessWindow &w)
{
    switch (cpl) {
#define SPDY_CASE(RR)                                                                                          \
    case RR:                                                                                                   \
        if constexpr (RR <= kRmaxLong && RR <= RCAP)                                                           \
            process_span<RR, MODE, MASKED, STORE_TABLE, ROOMY>(prev, cur, taps, krange, mask, MW, s, lane,     \
                                                               table_row, limit, w);                           \
        break;
        SPDY_CASE(1) SPDY_CASE(2) SPDY_CASE(3) SPDY_CASE(4) SPDY_CASE(5) SPDY_CASE(6)
        SPDY_CASE(7) SPDY_CASE(8) SPDY_CASE(9) SPDY_CASE(10) SPDY_CASE(11) SPDY_CASE(12)
        SPDY_CASE(13) SPDY_CASE(14) SPDY_CASE(15) SPDY_CASE(16) SPDY_CASE(17) SPDY_CASE(18)
        SPDY_CASE(19) SPDY_CASE(20) SPDY_CASE(21) SPDY_CASE(22) SPDY_CASE(23) SPDY_CASE(24)
        SPDY_CASE(25) SPDY_CASE(26) SPDY_CASE(27) SPDY_CASE(28) SPDY_CASE(29) SPDY_CASE(30) SPDY_CASE(31) SPDY_CASE(32) SPDY_CASE(33) SPDY_CASE(34) SPDY_CASE(35) SPDY_CASE(36)
        SPDY_CASE(37) SPDY_CASE(38) SPDY_CASE(39) SPDY_CASE(40) SPDY_CASE(41) SPDY_CASE(42) SPDY_CASE(43) SPDY_CASE(44) SPDY_CASE(45) SPDY_CASE(46) SPDY_CASE(47) SPDY_CASE(48)
#undef SPDY_CASE
        default: break;
    }
}

// The finished row goes from shared memory to the walk-back table as ONE bulk copy per layer, issued by one
// thread and carried out by the copy engine: the table stores then cost the warps no instructions and the
// load/store data path - the unit this kernel is bound by - no wavefronts.  Both addresses are 16-byte aligned
// and the size a multiple of 16 bytes (rows start on 128-cell boundaries of a 256-byte aligned table and
// are whole blocks of 32 cells long).  Protocol per layer: every thread that wrote the row makes its
// writes visible to the copy engine (bulk_copy_fence), the issuing thread waits until the engine has read
// the buffer that the next layer will overwrite (bulk_copy_wait_read: that copy was issued a whole layer
// earlier), the layer's barrier follows, then the issuing thread starts the copy of the row just finished.
__device__ __forceinline__ void bulk_copy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_copy_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_copy_row_to_table(void *table_row, const float *row, const int cells)
{
    const unsigned src = static_cast<unsigned>(__cvta_generic_to_shared(row));
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(table_row), "r"(src),
                 "r"(cells * 4)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// (value, t) merge with the lowest t among equal values.
__device__ __forceinline__ void warp_min_lowest_t(float &bv, int &bt)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int ot = __shfl_xor_sync(0xffffffffu, bt, off);
        if (ov < bv || (ov == bv && ot < bt)) {
            bv = ov;
            bt = ot;
        }
    }
}

// ----------------------------------------------------------------------------------------------
// One CTA per candidate
// ----------------------------------------------------------------------------------------------
//
// RCAP: the largest cells-per-lane this instantiation can run.  The registers a kernel needs grow
// with the largest unrolled pass, so plans whose passes are short use the RCAP = 8 build, which fits twice
// as many CTAs per SM.
//
// GROWS: keep the two row buffers in global memory (args.grows) instead of shared memory.  This is the
// fallback for bands too wide for one CTA's shared memory; the code is the same, the reads then go through
// L1/L2.  Writes of one layer are ordered before the reads of the next by the same per-layer __syncthreads().
//
// The passes of a layer are laid out on the host per warp (pass_ptr): lengths chosen by the slots that
// overlap them, dealt to the warps so that they arrive level at the one __syncthreads() per layer.
template <int MODE, int NT, int MINB, int RCAP, bool GROWS>
__global__ void __launch_bounds__(NT, MINB) spdy_forward_kernel(const FwdArgs args)
{
    constexpr bool ROWFMT = (MODE == MODE_ROW || MODE == MODE_ROW2);
    constexpr int NWARPS = NT / 32;
#ifdef SPDY_DEBUG_CHECKS
    constexpr bool BULK = false;  // the debug build stores every table cell itself, index-checked
#else
    constexpr bool BULK = ROWFMT && !GROWS;  // rows in shared memory, row-value table: bulk copy per layer
#endif
    constexpr bool ROOMY = NT * MINB <= 512 && !GROWS;  // 128 registers per thread
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *rows;
    int2 *tap_buf;
    if constexpr (GROWS) {
        rows = args.grows + static_cast<size_t>(blockIdx.x) * static_cast<size_t>(args.grows_stride);
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
    const int L = args.L, K = args.K;
    const int KS = (K + 1) & ~1;  // slots per staging buffer: even, so that slot pairs are 16-byte aligned
    const int MW = (K + 63) >> 6;
    const int64_t n_local = blockIdx.x;
    const int64_t n = args.n_first + n_local;
    const float INF = pos_inf();
    const int PAD = args.pad;

    // Both buffers start as +inf everywhere; D_0 is +0 at t = 0 (Eq. 3 via a virtual row 0).
    LayerDesc ld = args.layers[0];
    for (int i = tid; i < 2 * args.row_stride; i += NT) rows[i] = INF;
    for (int u = tid; u < ld.nslots; u += NT) tap_buf[u] = stage_slot(args, n, 0, u);
    int p0 = __ldg(args.pass_ptr + warp), p1 = __ldg(args.pass_ptr + warp + 1);
    __syncthreads();
    if (tid == 0) rows[PAD] = 0.0f;
    __syncthreads();

    for (int l = 0; l < L; ++l) {
        const float *prev = rows + (l & 1) * args.row_stride + PAD;
        float *cur = rows + ((l + 1) & 1) * args.row_stride + PAD;
        const int2 *taps = tap_buf + (l & 1) * KS;

        // Fetch the next layer's descriptor, pass range and slots early; the slots are parked in shared
        // memory after the passes.  (NT >= K is guaranteed by the host, so one thread per slot suffices.)
        LayerDesc ld_next = ld;
        int q0 = 0, q1 = 0;
        int2 next_tap = make_int2(0, 0);
        bool have_next = false;
        if (l + 1 < L) {
            ld_next = args.layers[l + 1];
            q0 = __ldg(args.pass_ptr + (l + 1) * NWARPS + warp);
            q1 = __ldg(args.pass_ptr + (l + 1) * NWARPS + warp + 1);
            have_next = tid < ld_next.nslots;
            if (have_next) next_tap = stage_slot(args, n, l + 1, tid);
        }

        unsigned char *row_base = static_cast<unsigned char *>(args.table) +
                                  (n_local * args.pitch + ld.rowoff) * (ROWFMT ? 4 : 1);
        AccessWindow w;
#ifdef SPDY_DEBUG_CHECKS
        w.read_lo = -PAD;
        w.read_hi = l == 0 ? args.row_stride - PAD : args.layers[l - 1].extent + args.layers[l - 1].fill;
        w.write_hi = ld.extent;
        w.table_hi = args.pitch - ld.rowoff;
        w.status = args.status;
        for (int i = tid; i < ld.extent; i += NT) cur[i] = __int_as_float(0x7fc00000);  // mark the new row unwritten
        __syncthreads();
#endif
        if constexpr (GROWS) {
            // (64 registers per thread: no room to hold the next pass's descriptor across a pass)
            for (int p = p0; p < p1; ++p) {
                const int2 pd = __ldg(reinterpret_cast<const int2 *>(args.passes + p));
                run_pass<MODE, RCAP, false, !BULK, ROOMY>(static_cast<unsigned>(pd.y) >> 24, prev, cur, taps, static_cast<unsigned>(pd.y),
                                            args.pass_masks + static_cast<size_t>(p) * MW, MW, pd.x, lane, row_base, 0, w);
            }
        } else {
            // The descriptor of the next pass is fetched while the current one runs.
            int2 pd_next = p0 < p1 ? __ldg(reinterpret_cast<const int2 *>(args.passes + p0)) : make_int2(0, 0);
            for (int p = p0; p < p1; ++p) {
                const int2 pd = pd_next;
                if (p + 1 < p1) pd_next = __ldg(reinterpret_cast<const int2 *>(args.passes + p + 1));
                run_pass<MODE, RCAP, false, !BULK, ROOMY>(static_cast<unsigned>(pd.y) >> 24, prev, cur, taps, static_cast<unsigned>(pd.y),
                                            args.pass_masks + static_cast<size_t>(p) * MW, MW, pd.x, lane, row_base, 0, w);
            }
        }
        // Cells [width, extent) of the new row were written as +inf by the passes (they saw only +inf
        // sources); `fill` more cells of +inf behind them cover every read of the next layer.
        for (int i = tid; i < ld.fill; i += NT) cur[ld.extent + i] = INF;
        if (have_next) tap_buf[((l + 1) & 1) * KS + tid] = next_tap;
        if constexpr (BULK) {
            bulk_copy_fence();
            if (tid == 0) bulk_copy_wait_read();
        }
        __syncthreads();
        if constexpr (BULK)
            if (tid == 0) bulk_copy_row_to_table(row_base, cur, ld.extent);
        ld = ld_next;
        p0 = q0;
        p1 = q1;
    }

    // min over t <= B of D_L[t], lowest t among equals (the band's upper end never exceeds B).
    if constexpr (BULK)
        if (tid == 0) bulk_copy_wait_read();  // the last row's copy must have left shared memory before the CTA does
    const float *last = rows + (L & 1) * args.row_stride + PAD;
    float bv = INF;
    int bt = 0x7fffffff;
    for (int t = tid; t < ld.width; t += NT) {
        const float v = last[t];
        if (v < bv) {
            bv = v;
            bt = t;
        }
    }
    warp_min_lowest_t(bv, bt);
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
        warp_min_lowest_t(bv, bt);
        if (lane == 0) {
            const bool feasible = bv < INF;
            args.cost[n] = feasible ? bv : INF;
            args.time_used[n] = feasible ? ld.lo + bt : -1;
        }
    }
}

// ----------------------------------------------------------------------------------------------
// One warp per candidate
// ----------------------------------------------------------------------------------------------
//
// For rows a pass or two wide (a budget of about a thousand buckets) a CTA per candidate spends more on
// its per-layer barrier and fixed costs than on cell updates.  Here every warp of a CTA owns a candidate
// outright: its own two row buffers and slot buffers in the CTA's shared memory, all passes of a layer, a
// __syncwarp() where the CTA kernel has a __syncthreads().  Warps never wait for one another.  The host
// offers this kernel only to plans whose layers have at most 64 shift slots (two staged per lane).
constexpr int kWarpKernelThreads = 128;

template <int MODE, int MINB, int RCAP>
__global__ void __launch_bounds__(kWarpKernelThreads, MINB) spdy_forward_warp_kernel(const FwdArgs args)
{
    constexpr bool ROWFMT = (MODE == MODE_ROW || MODE == MODE_ROW2);
    constexpr int NWARPS = kWarpKernelThreads / 32;
#ifdef SPDY_DEBUG_CHECKS
    constexpr bool BULK = false;
#else
    constexpr bool BULK = ROWFMT;  // row-value table: one bulk copy per layer and warp (see bulk_copy_row_to_table)
#endif
    constexpr bool ROOMY = MINB <= 4;  // 128 registers per thread
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t n_local = static_cast<int64_t>(blockIdx.x) * NWARPS + warp;
    if (n_local >= args.n_count) return;
    if (args.cand_flags && args.cand_flags[n_local] != args.which) return;
    const int L = args.L, K = args.K;
    const int KS = (K + 1) & ~1;
    const int MW = (K + 63) >> 6;
    const int64_t n = args.n_first + n_local;
    const float INF = pos_inf();
    const int PAD = args.pad;
    float *rows = reinterpret_cast<float *>(smem_raw) + static_cast<size_t>(warp) * 2 * args.row_stride;
    int2 *tap_buf = reinterpret_cast<int2 *>(reinterpret_cast<float *>(smem_raw) + static_cast<size_t>(NWARPS) * 2 * args.row_stride) +
                    static_cast<size_t>(warp) * 2 * KS;

    LayerDesc ld = args.layers[0];
    for (int i = lane; i < 2 * args.row_stride; i += 32) rows[i] = INF;
    for (int u = lane; u < ld.nslots; u += 32) tap_buf[u] = stage_slot(args, n, 0, u);
    int p0 = __ldg(args.pass_ptr), p1 = __ldg(args.pass_ptr + 1);
    __syncwarp();
    if (lane == 0) rows[PAD] = 0.0f;
    __syncwarp();

    for (int l = 0; l < L; ++l) {
        const float *prev = rows + (l & 1) * args.row_stride + PAD;
        float *cur = rows + ((l + 1) & 1) * args.row_stride + PAD;
        const int2 *taps = tap_buf + (l & 1) * KS;

        LayerDesc ld_next = ld;
        int q0 = 0, q1 = 0;
        int2 next_a = make_int2(0, 0), next_b = make_int2(0, 0);
        if (l + 1 < L) {
            ld_next = args.layers[l + 1];
            q0 = __ldg(args.pass_ptr + l + 1);
            q1 = __ldg(args.pass_ptr + l + 2);
            if (lane < ld_next.nslots) next_a = stage_slot(args, n, l + 1, lane);
            if (lane + 32 < ld_next.nslots) next_b = stage_slot(args, n, l + 1, lane + 32);
        }

        unsigned char *row_base = static_cast<unsigned char *>(args.table) +
                                  (n_local * args.pitch + ld.rowoff) * (ROWFMT ? 4 : 1);
        AccessWindow w;
#ifdef SPDY_DEBUG_CHECKS
        w.read_lo = -PAD;
        w.read_hi = l == 0 ? args.row_stride - PAD : args.layers[l - 1].extent + args.layers[l - 1].fill;
        w.write_hi = ld.extent;
        w.table_hi = args.pitch - ld.rowoff;
        w.status = args.status;
        for (int i = lane; i < ld.extent; i += 32) cur[i] = __int_as_float(0x7fc00000);
        __syncwarp();
#endif
        // The descriptor of the next pass is fetched while the current one runs.
        int2 pd_next = p0 < p1 ? __ldg(reinterpret_cast<const int2 *>(args.passes + p0)) : make_int2(0, 0);
        for (int p = p0; p < p1; ++p) {
            const int2 pd = pd_next;
            if (p + 1 < p1) pd_next = __ldg(reinterpret_cast<const int2 *>(args.passes + p + 1));
            run_pass<MODE, RCAP, false, !BULK, ROOMY>(static_cast<unsigned>(pd.y) >> 24, prev, cur, taps, static_cast<unsigned>(pd.y),
                                        args.pass_masks + static_cast<size_t>(p) * MW, MW, pd.x, lane, row_base, 0, w);
        }
        for (int i = lane; i < ld.fill; i += 32) cur[ld.extent + i] = INF;
        if (l + 1 < L) {
            if (lane < ld_next.nslots) tap_buf[((l + 1) & 1) * KS + lane] = next_a;
            if (lane + 32 < ld_next.nslots) tap_buf[((l + 1) & 1) * KS + lane + 32] = next_b;
        }
        if constexpr (BULK) {
            bulk_copy_fence();
            if (lane == 0) bulk_copy_wait_read();
        }
        __syncwarp();
        if constexpr (BULK)
            if (lane == 0) bulk_copy_row_to_table(row_base, cur, ld.extent);
        ld = ld_next;
        p0 = q0;
        p1 = q1;
    }

    if constexpr (BULK)
        if (lane == 0) bulk_copy_wait_read();
    const float *last = rows + (L & 1) * args.row_stride + PAD;
    float bv = INF;
    int bt = 0x7fffffff;
    for (int t = lane; t < ld.width; t += 32) {
        const float v = last[t];
        if (v < bv) {
            bv = v;
            bt = t;
        }
    }
    warp_min_lowest_t(bv, bt);
    if (lane == 0) {
        const bool feasible = bv < INF;
        args.cost[n] = feasible ? bv : INF;
        args.time_used[n] = feasible ? ld.lo + bt : -1;
    }
}

// ----------------------------------------------------------------------------------------------
// One candidate per thread-block cluster
// ----------------------------------------------------------------------------------------------
//
// For batches with fewer candidates than SMs (or on request) the band of every row is cut into C
// contiguous slices, one per CTA of a cluster.  Each CTA keeps its slice of the new row in its own shared
// memory (`out`, double buffered) and, before a layer, gathers the window of the previous row its slice
// depends on - its own slice plus up to max_k a_k cells to the left - from the `out` buffers of its cluster
// peers through distributed shared memory into a private window (`win`).  The cell updates then
// run on local shared memory exactly as in the single-CTA kernel.  One hardware cluster barrier
// per layer orders "slices of row l written" before "windows for row l+1 gathered"; every thread
// of every CTA reaches every barrier (there is no early exit), so the barrier cannot wait forever.
template <int MODE, int NT>
__global__ void __launch_bounds__(NT, 1) spdy_forward_cluster_kernel(const ClusterArgs cargs)
{
    namespace cg = cooperative_groups;
    constexpr bool ROWFMT = (MODE == MODE_ROW || MODE == MODE_ROW2);
    constexpr int NWARPS = NT / 32;
    constexpr int CAP = NT >= 512 ? 16 : kRmax;  // == cluster_cells_per_lane(NT), the host's figure
    static_assert(CAP <= kRmax, "pass bodies exist up to kRmax cells per lane");
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
#ifdef SPDY_DEBUG_CHECKS
                    if (src < 0 || src >= C || seg_lo - src * sd.prev_slice < 0 ||
                        seg_hi - src * sd.prev_slice > cargs.out_stride || seg_hi - sd.q0 > cargs.win_stride) {
                        if (tid == 0) atomicOr(args.status, STATUS_READ_RANGE);
                        continue;
                    }
#endif
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
        AccessWindow w;
#ifdef SPDY_DEBUG_CHECKS
        w.read_lo = sd.q0;
        w.read_hi = sd.q0 + sd.win_len;
        w.write_hi = sd.slice_hi;
        w.table_hi = args.pitch - ld.rowoff;
        w.status = args.status;
#endif
        // All passes of a slice have one length: pick the unrolled body once, outside the pass loop.
        switch (sd.cpl) {
#define SPDY_CASE(RR)                                                                                             \
    case RR:                                                                                                      \
        if constexpr (RR <= CAP)                                                                                  \
            for (int span = warp; span < sd.nspans; span += NWARPS) {                                             \
                const int p = sd.mask_off + span;                                                                 \
                const int2 pd = __ldg(reinterpret_cast<const int2 *>(args.passes + p));                           \
                process_span<RR, MODE, true>(prev, cur, taps, static_cast<unsigned>(pd.y),                        \
                                             args.pass_masks + static_cast<size_t>(p) * MW, MW, pd.x, lane,       \
                                             row_base, sd.slice_hi, w);                                           \
            }                                                                                                     \
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
    warp_min_lowest_t(bv, bt);
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
        warp_min_lowest_t(bv, bt);
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

// ----------------------------------------------------------------------------------------------
// Kernel tables: each forward mode is compiled in a translation unit of its own
// ----------------------------------------------------------------------------------------------

using FwdKernel = void (*)(const FwdArgs);
using ClusterKernel = void (*)(const ClusterArgs);

struct FwdVariant {
    int kind;     // KernelKind
    int mode;
    int threads;
    int rcap;
    FwdKernel fn;
};

struct ClusterVariant {
    int mode;
    int threads;
    ClusterKernel fn;
};

struct VariantList {
    const FwdVariant *fwd;
    int n_fwd;
    const ClusterVariant *cluster;
    int n_cluster;
};

VariantList variants_arg();
VariantList variants_arg_pred();
VariantList variants_arg_pair();
VariantList variants_row();
VariantList variants_row2();

// The standard set of builds of one mode.  FULL adds the rows-in-global build and the warp-per-candidate
// builds, which only the default cell update of each table format has.
#define SPDY_CTA_VARIANT(MODE, NT, MINB, RCAP) \
    FwdVariant { KERNEL_CTA, MODE, NT, RCAP, spdy_forward_kernel<MODE, NT, MINB, RCAP, false> }
// A 256-thread CTA of the pairwise argmin update (two register arrays of cells per lane) needs more than the
// 80 registers that three resident CTAs leave: it runs two per SM.  cells_per_lane_1024() is the longest pass
// a 1024-thread CTA (64 registers per thread) can unroll without spilling.
template <int MODE> constexpr int ctas_256() { return MODE == MODE_ARG_PAIR ? 2 : 3; }
#define SPDY_CTA_VARIANTS(MODE)                                                                                 \
    SPDY_CTA_VARIANT(MODE, 128, 4, long_pass_cap(MODE)), SPDY_CTA_VARIANT(MODE, 256, ctas_256<MODE>(), kRmax),    \
    SPDY_CTA_VARIANT(MODE, 512, 1, long_pass_cap(MODE)), SPDY_CTA_VARIANT(MODE, 1024, 1, cells_per_lane_1024(MODE)), \
    SPDY_CTA_VARIANT(MODE, 128, 6, 8), SPDY_CTA_VARIANT(MODE, 256, 3, 8),                                       \
    SPDY_CTA_VARIANT(MODE, 512, 1, 8), SPDY_CTA_VARIANT(MODE, 1024, 1, 8)
#define SPDY_FULL_VARIANTS(MODE)                                                                                \
    SPDY_CTA_VARIANTS(MODE),                                                                                    \
    FwdVariant{KERNEL_CTA_GLOBAL, MODE, 1024, global_rows_cap_1024(MODE),                                       \
               spdy_forward_kernel<MODE, 1024, 1, global_rows_cap_1024(MODE), true>},                           \
    FwdVariant{KERNEL_CTA_GLOBAL, MODE, 512, kRmax, spdy_forward_kernel<MODE, 512, 1, kRmax, true>},            \
    FwdVariant{KERNEL_WARP, MODE, kWarpKernelThreads, warp_short_cap(MODE),                                     \
               spdy_forward_warp_kernel<MODE, 8, warp_short_cap(MODE)>},                                        \
    FwdVariant{KERNEL_WARP, MODE, kWarpKernelThreads, long_pass_cap(MODE),                                      \
               spdy_forward_warp_kernel<MODE, 4, long_pass_cap(MODE)>}
#define SPDY_CLUSTER_VARIANTS(MODE) \
    ClusterVariant{MODE, 256, spdy_forward_cluster_kernel<MODE, 256>}, ClusterVariant{MODE, 512, spdy_forward_cluster_kernel<MODE, 512>}

}  // namespace spdy

#endif  // SPDY_DEVICE_CUH
