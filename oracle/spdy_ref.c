/*
 * CPU oracle for the SPDY dynamic program.  TEST INFRASTRUCTURE ONLY: it exists to check the
 * CUDA library and to serve as the timed CPU baseline; no product code path may call it.
 *
 * Plain, single-threaded, full-width rows, no blocking or band-limiting: the recurrence of
 * Section 3.2 (Eq. 2-3) carried out in the loop order of Algorithm 1 (Appendix A): layers, then
 * choices in ascending index, then time buckets; strict "<" update, so the lowest choice index
 * wins ties.  Arithmetic is fp32 with one add per cell (compile with -fno-fast-math
 * -ffp-contract=off; the x86-64 default keeps denormals).
 *
 * Readings adopted where the paper leaves room:
 *  - Eq. 2-3 are followed for the bucket range: a choice of time tau updates t = tau..B
 *    (Algorithm 1 prints the range as starting one bucket later, which would forbid a prefix
 *    of total time 0; Eq. 2 has no such exclusion).
 *  - Layer 1 goes through the same recurrence from a virtual row D_0 with D_0[0] = +0 and
 *    +inf elsewhere; this equals Algorithm 1's explicit seeding of row 1.
 *  - A choice with tau > B can never be used and is skipped.
 *  - The final argmin over t takes the lowest t among equal minima.
 *  - A problem with no profile inside the budget reports cost = +inf, time_used = -1 and a
 *    profile of 0xFF bytes.
 *
 * Pins (tests/test_oracle_pins.py): exhaustive enumeration of all K^L profiles, the knapsack
 * special case against a textbook 0/1 knapsack, closed forms (all-dense, infeasible, K = 1,
 * L = 1), monotonicity in B, and self-consistency invariants of the returned profile.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SPDY_REF_OK 0
#define SPDY_REF_BAD_ARG (-1)
#define SPDY_REF_NO_MEMORY (-2)
#define SPDY_REF_INTERNAL (-3)

/*
 * One candidate.  errors: [L][K] fp32, times: [L][K] int32 (>= 0), B >= 0.
 * D_work: 2*(B+1) floats, P_work: L*(B+1) bytes, both caller-provided scratch.
 */
int spdy_ref_solve_one(const float *errors, const int32_t *times, int32_t L, int32_t K, int32_t B,
                       uint8_t *profile, float *cost, int32_t *time_used, float *D_work,
                       uint8_t *P_work)
{
    if (!errors || !times || !profile || !cost || !time_used || !D_work || !P_work)
        return SPDY_REF_BAD_ARG;
    if (L < 1 || K < 1 || K > 255 || B < 0)
        return SPDY_REF_BAD_ARG;
    const size_t width = (size_t)B + 1;
    float *prev = D_work;
    float *cur = D_work + width;

    /* Virtual row D_0: zero layers take exactly zero time at zero error (Eq. 3). */
    for (size_t t = 0; t < width; ++t)
        prev[t] = INFINITY;
    prev[0] = 0.0f;

    for (int32_t l = 0; l < L; ++l) {
        uint8_t *P = P_work + (size_t)l * width;
        for (size_t t = 0; t < width; ++t) {
            cur[t] = INFINITY;
            P[t] = 0xFF;
        }
        for (int32_t k = 0; k < K; ++k) { /* "for s in S", ascending index */
            const int32_t tau = times[(size_t)l * K + k];
            if (tau < 0)
                return SPDY_REF_BAD_ARG;
            if (tau > B)
                continue;
            const float e = errors[(size_t)l * K + k];
            for (int32_t t = tau; t <= B; ++t) {
                const float v = prev[t - tau] + e; /* Eq. 2: E_{l-1}^{t - tau} + e */
                if (v < cur[t]) {
                    cur[t] = v;
                    P[t] = (uint8_t)k;
                }
            }
        }
        float *tmp = prev;
        prev = cur;
        cur = tmp;
    }

    /* min over t <= B of E_L^t, first (lowest) t among equals. */
    int32_t t_best = 0;
    float best = prev[0];
    for (int32_t t = 1; t <= B; ++t) {
        if (prev[t] < best) {
            best = prev[t];
            t_best = t;
        }
    }
    if (!(best < INFINITY)) {
        *cost = INFINITY;
        *time_used = -1;
        memset(profile, 0xFF, (size_t)L);
        return SPDY_REF_OK;
    }
    *cost = best;
    *time_used = t_best;

    /* Walk the choices back from the last layer (end of Algorithm 1). */
    int32_t t = t_best;
    for (int32_t l = L - 1; l >= 0; --l) {
        const uint8_t k = P_work[(size_t)l * width + (size_t)t];
        if (k == 0xFF || k >= K)
            return SPDY_REF_INTERNAL;
        profile[l] = k;
        t -= times[(size_t)l * K + k];
        if (t < 0)
            return SPDY_REF_INTERNAL;
    }
    return t == 0 ? SPDY_REF_OK : SPDY_REF_INTERNAL;
}

/*
 * Batch of N candidates sharing one timing table.  Candidates [first, first+count) are solved
 * one after another on the calling thread; outputs are indexed by the absolute candidate
 * number, so several host threads can work on disjoint ranges of the same arrays.
 */
int spdy_ref_solve_range(const float *errors, const int32_t *times, int32_t L, int32_t K, int32_t B,
                         int64_t first, int64_t count, uint8_t *profile, float *cost,
                         int32_t *time_used)
{
    if (count < 0 || first < 0 || L < 1 || K < 1 || B < 0)
        return SPDY_REF_BAD_ARG;
    if (count == 0)
        return SPDY_REF_OK;
    const size_t width = (size_t)B + 1;
    float *D = (float *)malloc(2 * width * sizeof(float));
    uint8_t *P = (uint8_t *)malloc((size_t)L * width);
    if (!D || !P) {
        free(D);
        free(P);
        return SPDY_REF_NO_MEMORY;
    }
    int rc = SPDY_REF_OK;
    for (int64_t n = first; n < first + count && rc == SPDY_REF_OK; ++n) {
        rc = spdy_ref_solve_one(errors + (size_t)n * L * K, times, L, K, B,
                                profile + (size_t)n * L, cost + n, time_used + n, D, P);
    }
    free(D);
    free(P);
    return rc;
}

/*
 * Full last row E_L^t for one candidate (t = 0..B), for tests that look at more than the
 * minimum (e.g. monotonicity of the prefix minimum in the budget).
 */
int spdy_ref_last_row(const float *errors, const int32_t *times, int32_t L, int32_t K, int32_t B,
                      float *row_out)
{
    if (!errors || !times || !row_out || L < 1 || K < 1 || B < 0)
        return SPDY_REF_BAD_ARG;
    const size_t width = (size_t)B + 1;
    float *D = (float *)malloc(2 * width * sizeof(float));
    if (!D)
        return SPDY_REF_NO_MEMORY;
    float *prev = D, *cur = D + width;
    for (size_t t = 0; t < width; ++t)
        prev[t] = INFINITY;
    prev[0] = 0.0f;
    for (int32_t l = 0; l < L; ++l) {
        for (size_t t = 0; t < width; ++t)
            cur[t] = INFINITY;
        for (int32_t k = 0; k < K; ++k) {
            const int32_t tau = times[(size_t)l * K + k];
            if (tau < 0 || tau > B)
                continue;
            const float e = errors[(size_t)l * K + k];
            for (int32_t t = tau; t <= B; ++t) {
                const float v = prev[t - tau] + e;
                if (v < cur[t])
                    cur[t] = v;
            }
        }
        float *tmp = prev;
        prev = cur;
        cur = tmp;
    }
    memcpy(row_out, prev, width * sizeof(float));
    free(D);
    return SPDY_REF_OK;
}
