// SPDY's search for the sensitivity coefficients (Section 3.3; Appendix B, Algorithm 4) with the dynamic
// programs of many trials solved as one batch.  Host logic in plain C++; the dynamic programs run through a
// solver callback or, by default, through the CUDA part of the library (coefficient input, host buffers).
//
// Algorithm 4 is sequential: every trial mutates the current best vector c* and replaces it when the
// mutated vector's profile evaluates better.  What a trial resamples (which entries, which values) does
// not depend on c*, so the proposals of all remaining trials of a neighbourhood size can be formed from
// the current c* at once and their dynamic programs solved as one batch.  The profiles are then evaluated
// one by one in trial order, stopping at the first improvement; the proposals behind it were built from a
// c* that is now stale and are rebuilt in the next batch.  Trial for trial this takes the same decisions
// as the sequential algorithm and calls the (expensive) evaluation exactly as often; only dynamic programs
// are solved speculatively.
#include "spdy_plan.h"

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

using namespace spdy;

namespace {

double seconds_since(const std::chrono::steady_clock::time_point &t0)
{
    return std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
}

}  // namespace

extern "C" int spdy_search(spdy_plan *plan, const float *c0_host, const float *phase1_host,
                           const spdy_search_options *opts, spdy_draw_fn draw, void *draw_user, spdy_eval_fn eval,
                           void *eval_user, spdy_solve_fn solve, void *solve_user, void *cuda_stream,
                           float *c_out_host, uint8_t *profile_out_host, spdy_search_result *result,
                           int32_t *accepted_d_host, int32_t *accepted_trial_host, int64_t accepted_capacity)
{
    if (!plan || !c0_host || !opts || !draw || !eval || !c_out_host || !profile_out_host || !result)
        return SPDY_ERR_INVALID_ARG;
    const int32_t L = plan->L, trials = opts->trials;
    const int64_t max_batch = opts->max_batch > 0 ? opts->max_batch : 65536;
    if (trials < 0 || opts->patience < 0 || !(opts->delta >= 0.0) || !(opts->delta <= 1.0) || (trials > 0 && !phase1_host) ||
        accepted_capacity < 0 || (accepted_capacity > 0 && (!accepted_d_host || !accepted_trial_host)))
        return SPDY_ERR_INVALID_ARG;
    if (!solve && (plan->device < 0 || !device_hooks() || !device_hooks()->solve_coeffs_host)) return SPDY_ERR_NO_DEVICE_CODE;
    std::memset(result, 0, sizeof(*result));

    try {
        std::vector<float> proposals;
        std::vector<uint8_t> profiles;
        std::vector<int32_t> idx(static_cast<size_t>(std::max(1, L)));
        std::vector<float> val(static_cast<size_t>(std::max(1, L)));
        std::vector<float> c_star(c0_host, c0_host + L);
        std::vector<uint8_t> prof_star(static_cast<size_t>(L), 0xFF);
        double best = 0.0;

        // Dynamic programs of `count` coefficient vectors, at most max_batch per call of the solver.
        auto solve_all = [&](int64_t count) -> int {
            profiles.resize(static_cast<size_t>(count) * L);
            const auto t0 = std::chrono::steady_clock::now();
            for (int64_t lo = 0; lo < count; lo += max_batch) {
                const int64_t n = std::min(max_batch, count - lo);
                const float *in = proposals.data() + static_cast<size_t>(lo) * L;
                uint8_t *out = profiles.data() + static_cast<size_t>(lo) * L;
                const int rc = solve ? solve(in, n, out, solve_user)
                                     : device_hooks()->solve_coeffs_host(plan, in, n, out, cuda_stream);
                if (rc != SPDY_OK) return rc;
                result->dp_batches += 1;
            }
            result->dp_candidates += count;
            result->dp_seconds += seconds_since(t0);
            return SPDY_OK;
        };
        auto evaluate = [&](const uint8_t *profile) {
            result->evals += 1;
            const auto t0 = std::chrono::steady_clock::now();
            const double v = eval(profile, L, eval_user);
            result->eval_seconds += seconds_since(t0);
            return v;
        };
        auto accept = [&](const float *c, const uint8_t *profile, double v, int32_t d, int32_t trial) {
            std::copy(c, c + L, c_star.begin());
            std::copy(profile, profile + L, prof_star.begin());
            best = v;
            if (result->accepted < accepted_capacity) {
                accepted_d_host[result->accepted] = d;
                accepted_trial_host[result->accepted] = trial;
            }
            result->accepted += 1;
        };

        // First loop of Algorithm 4: c0 and `trials` fresh samples, one batch, evaluated in order.
        proposals.assign(c0_host, c0_host + L);
        if (trials > 0) proposals.insert(proposals.end(), phase1_host, phase1_host + static_cast<size_t>(trials) * L);
        int rc = solve_all(1 + trials);
        if (rc != SPDY_OK) return rc;
        best = evaluate(profiles.data());
        std::copy(profiles.begin(), profiles.begin() + L, prof_star.begin());
        for (int32_t j = 0; j < trials; ++j) {
            const uint8_t *pr = profiles.data() + static_cast<size_t>(1 + j) * L;
            const double v = evaluate(pr);
            if (v < best) accept(phase1_host + static_cast<size_t>(j) * L, pr, v, 0, j);
        }

        // Second loop: neighbourhood sizes d = ceil(delta L) .. 1.  patience = 0 runs `trials` trials per
        // size as Algorithm 4 prints it; patience > 0 stops a size after that many trials in a row without
        // improvement, as the text of Section 3.3 says.
        for (int32_t d = static_cast<int32_t>(std::ceil(opts->delta * L)); d >= 1; --d) {
            int64_t j = 0, since_improved = 0;
            for (;;) {
                const int64_t remaining = opts->patience == 0 ? trials - j : opts->patience - since_improved;
                if (remaining <= 0) break;
                const int64_t count = std::min(remaining, max_batch);
                proposals.resize(static_cast<size_t>(count) * L);
                for (int64_t i = 0; i < count; ++i) {
                    float *row = proposals.data() + static_cast<size_t>(i) * L;
                    std::copy(c_star.begin(), c_star.end(), row);
                    draw(d, static_cast<int32_t>(j + i), idx.data(), val.data(), draw_user);
                    for (int32_t q = 0; q < d && q < L; ++q) {
                        if (idx[q] < 0 || idx[q] >= L) return SPDY_ERR_INVALID_ARG;
                        row[idx[q]] = val[q];
                    }
                }
                rc = solve_all(count);
                if (rc != SPDY_OK) return rc;
                int64_t improved_at = -1;
                for (int64_t i = 0; i < count; ++i) {
                    const uint8_t *pr = profiles.data() + static_cast<size_t>(i) * L;
                    const double v = evaluate(pr);
                    if (v < best) {
                        accept(proposals.data() + static_cast<size_t>(i) * L, pr, v, d, static_cast<int32_t>(j + i));
                        improved_at = i;
                        break;
                    }
                }
                if (improved_at >= 0) {
                    j += improved_at + 1;
                    since_improved = 0;
                } else {
                    j += count;
                    since_improved += count;
                }
            }
        }
        std::copy(c_star.begin(), c_star.end(), c_out_host);
        std::copy(prof_star.begin(), prof_star.end(), profile_out_host);
        result->loss = best;
    } catch (const std::bad_alloc &) {
        return SPDY_ERR_NO_MEMORY;
    }
    return SPDY_OK;
}
