/*
 * spdy_dp.h - C ABI of the batched SPDY dynamic program for NVIDIA B200 (sm_100a).
 *
 * The problem (Frantar & Alistarh, "SPDY: Accurate Pruning with Speedup Guarantees",
 * Section 3.1, Eq. 1): for each of L layers pick one of K choices so that the summed error is
 * minimal while the summed (integer, bucketed) time stays within a budget B.  Section 3.2
 * (Eq. 2-3) gives the exact dynamic program over "lowest error of the first l layers taking
 * exactly t buckets"; Appendix A (Algorithm 1) adds the choice table and the walk back from the
 * last layer that recovers the profile.  This library solves N such problems at once - the N
 * candidate error tables one step of the search of Section 3.3 / Algorithm 4 proposes - that
 * share one timing table.
 *
 * Semantics fixed here (bit-exact, fp32, round-to-nearest, one add per cell):
 *   D_0[0] = +0, D_0[t>0] = +inf;
 *   D_l[t] = min over k (ascending, strict "<": lowest k wins ties) of D_{l-1}[t - times[l][k]]
 *            + errors[n][l][k], over the choices with times[l][k] <= t;
 *   t*     = lowest t in [0, B] minimising D_L[t];   cost = D_L[t*];   time_used = t*;
 *   profile[l] = the winning k along the walk back from (L, t*).
 * A candidate with no profile of finite error inside the budget is not an error: it gets
 * cost = +inf, time_used = -1 and profile bytes 0xFF.
 *
 * Value domain: errors may be any finite fp32 or +inf (a choice that must not be taken);
 * NaN and -inf are invalid (results unspecified, no fault).  times are >= 0, may be 0, may repeat
 * and may exceed B (such a choice is unusable).  1 <= K <= 255, L >= 1, B >= 0, N >= 0.
 *
 * All functions return SPDY_OK (0) or a negative spdy_status; none throws, aborts or traps.
 * "host" / "device" below says where a pointer must point.  The library keeps no caller
 * pointer beyond the stream work it enqueued.
 */
#ifndef SPDY_DP_H
#define SPDY_DP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum spdy_status {
    SPDY_OK = 0,
    SPDY_ERR_INVALID_ARG = -1,        /* null pointer, size out of range, negative time, bad alignment */
    SPDY_ERR_WORKSPACE_TOO_SMALL = -2, /* workspace cannot hold even one candidate's table */
    SPDY_ERR_UNSUPPORTED = -3,        /* rows too wide for the largest launch shape on this device */
    SPDY_ERR_CUDA = -4,               /* a CUDA runtime call failed; see spdy_last_cuda_error() */
    SPDY_ERR_NO_MEMORY = -5,          /* host or device allocation failed */
    SPDY_ERR_INTERNAL = -6,           /* a self-check inside the kernels failed */
    SPDY_ERR_STATIC_LIMIT = -7,       /* spdy_solve_batch_static: problem exceeds its built-in scratch */
    SPDY_ERR_NO_DEVICE_CODE = -8      /* a device was asked of the host-only build of the library */
} spdy_status;

/*
 * What the forward kernel stores per live cell for the walk back.  Both give identical outputs.
 *   ROW_F32 keeps Algorithm 1's matrix D (the row values) and lets the walk back re-derive, at
 *   each of the L cells it visits, the lowest k whose fp32 sum D_{l-1}[t - times[l][k]] +
 *   errors[n][l][k] equals D_l[t] bit for bit.  The forward pass then needs only add + minimum
 *   per cell, merges choices of equal time unconditionally, and runs about 1.3x faster; the table is
 *   4 bytes per cell.
 *   ARG_U8 keeps Algorithm 1's matrix P (the winning choice index), one byte per cell, at the
 *   price of a compare and a select (taken over pairs of choices) per cell update on top of add and
 *   minimum: about 1.3x the forward time of ROW_F32.  Use it when workspace is scarce.
 *   Equal-time choices can be merged here only for candidates whose errors do not fall with the
 *   choice index inside any group of equal-time choices (always true for Eq. 4's errors with
 *   non-negative coefficients); a small kernel tests that per candidate, and the others run with one
 *   slot per choice.  The workspace then carries one extra 256 bytes per candidate.
 */
typedef enum spdy_table_format {
    SPDY_TABLE_DEFAULT = 0, /* let the plan choose (currently SPDY_TABLE_ROW_F32) */
    SPDY_TABLE_ARG_U8 = 1,
    SPDY_TABLE_ROW_F32 = 2
} spdy_table_format;

/* Which kernel family runs the forward pass when one CTA-sized unit works on a candidate. */
typedef enum spdy_kernel {
    SPDY_KERNEL_AUTO = 0, /* let the plan choose */
    SPDY_KERNEL_CTA = 1,  /* one CTA per candidate, one block barrier per layer */
    SPDY_KERNEL_WARP = 2  /* one warp per candidate, four candidates per CTA, no block barrier: for rows a
                             warp pass or two wide (a budget of about a thousand buckets) */
} spdy_kernel;

typedef struct spdy_options {
    int32_t table_format;  /* spdy_table_format */
    int32_t threads;       /* threads per CTA, 0 = choose; one of 128, 256, 512, 1024 and >= K */
    int32_t cluster;       /* CTAs cooperating on one candidate: 0 = choose, 1 = one CTA; 2, 4 or 8 = a
                              thread-block cluster that splits every row, which shortens the latency of
                              batches with fewer candidates than SMs.  1 also forbids the fallbacks for
                              rows too wide for one CTA's shared memory (UNSUPPORTED instead) */
    int32_t forward_mode;  /* 0 = choose.  Variants of the forward kernel's cell update, all with
                              identical results, for measurement: 1 compare+select (ARG_U8),
                              2 compare+predicated moves (ARG_U8), 3 fp32 minimum (ROW_F32),
                              4 packed adds + 3-input minimum over slot pairs (ROW_F32),
                              5 3-input minimum over slot pairs, the winner inside a pair settled once per
                              warp pass (ARG_U8) */
    int32_t rows_in_global; /* 1: keep the two dynamic-program rows in the workspace (global memory) rather than
                              in shared memory and read them through L1.  Chosen automatically when two rows
                              do not fit one CTA's shared memory (B of about 10^5 buckets and more); any width
                              runs.  One CTA of 1024 threads per candidate; not combinable with cluster > 1 */
    int32_t kernel;        /* spdy_kernel */
    int32_t schedule;      /* how a row is cut into warp passes.  Bits 0-7: 0 = the plan's choice (2 with the
                              fp32 table, 1 with the uint8 table); 1 = passes of one length per layer, dealt
                              round-robin; 2 = as many passes, cut where their costs are level (fewer updates
                              wasted on slots that overlap a pass only partly); 3 = passes sized by dynamic
                              programming and dealt to the warps by load (least waste, most passes, measured
                              slowest; for measurement).  Bits 8-15: upper limit of cells per lane per pass,
                              1..48 (0 = the kernel's own limit; for measurement) */
    int32_t auto_shape;    /* 0: when threads, cluster, rows_in_global and kernel are all 0 the plan also lays
                              out launch shapes for batches too small to fill the device (larger CTAs, clusters
                              of 2/4/8) and spdy_solve_batch picks by N; 1: never, one shape for every N */
} spdy_options;

/* Facts about a plan: shapes, the launch shape chosen, and work counts for measurement. */
typedef struct spdy_plan_info {
    int32_t L, K, B;
    int32_t feasible;       /* 0: sum of per-layer minimum times exceeds B, every candidate is infeasible */
    int32_t max_width;      /* widest live band, in cells */
    int32_t span;           /* most cells one warp processes per pass */
    int32_t threads;        /* threads per CTA */
    int32_t cluster;        /* CTAs per candidate */
    int32_t table_format;   /* resolved spdy_table_format */
    int32_t ctas_per_sm;    /* resident CTAs per SM the launch shape allows */
    int32_t sm_count;
    int32_t rows_in_global; /* 1 if the row buffers live in the workspace */
    int64_t smem_bytes;     /* dynamic shared memory per CTA */
    int64_t table_bytes_per_candidate; /* workspace one candidate needs: walk-back table (+ row buffers) */
    int64_t band_cells;     /* sum over layers of the live band width (cells written per candidate) */
    int64_t useful_updates; /* sum over (layer, choice) of cells whose source lies in the previous band */
    int64_t issued_updates; /* cell updates the kernel actually issues per candidate (span granularity) */
    int64_t nominal_updates;/* L*K*B per candidate, the unit of the headline metric */
    int64_t distinct_updates; /* like useful_updates after choices of a layer with equal times are merged
                                 into one shift: the cell updates the forward pass has to perform.  With the
                                 byte table this is the count for candidates that may be merged (see
                                 spdy_table_format); issued_updates is given for the same table set */
    int32_t launches_per_wave; /* kernels one wave of candidates launches (2, or 5 with the byte table's two table sets) */
    int32_t kernel;            /* spdy_kernel of the main launch shape (CTA also for clusters and rows in global memory) */
    int32_t forward_mode;      /* resolved cell-update variant (see spdy_options.forward_mode) */
    int32_t candidates_per_cta;/* 1, or 4 with one warp per candidate */
    int32_t alternates;        /* further launch shapes laid out for small batches (see spdy_options.auto_shape) */
    int32_t reserved1;
} spdy_plan_info;

typedef struct spdy_plan spdy_plan; /* opaque; owns only its own small host and device tables */

/*
 * Build a plan for one timing table and budget (Eq. 1's constraint; the live band of each DP
 * row follows from the per-layer minimum and maximum times).  Synchronous; small host work plus
 * one small host-to-device copy on `device`.
 *   times_host  host, [L][K] int32 row-major, read during the call only.
 *   device      CUDA device ordinal, or -1 for a host-only plan (info queries only; solving
 *               with it returns SPDY_ERR_INVALID_ARG).  The host-only build of the library
 *               (libspdy_plan_host.so: plans, helpers, no kernels) accepts -1 only.
 *   opts        host, may be NULL for defaults.
 *   *out        receives the plan; destroy with spdy_plan_destroy.
 * Errors: INVALID_ARG (null, L<1, K<1, K>255, B<0, a negative time, bad option), UNSUPPORTED
 * (band too wide for the launch shape the options pin), NO_MEMORY, CUDA.
 */
int spdy_plan_create(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B,
                     int device, const spdy_options *opts);
void spdy_plan_destroy(spdy_plan *plan);

/* Fill *info (host).  INVALID_ARG on null. */
int spdy_plan_get_info(const spdy_plan *plan, spdy_plan_info *info);

/* Per-layer live band [lo, lo+width) of row l (l = 1..L stored at index l-1); host arrays of L
 * int32 each, either may be NULL.  For an infeasible plan widths are 0. */
int spdy_plan_get_bands(const spdy_plan *plan, int32_t *lo_host, int32_t *width_host);

/*
 * Inspection of a plan's host tables, for tests and tools (no GPU work).  `which` selects the table set:
 * 0 = the main launch shape, -1 = the byte table's second set with merged equal-time choices (INVALID_ARG
 * if there is none), i >= 1 = the i-th launch shape for small batches.  The pointers stay valid until the
 * plan is destroyed.
 *   layers      [L][8] int32: width, row offset in the table, lo, smallest usable time, extent (cells the
 *               passes write, a multiple of 32), shift slots, fill (cells of +inf refilled behind the row:
 *               as far as the next layer reads beyond the extent), 0
 *   slots       [L][K][2] int32: (a, b) of each shift slot: it contributes to band cells a..b and reads the
 *               previous row at cell - a (the first layers[l][5] entries of a layer are valid)
 *   passes      [n_passes][2]: first cell, and u_lo | u_hi << 8 | dense << 16 | cells_per_lane << 24
 *   pass_masks  [n_passes][mask_words] uint64: bit u set = slot u overlaps the pass
 *   pass_ptr    [L * warps_per_candidate + 1]: the passes of (layer l, warp w) are pass_ptr[l*W+w] ..
 *               pass_ptr[l*W+w+1] (NULL for a cluster shape, whose passes are listed per slice)
 *   slices      [L][cluster][8] int32 for a cluster shape (slice_lo, slice_hi, cells per lane, passes, first
 *               pass, first window cell, window length, slice length of the previous row), else NULL
 * spdy_plan_verify re-derives on the host, for every layer, pass and slot of every table set of the plan, the
 * lowest and highest row-buffer cell a lane reads and the cells it writes, and checks them against the
 * buffers' extents and against the region known to hold the previous row or +inf (Algorithm 1's shifted
 * read D[l-1, t - t_l^s]): SPDY_OK, or SPDY_ERR_INTERNAL on the first violation.  Every plan is verified
 * this way when it is created.
 */
typedef struct spdy_plan_tables {
    int32_t L, K;
    int32_t kernel_kind;         /* 0 CTA per candidate, 1 CTA with rows in global memory, 2 cluster, 3 warp per candidate */
    int32_t threads, warps_per_candidate, cluster, forward_mode;
    int32_t max_cells_per_lane;  /* the kernel build's largest pass */
    int32_t row_stride, pad;     /* floats per row buffer; guard cells of +inf below cell 0 of a row */
    int32_t out_stride, win_stride; /* cluster shape: floats per slice buffer and per window */
    int32_t mask_words, n_passes;
    int64_t pitch;               /* table cells per candidate */
    const int32_t *layers;
    const int32_t *slots;
    const int32_t *passes;
    const uint64_t *pass_masks;
    const int32_t *pass_ptr;
    const int32_t *slices;
} spdy_plan_tables;
int spdy_plan_get_tables(const spdy_plan *plan, int32_t which, spdy_plan_tables *out);

/* Which table set spdy_solve_batch would run a batch of N candidates on, given `workspace_bytes` of
 * workspace: 0 = the main launch shape, i >= 1 = the i-th launch shape for small batches (the index
 * spdy_plan_get_tables takes).  Returns -1 for a null plan. */
int32_t spdy_plan_shape_for_batch(const spdy_plan *plan, int64_t N, size_t workspace_bytes);
int spdy_plan_verify(const spdy_plan *plan);

/* The walk-back table is Algorithm 1's L x (T+1) matrix (the O(L*T) memory of Section 3.2), kept per
 * candidate and cut down to the live band of each row.
 * Bytes of workspace that let N candidates run as a single wave.  Any workspace of at least
 * spdy_workspace_bytes(plan, 1) is accepted; a smaller-than-full one makes the batch run as
 * several waves on the stream.  Returns 0 for a null plan or N <= 0. */
size_t spdy_workspace_bytes(const spdy_plan *plan, int64_t N);

/*
 * Solve N candidates (Eq. 2-3 forward, final min over t <= B, walk back of Algorithm 1).
 * Asynchronous: enqueues kernels on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 * default stream) and returns; outputs are valid once the stream reaches that point.
 *   errors_dev     device, [N][L][K] fp32 row-major, 4-byte aligned.
 *   profile_dev    device, [N][L] uint8 out: choice index per layer (0xFF.. if infeasible).
 *   cost_dev       device, [N] fp32 out.
 *   time_used_dev  device, [N] int32 out (-1 if infeasible).
 *   workspace_dev  device, caller-owned scratch of workspace_bytes bytes, 256-byte aligned;
 *                  contents undefined afterwards; must not be shared by solves that overlap.
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, CUDA (launch failure).
 */
int spdy_solve_batch(const spdy_plan *plan, const float *errors_dev, int64_t N,
                     uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev,
                     void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/*
 * Same computation with HOST buffers (pageable or pinned): copies errors to the device, solves,
 * copies the three outputs back and waits for the stream.  Device staging memory is owned by
 * the plan and grows on demand (cudaMalloc on first use or growth), so one plan must not run
 * two host-buffer solves at the same time.  An error table larger than one wave of CTAs is uploaded in
 * a few chunks on a second, plan-owned stream (ordered after the work already queued on `cuda_stream`),
 * each chunk's kernels waiting only for their own chunk, so that with pinned host memory the upload
 * hides behind the kernels; chunk sizes follow the upload and solving rates the previous call on the plan
 * measured, and a table whose upload is cheaper than a chunk boundary goes up in one piece.
 */
int spdy_solve_batch_host(spdy_plan *plan, const float *errors_host, int64_t N,
                          uint8_t *profile_host, float *cost_host, int32_t *time_used_host,
                          void *cuda_stream);

/*
 * The same path with the errors of the search's error model (Section 3.3, Eq. 4) instead of a table:
 *   errors[n][l][i] = coeffs[n][l] * (i / (K - 1))^2,   i = 0 .. K-1 the choice index,
 * formed inside the kernels as ONE fp32 round-to-nearest multiply of the coefficient with
 * fp32((i / (K - 1))^2) (the square taken in fp64 and rounded once; K = 1 gives 0).  This is what one
 * evaluation of Algorithm 4 submits: a candidate is L coefficients rather than L*K errors, so the
 * input shrinks K-fold.  Results are bit-identical to spdy_solve_batch on the table that
 * spdy_quadratic_errors writes for the same coefficients.
 *   coeffs_dev   device, [N][L] fp32 (the paper draws them from [0, 1]; any finite value is accepted).
 * Everything else as for spdy_solve_batch / spdy_solve_batch_host.
 */
int spdy_solve_batch_coeffs(const spdy_plan *plan, const float *coeffs_dev, int64_t N,
                            uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev,
                            void *workspace_dev, size_t workspace_bytes, void *cuda_stream);
int spdy_solve_batch_coeffs_host(spdy_plan *plan, const float *coeffs_host, int64_t N,
                                 uint8_t *profile_host, float *cost_host, int32_t *time_used_host,
                                 void *cuda_stream);

/*
 * Eq. 4 written out: errors_dev[n][l][i] = coeffs_dev[n][l] * (i / (K - 1))^2 with the arithmetic stated
 * above.  Device pointers on the current device ([N][L] in, [N][L][K] out), asynchronous on
 * `cuda_stream`.  INVALID_ARG on null pointers or sizes < 1 (N = 0 is a no-op).
 */
int spdy_quadratic_errors(const float *coeffs_dev, int64_t N, int32_t L, int32_t K, float *errors_dev,
                          void *cuda_stream);

/*
 * Host-side helpers around the path (no GPU work).
 *
 * spdy_time_target: the execution-time target of a speedup target X (Section 3.1):
 *   T = T_dense / X - T_base, T_base the run time of everything pruning does not touch.
 *
 * spdy_bucketize_times: time discretisation of Section 3.2 - B buckets of width T / B, so that the
 *   budget T becomes B.  out[l][k] = round(times[l][k] * B / T) in fp64, to the nearest integer with
 *   halves away from zero (SPDY_ROUND_NEAREST) or upwards (SPDY_ROUND_UP; then a profile within B
 *   buckets is within T in real time).  times_host [L][K] fp64 >= 0, out_host [L][K] int32, both host.
 *   INVALID_ARG on null, T <= 0, B < 1, a negative or non-finite time, or a result beyond int32.
 *
 * spdy_uniform_profile: the "uniform" baseline of Section 4 - the lowest choice index k (choices in
 *   order of increasing sparsity) such that every layer at choice k fits the budget B; layers flagged
 *   in keep_dense_host ([L] bytes, may be NULL) stay at choice 0.  *choice_out = k or -1 if none fits,
 *   *total_out (may be NULL) = that profile's total time or -1.  times_host [L][K] int32 >= 0.
 */
typedef enum spdy_rounding { SPDY_ROUND_NEAREST = 0, SPDY_ROUND_UP = 1 } spdy_rounding;
double spdy_time_target(double t_dense, double speedup, double t_base);
int spdy_bucketize_times(const double *times_host, int32_t L, int32_t K, double T, int32_t B, int32_t rounding,
                         int32_t *out_host);
int spdy_uniform_profile(const int32_t *times_host, int32_t L, int32_t K, int32_t B, const uint8_t *keep_dense_host,
                         int32_t *choice_out, int64_t *total_out);

/*
 * SPDY's search for the sensitivity coefficients (Section 3.3; Appendix B, Algorithm 4) with the dynamic
 * programs of all pending trials solved as one batch.  Host loop; synchronous.
 *
 * Algorithm 4 samples c0 and `trials` more coefficient vectors, keeps the best, then for neighbourhood
 * sizes d = ceil(delta * L) .. 1 mutates the best vector c* in d random entries `trials` times per size,
 * accepting a mutation when its profile evaluates strictly better.  What a trial resamples does not depend
 * on c*, so this call forms the proposals of all remaining trials of a size from the current c* at once,
 * solves their dynamic programs (Eq. 4 errors, spdy_solve_batch_coeffs_host) as one batch and evaluates
 * the profiles in trial order up to the first improvement; the proposals behind it are rebuilt from the
 * new c*.  Decisions, result and the number of evaluations equal the sequential algorithm's.
 *
 *   plan         a plan for the timing table and budget (K = plan's K, L = plan's L)
 *   c0_host      [L] fp32, phase1_host [trials][L] fp32: the random vectors of the first loop (the caller
 *                draws them: the paper samples uniformly from [0, 1])
 *   opts         trials (Algorithm 4's k), delta (its neighbourhood fraction), patience: 0 = `trials` trials
 *                per size as Algorithm 4 prints it, p > 0 = stop a size after p trials in a row without
 *                improvement, as the text of Section 3.3 says; max_batch: most dynamic programs per solver
 *                call (0 = 65536)
 *   draw         called as draw(d, trial, indices[d], values[d], user): the d distinct entries (0 .. L-1) and
 *                their new values that trial `trial` of size d resamples; must not depend on earlier calls
 *   eval         eval(profile[L], L, user) -> the loss of that profile (Section 3.4: the calibration loss of
 *                the stitched model), lower is better; profile bytes 0xFF = infeasible, return +inf
 *   solve        NULL = this library on the plan's device; else solve(coeffs[n][L], n, profile[n][L], user)
 *                -> status, which lets the loop run against another solver (tests use the CPU oracle)
 *   c_out_host [L], profile_out_host [L], *result: the best vector, its profile, loss and counters
 *   accepted_d_host / accepted_trial_host [accepted_capacity], may be NULL with capacity 0: the accepted
 *                trials in order, d = 0 for the first loop; result->accepted counts all of them
 * Errors: INVALID_ARG, NO_MEMORY, NO_DEVICE_CODE (solve NULL on a host-only plan or build), the solver's.
 */
typedef double (*spdy_eval_fn)(const uint8_t *profile_host, int32_t L, void *user);
typedef void (*spdy_draw_fn)(int32_t d, int32_t trial, int32_t *indices_host, float *values_host, void *user);
typedef int (*spdy_solve_fn)(const float *coeffs_host, int64_t n, uint8_t *profile_host, void *user);
typedef struct spdy_search_options {
    int32_t trials;
    int32_t patience;
    double delta;
    int64_t max_batch;
} spdy_search_options;
typedef struct spdy_search_result {
    double loss;
    int64_t evals;         /* calls of eval */
    int64_t accepted;      /* accepted trials */
    int64_t dp_batches;    /* solver calls */
    int64_t dp_candidates; /* dynamic programs solved */
    double dp_seconds, eval_seconds;
} spdy_search_result;
int spdy_search(spdy_plan *plan, const float *c0_host, const float *phase1_host, const spdy_search_options *opts,
                spdy_draw_fn draw, void *draw_user, spdy_eval_fn eval, void *eval_user, spdy_solve_fn solve,
                void *solve_user, void *cuda_stream, float *c_out_host, uint8_t *profile_out_host,
                spdy_search_result *result, int32_t *accepted_d_host, int32_t *accepted_trial_host,
                int64_t accepted_capacity);

/*
 * One-shot form of the whole path, in the shape of the problem statement of Section 3.1 (Eq. 1: errors
 * e_l^s, times t_l^s, budget T in, one choice per layer out): errors[N][L][K], times[L][K], budget B ->
 * profile, cost, time_used, all device pointers on the current device.  Reads times back to
 * the host, builds a transient plan, allocates and frees its own workspace, and waits for the
 * stream before returning (synchronous).  Convenience for callers that solve once.
 */
int spdy_solve_batch_simple(const float *errors_dev, const int32_t *times_dev, int64_t N,
                            int32_t L, int32_t K, int32_t B, uint8_t *profile_dev, float *cost_dev,
                            int32_t *time_used_dev, void *cuda_stream);

/*
 * Read and clear the plan's device-side self-check word: the walk-back kernels set it if a table
 * entry is not a valid choice or the walk does not end at t = 0 (which would mean corrupted
 * scratch or invalid inputs such as NaN).  Waits for `cuda_stream`.  Returns SPDY_OK,
 * SPDY_ERR_INTERNAL if the word was set, or a CUDA error.
 */
int spdy_plan_check_status(spdy_plan *plan, void *cuda_stream);

/*
 * The same word, returned rather than judged: *word_host receives it (0 = nothing flagged) and it is
 * cleared.  Bit 0: the walk back met an invalid table entry.  The remaining bits are set only by the debug
 * build of the library (libspdy_dp_debug.so, compiled with SPDY_DEBUG_CHECKS), in which every row-buffer
 * and table access of the forward kernels tests its index first and a bad access is recorded and skipped
 * instead of performed: bit 1 = a read of the previous row (Algorithm 1's D[l-1, t - t_l^s]) outside the
 * cells known to hold the row or +inf, bit 2 = a read that returned the marker of a cell not yet written,
 * bit 3 = a store outside its row or table.  spdy_debug_checks_enabled() tells which build is loaded.
 */
int spdy_plan_status_word(spdy_plan *plan, void *cuda_stream, int32_t *word_host);
int spdy_debug_checks_enabled(void);

/*
 * Measurement aid.  With timing on, every spdy_solve_batch on this plan records CUDA events on
 * the solve's stream around the forward kernel(s) and around the walk-back kernel(s);
 * spdy_plan_last_timing waits for the last solve's events and returns the summed durations in
 * milliseconds (either pointer may be NULL).  Off by default; adds three event records per wave.
 * A plan with timing on must not run solves concurrently from several host threads.
 */
int spdy_plan_enable_timing(spdy_plan *plan, int on);
int spdy_plan_last_timing(spdy_plan *plan, float *forward_ms_host, float *walkback_ms_host);

/*
 * (No counterpart in the paper: a deployment convenience.)
 *
 * The same path - forward dynamic program, final minimum, walk back - for callers that are not
 * allowed to allocate device memory: code that runs under a framework which owns the whole
 * device heap and forbids side allocations, services that fix their memory footprint at start-up,
 * or a process that has already handed every free byte to another pool.  This call makes no CUDA
 * allocation of any kind (no cudaMalloc / cudaFree / pool or async allocation, no allocating
 * library routine); its only scratch is an array of SPDY_STATIC_SCRATCH_BYTES compiled into the
 * library, which every device that loads the library holds until the process exits.  The array
 * carries the plan's small tables and the walk-back table (one byte per live cell); a batch whose
 * table is larger runs as several waves.  The caller still passes every input and output.
 *
 *   errors_dev     device, [N][L][K] fp32.          times_host  host, [L][K] int32.
 *   profile_dev / cost_dev / time_used_dev          device outputs as for spdy_solve_batch.
 *
 * Behaviour to know about:
 *   - Works on the current device.  Synchronous: waits for `cuda_stream` before returning.
 *   - The first call on each device looks up the array's device address through the runtime
 *     (which may load the module); make that first call outside any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the last call left.  The
 *     only word that must start at zero, the self-check flag, is cleared on the stream at each
 *     call.  Two calls whose GPU work overlaps (different streams or host threads) race on the
 *     array: serialise them.
 *   - Limits: returns SPDY_ERR_STATIC_LIMIT when the plan tables plus ONE candidate's table do
 *     not fit the array, or when a row is too wide for a single CTA (the cluster variant is not
 *     offered here).  The BERT-base shape (L 72, K 42, B 10000) needs about 0.4 MB per candidate.
 * Other errors as for spdy_solve_batch (INVALID_ARG, CUDA, INTERNAL).
 */
#define SPDY_STATIC_SCRATCH_BYTES (64u << 20)
int spdy_solve_batch_static(const float *errors_dev, const int32_t *times_host, int64_t N, int32_t L,
                            int32_t K, int32_t B, uint8_t *profile_dev, float *cost_dev,
                            int32_t *time_used_dev, void *cuda_stream);

/* Size in bytes of the array spdy_solve_batch_static works in (SPDY_STATIC_SCRATCH_BYTES). */
size_t spdy_static_scratch_bytes(void);

/*
 * Measurement aid: the two ceilings of the forward pass (Eq. 2's update = one read of the previous row,
 * one add, one minimum) as this device delivers them, from two short probe kernels on the default
 * stream of `device` (about 50 ms; allocates and frees a small buffer; synchronous).
 *   *lds_reads_per_s          4-byte shared-memory reads per second, lane-consecutive, all SMs
 *   *cell_updates_alu_per_s   cell updates per second of the arithmetic alone (packed fp32 adds and
 *                             3-input minima on registers)
 * Either pointer may be NULL.  Errors: INVALID_ARG, NO_MEMORY, CUDA.
 */
int spdy_probe_peaks(int device, double *lds_reads_per_s, double *cell_updates_alu_per_s);

/* Static, human-readable text for a status code. */
const char *spdy_strerror(int status);

/* The cudaError_t value of the most recent failed CUDA call on this host thread (0 if none). */
int spdy_last_cuda_error(void);

/* Library version, major*1000 + minor. */
int spdy_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPDY_DP_H */
