// CUDA side of the C ABI: device state of a plan, launches of the forward kernels, the walk-back kernels
// (end of Appendix A, Algorithm 1), the host-buffer path, the peak probes and the entry point that
// allocates nothing.  The forward kernels live in spdy_device.cuh and are instantiated per cell-update
// mode in the spdy_fwd_*.cu files; the host side of a plan is spdy_plan.cpp.
#include "spdy_device.cuh"

#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

using namespace spdy;

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

// Everything a plan owns on the device (spdy_plan::dev).
struct spdy::DeviceSide {
    const FwdVariant *variant = nullptr;
    const ClusterVariant *cvariant = nullptr;
    // device tables: one allocation (`blob`), or a region of the static scratch when owns_blob is false
    bool owns_blob = true;
    unsigned char *blob = nullptr;
    int32_t *times = nullptr;
    LayerDesc *layers = nullptr;
    TapRange *slots = nullptr;
    uint8_t *slot_ptr = nullptr;
    uint8_t *slot_member = nullptr;
    unsigned long long *masks = nullptr;
    PassDesc *passes = nullptr;
    int32_t *pass_ptr = nullptr;
    int32_t *status = nullptr;
    SliceDesc *slices = nullptr;
    float *qtab = nullptr;
    // optional event timing of the last solve (three events per wave)
    bool timing = false;
    std::vector<cudaEvent_t> events;
    size_t events_used = 0;
    // host-buffer entry points: a second stream and events that let the upload of one chunk of
    // candidates overlap the kernels of the chunk before it
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t entry_event = nullptr;
    std::vector<cudaEvent_t> copy_events;
    // how fast the first chunk went up and how fast it was solved, timed in every chunked call: the ratio
    // sets how much larger than its predecessor a chunk may be for its upload to hide behind the kernels
    cudaEvent_t probe[4] = {nullptr, nullptr, nullptr, nullptr};
    double chunk_growth = 6.0;
    double upload_ms_per_byte = 0.0;  // 0 = not measured yet
    double first_wave_ms = 0.0;
    // staging for the host-buffer entry points
    unsigned char *arena = nullptr;
    size_t arena_bytes = 0;
};

namespace {

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
    if (!ok || t != 0) atomicOr(args.status, STATUS_WALK_BACK);
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
    if ((!ok || t != 0) && lane == 0) atomicOr(args.status, STATUS_WALK_BACK);
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
// Device state of a plan
// ----------------------------------------------------------------------------------------------

VariantList variants_of(int mode)
{
    switch (mode) {
        case MODE_ARG: return variants_arg();
        case MODE_ARG_PRED: return variants_arg_pred();
        case MODE_ARG_PAIR: return variants_arg_pair();
        case MODE_ROW: return variants_row();
        case MODE_ROW2: return variants_row2();
        default: return VariantList{nullptr, 0, nullptr, 0};
    }
}

void bind_tables(DeviceSide *d, const TableLayout &t, unsigned char *base)
{
    d->times = reinterpret_cast<int32_t *>(base + t.times);
    d->layers = reinterpret_cast<LayerDesc *>(base + t.layers);
    d->slots = reinterpret_cast<TapRange *>(base + t.slots);
    d->slot_ptr = base + t.slot_ptr;
    d->slot_member = base + t.slot_member;
    d->masks = reinterpret_cast<unsigned long long *>(base + t.masks);
    d->passes = reinterpret_cast<PassDesc *>(base + t.passes);
    d->pass_ptr = reinterpret_cast<int32_t *>(base + t.pass_ptr);
    d->status = reinterpret_cast<int32_t *>(base + t.status);
    d->slices = reinterpret_cast<SliceDesc *>(base + t.slices);
    d->qtab = reinterpret_cast<float *>(base + t.qtab);
}

int hook_limits(int device, DeviceLimits *out)
{
    int v = 0;
    SPDY_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, device));
    out->smem_per_sm = v;
    SPDY_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
    out->smem_per_block = v;
    SPDY_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device));
    out->sm_count = v;
    return SPDY_OK;
}

// Picks the kernel build of the plan's launch shape, raises its dynamic shared-memory limit and asks the
// driver how many CTAs (or clusters) fit.  The limit belongs to the kernel on the device, not to a plan:
// it is always set to the device's opt-in maximum less the kernel's static shared memory - every plan
// writes the same value - so that plans of different widths can live side by side.
int select_kernel(spdy_plan *p, DeviceSide *d)
{
    const VariantList list = variants_of(p->mode);
    const void *fn = nullptr;
    if (p->kind == KERNEL_CLUSTER) {
        for (int i = 0; i < list.n_cluster; ++i)
            if (list.cluster[i].threads == p->threads) d->cvariant = &list.cluster[i];
        if (!d->cvariant) return SPDY_ERR_UNSUPPORTED;
        fn = reinterpret_cast<const void *>(d->cvariant->fn);
    } else {
        for (int i = 0; i < list.n_fwd; ++i)
            if (list.fwd[i].kind == p->kind && list.fwd[i].threads == p->threads && list.fwd[i].rcap == p->rcap)
                d->variant = &list.fwd[i];
        if (!d->variant) return SPDY_ERR_UNSUPPORTED;
        fn = reinterpret_cast<const void *>(d->variant->fn);
    }
    cudaFuncAttributes fattr;
    SPDY_CUDA_TRY(cudaFuncGetAttributes(&fattr, fn));
    const int64_t max_dynamic = p->limits.smem_per_block - static_cast<int64_t>(fattr.sharedSizeBytes);
    if (p->smem_bytes > max_dynamic) return SPDY_ERR_UNSUPPORTED;
    SPDY_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(max_dynamic)));
    if (p->kind == KERNEL_CLUSTER) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(p->cluster), 1, 1);
        cfg.blockDim = dim3(static_cast<unsigned>(p->threads), 1, 1);
        cfg.dynamicSmemBytes = static_cast<size_t>(p->smem_bytes);
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = static_cast<unsigned>(p->cluster);
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        SPDY_CUDA_TRY(cudaOccupancyMaxActiveClusters(&clusters, d->cvariant->fn, &cfg));
        if (clusters < 1) return SPDY_ERR_UNSUPPORTED;
        p->ctas_per_sm = std::max(1, clusters * p->cluster / std::max(1, p->limits.sm_count));
    } else {
        int occ = 0;
        SPDY_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, d->variant->fn, p->threads,
                                                                    static_cast<size_t>(p->smem_bytes)));
        if (occ < 1) return SPDY_ERR_UNSUPPORTED;
        p->ctas_per_sm = occ;
    }
    return SPDY_OK;
}

void hook_release(spdy_plan *p)
{
    DeviceSide *d = p->dev;
    if (!d) return;
    {
        DeviceGuard guard;
        guard.enter(p->device);
        if (d->owns_blob && d->blob) cudaFree(d->blob);
        if (d->arena) cudaFree(d->arena);
        for (cudaEvent_t e : d->events) cudaEventDestroy(e);
        for (cudaEvent_t e : d->copy_events) cudaEventDestroy(e);
        if (d->entry_event) cudaEventDestroy(d->entry_event);
        for (cudaEvent_t e : d->probe)
            if (e) cudaEventDestroy(e);
        if (d->copy_stream) cudaStreamDestroy(d->copy_stream);
    }
    delete d;
    p->dev = nullptr;
}

int hook_attach(spdy_plan *p)
{
    DeviceSide *d = new (std::nothrow) DeviceSide();
    if (!d) return SPDY_ERR_NO_MEMORY;
    p->dev = d;
    DeviceGuard guard;
    int rc = guard.enter(p->device);
    if (rc == SPDY_OK) rc = select_kernel(p, d);
    if (rc == SPDY_OK) {
        const TableLayout t = table_layout(p);
        std::vector<unsigned char> host;
        try {
            pack_tables(p, t, host);
        } catch (const std::bad_alloc &) {
            rc = SPDY_ERR_NO_MEMORY;
        }
        if (rc == SPDY_OK) {
            cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&d->blob), t.total);
            if (err != cudaSuccess) {
                g_last_cuda_error = static_cast<int>(err);
                d->blob = nullptr;
                rc = err == cudaErrorMemoryAllocation ? SPDY_ERR_NO_MEMORY : SPDY_ERR_CUDA;
            }
        }
        if (rc == SPDY_OK) {
            cudaError_t err = cudaMemcpy(d->blob, host.data(), t.total, cudaMemcpyHostToDevice);
            if (err != cudaSuccess) {
                g_last_cuda_error = static_cast<int>(err);
                rc = SPDY_ERR_CUDA;
            }
            bind_tables(d, t, d->blob);
        }
    }
    if (rc != SPDY_OK) hook_release(p);
    return rc;
}

int hook_solve_coeffs_host(spdy_plan *p, const float *coeffs_host, int64_t n, uint8_t *profile_host, void *cuda_stream);

const DeviceHooks kHooks = {hook_limits, hook_attach, hook_release, hook_solve_coeffs_host};

struct HookRegistration {
    HookRegistration() { register_device_hooks(&kHooks); }
} g_hook_registration;

// The whole path for one batch; exactly one of errors_dev / coeffs_dev is non-null.
// phases: bit 0 = forward pass (and final minimum), bit 1 = walk back; the host-buffer path runs them
// separately so that one walk back serves several forward launches into one table.  `shape`: the table
// set to run (the plan itself or one of its launch shapes for small batches); null = choose by N.
int solve_impl(const spdy_plan *plan, const spdy_plan *shape, const float *errors_dev, const float *coeffs_dev, int64_t N,
               uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev, void *workspace_dev,
               size_t workspace_bytes, void *cuda_stream, bool keep_timing = false, int phases = 3)
{
    if (!plan || plan->device < 0 || !plan->dev || N < 0) return SPDY_ERR_INVALID_ARG;
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
    if (!shape) shape = pick_for_batch(plan, N, workspace_bytes);
    const size_t per = static_cast<size_t>(table_bytes_one(shape) + row_bytes_one(shape) + flag_bytes_one(shape));
    const int64_t wave = static_cast<int64_t>(std::min<size_t>(workspace_bytes / per, static_cast<size_t>(N)));
    if (wave < 1) return SPDY_ERR_WORKSPACE_TOO_SMALL;
    // The table pitch handed to the kernels is in cells; every candidate's table is 256-byte aligned.
    const int64_t pitch_cells = table_bytes_one(shape) / cell_bytes(shape);
    // Row buffers in global memory (wide-band fallback) follow the tables of the wave.
    float *grows = shape->kind == KERNEL_CTA_GLOBAL
                       ? reinterpret_cast<float *>(static_cast<unsigned char *>(workspace_dev) + wave * table_bytes_one(shape))
                       : nullptr;

    DeviceSide *timer = plan->dev;  // events and the self-check word belong to the public plan
    if (timer->timing && !keep_timing) timer->events_used = 0;
    for (int64_t first = 0; first < N; first += wave) {
        const int64_t count = std::min<int64_t>(wave, N - first);
        cudaEvent_t *ev = nullptr;
        if (timer->timing) {
            while (timer->events.size() < timer->events_used + 3) {
                cudaEvent_t e;
                SPDY_CUDA_TRY(cudaEventCreate(&e));
                timer->events.push_back(e);
            }
            ev = &timer->events[timer->events_used];
            timer->events_used += 3;
            SPDY_CUDA_TRY(cudaEventRecord(ev[0], stream));
        }
        // With a second (merged) table set every candidate of the wave gets a flag saying which set is
        // exact for it; both sets are then launched over the whole wave and every CTA / walk-back thread
        // runs only if its candidate carries the set's flag (the others leave at once).
        uint8_t *flags = nullptr;
        if (shape->merged) flags = static_cast<unsigned char *>(workspace_dev) + wave * (table_bytes_one(shape) + row_bytes_one(shape));
        if (shape->merged && (phases & 1)) {
            const DeviceSide *m = shape->merged->dev;
            const int bt = 128;
            spdy_monotone_flags_kernel<<<static_cast<unsigned>((count * 32 + bt - 1) / bt), bt, 0, stream>>>(
                errors_dev, coeffs_dev, m->qtab, m->layers, m->slot_ptr, m->slot_member, flags, first, count,
                plan->L, plan->K);
            SPDY_CUDA_TRY(cudaGetLastError());
        }
        auto forward = [&](const spdy_plan *tp, int which) -> int {
            const DeviceSide *td = tp->dev;
            FwdArgs fa;
            fa.errors = errors_dev;
            fa.coeffs = coeffs_dev;
            fa.qtab = td->qtab;
            fa.slots = td->slots;
            fa.slot_ptr = td->slot_ptr;
            fa.slot_member = td->slot_member;
            fa.layers = td->layers;
            fa.passes = td->passes;
            fa.pass_masks = td->masks;
            fa.pass_ptr = td->pass_ptr;
            fa.table = workspace_dev;
            fa.cost = cost_dev;
            fa.time_used = time_used_dev;
            fa.status = timer->status;
            fa.pitch = pitch_cells;
            fa.n_first = first;
            fa.n_count = count;
            fa.L = tp->L;
            fa.K = tp->K;
            fa.row_stride = tp->row_stride;
            fa.pad = tp->pad;
            fa.grows = grows;
            fa.grows_stride = row_bytes_one(shape) / 4;
            fa.cand_flags = flags;
            fa.which = which;
            // Grid x is limited to 2^31-1 CTAs, far above any wave that fits in memory.
            if (tp->kind == KERNEL_CLUSTER) {
                ClusterArgs ca;
                ca.f = fa;
                ca.slices = td->slices;
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
                SPDY_CUDA_TRY(cudaLaunchKernelEx(&cfg, td->cvariant->fn, ca));
            } else if (tp->kind == KERNEL_WARP) {
                const int per_cta = tp->threads / 32;
                td->variant->fn<<<static_cast<unsigned>((count + per_cta - 1) / per_cta), tp->threads,
                                  static_cast<size_t>(tp->smem_bytes), stream>>>(fa);
            } else {
                td->variant->fn<<<static_cast<unsigned>(count), tp->threads, static_cast<size_t>(tp->smem_bytes), stream>>>(fa);
            }
            SPDY_CUDA_TRY(cudaGetLastError());
            return SPDY_OK;
        };
        auto walk_back = [&](const spdy_plan *tp, int which) -> int {
            const DeviceSide *td = tp->dev;
            BackArgs ba;
            ba.errors = errors_dev;
            ba.coeffs = coeffs_dev;
            ba.qtab = td->qtab;
            ba.times = td->times;
            ba.layers = td->layers;
            ba.table = workspace_dev;
            ba.cost = cost_dev;
            ba.time_used = time_used_dev;
            ba.profile = profile_dev;
            ba.status = timer->status;  // one self-check word per public plan
            ba.pitch = pitch_cells;
            ba.n_first = first;
            ba.n_count = count;
            ba.L = tp->L;
            ba.K = tp->K;
            ba.cand_flags = flags;
            ba.which = which;
            ba.slot_ptr = tp->merge_first ? td->slot_ptr : nullptr;
            ba.slot_member = tp->merge_first ? td->slot_member : nullptr;
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
            if (shape->merged) lrc = forward(shape->merged, 1);
            if (lrc == SPDY_OK) lrc = forward(shape, 0);
            if (lrc != SPDY_OK) return lrc;
        }
        if (ev) SPDY_CUDA_TRY(cudaEventRecord(ev[1], stream));
        if (phases & 2) {
            if (shape->merged) lrc = walk_back(shape->merged, 1);
            if (lrc == SPDY_OK) lrc = walk_back(shape, 0);
            if (lrc != SPDY_OK) return lrc;
        }
        if (ev) SPDY_CUDA_TRY(cudaEventRecord(ev[2], stream));
    }
    return SPDY_OK;
}

// Host-buffer form of the path: the input is an error table ([N][L][K]) or, with `coeffs`, Eq. 4's
// coefficients ([N][L]).
int solve_host_impl(spdy_plan *plan, const float *errors_host, bool coeffs, int64_t N,
                    uint8_t *profile_host, float *cost_host, int32_t *time_used_host, void *cuda_stream)
{
    if (!plan || plan->device < 0 || !plan->dev || N < 0) return SPDY_ERR_INVALID_ARG;
    if (N == 0) return SPDY_OK;
    if (!errors_host || !profile_host || !cost_host || !time_used_host) return SPDY_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;
    DeviceSide *d = plan->dev;

    const size_t err_bytes = static_cast<size_t>(N) * plan->L * (coeffs ? 1 : plan->K) * sizeof(float);
    const size_t off_profile = round_up(err_bytes, 256);
    const size_t off_cost = off_profile + round_up(static_cast<size_t>(N) * plan->L, 256);
    const size_t off_time = off_cost + round_up(static_cast<size_t>(N) * 4, 256);
    const size_t off_ws = off_time + round_up(static_cast<size_t>(N) * 4, 256);
    // Cap the table at 16 GiB; larger batches run as waves.
    const size_t ws_full = plan->feasible ? spdy_workspace_bytes(plan, N) : 0;
    const size_t ws_unit = plan->feasible ? spdy_workspace_bytes(plan, 1) : 0;
    const size_t ws_cap = std::max<size_t>(ws_unit, static_cast<size_t>(16) << 30);
    const size_t ws_bytes = std::min(ws_full, ws_cap) / std::max<size_t>(ws_unit, 1) * ws_unit;
    const size_t total = off_ws + ws_bytes;
    if (total > d->arena_bytes) {
        if (d->arena) {
            SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
            SPDY_CUDA_TRY(cudaFree(d->arena));
            d->arena = nullptr;
            d->arena_bytes = 0;
        }
        cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&d->arena), total);
        if (err != cudaSuccess) {
            g_last_cuda_error = static_cast<int>(err);
            d->arena = nullptr;
            return err == cudaErrorMemoryAllocation ? SPDY_ERR_NO_MEMORY : SPDY_ERR_CUDA;
        }
        d->arena_bytes = total;
    }
    unsigned char *base = d->arena;
    float *d_err = reinterpret_cast<float *>(base);
    uint8_t *d_profile = base + off_profile;
    float *d_cost = reinterpret_cast<float *>(base + off_cost);
    int32_t *d_time = reinterpret_cast<int32_t *>(base + off_time);
    // One launch shape for the whole call, so that every chunk writes the table one walk back reads.
    const spdy_plan *shape = plan->feasible ? pick_for_batch(plan, N, ws_bytes) : plan;
    const size_t ws_one = plan->feasible
                              ? static_cast<size_t>(table_bytes_one(shape) + row_bytes_one(shape) + flag_bytes_one(shape))
                              : 0;
    // Everything from the first queued copy on runs inside `enqueue`: whatever makes it stop early, the
    // copies already queued still read the caller's host buffer, so every exit waits for both streams
    // before the error goes back to the caller (who may free or reuse the buffer on seeing it).
    bool chunked = false;
    size_t first_chunk_bytes = 1;
    auto enqueue = [&]() -> int {
        // An error table goes up in chunks of growing size on a second stream, so that every upload but the
        // first hides behind the kernels of the chunk before it.  The first chunk is one full wave of CTAs; each
        // further one may be larger than its predecessor by the ratio of solving time to upload time per
        // candidate, which the previous call on this plan measured on its first chunk (about 6 with a fast
        // host link, 2 to 3 with a slow one; 6 until measured).  Every chunk boundary costs a launch tail (and a
        // walk back, unless one serves all), so a remainder not much larger than the next chunk goes with it,
        // and coefficient input (K times smaller) goes up in one piece.
        const int64_t per_cand = static_cast<int64_t>(plan->L) * (coeffs ? 1 : plan->K);
        std::vector<int64_t> bounds(1, 0);
        {
            const int64_t per_cta = shape->kind == KERNEL_WARP ? shape->threads / 32 : 1;
            double size = static_cast<double>(std::max<int64_t>(1, static_cast<int64_t>(shape->ctas_per_sm) * shape->limits.sm_count *
                                                                       per_cta / std::max(1, shape->cluster)));
            if (coeffs) size = static_cast<double>(N);
            // A chunk boundary costs about half a wave of CTAs (the tail of one launch and the ramp of the next);
            // chunking saves at most the upload time of everything behind the first chunk.  Where a wave is long
            // and the table small (BERT-large shape: 3.8 ms against 1.3 ms) one piece is the better deal.
            if (d->upload_ms_per_byte > 0.0 && static_cast<double>(N) > size) {
                const double saved = (static_cast<double>(N) - size) * static_cast<double>(per_cand) * 4.0 * d->upload_ms_per_byte;
                if (saved < 0.5 * d->first_wave_ms) size = static_cast<double>(N);
            }
            while (bounds.back() < N) {
                const int64_t left = N - bounds.back();
                const int64_t take = static_cast<double>(left) <= 1.35 * size ? left : static_cast<int64_t>(size);
                bounds.push_back(bounds.back() + std::max<int64_t>(1, take));
                size *= d->chunk_growth;
            }
        }
        const size_t chunks = bounds.size() - 1;
        if (chunks > 1) {
            if (!d->copy_stream) SPDY_CUDA_TRY(cudaStreamCreateWithFlags(&d->copy_stream, cudaStreamNonBlocking));
            if (!d->entry_event) SPDY_CUDA_TRY(cudaEventCreateWithFlags(&d->entry_event, cudaEventDisableTiming));
            while (d->copy_events.size() < chunks) {
                cudaEvent_t e;
                SPDY_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
                d->copy_events.push_back(e);
            }
            // Work already queued on the caller's stream may still read the staging buffer.
            SPDY_CUDA_TRY(cudaEventRecord(d->entry_event, stream));
            SPDY_CUDA_TRY(cudaStreamWaitEvent(d->copy_stream, d->entry_event, 0));
            for (cudaEvent_t &e : d->probe)
                if (!e) SPDY_CUDA_TRY(cudaEventCreate(&e));
            for (size_t c = 0; c < chunks; ++c) {
                const int64_t first = bounds[c], count = bounds[c + 1] - bounds[c];
                if (c == 0) SPDY_CUDA_TRY(cudaEventRecord(d->probe[0], d->copy_stream));
                SPDY_CUDA_TRY(cudaMemcpyAsync(d_err + first * per_cand, errors_host + first * per_cand,
                                              static_cast<size_t>(count * per_cand) * sizeof(float),
                                              cudaMemcpyHostToDevice, d->copy_stream));
                if (c == 0) SPDY_CUDA_TRY(cudaEventRecord(d->probe[1], d->copy_stream));
                SPDY_CUDA_TRY(cudaEventRecord(d->copy_events[c], d->copy_stream));
            }
        } else {
            SPDY_CUDA_TRY(cudaMemcpyAsync(d_err, errors_host, err_bytes, cudaMemcpyHostToDevice, stream));
        }
        // When the whole batch's table fits the staging workspace (and nothing but tables lives there),
        // the chunks' forward passes write disjoint parts of it and ONE walk back follows: the walk back
        // is a latency chain of L steps whatever the number of candidates.
        const bool one_walk_back = chunks > 1 && plan->feasible && !shape->merged && shape->kind != KERNEL_CTA_GLOBAL &&
                                   ws_bytes >= ws_one * static_cast<size_t>(N);
        int lrc = SPDY_OK;
        for (size_t c = 0; c < chunks; ++c) {
            const int64_t first = bounds[c], count = bounds[c + 1] - bounds[c];
            if (chunks > 1) SPDY_CUDA_TRY(cudaStreamWaitEvent(stream, d->copy_events[c], 0));
            if (chunks > 1 && c <= 1) SPDY_CUDA_TRY(cudaEventRecord(d->probe[2 + c], stream));  // around chunk 0's kernels
            const float *in = d_err + first * per_cand;
            if (one_walk_back)
                lrc = solve_impl(plan, shape, coeffs ? nullptr : in, coeffs ? in : nullptr, count, d_profile + first * plan->L,
                                 d_cost + first, d_time + first, base + off_ws + static_cast<size_t>(first) * ws_one,
                                 static_cast<size_t>(count) * ws_one, stream, c > 0, 1);
            else
                lrc = solve_impl(plan, shape, coeffs ? nullptr : in, coeffs ? in : nullptr, count, d_profile + first * plan->L,
                                 d_cost + first, d_time + first, base + off_ws, ws_bytes, stream, c > 0);
            if (lrc != SPDY_OK) return lrc;
        }
        if (one_walk_back) {
            lrc = solve_impl(plan, shape, coeffs ? nullptr : d_err, coeffs ? d_err : nullptr, N, d_profile, d_cost, d_time,
                             base + off_ws, ws_bytes, stream, true, 2);
            if (lrc != SPDY_OK) return lrc;
        }
        SPDY_CUDA_TRY(cudaMemcpyAsync(profile_host, d_profile, static_cast<size_t>(N) * plan->L, cudaMemcpyDeviceToHost, stream));
        SPDY_CUDA_TRY(cudaMemcpyAsync(cost_host, d_cost, static_cast<size_t>(N) * 4, cudaMemcpyDeviceToHost, stream));
        SPDY_CUDA_TRY(cudaMemcpyAsync(time_used_host, d_time, static_cast<size_t>(N) * 4, cudaMemcpyDeviceToHost, stream));
        chunked = chunks > 1;
        first_chunk_bytes = static_cast<size_t>(bounds[1] * per_cand) * sizeof(float);
        return SPDY_OK;
    };
    rc = enqueue();
    if (rc != SPDY_OK) {
        if (d->copy_stream) cudaStreamSynchronize(d->copy_stream);
        cudaStreamSynchronize(stream);
        return rc;
    }
    SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
    if (chunked) {
        // (probe[3] was recorded after chunk 1's upload had arrived, i.e. it may include waiting for it: the
        // ratio then comes out too large by at most that wait, which the factor 0.85 and the bounds absorb)
        float up_ms = 0.f, solve_ms = 0.f;
        if (cudaEventElapsedTime(&up_ms, d->probe[0], d->probe[1]) == cudaSuccess &&
            cudaEventElapsedTime(&solve_ms, d->probe[2], d->probe[3]) == cudaSuccess && up_ms > 0.f && solve_ms > 0.f) {
            d->chunk_growth = std::min(8.0, std::max(1.5, 0.85 * static_cast<double>(solve_ms) / up_ms));
            d->upload_ms_per_byte = static_cast<double>(up_ms) / static_cast<double>(first_chunk_bytes);
            d->first_wave_ms = solve_ms;
        }
    }
    return SPDY_OK;
}

// The search's solver: coefficients up, profiles down, self-check word read.
int hook_solve_coeffs_host(spdy_plan *p, const float *coeffs_host, int64_t n, uint8_t *profile_host, void *cuda_stream)
{
    std::vector<float> cost;
    std::vector<int32_t> time_used;
    try {
        cost.resize(static_cast<size_t>(n));
        time_used.resize(static_cast<size_t>(n));
    } catch (const std::bad_alloc &) {
        return SPDY_ERR_NO_MEMORY;
    }
    int rc = solve_host_impl(p, coeffs_host, true, n, profile_host, cost.data(), time_used.data(), cuda_stream);
    if (rc == SPDY_OK) rc = spdy_plan_check_status(p, cuda_stream);
    return rc;
}

}  // namespace

extern "C" {

int spdy_last_cuda_error(void) { return g_last_cuda_error; }

int spdy_debug_checks_enabled(void)
{
#ifdef SPDY_DEBUG_CHECKS
    return 1;
#else
    return 0;
#endif
}

int spdy_solve_batch(const spdy_plan *plan, const float *errors_dev, int64_t N,
                     uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev,
                     void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    if (!errors_dev && N > 0) return SPDY_ERR_INVALID_ARG;
    return solve_impl(plan, nullptr, errors_dev, nullptr, N, profile_dev, cost_dev, time_used_dev, workspace_dev,
                      workspace_bytes, cuda_stream);
}

int spdy_solve_batch_coeffs(const spdy_plan *plan, const float *coeffs_dev, int64_t N,
                            uint8_t *profile_dev, float *cost_dev, int32_t *time_used_dev,
                            void *workspace_dev, size_t workspace_bytes, void *cuda_stream)
{
    if (!coeffs_dev && N > 0) return SPDY_ERR_INVALID_ARG;
    return solve_impl(plan, nullptr, nullptr, coeffs_dev, N, profile_dev, cost_dev, time_used_dev, workspace_dev,
                      workspace_bytes, cuda_stream);
}

int spdy_plan_enable_timing(spdy_plan *plan, int on)
{
    if (!plan || plan->device < 0 || !plan->dev) return SPDY_ERR_INVALID_ARG;
    plan->dev->timing = on != 0;
    plan->dev->events_used = 0;
    return SPDY_OK;
}

int spdy_plan_last_timing(spdy_plan *plan, float *forward_ms_host, float *walkback_ms_host)
{
    if (!plan || plan->device < 0 || !plan->dev || !plan->dev->timing) return SPDY_ERR_INVALID_ARG;
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;
    DeviceSide *d = plan->dev;
    float fwd = 0.f, back = 0.f;
    for (size_t i = 0; i + 3 <= d->events_used && i + 3 <= d->events.size(); i += 3) {
        SPDY_CUDA_TRY(cudaEventSynchronize(d->events[i + 2]));
        float a = 0.f, b = 0.f;
        SPDY_CUDA_TRY(cudaEventElapsedTime(&a, d->events[i], d->events[i + 1]));
        SPDY_CUDA_TRY(cudaEventElapsedTime(&b, d->events[i + 1], d->events[i + 2]));
        fwd += a;
        back += b;
    }
    if (forward_ms_host) *forward_ms_host = fwd;
    if (walkback_ms_host) *walkback_ms_host = back;
    return SPDY_OK;
}

int spdy_plan_status_word(spdy_plan *plan, void *cuda_stream, int32_t *word_host)
{
    if (!plan || plan->device < 0 || !plan->dev || !word_host) return SPDY_ERR_INVALID_ARG;
    DeviceGuard guard;
    int rc = guard.enter(plan->device);
    if (rc != SPDY_OK) return rc;
    int32_t word = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    SPDY_CUDA_TRY(cudaMemcpyAsync(&word, plan->dev->status, sizeof(word), cudaMemcpyDeviceToHost, stream));
    SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
    if (word != 0) {
        SPDY_CUDA_TRY(cudaMemsetAsync(plan->dev->status, 0, sizeof(word), stream));
        SPDY_CUDA_TRY(cudaStreamSynchronize(stream));
    }
    *word_host = word;
    return SPDY_OK;
}

int spdy_plan_check_status(spdy_plan *plan, void *cuda_stream)
{
    int32_t word = 0;
    int rc = spdy_plan_status_word(plan, cuda_stream, &word);
    if (rc != SPDY_OK) return rc;
    return word != 0 ? SPDY_ERR_INTERNAL : SPDY_OK;
}

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
    spdy_options opts = {};
    opts.auto_shape = N >= 300 ? 1 : 0;  // a batch that fills the device needs no launch shapes for small ones
    int rc = spdy_plan_create(&plan, times.data(), L, K, B, device, &opts);
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

}  // extern "C"

// ----------------------------------------------------------------------------------------------
// Entry point that performs no device allocation
// ----------------------------------------------------------------------------------------------

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

    // Host-side plan (bands, pass shapes) with the one-byte table so more candidates fit a wave; one table
    // set and one launch shape, whatever N.
    DeviceLimits limits;
    rc = hook_limits(device, &limits);
    if (rc != SPDY_OK) return rc;
    spdy_options opts = {};
    opts.table_format = SPDY_TABLE_ARG_U8;
    opts.cluster = 1;  // the cluster variant's wider rows would not leave room for a table anyway
    opts.auto_shape = 1;
    spdy_plan *p = nullptr;
    rc = create_host_plan(&p, times_host, L, K, B, device, &opts, limits, false);
    if (rc == SPDY_ERR_UNSUPPORTED) rc = SPDY_ERR_STATIC_LIMIT;
    if (rc != SPDY_OK) return rc;
    auto discard = [&]() {
        delete p->dev;  // host object only: its tables live in the static array
        p->dev = nullptr;
        destroy_host_plan(p);
    };
    DeviceSide *d = new (std::nothrow) DeviceSide();
    if (!d) {
        destroy_host_plan(p);
        return SPDY_ERR_NO_MEMORY;
    }
    d->owns_blob = false;
    p->dev = d;
    rc = select_kernel(p, d);
    if (rc == SPDY_ERR_UNSUPPORTED) rc = SPDY_ERR_STATIC_LIMIT;
    if (rc != SPDY_OK) {
        discard();
        return rc;
    }

    // The plan tables go to the front of the scratch, the walk-back table behind them.
    const TableLayout tl = table_layout(p);
    const size_t off_table = tl.total;
    const size_t one = p->feasible ? spdy_workspace_bytes(p, 1) : 0;
    if (off_table + one > kStaticScratchBytes) {
        discard();
        return SPDY_ERR_STATIC_LIMIT;
    }
    std::vector<unsigned char> host;
    try {
        pack_tables(p, tl, host);
    } catch (const std::bad_alloc &) {
        discard();
        return SPDY_ERR_NO_MEMORY;
    }
    bind_tables(d, tl, base);
    // The array keeps the previous call's contents; the image below overwrites every table and
    // carries a zero self-check word, the only thing that must start at zero.
    cudaError_t err = cudaMemcpyAsync(base, host.data(), tl.total, cudaMemcpyHostToDevice, stream);
    if (err != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(err);
        cudaStreamSynchronize(stream);
        discard();
        return SPDY_ERR_CUDA;
    }
    const size_t table_bytes = p->feasible ? (kStaticScratchBytes - off_table) / one * one : 0;
    rc = solve_impl(p, p, errors_dev, nullptr, N, profile_dev, cost_dev, time_used_dev, base + off_table,
                    table_bytes, stream);
    int32_t word = 0;
    if (rc == SPDY_OK) {
        err = cudaMemcpyAsync(&word, d->status, sizeof(word), cudaMemcpyDeviceToHost, stream);
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
    discard();  // host objects only: this plan owns no device memory
    return rc;
}

}  // extern "C"
