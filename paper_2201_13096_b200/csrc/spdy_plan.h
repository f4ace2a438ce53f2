// Host side of a plan: everything that follows from the timing table, the budget and the launch options
// alone - live bands, shift slots, warp passes, table layout, work counts - in plain C++ with no CUDA
// dependency, so that it builds and is tested with the host compiler only.  The CUDA part of the library
// (kernels, uploads, launches) sees a plan through this header and hangs its own state off `dev`.
//
// Section 3.2 (Eq. 2-3) and Appendix A (Algorithm 1) define the dynamic program the tables describe.
#ifndef SPDY_PLAN_H
#define SPDY_PLAN_H

#include "../../include/spdy_dp.h"

#include <cstdint>
#include <vector>

namespace spdy {

constexpr int kLibraryVersion = 2004;

// Most band cells one lane owns in one warp pass; the kernels unroll passes of 1..kRmax cells per lane.
constexpr int kRmax = 24;

// The builds with 128 registers per thread to themselves (128-thread CTAs at four per SM) and the cheapest
// cell update (packed add + 3-input minimum) unroll passes twice as long: every pass pays for its own
// 16-byte slot reads (about three data-path wavefronts per pair of slots), so half as many passes take
// 4 % off the traffic of the unit the kernel is bound by.
#ifdef SPDY_DEBUG_CHECKS
constexpr int kRmaxLong = 24;  // the index-checked pass bodies of 48 cells take minutes each to compile
#else
constexpr int kRmaxLong = 48;
#endif
constexpr int long_pass_cap(int mode) { return mode == 4 /* MODE_ROW2 */ ? kRmaxLong : kRmax; }

// Widest band (cells) for which the plan considers one warp per candidate when left to choose (it then
// takes it if at least three CTAs of four candidates fit an SM).
constexpr int kWarpKernelMaxWidth = 4096;

// How the forward kernel forms a cell and what it stores for the walk back.
enum ForwardMode {
    MODE_ARG = 1,       // compare + two selects per cell, byte table of winning choices
    MODE_ARG_PRED = 2,  // compare + two predicated moves per cell, byte table
    MODE_ROW = 3,       // value-only minimum, fp32 table of row values
    MODE_ROW2 = 4,      // value-only, two slots per step: packed f32x2 adds and 3-input minimum
    MODE_ARG_PAIR = 5   // byte table, two slots per step: 3-input minimum, index resolved from the outcome
};

// Longest pass (cells per lane) a 1024-thread CTA unrolls: 64 registers per thread bound it, and the pairwise
// argmin update keeps two register arrays per cell.
constexpr int cells_per_lane_1024(int mode) { return mode == MODE_ARG_PAIR ? 8 : 16; }

// Longest pass of a cluster's CTA: a 512-thread CTA has 128 registers per thread, which the masked stores of
// a slice plus 24 cells per lane exceed.
constexpr int cluster_cells_per_lane(int threads) { return threads >= 512 ? 16 : kRmax; }

// Longest pass of the 1024-thread kernel whose rows live in global memory (64 registers per thread, 64-bit
// row addresses).
constexpr int global_rows_cap_1024(int mode) { return mode == MODE_ARG_PAIR ? 7 : 11; }

// The warp-per-candidate kernel comes in two builds: passes of up to warp_short_cap() cells per lane in 64
// registers (8 CTAs of 128 threads per SM) and up to long_pass_cap() in 128 registers (4 CTAs).
constexpr int warp_short_cap(int mode) { return mode == MODE_ARG_PAIR ? 7 : 8; }
inline bool mode_is_row(int mode) { return mode == MODE_ROW || mode == MODE_ROW2; }
inline bool mode_is_arg(int mode) { return mode == MODE_ARG || mode == MODE_ARG_PRED || mode == MODE_ARG_PAIR; }

// Which kernel family runs the forward pass.
enum KernelKind {
    KERNEL_CTA = 0,      // one CTA per candidate, rows in shared memory
    KERNEL_CTA_GLOBAL = 1,  // one CTA of 1024 threads per candidate, rows in the workspace
    KERNEL_CLUSTER = 2,  // one thread-block cluster per candidate, every row cut into slices
    KERNEL_WARP = 3      // one warp per candidate (narrow rows), several candidates per CTA
};

// Row l (1-based; stored at index l-1) lives on the band [lo, lo + width).  A band cell is addressed
// by t_rel = t - lo.  The warp passes of a layer cover [0, extent), extent a multiple of 32 >= width;
// `rowoff` is where the row starts inside one candidate's table, in cells.
struct LayerDesc {
    int32_t width;
    uint32_t rowoff;
    int32_t lo;
    int32_t mn;       // smallest usable time of the layer: lo_l = lo_{l-1} + mn
    int32_t extent;   // cells the passes of the layer write (>= width; the excess holds +inf)
    int32_t nslots;   // shift slots of the layer (see TapRange)
    int32_t fill;     // cells of +inf written behind the row: as far as the next layer reads beyond `extent`
    int32_t reserved1;
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

// One warp pass: the 32 * cpl band cells starting at `start` (lane i owns cells start + i, start + i + 32,
// ...).  krange = u_lo | u_hi << 8 | dense << 16 | cpl << 24: the slots that overlap the pass lie in
// [u_lo, u_hi); when they are all of that range (dense) the kernel loops straight over it, otherwise it
// walks the set bits of the pass's mask words.
struct PassDesc {
    int32_t start;
    uint32_t krange;
};

inline int pass_cpl(const PassDesc &p) { return static_cast<int>(p.krange >> 24); }

// Cluster variant, per (layer, rank): the slice of the row a CTA owns and its window of the previous row.
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

// What the host needs to know about the device to pick a launch shape (B200 figures by default, so that
// a plan can be laid out and inspected without a device).
struct DeviceLimits {
    int64_t smem_per_sm = 233472;
    int64_t smem_per_block = 232448;
    int32_t sm_count = 148;
};

// Where each device table sits inside one 256-byte aligned block of `total` bytes.
struct TableLayout {
    size_t times = 0, layers = 0, slots = 0, slot_ptr = 0, slot_member = 0, masks = 0, passes = 0, pass_ptr = 0,
           status = 0, slices = 0, qtab = 0, total = 0;
};

struct DeviceSide;  // owned by the CUDA part of the library

}  // namespace spdy

struct spdy_plan {
    int32_t L = 0, K = 0, B = 0;
    int device = -1;
    bool feasible = false;
    int mode = spdy::MODE_ROW2;
    int kind = spdy::KERNEL_CTA;
    int threads = 128;       // threads per CTA
    int warps_per_cand = 4;  // warps that share one candidate (threads / 32, or 1 for KERNEL_WARP)
    int rcap = spdy::kRmax;  // largest cells-per-lane of any pass: selects the kernel build
    int cluster = 1;
    int table_format = SPDY_TABLE_ROW_F32;
    int ctas_per_sm = 0;
    int schedule = 0;        // resolved pass schedule: 1 uniform, 2 levelled, 3 cost-sized (see spdy_plan.cpp)
    int pass_cap = 0;        // upper limit of cells per lane per pass asked for by the options (0 = the kernel's)
    spdy::DeviceLimits limits;
    int64_t smem_bytes = 0;
    int32_t row_stride = 0, pad = 0;  // floats per row buffer; +inf guard cells below cell 0 of a row
    // Byte table only: `merged` is a second plan over the same rows and passes whose slots are groups
    // of equal-time choices (ordered by their lowest member); candidates for which that is exact run
    // on it, the others on this plan.  `merge_first` marks such a second plan.
    bool merge_first = false;
    spdy_plan *merged = nullptr;
    // Launch shapes for batches too small to fill the device with the main shape (see pick_for_batch).
    std::vector<spdy_plan *> alternates;
    bool is_alternate = false;
    int64_t pitch = 0;  // table cells per candidate
    int64_t band_cells = 0, useful_updates = 0, distinct_updates = 0, issued_updates = 0;
    int32_t max_width = 0;
    std::vector<int32_t> times;
    std::vector<float> qtab;                // [K] squares of Eq. 4
    std::vector<spdy::LayerDesc> layers;
    std::vector<spdy::TapRange> taps;       // [L][K] by choice
    std::vector<spdy::TapRange> slots;      // [L][K] by shift slot (first layers[l].nslots valid)
    std::vector<uint8_t> slot_ptr;          // [L][K+1]
    std::vector<uint8_t> slot_member;       // [L][K]
    std::vector<spdy::PassDesc> passes;     // warp passes, grouped by (layer, warp)
    std::vector<uint64_t> pass_masks;       // [passes][mask words]: one bit per slot that overlaps the pass
    std::vector<int32_t> pass_ptr;          // [L * warps_per_cand + 1]: passes of (layer l, warp w) are
                                            // passes[pass_ptr[l*W + w] .. pass_ptr[l*W + w + 1])
    std::vector<spdy::SliceDesc> slices;    // cluster variant: [L][cluster]
    int32_t out_stride = 0, win_stride = 0;
    spdy::DeviceSide *dev = nullptr;
};

namespace spdy {

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline int mask_words(const spdy_plan *p) { return (p->K + 63) / 64; }
inline int64_t cell_bytes(const spdy_plan *p) { return p->table_format == SPDY_TABLE_ROW_F32 ? 4 : 1; }

// Workspace one candidate needs: its walk-back table, and its two row buffers when those live in
// global memory; one flag block per candidate when two table sets share the batch.  Multiples of 256 bytes.
int64_t table_bytes_one(const spdy_plan *p);
int64_t row_bytes_one(const spdy_plan *p);
int64_t flag_bytes_one(const spdy_plan *p);

// Lays a plan out on the host: validates, builds bands, slots, passes and the launch shape.  `*out` owns
// no device state afterwards (dev == nullptr).  merge_first: see spdy_plan::merge_first.
int create_host_plan(spdy_plan **out, const int32_t *times_host, int32_t L, int32_t K, int32_t B, int device,
                     const spdy_options *opts, const DeviceLimits &limits, bool merge_first);
void destroy_host_plan(spdy_plan *p);  // host members only; does not touch `dev`, `merged` or `alternates`

// Exhaustive host-side check of the plan's index arithmetic: every shared-memory (or row-buffer) cell a
// lane can read or write and every table cell it stores lies inside its buffer, and every read outside
// the previous row's band lands on a cell that holds +inf.  SPDY_OK or SPDY_ERR_INTERNAL.
int verify_plan(const spdy_plan *p);

TableLayout table_layout(const spdy_plan *p);
void pack_tables(const spdy_plan *p, const TableLayout &t, std::vector<unsigned char> &host);

// The table set (this plan or one of its alternates) that should run a batch of N candidates inside a
// workspace of `workspace_bytes`.
const spdy_plan *pick_for_batch(const spdy_plan *p, int64_t N, size_t workspace_bytes);

// Hooks the CUDA part registers when it is linked in; absent in the host-only build.
struct DeviceHooks {
    int (*limits)(int device, DeviceLimits *out);
    int (*attach)(spdy_plan *p);    // set kernel attributes, verify occupancy, upload the tables
    void (*release)(spdy_plan *p);  // free everything behind p->dev
    // Eq. 4 coefficients [n][L] in host memory -> profiles [n][L] in host memory (the search's solver)
    int (*solve_coeffs_host)(spdy_plan *p, const float *coeffs_host, int64_t n, uint8_t *profile_host, void *cuda_stream);
};
void register_device_hooks(const DeviceHooks *hooks);
const DeviceHooks *device_hooks();

}  // namespace spdy

#endif  // SPDY_PLAN_H
