// C-ABI library of the module-wise outer synchronisation (see include/dipaco.h).
// Host side: argument checks, planning (plan.hpp), table upload, kernel launches (kernels.cuh).
#include "../../include/dipaco.h"

#if defined(__SSE2__)
#include <emmintrin.h>
#endif
#include <condition_variable>
#include <cstring>
#include <exception>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "kernels.cuh"
#include "plan.hpp"

using namespace dipaco;

namespace {

constexpr int STAGING_SLOTS = 4;
constexpr size_t SMEM_LIMIT = 227 * 1024;  // opt-in dynamic shared memory per CTA on sm_100
constexpr size_t SMEM_PER_SM = 228 * 1024;
constexpr size_t SMEM_CTA_RESERVE = 1024;  // per-CTA reservation the driver adds
constexpr int64_t RAGGED_TILE = 256;       // split granularity of the scalar kernel: one element per thread
constexpr int64_t SHIFT_TILE = 2048;       // 256 threads * 8 elements: one CTA step of the shifted vector kernel
constexpr int MAX_COUNTERS = 256;          // work counters (one per bulk launch of an upload)

enum SyncState { STATE_IDLE = 0, STATE_ACCUMULATING = 1 };

struct Staging {
    void *host = nullptr;
    size_t capacity = 0;
    cudaEvent_t done = nullptr;
    bool in_flight = false;
};

// One kernel launch worth of tables inside a packed upload.
struct PackedLaunch {
    size_t passes_off = 0, contribs_off = 0, members_off = 0;
    size_t bulk_segs_off = 0, bulk_first_off = 0, rag_segs_off = 0, rag_first_off = 0;
    size_t shv_segs_off = 0, shv_first_off = 0;  // ranges of the shifted vector kernel (misaligned modules)
    int bulk_ctas = 0, rag_ctas = 0, shv_ctas = 0;
    int io_arrays = 2;
    int units = 2;                        // 16-byte units per compute thread and tile of this launch
    bool aligned_kernel_is_vector = false;
    bool shifted = false;                 // some path buffer of a bulk pass sits inside a 16-byte unit
    int num_passes = 0, total_items = 0;  // dynamic scheduling of the bulk-copy kernel
    double mean_contributors = 0.0;       // per element of the bulk range
};

struct HostMode;  // state of dipaco_outer_sync_host (host_mode.inl)

// Half the hardware threads, at most four.  Measured on a 16-core host beside a running upload
// (90 GB each step): three or four threads with streaming stores keep up with the link, more of
// them take memory bandwidth from the upload's DMA reads and the step gets slower again
// (1.73 s with 3-4 threads, 1.82 s with 5-6, 1.95 s with 8, 2.00 s with none).
int default_host_threads()
{
    const unsigned hw = std::thread::hardware_concurrency();
    return (int)std::min(4u, std::max(1u, hw / 2));
}

} // namespace

struct dipaco_ctx {
    Grid grid;
    float lr = 0.f, mu = 0.f;
    int optimizer = DIPACO_OPT_NESTEROV;
    int input_kind = DIPACO_INPUT_COPIES;
    // Adam family
    float *second_moment = nullptr;
    float *second_moment_staged = nullptr;  // host mode: device copy that the kernels use instead
    double adam_b1 = 0.9, adam_b2 = 0.999, adam_eps = 1e-8, adam_wd = 0.0;
    int adam_step = 0;  // 0 = no bias correction
    int dtype = DIPACO_F32;
    int elem_size = 4;
    int device = -1;
    int sm_count = 0;
    int kernel = DIPACO_KERNEL_AUTO;
    int ctas_per_sm = 1, stages = 10, units = 2;  // bulk-copy kernel tuning (measured on B200)
    int io_slots = 3;                            // buffers of theta/momentum/result tiles
    int64_t item_bytes = 2 * 1024 * 1024;        // most traffic of one dynamic work item
    int items_per_cta = 64;                      // least number of items per CTA that a launch is cut into
    int64_t launches = 0;
    int64_t host_unit_bytes = (int64_t)512 << 20;  // staged bytes (each way) of one unit in host mode
    int host_threads = default_host_threads();     // host threads that fan results out (0 = none)

    void *dev_tables = nullptr;
    size_t dev_tables_capacity = 0;
    Staging staging[STAGING_SLOTS];
    int staging_next = 0;
    std::vector<unsigned char> last_blob;  // tables currently in dev_tables (skip identical uploads)
    float *partial = nullptr;
    void *cast_scratch = nullptr;  // cast(theta') per module in the path dtype (chunk API, bf16 paths)
    bool cast_scratch_tried = false;
    int *error_word = nullptr;
    int *counters = nullptr;  // MAX_COUNTERS work counters for the bulk-copy kernel
    bool smem_attr_set[2][3][2] = {};  // [path type][units per thread][shifted variant]

    // round state of the incremental API
    int state = STATE_IDLE;
    float *theta = nullptr, *momentum = nullptr;
    cudaStream_t stream = nullptr;
    cudaStream_t last_stream = nullptr;
    std::vector<ModuleCoeffs> coeffs;
    int next_chunk = 0;

    HostMode *host_mode = nullptr;

    // Plan of the last dipaco_outer_sync, kept while its tables are the ones on the device: a call
    // with the same buffers, mask and settings launches again without planning or uploading.
    uint64_t settings_version = 1;           // bumped by every dipaco_set_*
    std::vector<unsigned char> plan_key;     // settings version, buffers, mask of the kept plan
    std::vector<PackedLaunch> plan_launches;
    bool plan_valid = false;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// Diagnostic kernel (dipaco_selftest_wait_expiry): one thread waits, with the given limit, on a
// barrier phase that nothing will ever complete.  No copy is in flight and no other thread takes
// part, so the only effect is what a pipeline CTA that gave up leaves behind: a code in the error
// word and a work counter that is not back at zero.
__global__ void wait_expiry_kernel(int *error_word, int *work_counter, unsigned long long limit_ns)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!bounded_wait(&bar, 0, error_word, 9, limit_ns)) atomicAdd(work_counter, 1);
    }
}


void compute_all_coeffs(dipaco_ctx *ctx, const uint8_t *reported)
{
    ctx->coeffs.resize(ctx->grid.modules.size());
    for (size_t id = 0; id < ctx->grid.modules.size(); ++id)
        module_coeffs(ctx->grid, ctx->grid.modules[id], reported, ctx->coeffs[id]);
}

int tile_units(const dipaco_ctx *ctx)
{
    return ctx->units > 0 ? ctx->units : 2;
}

// Elements of one tile of `units` 16-byte units per compute thread.
int64_t tile_elems_of(const dipaco_ctx *ctx, int units)
{
    const int ue = ctx->dtype == DIPACO_BF16 ? 8 : 4;
    return (int64_t)BULK_COMPUTE_THREADS * ue * units;
}

// The tile of the configured tuning (launches that need more fp32 tiles per buffer than fit may
// fall back to a smaller one, which always divides this one).
int64_t tile_elems(const dipaco_ctx *ctx)
{
    return tile_elems_of(ctx, tile_units(ctx));
}

// Shared memory of one bulk-kernel CTA for a given tile and depth.
size_t bulk_smem_bytes(const dipaco_ctx *ctx, int units, int stages, int io_arrays, int io_slots,
                       bool shifted = true)
{
    const size_t tile = (size_t)tile_elems_of(ctx, units);
    const size_t stage = tile * ctx->elem_size;
    // (the kernel variant for shifted path buffers loads 16 bytes more into every ring slot)
    size_t bytes = (size_t)stages * (stage + (shifted ? 16 : 0)) + (size_t)io_slots * io_arrays * tile * 4;
    if (ctx->elem_size != 4) bytes += (size_t)io_slots * stage;
    return bytes + sizeof(BulkShared) + 128;
}

int pick_stages(const dipaco_ctx *ctx, int units, int io_arrays, int io_slots, bool shifted = true)
{
    const size_t budget =
        std::min(SMEM_LIMIT, SMEM_PER_SM / (size_t)ctx->ctas_per_sm - 2 * SMEM_CTA_RESERVE);
    int best = 0;
    for (int s = 2; s <= BULK_MAX_STAGES; ++s)
        if (bulk_smem_bytes(ctx, units, s, io_arrays, io_slots, shifted) <= budget) best = s;
    if (ctx->stages > 0) return ctx->stages <= best ? ctx->stages : best;
    return best;
}

// Units per thread for a launch that stages io_arrays fp32 tiles per buffer: the configured
// value, or the next smaller one that still leaves a ring of two stages beside two buffers
// (the partial sum of a chunk walk and the second moment of the Adam family each add a tile
// that the tuning may not have been chosen for).  0 = nothing fits.
int fit_units(const dipaco_ctx *ctx, int io_arrays)
{
    for (int nu = tile_units(ctx); nu >= 1; nu /= 2)
        if (pick_stages(ctx, nu, io_arrays, 2) >= 2) return nu;
    return 0;
}

struct PtrLookup {
    void *const *ptrs;  // device pointers of path copies
    int first_path;     // ptrs[0] belongs to this path id
    int count;
    void *get(int path) const
    {
        const int i = path - first_path;
        return (i >= 0 && i < count) ? ptrs[i] : nullptr;
    }
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Serialise the tables of one launch into `blob` (appending) and describe them in `out`.
// extra_dst: optional raw destinations appended to a pass's member list (keyed by pass index).
int pack_launch(dipaco_ctx *ctx, const std::vector<PassSpec> &specs, const PtrLookup &lookup,
                const std::vector<std::vector<void *>> *extra_dst, const float *theta,
                const float *momentum, std::vector<unsigned char> &blob, PackedLaunch &out)
{
    const Grid &g = ctx->grid;
    const int es = ctx->elem_size;
    std::vector<PassDev> passes(specs.size());
    std::vector<ContribDev> contribs;
    std::vector<void *> members;
    std::vector<int64_t> bulk_begin(specs.size(), 0), bulk_end(specs.size(), 0);
    std::vector<int64_t> shv_begin(specs.size(), 0), shv_end(specs.size(), 0);
    // ranges of the one-element-per-thread kernel: a pass can have one before and one after its
    // vector range
    std::vector<int32_t> rag_pass;
    std::vector<int64_t> rag_begin, rag_end;
    auto add_ragged = [&](size_t pass, int64_t b, int64_t e) {
        if (b >= e) return;
        rag_pass.push_back((int32_t)pass);
        rag_begin.push_back(b);
        rag_end.push_back(e);
    };
    bool any_shifted = false;  // a bulk pass with a path buffer inside a 16-byte unit
    bool any_partial = false;
    for (const PassSpec &sp : specs)
        if (sp.flags & (PASS_PARTIAL_IN | PASS_PARTIAL_OUT)) any_partial = true;
    const int io_arrays = (any_partial ? 3 : 2) + (ctx->optimizer == DIPACO_OPT_ADAM ? 1 : 0);
    const int units = ctx->kernel == DIPACO_KERNEL_AUTO ? fit_units(ctx, io_arrays) : tile_units(ctx);
    if (units < 1) return DIPACO_EINVAL;
    const int64_t tile = tile_elems_of(ctx, units);

    for (size_t i = 0; i < specs.size(); ++i) {
        const PassSpec &sp = specs[i];
        const ModuleGeom &m = g.modules[sp.module];
        PassDev &pd = passes[i];
        pd.theta_off = m.theta_off;
        pd.partial_off = m.partial_off >= 0 ? m.partial_off : 0;
        pd.cast_off = m.cast_off;
        pd.flags = sp.flags;
        pd.scale = sp.scale;
        pd.item_first = 0;
        pd.tiles_per_item = 1;
        pd.bulk_tiles = 0;
        pd.bulk_begin = 0;
        pd.bulk_end = 0;
        if ((sp.flags & (PASS_PARTIAL_IN | PASS_PARTIAL_OUT)) && (m.partial_off < 0 || !ctx->partial))
            return DIPACO_ESTATE;
        if (((sp.flags & PASS_CAST_IN) || sp.cast_out) && !ctx->cast_scratch) return DIPACO_ESTATE;
        bool aligned = ((uintptr_t)(theta + m.theta_off) % 16 == 0) &&
                       ((uintptr_t)(momentum + m.theta_off) % 16 == 0);
        // Can an element range be cut so that every tile (or thread) starts 16-byte aligned in
        // all arrays that are not path buffers at once?  Ranges start where theta is 32-byte
        // aligned, i.e. at elements k with (state_pos + k) % 8 == 0; the other fp32 arrays must
        // then sit at the same place within a 16-byte unit as theta, and the cast scratch (path
        // type) at the same element position within its unit.
        const uintptr_t state_pos = ((uintptr_t)(theta + m.theta_off) % 32) / 4;  // in elements
        const uintptr_t state_rem = (uintptr_t)(theta + m.theta_off) % 16;
        bool state_congruent = (uintptr_t)(momentum + m.theta_off) % 16 == state_rem;
        if (ctx->optimizer == DIPACO_OPT_ADAM) {
            const float *v = ctx->second_moment_staged ? ctx->second_moment_staged : ctx->second_moment;
            aligned = aligned && ((uintptr_t)(v + m.theta_off) % 16 == 0);
            state_congruent = state_congruent && (uintptr_t)(v + m.theta_off) % 16 == state_rem;
        }
        if (sp.flags & (PASS_PARTIAL_IN | PASS_PARTIAL_OUT)) {
            aligned = aligned && ((uintptr_t)(ctx->partial + m.partial_off) % 16 == 0);
            state_congruent = state_congruent && (uintptr_t)(ctx->partial + m.partial_off) % 16 == state_rem;
        }
        if ((sp.flags & PASS_CAST_IN) || sp.cast_out) {
            const uintptr_t cast_addr = (uintptr_t)ctx->cast_scratch + (uintptr_t)m.cast_off * es;
            aligned = aligned && cast_addr % 16 == 0;
            state_congruent = state_congruent && cast_addr % 16 == (state_pos * es) % 16;
        }
        pd.contrib_begin = (int)contribs.size();
        for (size_t j = 0; j < sp.contributors.size(); ++j) {
            char *base = static_cast<char *>(lookup.get(sp.contributors[j]));
            if (!base) return DIPACO_EINVAL;
            ContribDev c;
            c.src = base + m.path_off * es;
            c.coeff = sp.coeff[j];
            c.pad = 0;
            aligned = aligned && ((uintptr_t)c.src % 16 == 0);
            contribs.push_back(c);
        }
        pd.contrib_count = (int)sp.contributors.size();
        pd.member_begin = (int)members.size();
        for (int path : sp.members) {
            char *base = static_cast<char *>(lookup.get(path));
            if (!base) return DIPACO_EINVAL;
            void *dst = base + m.path_off * es;
            aligned = aligned && ((uintptr_t)dst % 16 == 0);
            members.push_back(dst);
        }
        if (sp.cast_out)  // the module's slot in the cast scratch is one more destination
            members.push_back(static_cast<char *>(ctx->cast_scratch) + m.cast_off * es);
        if (extra_dst && i < extra_dst->size())
            for (void *dst : (*extra_dst)[i]) {
                aligned = aligned && ((uintptr_t)dst % 16 == 0);
                members.push_back(dst);
            }
        pd.member_count = (int)members.size() - pd.member_begin;
        pd.aligned_members = pd.member_count;

        // The vector kernel takes full tiles; the bulk-copy kernel also takes a partial last tile
        // as long as it is a whole number of 16-byte units of path data.
        const int64_t lo = sp.begin, hi = sp.end < 0 ? m.numel : sp.end;
        if (lo < 0 || hi > m.numel || lo > hi) return DIPACO_EINVAL;
        // a range that does not start on a 16-byte unit of both theta and the path data is
        // handled like a misaligned module
        const int64_t unit = 16 / es;
        if (lo % unit != 0) aligned = false;
        int64_t full = 0;
        if (aligned && ctx->kernel == DIPACO_KERNEL_VECTOR) full = (hi - lo) / tile * tile;
        if (aligned && ctx->kernel == DIPACO_KERNEL_AUTO) full = (hi - lo) / unit * unit;
        bulk_begin[i] = lo; bulk_end[i] = lo + full;
        if (!aligned && state_congruent && ctx->kernel != DIPACO_KERNEL_SCALAR) {
            // Path buffers at odd element offsets (or a range that starts inside a 16-byte unit).
            // The range of the vector or bulk-copy kernel starts at the first element at which
            // theta is 32-byte aligned.  Both read the aligned 16-byte units around the data, so
            // the last 8 elements of the range stay with the one-element kernel: no load reaches
            // past the module's slot in a path buffer.
            const int64_t first = lo + (int64_t)((8 - (state_pos + (uintptr_t)(lo % 8)) % 8) % 8);
            int64_t covered = 0;
            if (hi - 8 > first)
                covered = ctx->kernel == DIPACO_KERNEL_VECTOR ? (hi - 8 - first) / SHIFT_TILE * SHIFT_TILE
                                                              : (hi - 8 - first) / unit * unit;
            if (covered > 0) {
                // Destinations with the same position inside a 16-byte unit (at the range's
                // tiles) next to each other, the aligned ones first: both kernels rebuild their
                // realigned units only when that position changes, and the bulk-copy kernel
                // writes the aligned ones with bulk stores.  The order has no effect on results.
                const uintptr_t at_first = (uintptr_t)first * (uintptr_t)es;
                auto shift_of = [at_first](void *x) { return ((uintptr_t)x + at_first) & 15u; };
                std::stable_sort(members.begin() + pd.member_begin, members.end(),
                                 [&](void *x, void *y) { return shift_of(x) < shift_of(y); });
                int n_aligned = 0;
                while (n_aligned < pd.member_count && shift_of(members[(size_t)(pd.member_begin + n_aligned)]) == 0)
                    ++n_aligned;
                pd.aligned_members = n_aligned;
                if (ctx->kernel == DIPACO_KERNEL_VECTOR) {
                    shv_begin[i] = first;
                    shv_end[i] = first + covered;
                    bulk_begin[i] = bulk_end[i] = lo;
                } else {
                    bulk_begin[i] = first;
                    bulk_end[i] = first + covered;
                    any_shifted = true;
                }
                add_ragged(i, lo, first);
                add_ragged(i, first + covered, hi);
                continue;
            }
        }
        add_ragged(i, lo + full, hi);
    }

    std::vector<Segment> bulk_segs, rag_segs, shv_segs;
    std::vector<int32_t> bulk_first, rag_first, shv_first;
    const bool vector_kernel = ctx->kernel == DIPACO_KERNEL_VECTOR;
    int bulk_ctas = ctx->sm_count * (vector_kernel ? 8 : ctx->ctas_per_sm);
    int64_t bulk_tiles = 0, rag_tiles = 0, shv_tiles = 0;
    double bulk_bytes = 0.0, contrib_elems = 0.0, bulk_elems = 0.0;
    for (size_t i = 0; i < specs.size(); ++i) {
        contrib_elems += (double)specs[i].contributors.size() * (double)(bulk_end[i] - bulk_begin[i]);
        bulk_elems += (double)(bulk_end[i] - bulk_begin[i]);
        bulk_tiles += (bulk_end[i] - bulk_begin[i] + tile - 1) / tile;
        bulk_bytes += pass_cost_per_elem(specs[i], es) * (double)(bulk_end[i] - bulk_begin[i]);
        shv_tiles += (shv_end[i] - shv_begin[i]) / SHIFT_TILE;
    }
    for (size_t r = 0; r < rag_begin.size(); ++r)
        rag_tiles += (rag_end[r] - rag_begin[r] + RAGGED_TILE - 1) / RAGGED_TILE;
    if (bulk_tiles < bulk_ctas) bulk_ctas = (int)bulk_tiles;
    int rag_ctas = (int)std::min<int64_t>(rag_tiles, (int64_t)ctx->sm_count * 8);
    int64_t total_items = 0;
    if (bulk_ctas > 0 && vector_kernel) {
        split_segments(specs, bulk_begin, bulk_end, es, tile, bulk_ctas, bulk_segs, bulk_first);
    } else if (bulk_ctas > 0) {
        // Work items of about equal traffic, small enough that every CTA draws many of them.
        const double target =
            std::min((double)ctx->item_bytes, bulk_bytes / ((double)bulk_ctas * (double)ctx->items_per_cta));
        for (size_t i = 0; i < specs.size(); ++i) {
            const int64_t ntiles = (bulk_end[i] - bulk_begin[i] + tile - 1) / tile;
            const double per_tile = pass_cost_per_elem(specs[i], es) * (double)tile;
            int64_t tpi = (int64_t)std::floor(target / per_tile + 0.5);
            if (tpi < 1) tpi = 1;
            if (tpi > (1 << 20)) tpi = 1 << 20;
            passes[i].item_first = (int)total_items;
            passes[i].tiles_per_item = (int)tpi;
            passes[i].bulk_tiles = ntiles;
            passes[i].bulk_begin = bulk_begin[i];
            passes[i].bulk_end = bulk_end[i];
            total_items += (ntiles + tpi - 1) / tpi;
        }
        if (total_items > 0x7fff0000) return DIPACO_EINVAL;
        if (total_items < bulk_ctas) bulk_ctas = (int)total_items;
    }
    if (rag_ctas > 0)
        split_segments(specs, rag_begin, rag_end, es, RAGGED_TILE, rag_ctas, rag_segs, rag_first, &rag_pass);
    const int shv_ctas = (int)std::min<int64_t>(shv_tiles, (int64_t)ctx->sm_count * 8);
    if (shv_ctas > 0)
        split_segments(specs, shv_begin, shv_end, es, SHIFT_TILE, shv_ctas, shv_segs, shv_first);

    auto append = [&](const void *src, size_t bytes) -> size_t {
        const size_t off = align_up(blob.size(), 16);
        blob.resize(off + bytes);
        if (bytes) std::memcpy(blob.data() + off, src, bytes);
        return off;
    };
    out.passes_off = append(passes.data(), passes.size() * sizeof(PassDev));
    out.contribs_off = append(contribs.data(), contribs.size() * sizeof(ContribDev));
    out.members_off = append(members.data(), members.size() * sizeof(void *));
    static_assert(sizeof(Segment) == sizeof(SegmentDev), "segment layouts must match");
    out.bulk_segs_off = append(bulk_segs.data(), bulk_segs.size() * sizeof(Segment));
    out.bulk_first_off = append(bulk_first.data(), bulk_first.size() * sizeof(int32_t));
    out.rag_segs_off = append(rag_segs.data(), rag_segs.size() * sizeof(Segment));
    out.rag_first_off = append(rag_first.data(), rag_first.size() * sizeof(int32_t));
    out.shv_segs_off = append(shv_segs.data(), shv_segs.size() * sizeof(Segment));
    out.shv_first_off = append(shv_first.data(), shv_first.size() * sizeof(int32_t));
    out.bulk_ctas = bulk_ctas;
    out.rag_ctas = rag_ctas;
    out.shv_ctas = shv_ctas;
    out.io_arrays = io_arrays;
    out.units = units;
    out.aligned_kernel_is_vector = vector_kernel;
    out.shifted = any_shifted;
    out.num_passes = (int)passes.size();
    out.total_items = (int)total_items;
    out.mean_contributors = bulk_elems > 0.0 ? contrib_elems / bulk_elems : 0.0;
    return DIPACO_OK;
}

// Copy a packed blob to the device through a pinned staging slot (asynchronous on `stream`).
int upload_blob(dipaco_ctx *ctx, const std::vector<unsigned char> &blob, cudaStream_t stream)
{
    const size_t bytes = std::max<size_t>(blob.size(), 16);
    if (ctx->dev_tables && blob.size() == ctx->last_blob.size() &&
        std::memcmp(blob.data(), ctx->last_blob.data(), blob.size()) == 0)
        return DIPACO_OK;  // same pointers, mask and weights as the previous call
    ctx->last_blob.clear();
    ctx->plan_valid = false;  // the device tables are about to change
    if (bytes > ctx->dev_tables_capacity) {
        // grow: wait for earlier work that may still read the old tables
        if (cudaStreamSynchronize(stream) != cudaSuccess) return DIPACO_ECUDA;
        if (ctx->last_stream && ctx->last_stream != stream &&
            cudaStreamSynchronize(ctx->last_stream) != cudaSuccess)
            return DIPACO_ECUDA;
        if (ctx->dev_tables) cudaFree(ctx->dev_tables);
        ctx->dev_tables = nullptr;
        const size_t cap = align_up(bytes * 2, 4096);
        if (cudaMalloc(&ctx->dev_tables, cap) != cudaSuccess) {
            ctx->dev_tables_capacity = 0;
            return DIPACO_ENOMEM;
        }
        ctx->dev_tables_capacity = cap;
    }
    Staging &st = ctx->staging[ctx->staging_next];
    ctx->staging_next = (ctx->staging_next + 1) % STAGING_SLOTS;
    if (st.in_flight) {
        if (cudaEventSynchronize(st.done) != cudaSuccess) return DIPACO_ECUDA;
        st.in_flight = false;
    }
    if (bytes > st.capacity) {
        if (st.host) cudaFreeHost(st.host);
        st.host = nullptr;
        st.capacity = 0;
        const size_t cap = align_up(bytes * 2, 4096);
        if (cudaMallocHost(&st.host, cap) != cudaSuccess) return DIPACO_ENOMEM;
        st.capacity = cap;
    }
    if (!st.done && cudaEventCreateWithFlags(&st.done, cudaEventDisableTiming) != cudaSuccess)
        return DIPACO_ECUDA;
    std::memcpy(st.host, blob.data(), blob.size());
    if (cudaMemcpyAsync(ctx->dev_tables, st.host, bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return DIPACO_ECUDA;
    if (cudaEventRecord(st.done, stream) != cudaSuccess) return DIPACO_ECUDA;
    st.in_flight = true;
    ctx->last_blob = blob;
    return DIPACO_OK;
}

template <typename PathT, int NU, bool SHIFTED>
int launch_bulk_t(dipaco_ctx *ctx, const LaunchParams &lp, int ctas, int stages, int io_arrays, int io_slots,
                  size_t smem, cudaStream_t stream)
{
    bool &attr_set = ctx->smem_attr_set[sizeof(PathT) == 2 ? 1 : 0][NU == 1 ? 0 : (NU == 2 ? 1 : 2)][SHIFTED ? 1 : 0];
    if (!attr_set) {
        if (cudaFuncSetAttribute(sync_bulk_kernel<PathT, NU, SHIFTED>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)SMEM_LIMIT) != cudaSuccess)
            return DIPACO_ECUDA;
        attr_set = true;
    }
    sync_bulk_kernel<PathT, NU, SHIFTED><<<ctas, SHIFTED ? BULK_SHIFTED_THREADS : BULK_THREADS, smem, stream>>>(
        lp, stages, io_arrays, io_slots);
    return cudaGetLastError() == cudaSuccess ? DIPACO_OK : DIPACO_ECUDA;
}

template <typename PathT, bool SHIFTED>
int launch_bulk_units(dipaco_ctx *ctx, const LaunchParams &lp, int ctas, int stages, int io_arrays,
                      int io_slots, size_t smem, int nu, cudaStream_t stream)
{
    if (nu == 1) return launch_bulk_t<PathT, 1, SHIFTED>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, stream);
    if (nu == 2) return launch_bulk_t<PathT, 2, SHIFTED>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, stream);
    return launch_bulk_t<PathT, 4, SHIFTED>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, stream);
}

int launch_bulk(dipaco_ctx *ctx, const LaunchParams &lp, int ctas, int io_arrays, int nu,
                double mean_contributors, bool shifted, cudaStream_t stream)
{
    // Shared memory is split between the ring of path tiles and the theta/momentum/result
    // buffers.  Launches dominated by many-contributor modules need the ring depth (10 stages
    // measured best), launches with few contributors per module need the extra buffers.
    const int wanted = ctx->stages > 0 ? std::min(ctx->stages, 10) : 10;
    const int min_stages = mean_contributors >= 8.0 ? wanted : std::min(wanted, 6);
    int io_slots = ctx->io_slots;
    while (io_slots > 2 && pick_stages(ctx, nu, io_arrays, io_slots, shifted) < min_stages) --io_slots;
    const int stages = pick_stages(ctx, nu, io_arrays, io_slots, shifted);
    if (stages < 2) return DIPACO_EINVAL;
    const size_t smem = bulk_smem_bytes(ctx, nu, stages, io_arrays, io_slots, shifted);
    if (ctx->dtype == DIPACO_BF16)
        return shifted ? launch_bulk_units<__nv_bfloat16, true>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, nu, stream)
                       : launch_bulk_units<__nv_bfloat16, false>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, nu, stream);
    return shifted ? launch_bulk_units<float, true>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, nu, stream)
                   : launch_bulk_units<float, false>(ctx, lp, ctas, stages, io_arrays, io_slots, smem, nu, stream);
}

int launch_packed(dipaco_ctx *ctx, const PackedLaunch &pl, float *theta, float *momentum,
                  int *work_counter, cudaStream_t stream)
{
    const char *base = static_cast<const char *>(ctx->dev_tables);
    LaunchParams lp;
    lp.theta = theta;
    lp.momentum = momentum;
    lp.partial = ctx->partial;
    lp.cast_scratch = ctx->cast_scratch;
    lp.passes = reinterpret_cast<const PassDev *>(base + pl.passes_off);
    lp.contribs = reinterpret_cast<const ContribDev *>(base + pl.contribs_off);
    lp.members = reinterpret_cast<void *const *>(base + pl.members_off);
    const bool adam = ctx->optimizer == DIPACO_OPT_ADAM;
    lp.rule.lr = ctx->lr;
    lp.rule.mu = ctx->mu;
    lp.rule.optimizer = ctx->optimizer;
    lp.rule.b1 = (float)ctx->adam_b1;
    lp.rule.one_minus_b1 = (float)(1.0 - ctx->adam_b1);
    lp.rule.b2 = (float)ctx->adam_b2;
    lp.rule.one_minus_b2 = (float)(1.0 - ctx->adam_b2);
    lp.rule.eps = (float)ctx->adam_eps;
    lp.rule.decay = (float)(1.0 - (double)ctx->lr * ctx->adam_wd);
    lp.rule.inv_c1 = ctx->adam_step > 0 ? (float)(1.0 / (1.0 - std::pow(ctx->adam_b1, ctx->adam_step))) : 1.0f;
    lp.rule.inv_c2 = ctx->adam_step > 0 ? (float)(1.0 / (1.0 - std::pow(ctx->adam_b2, ctx->adam_step))) : 1.0f;
    lp.second_moment = !adam ? nullptr
                             : (ctx->second_moment_staged ? ctx->second_moment_staged : ctx->second_moment);
    lp.input_kind = ctx->input_kind;
    lp.v_index = pl.io_arrays - 1;
    lp.error_word = ctx->error_word;
    lp.num_passes = pl.num_passes;
    lp.total_items = pl.total_items;
    lp.work_counter = work_counter;
    if (pl.bulk_ctas > 0) {
        lp.segs = reinterpret_cast<const SegmentDev *>(base + pl.bulk_segs_off);
        lp.cta_first = reinterpret_cast<const int *>(base + pl.bulk_first_off);
        int rc = DIPACO_OK;
        if (pl.aligned_kernel_is_vector) {
            if (ctx->dtype == DIPACO_BF16)
                sync_direct_kernel<__nv_bfloat16, 8><<<pl.bulk_ctas, 256, 0, stream>>>(lp);
            else
                sync_direct_kernel<float, 8><<<pl.bulk_ctas, 256, 0, stream>>>(lp);
            if (cudaGetLastError() != cudaSuccess) rc = DIPACO_ECUDA;
        } else {
            rc = launch_bulk(ctx, lp, pl.bulk_ctas, pl.io_arrays, pl.units, pl.mean_contributors, pl.shifted, stream);
        }
        if (rc != DIPACO_OK) return rc;
        ++ctx->launches;
    }
    if (pl.shv_ctas > 0) {
        lp.segs = reinterpret_cast<const SegmentDev *>(base + pl.shv_segs_off);
        lp.cta_first = reinterpret_cast<const int *>(base + pl.shv_first_off);
        if (ctx->dtype == DIPACO_BF16)
            sync_direct_kernel<__nv_bfloat16, 8, true><<<pl.shv_ctas, 256, 0, stream>>>(lp);
        else
            sync_direct_kernel<float, 8, true><<<pl.shv_ctas, 256, 0, stream>>>(lp);
        if (cudaGetLastError() != cudaSuccess) return DIPACO_ECUDA;
        ++ctx->launches;
    }
    if (pl.rag_ctas > 0) {
        lp.segs = reinterpret_cast<const SegmentDev *>(base + pl.rag_segs_off);
        lp.cta_first = reinterpret_cast<const int *>(base + pl.rag_first_off);
        if (ctx->dtype == DIPACO_BF16)
            sync_direct_kernel<__nv_bfloat16, 1><<<pl.rag_ctas, 256, 0, stream>>>(lp);
        else
            sync_direct_kernel<float, 1><<<pl.rag_ctas, 256, 0, stream>>>(lp);
        if (cudaGetLastError() != cudaSuccess) return DIPACO_ECUDA;
        ++ctx->launches;
    }
    return DIPACO_OK;
}

// Plan, upload and launch a list of launches that share one upload.
struct LaunchRequest {
    std::vector<PassSpec> specs;
    PtrLookup lookup;
    std::vector<std::vector<void *>> extra_dst;
};

int launch_all(dipaco_ctx *ctx, const std::vector<PackedLaunch> &packed, float *theta, float *momentum,
               cudaStream_t stream)
{
    for (size_t i = 0; i < packed.size(); ++i) {
        // every bulk launch leaves its pair of counters at zero again, so pairs can be reused
        // by later launches on the same stream
        const int c = (int)(i % MAX_COUNTERS);
        const int rc = launch_packed(ctx, packed[i], theta, momentum, ctx->counters + 2 * c, stream);
        if (rc != DIPACO_OK) return rc;
    }
    ctx->last_stream = stream;
    return DIPACO_OK;
}

int run_launches(dipaco_ctx *ctx, std::vector<LaunchRequest> &reqs, float *theta, float *momentum,
                 cudaStream_t stream, std::vector<PackedLaunch> *keep = nullptr)
{
    std::vector<unsigned char> blob;
    std::vector<PackedLaunch> packed(reqs.size());
    for (size_t i = 0; i < reqs.size(); ++i) {
        const int rc = pack_launch(ctx, reqs[i].specs, reqs[i].lookup,
                                   reqs[i].extra_dst.empty() ? nullptr : &reqs[i].extra_dst, theta,
                                   momentum, blob, packed[i]);
        if (rc != DIPACO_OK) return rc;
    }
    int rc = upload_blob(ctx, blob, stream);
    if (rc != DIPACO_OK) return rc;
    rc = launch_all(ctx, packed, theta, momentum, stream);
    if (rc == DIPACO_OK && keep) *keep = std::move(packed);
    return rc;
}

bool valid_ptr_array(void *const *ptrs, int n)
{
    if (!ptrs) return false;
    for (int i = 0; i < n; ++i)
        if (!ptrs[i]) return false;
    return true;
}

int chunk_first(const Grid &g, int c) { return c * g.chunk_paths; }
int chunk_count(const Grid &g, int c) { return std::min(g.chunk_paths, g.P - c * g.chunk_paths); }

} // namespace

#include "host_mode.inl"

// ------------------------------------------------------------------------------------------ C ABI

extern "C" {

int dipaco_create(dipaco_ctx **out, int32_t num_levels, const int32_t *modules_per_level,
                  const int64_t *level_numel, int32_t num_paths, const int32_t *path_to_module,
                  const float *path_weights, float outer_lr, float outer_momentum,
                  int32_t path_dtype, int32_t chunk_paths, int32_t device)
{
    if (!out) return DIPACO_EINVAL;
    *out = nullptr;
    if (path_dtype != DIPACO_F32 && path_dtype != DIPACO_BF16) return DIPACO_EINVAL;
    if (!std::isfinite(outer_lr) || !std::isfinite(outer_momentum)) return DIPACO_EINVAL;
    if (device < -1) return DIPACO_EINVAL;
    dipaco_ctx *ctx = new (std::nothrow) dipaco_ctx();
    if (!ctx) return DIPACO_ENOMEM;
    try {
        if (!build_grid(ctx->grid, num_levels, modules_per_level, level_numel, num_paths,
                        path_to_module, path_weights, chunk_paths)) {
            delete ctx;
            return DIPACO_EINVAL;
        }
    } catch (const std::bad_alloc &) {
        delete ctx;
        return DIPACO_ENOMEM;
    }
    ctx->lr = outer_lr;
    ctx->mu = outer_momentum;
    ctx->dtype = path_dtype;
    ctx->elem_size = path_dtype == DIPACO_BF16 ? 2 : 4;
    ctx->device = device;
    if (device >= 0) {
        int count = 0;
        if (cudaGetDeviceCount(&count) != cudaSuccess || device >= count) {
            delete ctx;
            return DIPACO_ECUDA;
        }
        DeviceGuard guard(device);
        if (!guard.ok ||
            cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            delete ctx;
            return DIPACO_ECUDA;
        }
        if (cudaMalloc(&ctx->error_word, sizeof(int)) != cudaSuccess ||
            cudaMemset(ctx->error_word, 0, sizeof(int)) != cudaSuccess ||
            cudaMalloc(&ctx->counters, 2 * MAX_COUNTERS * sizeof(int)) != cudaSuccess ||
            cudaMemset(ctx->counters, 0, 2 * MAX_COUNTERS * sizeof(int)) != cudaSuccess) {
            dipaco_destroy(ctx);
            return DIPACO_ENOMEM;
        }
        if (ctx->grid.scratch_elems > 0 &&
            cudaMalloc(&ctx->partial, (size_t)ctx->grid.scratch_elems * sizeof(float)) != cudaSuccess) {
            cudaGetLastError();
            dipaco_destroy(ctx);
            return DIPACO_ENOMEM;
        }
    }
    *out = ctx;
    return DIPACO_OK;
}

int dipaco_destroy(dipaco_ctx *ctx)
{
    if (!ctx) return DIPACO_EINVAL;
    int rc = DIPACO_OK;
    if (ctx->device >= 0) {
        DeviceGuard guard(ctx->device);
        if (ctx->last_stream || ctx->stream) {
            if (cudaStreamSynchronize(ctx->last_stream ? ctx->last_stream : ctx->stream) != cudaSuccess)
                rc = DIPACO_ECUDA;
        }
        host_mode_release(ctx);
        for (Staging &st : ctx->staging) {
            if (st.done) cudaEventDestroy(st.done);
            if (st.host) cudaFreeHost(st.host);
        }
        if (ctx->dev_tables) cudaFree(ctx->dev_tables);
        if (ctx->partial) cudaFree(ctx->partial);
        if (ctx->cast_scratch) cudaFree(ctx->cast_scratch);
        if (ctx->error_word) cudaFree(ctx->error_word);
        if (ctx->counters) cudaFree(ctx->counters);
    }
    delete ctx;
    return rc;
}

int dipaco_set_weights(dipaco_ctx *ctx, const float *path_weights)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    if (path_weights) {
        for (int i = 0; i < ctx->grid.P; ++i)
            if (!(path_weights[i] >= 0.0f) || !std::isfinite(path_weights[i])) return DIPACO_EINVAL;
        ctx->grid.weights.assign(path_weights, path_weights + ctx->grid.P);
    } else {
        ctx->grid.weights.clear();
    }
    return DIPACO_OK;
}

int dipaco_set_module_scale(dipaco_ctx *ctx, const float *module_scale)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    if (module_scale) {
        const size_t n = ctx->grid.modules.size();
        for (size_t i = 0; i < n; ++i)
            if (!std::isfinite(module_scale[i])) return DIPACO_EINVAL;
        ctx->grid.module_scale.assign(module_scale, module_scale + n);
    } else {
        ctx->grid.module_scale.clear();
    }
    return DIPACO_OK;
}

int dipaco_set_level_sync(dipaco_ctx *ctx, const uint8_t *level_sync)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    if (level_sync) ctx->grid.level_sync.assign(level_sync, level_sync + ctx->grid.L);
    else ctx->grid.level_sync.clear();
    return DIPACO_OK;
}

int dipaco_set_optimizer(dipaco_ctx *ctx, int32_t optimizer)
{
    if (!ctx || optimizer < DIPACO_OPT_NESTEROV || optimizer > DIPACO_OPT_ADAM) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    if (optimizer == DIPACO_OPT_ADAM && !ctx->second_moment) return DIPACO_ESTATE;  // dipaco_set_adam first
    ctx->optimizer = optimizer;
    ctx->grid.second_moment = optimizer == DIPACO_OPT_ADAM;
    return DIPACO_OK;
}

int dipaco_set_adam(dipaco_ctx *ctx, float *second_moment, float beta1, float beta2, float eps,
                    float weight_decay, int32_t step)
{
    if (!ctx || !second_moment || step < 0) return DIPACO_EINVAL;
    if (!(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f)) return DIPACO_EINVAL;
    if (!(eps >= 0.0f) || !std::isfinite(eps) || !std::isfinite(weight_decay)) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    ctx->second_moment = second_moment;
    ctx->adam_b1 = beta1;
    ctx->adam_b2 = beta2;
    ctx->adam_eps = eps;
    ctx->adam_wd = weight_decay;
    ctx->adam_step = step;
    ctx->optimizer = DIPACO_OPT_ADAM;
    ctx->grid.second_moment = true;
    return DIPACO_OK;
}

int dipaco_set_input_kind(dipaco_ctx *ctx, int32_t input_kind)
{
    if (!ctx || (input_kind != DIPACO_INPUT_COPIES && input_kind != DIPACO_INPUT_GRADIENTS))
        return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    ctx->input_kind = input_kind;
    return DIPACO_OK;
}

int dipaco_set_shard(dipaco_ctx *ctx, int32_t shard_index, int32_t shard_count)
{
    if (!ctx || shard_count < 1 || shard_index < 0 || shard_index >= shard_count) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    ctx->grid.shard_index = shard_index;
    ctx->grid.shard_count = shard_count;
    return DIPACO_OK;
}

int dipaco_set_kernel(dipaco_ctx *ctx, int32_t kernel)
{
    if (!ctx || kernel < DIPACO_KERNEL_AUTO || kernel > DIPACO_KERNEL_SCALAR) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    ctx->kernel = kernel;
    return DIPACO_OK;
}

int dipaco_set_tuning(dipaco_ctx *ctx, int32_t ctas_per_sm, int32_t stages, int32_t units_per_thread,
                      int32_t io_slots)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    if (ctas_per_sm < 0 || ctas_per_sm > 8 || stages < 0 || stages == 1 || stages > BULK_MAX_STAGES)
        return DIPACO_EINVAL;
    if (units_per_thread != 0 && units_per_thread != 1 && units_per_thread != 2 && units_per_thread != 4)
        return DIPACO_EINVAL;
    if (io_slots != 0 && (io_slots < 2 || io_slots > BULK_MAX_IO_SLOTS)) return DIPACO_EINVAL;
    const int old_ctas = ctx->ctas_per_sm, old_units = ctx->units, old_stages = ctx->stages;
    if (ctas_per_sm) ctx->ctas_per_sm = ctas_per_sm;
    if (units_per_thread) ctx->units = units_per_thread;
    ctx->stages = 0;
    // chunked contexts stage a third fp32 tile (the partial sum) per buffer
    const int io_arrays = (ctx->grid.num_chunks > 1 ? 3 : 2) + (ctx->optimizer == DIPACO_OPT_ADAM ? 1 : 0);
    const int nu = tile_units(ctx);
    const bool fits = pick_stages(ctx, nu, io_arrays, 2) >= 2 && (!stages || stages <= pick_stages(ctx, nu, io_arrays, 2));
    if (!fits) {
        ctx->ctas_per_sm = old_ctas;
        ctx->units = old_units;
        ctx->stages = old_stages;
        return DIPACO_EINVAL;
    }
    ctx->stages = stages ? stages : old_stages;
    if (io_slots) ctx->io_slots = io_slots;
    return DIPACO_OK;
}

int dipaco_set_work_items(dipaco_ctx *ctx, int64_t max_item_bytes, int32_t items_per_cta)
{
    if (!ctx || max_item_bytes < 0 || items_per_cta < 0 || items_per_cta > 4096) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    if (max_item_bytes) ctx->item_bytes = max_item_bytes;
    if (items_per_cta) ctx->items_per_cta = items_per_cta;
    return DIPACO_OK;
}

int dipaco_set_host_threads(dipaco_ctx *ctx, int32_t threads)
{
    if (!ctx || threads < -1 || threads > 256) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    ctx->host_threads = threads < 0 ? default_host_threads() : threads;
    return DIPACO_OK;
}

int dipaco_set_host_unit_bytes(dipaco_ctx *ctx, int64_t bytes)
{
    if (!ctx || bytes < 0) return DIPACO_EINVAL;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    ++ctx->settings_version;
    ctx->host_unit_bytes = bytes == 0 ? (int64_t)512 << 20 : bytes;
    return DIPACO_OK;
}

int dipaco_sync_begin(dipaco_ctx *ctx, float *theta, float *momentum, const uint8_t *reported,
                      void *cuda_stream)
{
    if (!ctx || !theta || !momentum) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    if (ctx->grid.chunk_paths <= 0) return DIPACO_ESTATE;
    try {
        compute_all_coeffs(ctx, reported);
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
    // bf16 copies: the write-back launches of this API read cast(theta') (2 bytes per parameter)
    // from a scratch that the finishing passes fill, instead of fp32 theta'.  Allocated on the
    // first round; without it (no memory) the write-back reads theta' as before.
    if (ctx->elem_size != 4 && !ctx->cast_scratch && !ctx->cast_scratch_tried && ctx->grid.cast_elems > 0) {
        ctx->cast_scratch_tried = true;
        DeviceGuard guard(ctx->device);
        if (!guard.ok) return DIPACO_ECUDA;
        if (cudaMalloc(&ctx->cast_scratch, (size_t)ctx->grid.cast_elems * ctx->elem_size) != cudaSuccess) {
            cudaGetLastError();
            ctx->cast_scratch = nullptr;
        }
    }
    ctx->theta = theta;
    ctx->momentum = momentum;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->next_chunk = 0;
    ctx->state = STATE_ACCUMULATING;
    return DIPACO_OK;
}

int dipaco_sync_accumulate(dipaco_ctx *ctx, int32_t chunk_index, void *const *chunk_ptrs)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_ACCUMULATING) return DIPACO_ESTATE;
    if (chunk_index != ctx->next_chunk || chunk_index >= ctx->grid.num_chunks) return DIPACO_ESTATE;
    const int n = chunk_count(ctx->grid, chunk_index);
    if (!valid_ptr_array(chunk_ptrs, n)) return DIPACO_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DIPACO_ECUDA;
    try {
        std::vector<LaunchRequest> reqs(1);
        plan_accumulate(ctx->grid, ctx->coeffs, chunk_index, reqs[0].specs, false,
                        ctx->cast_scratch != nullptr);
        reqs[0].lookup = PtrLookup{chunk_ptrs, chunk_first(ctx->grid, chunk_index), n};
        if (!reqs[0].specs.empty()) {
            const int rc = run_launches(ctx, reqs, ctx->theta, ctx->momentum, ctx->stream);
            if (rc != DIPACO_OK) return rc;
        }
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
    ++ctx->next_chunk;
    return DIPACO_OK;
}

int dipaco_sync_writeback(dipaco_ctx *ctx, int32_t chunk_index, void *const *chunk_ptrs)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_ACCUMULATING || ctx->next_chunk != ctx->grid.num_chunks) return DIPACO_ESTATE;
    if (chunk_index < 0 || chunk_index >= ctx->grid.num_chunks) return DIPACO_EINVAL;
    const int n = chunk_count(ctx->grid, chunk_index);
    if (!valid_ptr_array(chunk_ptrs, n)) return DIPACO_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DIPACO_ECUDA;
    try {
        std::vector<LaunchRequest> reqs(1);
        plan_writeback(ctx->grid, ctx->coeffs, chunk_index, false, reqs[0].specs,
                       ctx->cast_scratch != nullptr);
        reqs[0].lookup = PtrLookup{chunk_ptrs, chunk_first(ctx->grid, chunk_index), n};
        if (!reqs[0].specs.empty()) {
            const int rc = run_launches(ctx, reqs, ctx->theta, ctx->momentum, ctx->stream);
            if (rc != DIPACO_OK) return rc;
        }
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
    return DIPACO_OK;
}

int dipaco_sync_end(dipaco_ctx *ctx)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_ACCUMULATING) return DIPACO_ESTATE;
    const bool complete = ctx->next_chunk == ctx->grid.num_chunks;
    ctx->state = STATE_IDLE;
    return complete ? DIPACO_OK : DIPACO_ESTATE;
}

int dipaco_outer_sync(dipaco_ctx *ctx, float *theta, float *momentum, void *const *path_ptrs,
                      const uint8_t *reported, void *cuda_stream)
{
    if (!ctx || !theta || !momentum) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    if (!valid_ptr_array(path_ptrs, ctx->grid.P)) return DIPACO_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DIPACO_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const Grid &g = ctx->grid;
    try {
        // Same settings, buffers and mask as the previous call, and its tables are still the ones
        // on the device: launch again, nothing to plan or upload.
        const size_t P = (size_t)g.P;
        std::vector<unsigned char> key(sizeof(uint64_t) + 3 * sizeof(void *) + 1 + P + P * sizeof(void *));
        {
            unsigned char *k = key.data();
            const void *fixed[3] = {theta, momentum, ctx->second_moment};
            std::memcpy(k, &ctx->settings_version, sizeof(uint64_t)); k += sizeof(uint64_t);
            std::memcpy(k, fixed, sizeof fixed); k += sizeof fixed;
            *k++ = reported ? 1 : 0;
            if (reported) for (size_t i = 0; i < P; ++i) k[i] = reported[i] ? 1 : 0;
            else std::memset(k, 1, P);
            k += P;
            std::memcpy(k, path_ptrs, P * sizeof(void *));
        }
        if (ctx->plan_valid && key == ctx->plan_key)
            return launch_all(ctx, ctx->plan_launches, theta, momentum, stream);
        ctx->plan_valid = false;

        compute_all_coeffs(ctx, reported);
        std::vector<LaunchRequest> reqs;
        const PtrLookup all_paths{path_ptrs, 0, g.P};
        if (g.num_chunks <= 1) {
            reqs.resize(1);
            plan_resident(g, ctx->coeffs, reqs[0].specs);
            reqs[0].lookup = all_paths;
        } else {
            // Walk the chunks in ascending order.  Every path copy is on the device here, so the
            // pass that finishes a module hands cast(theta') to all its paths at once, whatever
            // their chunk; modules that nobody updates are refilled in the first launch.
            for (int c = 0; c < g.num_chunks; ++c) {
                LaunchRequest r;
                plan_accumulate(g, ctx->coeffs, c, r.specs, true);
                r.lookup = all_paths;
                if (!r.specs.empty()) reqs.push_back(std::move(r));
            }
            LaunchRequest refill;
            plan_refill_unchanged(g, ctx->coeffs, refill.specs);
            refill.lookup = all_paths;
            if (!refill.specs.empty()) {
                if (reqs.empty()) reqs.push_back(std::move(refill));
                else
                    for (PassSpec &sp : refill.specs) reqs[0].specs.push_back(std::move(sp));
            }
        }
        bool any = false;
        for (auto &r : reqs) any = any || !r.specs.empty();
        if (!any) return DIPACO_OK;
        const int rc = run_launches(ctx, reqs, theta, momentum, stream, &ctx->plan_launches);
        if (rc == DIPACO_OK) {
            ctx->plan_key = std::move(key);
            ctx->plan_valid = true;
        }
        return rc;
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
}

int dipaco_outer_sync_host(dipaco_ctx *ctx, float *theta_host, float *momentum_host,
                           void *const *path_ptrs_host, const uint8_t *reported, void *cuda_stream)
{
    if (!ctx || !theta_host || !momentum_host) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    if (ctx->grid.chunk_paths <= 0) return DIPACO_ESTATE;
    if (!valid_ptr_array(path_ptrs_host, ctx->grid.P)) return DIPACO_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DIPACO_ECUDA;
    try {
        return host_mode_sync(ctx, theta_host, momentum_host, path_ptrs_host, reported,
                              static_cast<cudaStream_t>(cuda_stream));
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    } catch (const std::exception &) {
        return DIPACO_ENOMEM;  // the host threads could not be created: a resource limit
    }
}

int dipaco_plan_shard(const dipaco_ctx *ctx, int32_t shard_index, int32_t shard_count, int32_t level,
                      int64_t *begin, int64_t *end)
{
    if (!ctx || shard_count < 1 || shard_index < 0 || shard_index >= shard_count || level < 0 ||
        level >= ctx->grid.L)
        return DIPACO_EINVAL;
    int64_t lo = 0, hi = 0;
    Grid::slab_bounds(ctx->grid.N[(size_t)level], shard_index, shard_count, lo, hi);
    if (begin) *begin = lo;
    if (end) *end = hi;
    return DIPACO_OK;
}

int dipaco_create_shard(dipaco_ctx **out, const dipaco_ctx *whole, int32_t shard_index,
                        int32_t shard_count, int32_t device)
{
    if (!out) return DIPACO_EINVAL;
    *out = nullptr;
    if (!whole || shard_count < 1 || shard_index < 0 || shard_index >= shard_count) return DIPACO_EINVAL;
    const Grid &g = whole->grid;
    if (g.shard_count != 1) return DIPACO_ESTATE;  // a shard of a shard is not defined
    try {
        std::vector<int64_t> slab((size_t)g.L);
        for (int l = 0; l < g.L; ++l) {
            int64_t lo = 0, hi = 0;
            Grid::slab_bounds(g.N[(size_t)l], shard_index, shard_count, lo, hi);
            slab[(size_t)l] = hi - lo;
        }
        std::vector<int32_t> K(g.K.begin(), g.K.end()), table(g.table.begin(), g.table.end());
        dipaco_ctx *ctx = nullptr;
        const int rc = dipaco_create(&ctx, g.L, K.data(), slab.data(), g.P, table.data(),
                                     g.weights.empty() ? nullptr : g.weights.data(), whole->lr, whole->mu,
                                     whole->dtype, g.chunk_paths, device);
        if (rc != DIPACO_OK) return rc;
        ctx->grid.module_scale = g.module_scale;
        ctx->grid.level_sync = g.level_sync;
        ctx->input_kind = whole->input_kind;
        ctx->kernel = whole->kernel;
        ctx->ctas_per_sm = whole->ctas_per_sm;
        ctx->stages = whole->stages;
        ctx->units = whole->units;
        ctx->io_slots = whole->io_slots;
        ctx->item_bytes = whole->item_bytes;
        ctx->items_per_cta = whole->items_per_cta;
        ctx->host_unit_bytes = whole->host_unit_bytes;
        ctx->host_threads = whole->host_threads;
        // the Adam family needs the shard's own second-moment array: dipaco_set_adam on the shard
        ctx->optimizer = whole->optimizer == DIPACO_OPT_ADAM ? DIPACO_OPT_NESTEROV : whole->optimizer;
        *out = ctx;
        return DIPACO_OK;
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
}

int dipaco_selftest_wait_expiry(dipaco_ctx *ctx, int64_t limit_ns, void *cuda_stream)
{
    if (!ctx || limit_ns < 1 || limit_ns > 1000000000ll) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    if (ctx->state != STATE_IDLE) return DIPACO_ESTATE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DIPACO_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    wait_expiry_kernel<<<1, 32, 0, stream>>>(ctx->error_word, ctx->counters,
                                             (unsigned long long)limit_ns);
    if (cudaGetLastError() != cudaSuccess) return DIPACO_ECUDA;
    ctx->last_stream = stream;
    return DIPACO_OK;
}

int dipaco_device_status(dipaco_ctx *ctx)
{
    if (!ctx) return DIPACO_EINVAL;
    if (ctx->device < 0) return DIPACO_ENODEV;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DIPACO_ECUDA;
    cudaStream_t s = ctx->last_stream ? ctx->last_stream : ctx->stream;
    if (cudaStreamSynchronize(s) != cudaSuccess) return DIPACO_ECUDA;
    int word = 0;
    if (cudaMemcpy(&word, ctx->error_word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return DIPACO_ECUDA;
    if (word != 0) {
        cudaMemset(ctx->error_word, 0, sizeof(int));
        cudaMemset(ctx->counters, 0, 2 * MAX_COUNTERS * sizeof(int));  // a kernel that gave up did not re-arm them
        return DIPACO_ETIMEOUT;
    }
    return DIPACO_OK;
}

int64_t dipaco_launch_count(const dipaco_ctx *ctx) { return ctx ? ctx->launches : 0; }

int dipaco_plan_module(const dipaco_ctx *ctx, int32_t level, int32_t module, const uint8_t *reported,
                       int32_t *num_members, int32_t *members, int32_t *num_contributors,
                       int32_t *contributors, float *coeff, int32_t *will_update)
{
    if (!ctx || level < 0 || level >= ctx->grid.L || module < 0 || module >= ctx->grid.K[level])
        return DIPACO_EINVAL;
    try {
        const ModuleGeom &m = ctx->grid.modules[ctx->grid.module_id(level, module)];
        ModuleCoeffs mc;
        module_coeffs(ctx->grid, m, reported, mc);
        if (num_members) *num_members = (int32_t)m.members.size();
        if (members) std::copy(m.members.begin(), m.members.end(), members);
        if (num_contributors) *num_contributors = (int32_t)mc.contributors.size();
        if (contributors) std::copy(mc.contributors.begin(), mc.contributors.end(), contributors);
        if (coeff) std::copy(mc.coeff.begin(), mc.coeff.end(), coeff);
        if (will_update) *will_update = mc.update ? 1 : 0;
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
    return DIPACO_OK;
}

int dipaco_plan_offsets(const dipaco_ctx *ctx, int32_t level, int32_t module, int64_t *theta_offset,
                        int64_t *path_offset, int64_t *numel)
{
    if (!ctx || level < 0 || level >= ctx->grid.L || module < 0 || module >= ctx->grid.K[level])
        return DIPACO_EINVAL;
    const ModuleGeom &m = ctx->grid.modules[ctx->grid.module_id(level, module)];
    if (theta_offset) *theta_offset = m.theta_off;
    if (path_offset) *path_offset = m.path_off;
    if (numel) *numel = m.numel;
    return DIPACO_OK;
}

int dipaco_plan_chunks(const dipaco_ctx *ctx, int32_t *num_chunks, int64_t *scratch_elems)
{
    if (!ctx) return DIPACO_EINVAL;
    if (num_chunks) *num_chunks = ctx->grid.num_chunks;
    if (scratch_elems) *scratch_elems = ctx->grid.scratch_elems;
    return DIPACO_OK;
}

int dipaco_plan_traffic(const dipaco_ctx *ctx, const uint8_t *reported, int64_t *bytes,
                        int32_t *launches)
{
    if (!ctx) return DIPACO_EINVAL;
    try {
        const Grid &g = ctx->grid;
        std::vector<ModuleCoeffs> mc(g.modules.size());
        for (size_t id = 0; id < mc.size(); ++id) module_coeffs(g, g.modules[id], reported, mc[id]);
        double total = 0.0;
        int count = 0;
        std::vector<PassSpec> specs;
        auto add = [&]() {
            if (specs.empty()) return;
            ++count;
            for (const PassSpec &sp : specs)
                total += pass_cost_per_elem(sp, ctx->elem_size) *
                         (double)((sp.end < 0 ? g.modules[sp.module].numel : sp.end) - sp.begin);
        };
        if (g.num_chunks <= 1) {
            plan_resident(g, mc, specs);
            add();
        } else {
            // as dipaco_outer_sync walks them: the refill passes ride in the first launch
            std::vector<PassSpec> refill;
            plan_refill_unchanged(g, mc, refill);
            bool first = true;
            for (int c = 0; c < g.num_chunks; ++c) {
                plan_accumulate(g, mc, c, specs, true);
                if (specs.empty()) continue;
                if (first)
                    for (PassSpec &sp : refill) specs.push_back(sp);
                first = false;
                add();
            }
            if (first) { specs = refill; add(); }
        }
        if (bytes) *bytes = (int64_t)total;
        if (launches) *launches = count;
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
    return DIPACO_OK;
}

int dipaco_plan_split(const dipaco_ctx *ctx, const uint8_t *reported, int32_t num_ctas, int64_t tile,
                      int32_t capacity, int32_t *seg_level, int32_t *seg_module, int64_t *seg_begin,
                      int64_t *seg_end, int32_t *cta_first)
{
    if (!ctx || num_ctas < 1 || tile < 1 || capacity < 0) return DIPACO_EINVAL;
    try {
        std::vector<ModuleCoeffs> mc(ctx->grid.modules.size());
        for (size_t id = 0; id < mc.size(); ++id)
            module_coeffs(ctx->grid, ctx->grid.modules[id], reported, mc[id]);
        std::vector<PassSpec> specs;
        plan_resident(ctx->grid, mc, specs);
        std::vector<int64_t> begin(specs.size(), 0), end(specs.size(), 0);
        for (size_t i = 0; i < specs.size(); ++i)
            end[i] = ctx->grid.modules[specs[i].module].numel / tile * tile;
        std::vector<Segment> segs;
        std::vector<int32_t> first;
        split_segments(specs, begin, end, ctx->elem_size, tile, num_ctas, segs, first);
        if ((int64_t)segs.size() > capacity) return DIPACO_EINVAL;
        for (size_t s = 0; s < segs.size(); ++s) {
            const ModuleGeom &m = ctx->grid.modules[specs[segs[s].pass].module];
            if (seg_level) seg_level[s] = m.level;
            if (seg_module) seg_module[s] = m.index;
            if (seg_begin) seg_begin[s] = segs[s].begin;
            if (seg_end) seg_end[s] = segs[s].end;
        }
        if (cta_first)
            for (int b = 0; b <= num_ctas; ++b) cta_first[b] = first[(size_t)b];
        return (int)segs.size();
    } catch (const std::bad_alloc &) {
        return DIPACO_ENOMEM;
    }
}

const char *dipaco_strerror(int status)
{
    switch (status) {
    case DIPACO_OK: return "ok";
    case DIPACO_EINVAL: return "invalid argument";
    case DIPACO_ECUDA: return "CUDA runtime call failed";
    case DIPACO_ENOMEM: return "out of memory";
    case DIPACO_ESTATE: return "call not allowed in this state";
    case DIPACO_ETIMEOUT: return "a bounded wait inside a kernel ran out";
    case DIPACO_ENODEV: return "context has no device (plan only)";
    case DIPACO_ELIMIT: return "size exceeds the fixed limit of this entry point";
    default: return "unknown status";
    }
}

} // extern "C"
