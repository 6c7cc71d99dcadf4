// dipaco_outer_sync_host: the synchronisation for state kept in host memory.
// Included by dipaco.cu (inside its translation unit, after the launch helpers).
//
// Slab-ordered streaming.  The work is cut into units: an element range [a, b) of one module
// together with that range of EVERY reporting copy of the module.  A unit is therefore complete
// in itself: one fused pass (reduce in ascending path id + optimiser step + cast) finishes it, no
// partial sums are carried, and its result can leave the device at once.  Per unit:
//     H2D     theta[a:b], m[a:b] and the [a:b) piece of each reporting copy -> rows of an input buffer
//     kernel  the resident-mode pass on [a, b), reading the staged rows, writing theta', m' in
//             place and cast(theta') once per path of the module into the rows of an output buffer
//     D2H     theta'[a:b], m'[a:b], and each output row into its path's slot
// Streams for upload, kernel and download and a ring of three buffer sets overlap the upload of
// later units with the kernel and the download of earlier ones.  The download of a unit can only
// start once the unit is uploaded and reduced, so a step takes (bytes of the busier direction /
// PCIe rate) + about one unit's transfer time: units are kept small (dipaco_set_host_unit_bytes,
// 512 MiB by default), whatever the module's size.
// Every path of a module receives the SAME cast(theta').  With host threads (dipaco_set_host_threads,
// on by default) that piece crosses PCIe once per unit, into a small pinned bounce buffer, and a
// pool of host threads copies it into the slot of every path while later units upload: the
// device->host traffic shrinks from one copy per path to one per module, and the upload, which
// cannot shrink (every reporting copy is different data), has the link almost to itself.  With
// zero host threads the kernel writes one output row per path and all of them are downloaded.  Everything a unit's kernel needs besides the data (its tables) is uploaded
// once, before the first unit, so no small copy queues behind the bulk uploads.  Pieces of path
// copies that lie equally spaced in host memory (copies carved from one allocation) move as one
// strided 2-D copy per run instead of one copy per path.  Staging memory: at most chunk_paths
// path copies in total.  Paths that did not report are never uploaded.  Bitwise identical to the
// resident mode: same pass, same order.

namespace {

constexpr int HOST_BUFFERS = 3;
constexpr size_t HOST_BOUNCE_BYTES = (size_t)64 << 20;  // pinned landing buffer of one unit's cast piece

// Copy for destinations that will not be read again soon: streaming (non-temporal) stores write
// whole cache lines without first reading them, which halves the memory traffic of the fan-out
// and leaves more of the host's memory bandwidth to the PCIe uploads running beside it.
inline void copy_streaming(char *dst, const char *src, size_t n)
{
#if defined(__SSE2__)
    if (reinterpret_cast<uintptr_t>(dst) % 16 == 0) {
        size_t i = 0;
        for (; i + 64 <= n; i += 64) {
            const __m128i a = _mm_loadu_si128(reinterpret_cast<const __m128i *>(src + i));
            const __m128i b = _mm_loadu_si128(reinterpret_cast<const __m128i *>(src + i + 16));
            const __m128i c = _mm_loadu_si128(reinterpret_cast<const __m128i *>(src + i + 32));
            const __m128i d = _mm_loadu_si128(reinterpret_cast<const __m128i *>(src + i + 48));
            _mm_stream_si128(reinterpret_cast<__m128i *>(dst + i), a);
            _mm_stream_si128(reinterpret_cast<__m128i *>(dst + i + 16), b);
            _mm_stream_si128(reinterpret_cast<__m128i *>(dst + i + 32), c);
            _mm_stream_si128(reinterpret_cast<__m128i *>(dst + i + 48), d);
        }
        if (i < n) std::memcpy(dst + i, src + i, n - i);
        _mm_sfence();  // streaming stores are weakly ordered: make them visible before completion is signalled
        return;
    }
#endif
    std::memcpy(dst, src, n);
}

// A pool of host threads that copies one source piece into many destinations.  run() is called
// from a CUDA host-function callback (no CUDA call is made in here): thread t copies byte range t
// of T of the piece into every destination, so its share of the source stays in its cache.
class ReplicatePool {
public:
    struct Job {
        const char *src = nullptr;
        size_t bytes = 0;
        std::vector<char *> dst;
    };
    explicit ReplicatePool(int threads)
    {
        try {
            for (int t = 0; t < threads; ++t) workers_.emplace_back([this, t, threads] { work(t, threads); });
        } catch (...) {
            shut_down();  // a thread could not be created: end the ones that were, then report
            throw;
        }
    }
    ~ReplicatePool() { shut_down(); }
    int size() const { return (int)workers_.size(); }
    void run(const Job &job)
    {
        std::unique_lock<std::mutex> lock(mutex_);
        job_ = &job;
        remaining_ = (int)workers_.size();
        ++generation_;
        wake_.notify_all();
        done_.wait(lock, [this] { return remaining_ == 0; });
        job_ = nullptr;
    }

private:
    void shut_down()
    {
        {
            std::lock_guard<std::mutex> lock(mutex_);
            stop_ = true;
        }
        wake_.notify_all();
        for (std::thread &w : workers_) w.join();
        workers_.clear();
    }
    void work(int t, int threads)
    {
        unsigned long long seen = 0;
        for (;;) {
            const Job *job;
            {
                std::unique_lock<std::mutex> lock(mutex_);
                wake_.wait(lock, [&] { return stop_ || generation_ != seen; });
                if (stop_) return;
                seen = generation_;
                job = job_;
            }
            // shares cut at 64-byte boundaries
            const size_t lines = (job->bytes + 63) / 64;
            const size_t lo = std::min(job->bytes, lines * (size_t)t / threads * 64);
            const size_t hi = std::min(job->bytes, lines * (size_t)(t + 1) / threads * 64);
            if (hi > lo)
                for (char *d : job->dst) copy_streaming(d + lo, job->src + lo, hi - lo);
            {
                std::lock_guard<std::mutex> lock(mutex_);
                if (--remaining_ == 0) done_.notify_all();
            }
        }
    }
    std::vector<std::thread> workers_;
    std::mutex mutex_;
    std::condition_variable wake_, done_;
    const Job *job_ = nullptr;
    unsigned long long generation_ = 0;
    int remaining_ = 0;
    bool stop_ = false;
};

struct ReplicateCall {
    ReplicatePool *pool;
    ReplicatePool::Job job;
};

void CUDART_CB replicate_callback(void *data)
{
    ReplicateCall *call = static_cast<ReplicateCall *>(data);
    call->pool->run(call->job);
}

// One streamed unit: elements [a, b) of one module.
struct HostUnit {
    int module;
    int64_t a, b;
};

struct HostMode {
    float *theta_d = nullptr, *momentum_d = nullptr;  // full module state on the device
    float *second_d = nullptr;                        // second moment (Adam family), on demand
    char *stage_in[HOST_BUFFERS] = {};                // rows: staged pieces of reporting copies
    char *stage_out[HOST_BUFFERS] = {};               // rows: cast(theta') for every path of the module
    size_t stage_bytes = 0;                           // size of each of those buffers
    size_t max_pitch = 0;                             // largest pitch a 2-D copy accepts
    char *bounce[HOST_BUFFERS] = {};                  // pinned host: one unit's cast piece lands here
    ReplicatePool *pool = nullptr;                    // host threads that fan the piece out
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    cudaStream_t fan_stream = nullptr;                // carries the host-function callbacks
    cudaEvent_t fan_done[HOST_BUFFERS] = {};          // piece copied to every path: bounce reusable
    cudaEvent_t in_ready[HOST_BUFFERS] = {};     // upload of the unit in this buffer finished
    cudaEvent_t kernel_done[HOST_BUFFERS] = {};  // kernel finished: input reusable, output ready
    cudaEvent_t out_done[HOST_BUFFERS] = {};     // download finished: output buffer reusable
    cudaEvent_t main_ready = nullptr;
};

void host_mode_free_staging(HostMode *h)
{
    for (int b = 0; b < HOST_BUFFERS; ++b) {
        if (h->stage_in[b]) cudaFree(h->stage_in[b]);
        if (h->stage_out[b]) cudaFree(h->stage_out[b]);
        h->stage_in[b] = h->stage_out[b] = nullptr;
    }
    h->stage_bytes = 0;
}

void host_mode_release(dipaco_ctx *ctx)
{
    HostMode *h = ctx->host_mode;
    if (!h) return;
    if (h->in_stream) cudaStreamSynchronize(h->in_stream);
    if (h->out_stream) cudaStreamSynchronize(h->out_stream);
    if (h->fan_stream) cudaStreamSynchronize(h->fan_stream);
    delete h->pool;
    h->pool = nullptr;
    for (int b = 0; b < HOST_BUFFERS; ++b) {
        if (h->bounce[b]) cudaFreeHost(h->bounce[b]);
        if (h->fan_done[b]) cudaEventDestroy(h->fan_done[b]);
    }
    if (h->fan_stream) cudaStreamDestroy(h->fan_stream);
    if (h->theta_d) cudaFree(h->theta_d);
    if (h->momentum_d) cudaFree(h->momentum_d);
    if (h->second_d) cudaFree(h->second_d);
    host_mode_free_staging(h);
    for (int b = 0; b < HOST_BUFFERS; ++b) {
        if (h->in_ready[b]) cudaEventDestroy(h->in_ready[b]);
        if (h->kernel_done[b]) cudaEventDestroy(h->kernel_done[b]);
        if (h->out_done[b]) cudaEventDestroy(h->out_done[b]);
    }
    if (h->main_ready) cudaEventDestroy(h->main_ready);
    if (h->in_stream) cudaStreamDestroy(h->in_stream);
    if (h->out_stream) cudaStreamDestroy(h->out_stream);
    delete h;
    ctx->host_mode = nullptr;
}

int host_mode_prepare(dipaco_ctx *ctx)
{
    if (ctx->host_mode) return DIPACO_OK;
    const Grid &g = ctx->grid;
    HostMode *h = new (std::nothrow) HostMode();
    if (!h) return DIPACO_ENOMEM;
    ctx->host_mode = h;
    const size_t module_bytes = std::max<size_t>((size_t)g.module_params * sizeof(float), 16);
    if (cudaMalloc(&h->theta_d, module_bytes) != cudaSuccess ||
        cudaMalloc(&h->momentum_d, module_bytes) != cudaSuccess) {
        cudaGetLastError();
        host_mode_release(ctx);
        return DIPACO_ENOMEM;
    }
    int pitch = 0;
    bool ok = cudaDeviceGetAttribute(&pitch, cudaDevAttrMaxPitch, ctx->device) == cudaSuccess &&
              cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&h->out_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&h->fan_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&h->main_ready, cudaEventDisableTiming) == cudaSuccess;
    for (int b = 0; ok && b < HOST_BUFFERS; ++b)
        ok = cudaEventCreateWithFlags(&h->fan_done[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->in_ready[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->kernel_done[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->out_done[b], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        host_mode_release(ctx);
        return DIPACO_ECUDA;
    }
    h->max_pitch = pitch > 0 ? (size_t)pitch : 0;
    return DIPACO_OK;
}

// Staged rows of a unit: one per reporting copy on the way in; on the way out one per path of the
// module, or a single one when host threads fan it out.
size_t host_unit_rows(const dipaco_ctx *ctx, size_t id, bool fan_out)
{
    const size_t in = ctx->coeffs[id].contributors.size();
    const size_t out = fan_out ? 1 : ctx->grid.modules[id].members.size();
    return std::max<size_t>(std::max(in, out), 1);
}

// Cut the round into units of at most `cap` staged bytes each way (but at least one tile of every
// row), starting on tile boundaries; with fan-out a unit's piece also has to fit the bounce
// buffer.  Returns the bytes one staging buffer has to hold.
size_t plan_host_units(const dipaco_ctx *ctx, size_t cap, bool fan_out, std::vector<HostUnit> &units)
{
    const Grid &g = ctx->grid;
    const int es = ctx->elem_size;
    const int64_t tile = tile_elems(ctx);
    size_t need = 256;
    units.clear();
    for (size_t id = 0; id < g.modules.size(); ++id) {
        const ModuleGeom &m = g.modules[id];
        if (m.members.empty() || m.numel == 0 || !g.synced(m)) continue;
        const size_t rows = host_unit_rows(ctx, id, fan_out);
        // a tile's bytes are a multiple of the 256-byte row stride
        size_t fit = cap / (rows * (size_t)es);
        if (fan_out) fit = std::min(fit, HOST_BOUNCE_BYTES / (size_t)es);
        const int64_t slab = std::max<int64_t>(tile, (int64_t)fit / tile * tile);
        int64_t lo = 0, hi = m.numel;
        g.shard_range(m, lo, hi);
        for (int64_t a = lo; a < hi; a += slab) {
            const int64_t b = std::min(hi, a + slab);
            units.push_back(HostUnit{(int)id, a, b});
            need = std::max(need, rows * align_up((size_t)(b - a) * es, 256));
        }
    }
    return need;
}

// The allocation that contains a host pointer, through the driver's address-range query (looked
// up at run time, so the library does not link against the driver).  False for memory the driver
// does not know (pageable) or when the query is not available.
typedef int (*AddressRangeFn)(unsigned long long *base, size_t *size, unsigned long long ptr);

bool host_allocation_of(const void *p, uintptr_t &begin, uintptr_t &end)
{
    static AddressRangeFn query = []() -> AddressRangeFn {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult found;
        if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &found) != cudaSuccess ||
            found != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return reinterpret_cast<AddressRangeFn>(fn);
    }();
    if (!query) return false;
    unsigned long long base = 0;
    size_t size = 0;
    if (query(&base, &size, (unsigned long long)reinterpret_cast<uintptr_t>(p)) != 0 || size == 0) return false;
    begin = (uintptr_t)base;
    end = (uintptr_t)base + size;
    return true;
}

// Copy `width` bytes between each host pointer and the matching device row (row j at
// dev + j * dev_pitch).  Host pointers that are equally spaced inside ONE allocation (copies
// carved out of one block of pinned memory) go as one strided 2-D copy per run, all others one
// by one: a strided copy must not reach across separate allocations, even when they happen to
// lie equally spaced.
int copy_rows(bool to_device, char *dev, size_t dev_pitch, const std::vector<char *> &host, size_t width,
              size_t max_pitch, cudaStream_t stream)
{
    const size_t n = host.size();
    size_t j = 0;
    while (j < n) {
        size_t k = j + 1;
        ptrdiff_t stride = 0;
        if (k < n) {
            stride = host[k] - host[j];
            uintptr_t lo = 0, hi = 0;
            if (stride >= (ptrdiff_t)width && (size_t)stride <= max_pitch && dev_pitch <= max_pitch &&
                host_allocation_of(host[j], lo, hi))
                while (k < n && host[k] - host[k - 1] == stride &&
                       reinterpret_cast<uintptr_t>(host[k]) + width <= hi)
                    ++k;
        }
        cudaError_t err;
        if (k - j >= 2) {
            err = to_device
                      ? cudaMemcpy2DAsync(dev + j * dev_pitch, dev_pitch, host[j], (size_t)stride, width, k - j,
                                          cudaMemcpyHostToDevice, stream)
                      : cudaMemcpy2DAsync(host[j], (size_t)stride, dev + j * dev_pitch, dev_pitch, width, k - j,
                                          cudaMemcpyDeviceToHost, stream);
        } else {
            k = j + 1;
            err = to_device ? cudaMemcpyAsync(dev + j * dev_pitch, host[j], width, cudaMemcpyHostToDevice, stream)
                            : cudaMemcpyAsync(host[j], dev + j * dev_pitch, width, cudaMemcpyDeviceToHost, stream);
        }
        if (err != cudaSuccess) return DIPACO_ECUDA;
        j = k;
    }
    return DIPACO_OK;
}

int host_mode_sync(dipaco_ctx *ctx, float *theta_host, float *momentum_host,
                   void *const *path_ptrs_host, const uint8_t *reported, cudaStream_t stream)
{
    int rc = host_mode_prepare(ctx);
    if (rc != DIPACO_OK) return rc;
    HostMode *h = ctx->host_mode;
    const Grid &g = ctx->grid;
    const int es = ctx->elem_size;
    compute_all_coeffs(ctx, reported);
    // Adam family: the caller's second moment is a host array here; the kernels get a device copy
    const bool adam = ctx->optimizer == DIPACO_OPT_ADAM;
    float *second_host = ctx->second_moment;
    if (adam && !h->second_d &&
        cudaMalloc(&h->second_d, std::max<size_t>((size_t)g.module_params * sizeof(float), 16)) != cudaSuccess) {
        cudaGetLastError();
        return DIPACO_ENOMEM;
    }
    struct StagedSecondMoment {  // the kernels see the device copy for the duration of this call
        dipaco_ctx *c;
        StagedSecondMoment(dipaco_ctx *ctx_, float *p) : c(ctx_) { c->second_moment_staged = p; }
        ~StagedSecondMoment() { c->second_moment_staged = nullptr; }
    } staged(ctx, adam ? h->second_d : nullptr);

    // ---- cut the round into units; staging: input and output rows, HOST_BUFFERS of each, together
    // at most chunk_paths path copies
    const size_t bound = (size_t)g.chunk_paths * (size_t)g.params_per_path * es / (2 * HOST_BUFFERS);
    const size_t cap = std::max<size_t>(std::min(bound, (size_t)ctx->host_unit_bytes), 256);
    const bool fan_out = ctx->host_threads > 0;
    std::vector<HostUnit> units;
    const size_t need = plan_host_units(ctx, cap, fan_out, units);
    if (units.empty()) return DIPACO_OK;
    if (fan_out) {
        if (h->pool && h->pool->size() != ctx->host_threads) {
            if (cudaStreamSynchronize(h->fan_stream) != cudaSuccess) return DIPACO_ECUDA;
            delete h->pool;
            h->pool = nullptr;
        }
        if (!h->pool) h->pool = new ReplicatePool(ctx->host_threads);
        for (int b = 0; b < HOST_BUFFERS; ++b)
            if (!h->bounce[b] && cudaMallocHost(&h->bounce[b], HOST_BOUNCE_BYTES) != cudaSuccess) {
                cudaGetLastError();
                h->bounce[b] = nullptr;
                return DIPACO_ENOMEM;
            }
    }
    if (need > h->stage_bytes) {
        if (cudaStreamSynchronize(h->in_stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess ||
            cudaStreamSynchronize(h->out_stream) != cudaSuccess)
            return DIPACO_ECUDA;
        host_mode_free_staging(h);
        const size_t bytes = align_up(need, 4096);
        for (int b = 0; b < HOST_BUFFERS; ++b)
            if (cudaMalloc(&h->stage_in[b], bytes) != cudaSuccess || cudaMalloc(&h->stage_out[b], bytes) != cudaSuccess) {
                cudaGetLastError();
                host_mode_free_staging(h);
                return DIPACO_ENOMEM;
            }
        h->stage_bytes = bytes;
    }

    // Whatever way this function is left from here on, no copy may still be running into (or out
    // of) the caller's host buffers: the call is synchronous, and after an error the caller is
    // free to release them at once.
    std::vector<ReplicateCall> fan_calls(units.size());  // outlive the callbacks: declared before the drain
    struct DrainOnExit {
        HostMode *h;
        cudaStream_t main;
        ~DrainOnExit()
        {
            cudaStreamSynchronize(h->in_stream);
            cudaStreamSynchronize(main);
            cudaStreamSynchronize(h->out_stream);
            cudaStreamSynchronize(h->fan_stream);
        }
    } drain{h, stream};

    // ---- the tables of every unit's kernel, packed and uploaded once.  A staged row stands in
    // for a path copy through a virtual base pointer: base + (path_off + k) * es lands on the row
    // for k in [a, b).
    std::vector<LaunchRequest> reqs(units.size());
    std::vector<std::vector<void *>> row_of_path(units.size());
    for (size_t u = 0; u < units.size(); ++u) {
        const size_t id = (size_t)units[u].module;
        const ModuleGeom &m = g.modules[id];
        const ModuleCoeffs &mc = ctx->coeffs[id];
        const int64_t a = units[u].a, b = units[u].b;
        const int buf = (int)(u % HOST_BUFFERS);
        const size_t pitch = align_up((size_t)(b - a) * es, 256);
        std::vector<void *> &by_path = row_of_path[u];
        by_path.assign((size_t)g.P, nullptr);
        for (size_t j = 0; j < mc.contributors.size(); ++j)
            by_path[(size_t)mc.contributors[j]] = reinterpret_cast<void *>(
                reinterpret_cast<uintptr_t>(h->stage_in[buf] + j * pitch) - (uintptr_t)(m.path_off + a) * es);
        PassSpec sp;
        sp.module = (int)id;
        sp.flags = mc.update ? PASS_UPDATE : 0;
        sp.second_moment = mc.update && g.second_moment;
        sp.scale = g.scale_of(id);
        sp.contributors = mc.contributors;
        sp.coeff = mc.coeff;
        sp.begin = a;
        sp.end = b;
        reqs[u].specs.push_back(std::move(sp));
        std::vector<void *> rows(fan_out ? 1 : m.members.size());
        for (size_t j = 0; j < rows.size(); ++j)
            rows[j] = reinterpret_cast<void *>(reinterpret_cast<uintptr_t>(h->stage_out[buf] + j * pitch) -
                                               (uintptr_t)a * es);
        reqs[u].extra_dst.push_back(std::move(rows));
        reqs[u].lookup = PtrLookup{by_path.data(), 0, g.P};
    }
    std::vector<unsigned char> blob;
    std::vector<PackedLaunch> packed(units.size());
    for (size_t u = 0; u < units.size(); ++u) {
        rc = pack_launch(ctx, reqs[u].specs, reqs[u].lookup, &reqs[u].extra_dst, h->theta_d, h->momentum_d,
                         blob, packed[u]);
        if (rc != DIPACO_OK) return rc;
    }
    rc = upload_blob(ctx, blob, stream);
    if (rc != DIPACO_OK) return rc;

    // the side streams must not run ahead of work queued earlier on the caller's stream
    if (cudaEventRecord(h->main_ready, stream) != cudaSuccess ||
        cudaStreamWaitEvent(h->in_stream, h->main_ready, 0) != cudaSuccess ||
        cudaStreamWaitEvent(h->out_stream, h->main_ready, 0) != cudaSuccess ||
        cudaStreamWaitEvent(h->fan_stream, h->main_ready, 0) != cudaSuccess)
        return DIPACO_ECUDA;

    std::vector<char *> host_rows;
    for (size_t u = 0; u < units.size(); ++u) {
        const size_t id = (size_t)units[u].module;
        const ModuleGeom &m = g.modules[id];
        const ModuleCoeffs &mc = ctx->coeffs[id];
        const int64_t a = units[u].a, b = units[u].b;
        const int buf = (int)(u % HOST_BUFFERS);
        const size_t piece = (size_t)(b - a) * es;
        const size_t pitch = align_up(piece, 256);
        const size_t fbytes = (size_t)(b - a) * sizeof(float);
        const size_t slot_off = (size_t)(m.path_off + a) * es;

        // ---- upload (in_stream): wait until the kernel that last read this input buffer is done
        if (u >= HOST_BUFFERS && cudaStreamWaitEvent(h->in_stream, h->kernel_done[buf], 0) != cudaSuccess)
            return DIPACO_ECUDA;
        if (cudaMemcpyAsync(h->theta_d + m.theta_off + a, theta_host + m.theta_off + a, fbytes,
                            cudaMemcpyHostToDevice, h->in_stream) != cudaSuccess)
            return DIPACO_ECUDA;
        if (mc.update &&
            cudaMemcpyAsync(h->momentum_d + m.theta_off + a, momentum_host + m.theta_off + a, fbytes,
                            cudaMemcpyHostToDevice, h->in_stream) != cudaSuccess)
            return DIPACO_ECUDA;
        if (mc.update && adam &&
            cudaMemcpyAsync(h->second_d + m.theta_off + a, second_host + m.theta_off + a, fbytes,
                            cudaMemcpyHostToDevice, h->in_stream) != cudaSuccess)
            return DIPACO_ECUDA;
        host_rows.clear();
        for (int i : mc.contributors) host_rows.push_back(static_cast<char *>(path_ptrs_host[i]) + slot_off);
        rc = copy_rows(true, h->stage_in[buf], pitch, host_rows, piece, h->max_pitch, h->in_stream);
        if (rc != DIPACO_OK) return rc;
        if (cudaEventRecord(h->in_ready[buf], h->in_stream) != cudaSuccess ||
            cudaStreamWaitEvent(stream, h->in_ready[buf], 0) != cudaSuccess)
            return DIPACO_ECUDA;

        // ---- kernel (caller's stream): the output buffer must have been downloaded
        if (u >= HOST_BUFFERS && cudaStreamWaitEvent(stream, h->out_done[buf], 0) != cudaSuccess)
            return DIPACO_ECUDA;
        rc = launch_packed(ctx, packed[u], h->theta_d, h->momentum_d,
                           ctx->counters + 2 * (int)(u % MAX_COUNTERS), stream);
        if (rc != DIPACO_OK) return rc;
        ctx->last_stream = stream;
        if (cudaEventRecord(h->kernel_done[buf], stream) != cudaSuccess ||
            cudaStreamWaitEvent(h->out_stream, h->kernel_done[buf], 0) != cudaSuccess)
            return DIPACO_ECUDA;

        // ---- download (out_stream)
        if (mc.update) {
            if (cudaMemcpyAsync(theta_host + m.theta_off + a, h->theta_d + m.theta_off + a, fbytes,
                                cudaMemcpyDeviceToHost, h->out_stream) != cudaSuccess ||
                cudaMemcpyAsync(momentum_host + m.theta_off + a, h->momentum_d + m.theta_off + a,
                                fbytes, cudaMemcpyDeviceToHost, h->out_stream) != cudaSuccess)
                return DIPACO_ECUDA;
            if (adam &&
                cudaMemcpyAsync(second_host + m.theta_off + a, h->second_d + m.theta_off + a, fbytes,
                                cudaMemcpyDeviceToHost, h->out_stream) != cudaSuccess)
                return DIPACO_ECUDA;
        }
        host_rows.clear();
        for (int i : m.members) host_rows.push_back(static_cast<char *>(path_ptrs_host[i]) + slot_off);
        if (!fan_out || host_rows.size() == 1) {
            // one output row per path (or the only path's row) straight into place
            rc = copy_rows(false, h->stage_out[buf], pitch, host_rows, piece, h->max_pitch, h->out_stream);
            if (rc != DIPACO_OK) return rc;
            if (cudaEventRecord(h->out_done[buf], h->out_stream) != cudaSuccess) return DIPACO_ECUDA;
        } else {
            // the single output row lands in the bounce buffer (once the fan-out that last used it
            // is done) and host threads copy it into every path's slot
            if (u >= HOST_BUFFERS && cudaStreamWaitEvent(h->out_stream, h->fan_done[buf], 0) != cudaSuccess)
                return DIPACO_ECUDA;
            if (cudaMemcpyAsync(h->bounce[buf], h->stage_out[buf], piece, cudaMemcpyDeviceToHost,
                                h->out_stream) != cudaSuccess ||
                cudaEventRecord(h->out_done[buf], h->out_stream) != cudaSuccess ||
                cudaStreamWaitEvent(h->fan_stream, h->out_done[buf], 0) != cudaSuccess)
                return DIPACO_ECUDA;
            ReplicateCall &call = fan_calls[u];
            call.pool = h->pool;
            call.job.src = h->bounce[buf];
            call.job.bytes = piece;
            call.job.dst = host_rows;
            if (cudaLaunchHostFunc(h->fan_stream, replicate_callback, &call) != cudaSuccess) return DIPACO_ECUDA;
        }
        if (fan_out && cudaEventRecord(h->fan_done[buf], h->fan_stream) != cudaSuccess) return DIPACO_ECUDA;
    }
    if (cudaStreamSynchronize(h->in_stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess ||
        cudaStreamSynchronize(h->out_stream) != cudaSuccess ||
        cudaStreamSynchronize(h->fan_stream) != cudaSuccess)
        return DIPACO_ECUDA;
    return DIPACO_OK;
}

} // namespace
