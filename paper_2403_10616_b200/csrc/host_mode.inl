// dipaco_outer_sync_host: the synchronisation for state kept in host memory.
// Included by dipaco.cu (inside its translation unit, after the launch helpers).
//
// Slab-ordered streaming.  The work is cut into units: an element range [a, b) of one module
// together with that range of EVERY reporting copy of the module.  A unit is therefore complete
// in itself: one fused pass (reduce in ascending path id + Nesterov + cast) finishes it, no
// partial sums are carried, and its result can leave the device at once.  Per unit:
//     H2D  theta[a:b], m[a:b] and the [a:b) piece of each reporting copy  -> staging buffer
//     kernel  the resident-mode pass on [a, b), reading the staged pieces, writing theta', m'
//             in place and cast(theta') into a small output buffer
//     D2H  theta'[a:b], m'[a:b], and the output buffer into the slot of every path of the module
// Units are double-buffered over three streams, so the upload of unit n+1, the kernel of unit n
// and the download of unit n-1 overlap; a step costs about max(H2D bytes, D2H bytes) / PCIe rate.
// The first units are small and double in size up to the steady size, and the last ones halve
// again, so that the time before the first kernel (nothing overlaps the first upload) and after the
// last one (nothing overlaps the last download) stays in the millisecond range.
// The staging memory is bounded by chunk_paths path copies.  Paths that did not report are never
// uploaded.  Bitwise identical to the resident mode: same pass, same order.

namespace {

struct HostMode {
    float *theta_d = nullptr, *momentum_d = nullptr;  // full module state on the device
    float *second_d = nullptr;                        // second moment (Adam family), on demand
    char *stage_in[2] = {nullptr, nullptr};           // staged pieces of path copies
    char *stage_out[2] = {nullptr, nullptr};          // cast(theta') of the unit (bf16 paths)
    size_t stage_in_bytes = 0, stage_out_bytes = 0;
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    cudaEvent_t in_ready[2] = {nullptr, nullptr};    // upload of the unit in this buffer finished
    cudaEvent_t kernel_done[2] = {nullptr, nullptr}; // kernel finished: input reusable, output ready
    cudaEvent_t out_done[2] = {nullptr, nullptr};    // download finished: output buffer reusable
    cudaEvent_t main_ready = nullptr;
};

void host_mode_release(dipaco_ctx *ctx)
{
    HostMode *h = ctx->host_mode;
    if (!h) return;
    if (h->in_stream) cudaStreamSynchronize(h->in_stream);
    if (h->out_stream) cudaStreamSynchronize(h->out_stream);
    if (h->theta_d) cudaFree(h->theta_d);
    if (h->momentum_d) cudaFree(h->momentum_d);
    if (h->second_d) cudaFree(h->second_d);
    for (int b = 0; b < 2; ++b) {
        if (h->stage_in[b]) cudaFree(h->stage_in[b]);
        if (h->stage_out[b]) cudaFree(h->stage_out[b]);
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
    const int es = ctx->elem_size;
    const size_t module_bytes = std::max<size_t>((size_t)g.module_params * sizeof(float), 16);
    // two input buffers that together hold chunk_paths path copies
    const size_t tile_bytes = (size_t)tile_elems(ctx) * es;
    size_t in_bytes = (size_t)g.chunk_paths * (size_t)g.params_per_path * es / 2;
    size_t max_contrib = 1;
    int64_t max_numel = 1;
    for (const ModuleGeom &m : g.modules) {
        max_contrib = std::max(max_contrib, m.members.size());
        max_numel = std::max(max_numel, m.numel);
    }
    in_bytes = std::max(in_bytes, max_contrib * tile_bytes);  // at least one tile of every copy
    h->stage_in_bytes = align_up(in_bytes, 256);
    // the largest unit is bounded by a whole module and by stage_in_bytes / (1 copy)
    const size_t out_elems = std::min<size_t>((size_t)max_numel, h->stage_in_bytes / es);
    h->stage_out_bytes = align_up(std::max<size_t>(out_elems * es, 256), 256);
    bool ok = cudaMalloc(&h->theta_d, module_bytes) == cudaSuccess &&
              cudaMalloc(&h->momentum_d, module_bytes) == cudaSuccess;
    for (int b = 0; ok && b < 2; ++b) {
        ok = cudaMalloc(&h->stage_in[b], h->stage_in_bytes) == cudaSuccess;
        if (ok && es != 4) ok = cudaMalloc(&h->stage_out[b], h->stage_out_bytes) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        host_mode_release(ctx);
        return DIPACO_ENOMEM;
    }
    ok = cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking) == cudaSuccess &&
         cudaStreamCreateWithFlags(&h->out_stream, cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->main_ready, cudaEventDisableTiming) == cudaSuccess;
    for (int b = 0; ok && b < 2; ++b)
        ok = cudaEventCreateWithFlags(&h->in_ready[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->kernel_done[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->out_done[b], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        host_mode_release(ctx);
        return DIPACO_ECUDA;
    }
    return DIPACO_OK;
}

// One streamed unit: elements [a, b) of one module.
struct HostUnit {
    int module;
    int64_t a, b;
};

constexpr size_t HOST_RAMP_BASE = (size_t)16 << 20;  // bytes one direction moves in the first / last unit

// Cut the round into units.  Steady size: every reporting copy's piece fits one input buffer, the
// cast piece fits the output buffer, and the upload stays under the configured cap.  Unit k from
// the start and unit k from the end move at most HOST_RAMP_BASE * 2^k bytes in either direction.
int plan_host_units(const dipaco_ctx *ctx, const HostMode *h, std::vector<HostUnit> &units)
{
    const Grid &g = ctx->grid;
    const int es = ctx->elem_size;
    const int64_t tile = tile_elems(ctx);
    units.clear();
    auto bytes_per_elem = [&](size_t id) -> size_t {
        const size_t up = ctx->coeffs[id].contributors.size(), down = g.modules[id].members.size();
        return std::max(up, down) * (size_t)es + 2 * sizeof(float);
    };
    auto ramp_elems = [&](size_t id, size_t k) -> int64_t {
        const size_t cap = HOST_RAMP_BASE << std::min<size_t>(k, 24);
        return std::max<int64_t>(tile, (int64_t)(cap / bytes_per_elem(id)) / tile * tile);
    };
    for (size_t id = 0; id < g.modules.size(); ++id) {
        const ModuleGeom &m = g.modules[id];
        const ModuleCoeffs &mc = ctx->coeffs[id];
        if (m.members.empty() || m.numel == 0 || !g.synced(m)) continue;
        const size_t ncon = mc.contributors.size();
        const size_t in_budget = std::max<size_t>(std::min(h->stage_in_bytes, (size_t)ctx->host_unit_bytes),
                                                  ncon * (size_t)tile * es);
        int64_t slab = m.numel;
        if (ncon > 0 && ncon * align_up((size_t)m.numel * es, 256) > in_budget) {
            const int64_t fit = (int64_t)(in_budget / (ncon * (size_t)es));
            slab = fit / tile * tile;  // a tile's bytes are a multiple of the 256-byte piece stride
        }
        if ((size_t)slab * es > h->stage_out_bytes)
            slab = (int64_t)(h->stage_out_bytes / (size_t)es) / tile * tile;
        if (slab < 1) return DIPACO_ENOMEM;
        int64_t lo = 0, hi = m.numel;
        g.shard_range(m, lo, hi);
        for (int64_t a = lo; a < hi;) {
            const int64_t n = std::min(slab, ramp_elems(id, units.size()));
            const int64_t b = std::min(hi, a + n);
            units.push_back(HostUnit{(int)id, a, b});
            a = b;
        }
    }
    // the same ramp from the end: split the last units until unit k from the end fits its cap
    std::vector<HostUnit> tail;
    while (!units.empty() && tail.size() < 24) {
        HostUnit &u = units.back();
        const int64_t cap = ramp_elems((size_t)u.module, tail.size());
        if (u.b - u.a > cap) {
            const int64_t cut = (u.b - cap) / tile * tile;  // unit starts stay on tile boundaries
            if (cut > u.a) {
                tail.push_back(HostUnit{u.module, cut, u.b});
                u.b = cut;
                continue;
            }
        }
        const bool steady = (size_t)cap * bytes_per_elem((size_t)u.module) >= h->stage_in_bytes;
        tail.push_back(u);
        units.pop_back();
        if (steady) break;
    }
    units.insert(units.end(), tail.rbegin(), tail.rend());
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
    const int64_t tile = tile_elems(ctx);
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

    // Whatever way this function is left, no copy may still be running into (or out of) the
    // caller's host buffers: the call is synchronous, and after an error the caller is free to
    // release them at once.
    struct DrainOnExit {
        HostMode *h;
        cudaStream_t main;
        ~DrainOnExit()
        {
            cudaStreamSynchronize(h->in_stream);
            cudaStreamSynchronize(main);
            cudaStreamSynchronize(h->out_stream);
        }
    } drain{h, stream};

    // the side streams must not run ahead of work queued earlier on the caller's stream
    if (cudaEventRecord(h->main_ready, stream) != cudaSuccess ||
        cudaStreamWaitEvent(h->in_stream, h->main_ready, 0) != cudaSuccess ||
        cudaStreamWaitEvent(h->out_stream, h->main_ready, 0) != cudaSuccess)
        return DIPACO_ECUDA;

    std::vector<void *> by_path((size_t)g.P, nullptr);
    std::vector<HostUnit> units;
    rc = plan_host_units(ctx, h, units);
    if (rc != DIPACO_OK) return rc;
    long long unit_index = 0;
    for (const HostUnit &unit : units) {
        {
            const size_t id = (size_t)unit.module;
            const ModuleGeom &m = g.modules[id];
            const ModuleCoeffs &mc = ctx->coeffs[id];
            const size_t ncon = mc.contributors.size();
            const int64_t a = unit.a, b = unit.b;
            const int buf = (int)(unit_index & 1);
            const size_t piece = (size_t)(b - a) * es;
            const size_t piece_stride = align_up(piece, 256);
            const size_t fbytes = (size_t)(b - a) * sizeof(float);

            // ---- upload (in_stream): wait until the kernel of unit n-2 released this buffer
            if (unit_index >= 2 && cudaStreamWaitEvent(h->in_stream, h->kernel_done[buf], 0) != cudaSuccess)
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
            for (size_t j = 0; j < ncon; ++j) {
                const int i = mc.contributors[j];
                char *dst = h->stage_in[buf] + j * piece_stride;
                const char *src = static_cast<const char *>(path_ptrs_host[i]) + (size_t)(m.path_off + a) * es;
                if (cudaMemcpyAsync(dst, src, piece, cudaMemcpyHostToDevice, h->in_stream) != cudaSuccess)
                    return DIPACO_ECUDA;
                // virtual base: base + (path_off + k) * es lands on the staged piece for k in [a, b)
                by_path[(size_t)i] = reinterpret_cast<void *>(reinterpret_cast<uintptr_t>(dst) -
                                                              (uintptr_t)(m.path_off + a) * es);
            }
            if (cudaEventRecord(h->in_ready[buf], h->in_stream) != cudaSuccess ||
                cudaStreamWaitEvent(stream, h->in_ready[buf], 0) != cudaSuccess)
                return DIPACO_ECUDA;

            // ---- kernel (caller's stream): the output buffer must have been downloaded
            if (unit_index >= 2 && cudaStreamWaitEvent(stream, h->out_done[buf], 0) != cudaSuccess)
                return DIPACO_ECUDA;
            const bool need_kernel = mc.update || es != 4;
            if (need_kernel) {
                std::vector<LaunchRequest> reqs(1);
                PassSpec sp;
                sp.module = (int)id;
                sp.flags = mc.update ? PASS_UPDATE : 0;
                sp.scale = g.scale_of(id);
                sp.contributors = mc.contributors;
                sp.coeff = mc.coeff;
                sp.begin = a;
                sp.end = b;
                reqs[0].specs.push_back(std::move(sp));
                if (es != 4)
                    reqs[0].extra_dst.push_back({reinterpret_cast<void *>(
                        reinterpret_cast<uintptr_t>(h->stage_out[buf]) - (uintptr_t)a * es)});
                reqs[0].lookup = PtrLookup{by_path.data(), 0, g.P};
                rc = run_launches(ctx, reqs, h->theta_d, h->momentum_d, stream);
                if (rc != DIPACO_OK) return rc;
            }
            for (size_t j = 0; j < ncon; ++j) by_path[(size_t)mc.contributors[j]] = nullptr;
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
            const char *out_src = es != 4 ? h->stage_out[buf]
                                          : reinterpret_cast<const char *>(h->theta_d + m.theta_off + a);
            for (int i : m.members) {
                char *dst = static_cast<char *>(path_ptrs_host[i]) + (size_t)(m.path_off + a) * es;
                if (cudaMemcpyAsync(dst, out_src, piece, cudaMemcpyDeviceToHost, h->out_stream) != cudaSuccess)
                    return DIPACO_ECUDA;
            }
            if (cudaEventRecord(h->out_done[buf], h->out_stream) != cudaSuccess) return DIPACO_ECUDA;
            ++unit_index;
        }
    }
    if (cudaStreamSynchronize(h->in_stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess ||
        cudaStreamSynchronize(h->out_stream) != cudaSuccess)
        return DIPACO_ECUDA;
    return DIPACO_OK;
}

} // namespace
