// dipaco_outer_sync_host: the synchronisation for state kept in host memory.
// Included by dipaco.cu (inside its translation unit, after the launch helpers).
//
// Reporting path copies are streamed host -> device in chunks of chunk_paths through two device
// buffers (the copy of chunk c+1 overlaps the kernel of chunk c).  The chunk kernels only read
// the copies; as soon as a module's last reporting path has been accumulated the module is
// updated, its value is cast once into a device array shaped like theta (bf16 paths only) and
// copied device -> host into the slot of every path through the module, while later chunks are
// still being uploaded.  Paths that did not report are never uploaded.

namespace {

struct HostMode {
    float *theta_d = nullptr, *momentum_d = nullptr;
    void *chunk_buf[2] = {nullptr, nullptr};
    void *cast_d = nullptr;  // module values in the path dtype (bf16 paths only)
    cudaStream_t copy_stream = nullptr, d2h_stream = nullptr;
    cudaEvent_t h2d_done[2] = {nullptr, nullptr};
    cudaEvent_t buf_free[2] = {nullptr, nullptr};
    cudaEvent_t main_ready = nullptr;
    std::vector<cudaEvent_t> finalised;  // one per chunk + one for the modules nobody reported to
};

void host_mode_release(dipaco_ctx *ctx)
{
    HostMode *h = ctx->host_mode;
    if (!h) return;
    if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
    if (h->d2h_stream) cudaStreamSynchronize(h->d2h_stream);
    if (h->theta_d) cudaFree(h->theta_d);
    if (h->momentum_d) cudaFree(h->momentum_d);
    for (int b = 0; b < 2; ++b) {
        if (h->chunk_buf[b]) cudaFree(h->chunk_buf[b]);
        if (h->h2d_done[b]) cudaEventDestroy(h->h2d_done[b]);
        if (h->buf_free[b]) cudaEventDestroy(h->buf_free[b]);
    }
    if (h->cast_d) cudaFree(h->cast_d);
    if (h->main_ready) cudaEventDestroy(h->main_ready);
    for (cudaEvent_t e : h->finalised)
        if (e) cudaEventDestroy(e);
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    if (h->d2h_stream) cudaStreamDestroy(h->d2h_stream);
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
    const size_t path_bytes = align_up((size_t)g.params_per_path * ctx->elem_size, 256);
    const size_t chunk_bytes = std::max<size_t>(path_bytes * (size_t)g.chunk_paths, 16);
    bool ok = cudaMalloc(&h->theta_d, module_bytes) == cudaSuccess &&
              cudaMalloc(&h->momentum_d, module_bytes) == cudaSuccess &&
              cudaMalloc(&h->chunk_buf[0], chunk_bytes) == cudaSuccess &&
              cudaMalloc(&h->chunk_buf[1], chunk_bytes) == cudaSuccess;
    if (ok && ctx->elem_size != 4)
        ok = cudaMalloc(&h->cast_d, std::max<size_t>((size_t)g.module_params * ctx->elem_size, 16)) ==
             cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        host_mode_release(ctx);
        return DIPACO_ENOMEM;
    }
    ok = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) == cudaSuccess &&
         cudaStreamCreateWithFlags(&h->d2h_stream, cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->main_ready, cudaEventDisableTiming) == cudaSuccess;
    for (int b = 0; ok && b < 2; ++b)
        ok = cudaEventCreateWithFlags(&h->h2d_done[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->buf_free[b], cudaEventDisableTiming) == cudaSuccess;
    h->finalised.assign((size_t)g.num_chunks + 1, nullptr);
    for (size_t i = 0; ok && i < h->finalised.size(); ++i)
        ok = cudaEventCreateWithFlags(&h->finalised[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        host_mode_release(ctx);
        return DIPACO_ECUDA;
    }
    return DIPACO_OK;
}

// Cast the given modules' current theta into cast_d (bf16 paths) on `stream`, then copy the new
// value of each module to the host: theta', m' (if updated) and the slot of every member path.
int host_mode_emit(dipaco_ctx *ctx, const std::vector<int> &module_ids, bool updated,
                   float *theta_host, float *momentum_host, void *const *path_ptrs_host,
                   cudaStream_t stream, cudaEvent_t done_event)
{
    HostMode *h = ctx->host_mode;
    const Grid &g = ctx->grid;
    const int es = ctx->elem_size;
    if (module_ids.empty()) return DIPACO_OK;
    if (h->cast_d) {
        std::vector<LaunchRequest> reqs(1);
        for (int id : module_ids) {
            PassSpec sp;
            sp.module = id;
            sp.flags = 0;
            reqs[0].specs.push_back(sp);
            reqs[0].extra_dst.push_back(
                {static_cast<char *>(h->cast_d) + (size_t)g.modules[id].theta_off * es});
        }
        reqs[0].lookup = PtrLookup{nullptr, 0, 0};
        const int rc = run_launches(ctx, reqs, h->theta_d, h->momentum_d, stream);
        if (rc != DIPACO_OK) return rc;
    }
    if (cudaEventRecord(done_event, stream) != cudaSuccess) return DIPACO_ECUDA;
    if (cudaStreamWaitEvent(h->d2h_stream, done_event, 0) != cudaSuccess) return DIPACO_ECUDA;
    for (int id : module_ids) {
        const ModuleGeom &m = g.modules[id];
        const size_t fbytes = (size_t)m.numel * sizeof(float);
        if (updated) {
            if (cudaMemcpyAsync(theta_host + m.theta_off, h->theta_d + m.theta_off, fbytes,
                                cudaMemcpyDeviceToHost, h->d2h_stream) != cudaSuccess ||
                cudaMemcpyAsync(momentum_host + m.theta_off, h->momentum_d + m.theta_off, fbytes,
                                cudaMemcpyDeviceToHost, h->d2h_stream) != cudaSuccess)
                return DIPACO_ECUDA;
        }
        const char *src = h->cast_d ? static_cast<const char *>(h->cast_d) + (size_t)m.theta_off * es
                                    : reinterpret_cast<const char *>(h->theta_d + m.theta_off);
        for (int i : m.members) {
            char *dst = static_cast<char *>(path_ptrs_host[i]) + (size_t)m.path_off * es;
            if (cudaMemcpyAsync(dst, src, (size_t)m.numel * es, cudaMemcpyDeviceToHost,
                                h->d2h_stream) != cudaSuccess)
                return DIPACO_ECUDA;
        }
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
    const size_t module_bytes = (size_t)g.module_params * sizeof(float);
    const size_t path_bytes = (size_t)g.params_per_path * es;
    const size_t path_stride = align_up(path_bytes, 256);
    compute_all_coeffs(ctx, reported);

    if (module_bytes > 0 &&
        (cudaMemcpyAsync(h->theta_d, theta_host, module_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
         cudaMemcpyAsync(h->momentum_d, momentum_host, module_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess))
        return DIPACO_ECUDA;
    // the side streams must not run ahead of work queued earlier on the caller's stream
    if (cudaEventRecord(h->main_ready, stream) != cudaSuccess ||
        cudaStreamWaitEvent(h->copy_stream, h->main_ready, 0) != cudaSuccess ||
        cudaStreamWaitEvent(h->d2h_stream, h->main_ready, 0) != cudaSuccess)
        return DIPACO_ECUDA;

    std::vector<void *> chunk_ptrs((size_t)g.chunk_paths);
    for (int c = 0; c < g.num_chunks; ++c) {
        const int b = c & 1;
        const int first = chunk_first(g, c), n = chunk_count(g, c);
        if (c >= 2 && cudaStreamWaitEvent(h->copy_stream, h->buf_free[b], 0) != cudaSuccess)
            return DIPACO_ECUDA;
        for (int j = 0; j < n; ++j) {
            chunk_ptrs[(size_t)j] = static_cast<char *>(h->chunk_buf[b]) + (size_t)j * path_stride;
            const int i = first + j;
            if (reported && !reported[i]) continue;
            if (path_bytes > 0 &&
                cudaMemcpyAsync(chunk_ptrs[(size_t)j], path_ptrs_host[i], path_bytes,
                                cudaMemcpyHostToDevice, h->copy_stream) != cudaSuccess)
                return DIPACO_ECUDA;
        }
        if (cudaEventRecord(h->h2d_done[b], h->copy_stream) != cudaSuccess ||
            cudaStreamWaitEvent(stream, h->h2d_done[b], 0) != cudaSuccess)
            return DIPACO_ECUDA;

        std::vector<LaunchRequest> reqs(1);
        plan_accumulate(g, ctx->coeffs, c, reqs[0].specs);
        std::vector<int> done_here;
        for (PassSpec &sp : reqs[0].specs) {
            sp.members.clear();  // results leave through the cast array, not the chunk buffers
            if (sp.flags & PASS_UPDATE) done_here.push_back(sp.module);
        }
        reqs[0].lookup = PtrLookup{chunk_ptrs.data(), first, n};
        if (!reqs[0].specs.empty()) {
            rc = run_launches(ctx, reqs, h->theta_d, h->momentum_d, stream);
            if (rc != DIPACO_OK) return rc;
        }
        if (cudaEventRecord(h->buf_free[b], stream) != cudaSuccess) return DIPACO_ECUDA;
        rc = host_mode_emit(ctx, done_here, true, theta_host, momentum_host, path_ptrs_host, stream,
                            h->finalised[(size_t)c]);
        if (rc != DIPACO_OK) return rc;
    }
    // modules nobody reported to: theta and m stay, their copies are reset to cast(theta)
    std::vector<int> untouched;
    for (size_t id = 0; id < g.modules.size(); ++id)
        if (!ctx->coeffs[id].update && !g.modules[id].members.empty() && g.modules[id].numel > 0)
            untouched.push_back((int)id);
    rc = host_mode_emit(ctx, untouched, false, theta_host, momentum_host, path_ptrs_host, stream,
                        h->finalised[(size_t)g.num_chunks]);
    if (rc != DIPACO_OK) return rc;

    if (cudaStreamSynchronize(h->copy_stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess ||
        cudaStreamSynchronize(h->d2h_stream) != cudaSuccess)
        return DIPACO_ECUDA;
    return DIPACO_OK;
}

} // namespace
