// dipaco_module_sync_static: the chunked synchronisation of one module with its partial-sum
// scratch in a static device array, for callers that must not allocate (see include/dipaco.h).
// The static array, its one-time address look-up and the kernels that use it live in this file.
#include "../../include/dipaco.h"

#include <cmath>

#include "kernels.cuh"

using namespace dipaco;

namespace {

constexpr int STATIC_MAX_CHUNK = 32;   // path pointers carried in the kernel arguments

// Partial sums between chunks.  Every GPU on which this module has been loaded (at the latest by
// the first call of the entry point there) holds these 16 MiB until the process exits.
static __device__ __align__(256) float g_static_partial[DIPACO_STATIC_MAX_NUMEL];

struct StaticAccumulateArgs {
    float *theta;
    float *momentum;
    float *partial;
    long long numel;
    const void *src[STATIC_MAX_CHUNK];
    float coeff[STATIC_MAX_CHUNK];
    int count;
    int flags;  // KPASS_*
    float lr, mu;
};

struct StaticWritebackArgs {
    const float *theta;
    long long numel;
    void *dst[STATIC_MAX_CHUNK];
    int count;
};

// One element per thread, any alignment; the same arithmetic (sync_accumulate, sync_update) and
// the same order as the context-based kernels.
template <typename PathT>
__global__ void __launch_bounds__(256) static_accumulate_kernel(StaticAccumulateArgs a)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < a.numel; k += stride) {
        const float th = a.theta[k];
        float acc = (a.flags & KPASS_PARTIAL_IN) ? a.partial[k] : 0.0f;
        for (int j = 0; j < a.count; ++j)
            acc = sync_accumulate(acc, a.coeff[j], th,
                                  PathIO<PathT>::load(static_cast<const PathT *>(a.src[j]) + k), 0);
        if (a.flags & KPASS_PARTIAL_OUT) a.partial[k] = acc;
        if (a.flags & KPASS_UPDATE) {
            float t1, m1, unused = 0.0f;
            UpdateRule rule = {};
            rule.lr = a.lr;
            rule.mu = a.mu;
            rule.optimizer = KOPT_NESTEROV;
            sync_update(th, a.momentum[k], unused, acc, 1.0f, rule, t1, m1);
            a.theta[k] = t1;
            a.momentum[k] = m1;
        }
    }
}

template <typename PathT>
__global__ void __launch_bounds__(256) static_writeback_kernel(StaticWritebackArgs a)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < a.numel; k += stride) {
        const float v = a.theta[k];
        for (int j = 0; j < a.count; ++j) PathIO<PathT>::store(static_cast<PathT *>(a.dst[j]) + k, v);
    }
}

// With that device current: the device address of the static array.  In host code the array's
// name is only a handle for this look-up, never a pointer a kernel may use.  The look-up is
// repeated on every call (it is cheap and allocates nothing once the module is loaded), so a
// primary context that the application destroyed and re-created is followed.  The very first
// look-up on a device makes the CUDA runtime load this file's module there, which is when the
// array's 16 MiB are reserved: that can fail on a device whose memory is already exhausted.
int static_setup(int device, float **partial, int *sm_count)
{
    void *addr = nullptr;
    const cudaError_t err = cudaGetSymbolAddress(&addr, g_static_partial);
    if (err != cudaSuccess || !addr) {
        cudaGetLastError();  // leave no sticky error behind for the caller's next runtime call
        return err == cudaErrorMemoryAllocation ? DIPACO_ENOMEM : DIPACO_ECUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) {
        cudaGetLastError();
        return DIPACO_ECUDA;
    }
    *partial = static_cast<float *>(addr);
    *sm_count = sms;
    return DIPACO_OK;
}

struct CurrentDevice {
    int prev = -1;
    bool ok = true;
    explicit CurrentDevice(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~CurrentDevice()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

bool path_reports(const uint8_t *reported, int i) { return !reported || reported[i]; }
double path_weight(const float *weights, int i) { return weights ? (double)weights[i] : 1.0; }

} // namespace

extern "C" int dipaco_module_sync_static(float *theta, float *momentum, int64_t numel,
                                         int32_t num_paths, void *const *copy_ptrs,
                                         const float *path_weights, const uint8_t *reported,
                                         float outer_lr, float outer_momentum, int32_t path_dtype,
                                         int32_t chunk_paths, int32_t device, void *cuda_stream)
{
    if (!theta || !momentum || !copy_ptrs || num_paths < 1 || numel < 0) return DIPACO_EINVAL;
    if (path_dtype != DIPACO_F32 && path_dtype != DIPACO_BF16) return DIPACO_EINVAL;
    if (chunk_paths < 1 || chunk_paths > STATIC_MAX_CHUNK) return DIPACO_EINVAL;
    if (device < 0) return DIPACO_EINVAL;
    if (!std::isfinite(outer_lr) || !std::isfinite(outer_momentum)) return DIPACO_EINVAL;
    if (numel > (int64_t)DIPACO_STATIC_MAX_NUMEL) return DIPACO_ELIMIT;
    for (int i = 0; i < num_paths; ++i) {
        if (!copy_ptrs[i]) return DIPACO_EINVAL;
        if (path_weights && (!(path_weights[i] >= 0.0f) || !std::isfinite(path_weights[i])))
            return DIPACO_EINVAL;
    }
    if (numel == 0) return DIPACO_OK;

    CurrentDevice guard(device);
    if (!guard.ok) return DIPACO_ECUDA;
    float *partial = nullptr;
    int sm_count = 0;
    const int rc = static_setup(device, &partial, &sm_count);
    if (rc != DIPACO_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // total weight of the reporting copies and the chunks that hold the first / last of them
    double total = 0.0;
    int first_rep = -1, last_rep = -1;
    for (int i = 0; i < num_paths; ++i)
        if (path_reports(reported, i)) {
            total += path_weight(path_weights, i);
            if (first_rep < 0) first_rep = i;
            last_rep = i;
        }
    const bool update = first_rep >= 0 && total > 0.0;
    const int num_chunks = (num_paths + chunk_paths - 1) / chunk_paths;
    const long long blocks_needed = (numel + 255) / 256;
    const int grid = (int)(blocks_needed < (long long)sm_count * 8 ? blocks_needed : (long long)sm_count * 8);

    if (update) {
        const int first_chunk = first_rep / chunk_paths, last_chunk = last_rep / chunk_paths;
        for (int c = first_chunk; c <= last_chunk; ++c) {
            StaticAccumulateArgs a;
            a.theta = theta;
            a.momentum = momentum;
            a.partial = partial;
            a.numel = numel;
            a.count = 0;
            a.lr = outer_lr;
            a.mu = outer_momentum;
            const int stop = (c + 1) * chunk_paths < num_paths ? (c + 1) * chunk_paths : num_paths;
            for (int i = c * chunk_paths; i < stop; ++i)
                if (path_reports(reported, i)) {
                    a.src[a.count] = copy_ptrs[i];
                    a.coeff[a.count] = (float)(path_weight(path_weights, i) / total);
                    ++a.count;
                }
            if (a.count == 0) continue;
            // the first chunk starts from zero, so the array's old contents are never read
            a.flags = (c > first_chunk ? KPASS_PARTIAL_IN : 0) |
                      (c == last_chunk ? KPASS_UPDATE : KPASS_PARTIAL_OUT);
            if (path_dtype == DIPACO_BF16)
                static_accumulate_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(a);
            else
                static_accumulate_kernel<float><<<grid, 256, 0, stream>>>(a);
            if (cudaGetLastError() != cudaSuccess) return DIPACO_ECUDA;
        }
    }
    for (int c = 0; c < num_chunks; ++c) {
        StaticWritebackArgs w;
        w.theta = theta;
        w.numel = numel;
        w.count = 0;
        const int stop = (c + 1) * chunk_paths < num_paths ? (c + 1) * chunk_paths : num_paths;
        for (int i = c * chunk_paths; i < stop; ++i) w.dst[w.count++] = copy_ptrs[i];
        if (path_dtype == DIPACO_BF16)
            static_writeback_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(w);
        else
            static_writeback_kernel<float><<<grid, 256, 0, stream>>>(w);
        if (cudaGetLastError() != cudaSuccess) return DIPACO_ECUDA;
    }
    return DIPACO_OK;
}
