// Device code of the outer synchronisation (DiPaCo, Algorithm 1, outer loop + re-dispatch).
//
// Three kernel families share one arithmetic definition (sync_accumulate, sync_update), so they
// give bitwise identical results:
//   sync_direct_kernel<PathT,1>   one element per thread, any alignment (ragged tails, odd offsets)
//   sync_direct_kernel<PathT,8>   128-bit register loads/stores on 16-byte aligned full tiles
//   sync_direct_kernel<PathT,8,true>  the same for path buffers at any element alignment, each
//                                 with its own: 128-bit accesses to the aligned units around the
//                                 data, funnel shifts, and a warp shuffle to realign the stores
//   sync_bulk_kernel<PathT,NU>    persistent, warp-specialised: a scheduler warp draws work items
//                                 from a counter, one warp streams tiles into a shared-memory
//                                 ring with bulk async copies (TMA, 1-D), eight warps reduce and
//                                 apply the optimiser step, one warp scatters the result tile to
//                                 every path with bulk stores from shared memory.
//   sync_bulk_kernel<PathT,NU,true>  the same for path buffers at any element alignment: tiles
//                                 loaded from the aligned address at or before them and cut out
//                                 of neighbouring 16-byte units; shifted destinations written in
//                                 realigned units by four store warps.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dipaco {

enum : int {
    KPASS_UPDATE = 1,
    KPASS_PARTIAL_IN = 2,
    KPASS_PARTIAL_OUT = 4,
    KPASS_CAST_IN = 8,  // write-back only pass: cast(theta') is read from the cast scratch (path
                        // dtype) instead of being derived from fp32 theta'
};

struct PassDev {
    long long theta_off;    // elements into theta / momentum
    long long partial_off;  // elements into the partial-sum scratch (valid with PARTIAL flags)
    long long cast_off;     // elements into the cast scratch (valid with KPASS_CAST_IN)
    int contrib_begin, contrib_count;
    int member_begin, member_count;
    int aligned_members;  // bulk-copy kernel: the first so many members are 16-byte aligned at the
                          // pass's tiles (the host puts them first), the others sit inside a unit
    int flags;
    // dynamic scheduling of the bulk-copy kernel: this pass owns work items
    // [item_first, item_first + ceil(bulk_tiles / tiles_per_item)), each a run of full tiles
    int item_first;
    int tiles_per_item;
    float scale;  // factor on the finished outer gradient (Section 2.7, norm rescaling); 1 = none
    long long bulk_tiles;
    long long bulk_begin;  // element range [bulk_begin, bulk_end) of the module that the bulk-copy
    long long bulk_end;    // kernel covers: whole 16-byte units of path data; the last tile of the
                           // pass may be partial
};

struct ContribDev {
    const void *src;  // start of the module's slot inside the contributor's path copy
    float coeff;      // c_i = w_i / W
    int pad;
};

struct SegmentDev {
    int pass, pad;
    long long begin, end;  // element range inside the module
};

enum : int { KOPT_NESTEROV = 0, KOPT_MOMENTUM = 1, KOPT_SGD = 2, KOPT_ADAM = 3 };

struct UpdateRule {
    float lr, mu;
    int optimizer;  // KOPT_*
    // Adam family (constants rounded once from double on the host)
    float b1, one_minus_b1, b2, one_minus_b2;
    float eps;
    float decay;    // 1 - lr * weight_decay
    float inv_c1, inv_c2;  // reciprocals of the bias corrections 1 - b^t, or 1
};

struct LaunchParams {
    float *theta;
    float *momentum;
    float *partial;
    const void *cast_scratch;  // cast(theta') of finished modules in the path dtype (chunk API)
    const PassDev *passes;
    const ContribDev *contribs;
    void *const *members;  // start of the module's slot inside each member path copy
    const SegmentDev *segs;
    const int *cta_first;  // [gridDim.x + 1]
    UpdateRule rule;       // outer optimiser and its constants
    float *second_moment;  // Adam family only: v, same layout as theta
    int input_kind;        // 0: path buffers hold copies of the modules, 1: they hold gradients
    int v_index;           // bulk-copy kernel: which fp32 tile of a buffer carries v
    int *error_word;
    // bulk-copy kernel only
    int num_passes;
    int total_items;
    int *work_counter;  // [0]: next work item, [1]: CTAs that finished drawing; both zero before the
                        // launch, and reset to zero by the last CTA so the next launch can reuse them
};

// ------------------------------------------------------------------------------------------
// The arithmetic, written once (sync_accumulate, sync_update).  Explicit intrinsics: no contraction
// or reassociation choices are left to the compiler, so every kernel family rounds identically.

__device__ __forceinline__ float sync_accumulate(float acc, float c, float theta, float x, int input_kind)
{
    // acc + c * (theta - x): one term of the outer gradient (Algorithm 1, outer-gradient line);
    // acc + c * x when the buffers hold gradients (Section 4.5, module-wise gradient aggregation)
    const float d = input_kind ? x : __fsub_rn(theta, x);
    return __fmaf_rn(c, d, acc);
}

__device__ __forceinline__ void sync_update(float theta, float m, float &v, float sum, float scale,
                                            const UpdateRule &r, float &theta_new, float &m_new)
{
    // Delta = scale * sum, then the outer optimiser step:
    //   Nesterov   m' = mu*m + Delta ; theta' = theta - lr*(Delta + mu*m')
    //   heavy ball m' = mu*m + Delta ; theta' = theta - lr*m'
    //   SGD        m' = m            ; theta' = theta - lr*Delta
    //   Adam       m' = b1*m + (1-b1)*Delta ; v' = b2*v + (1-b2)*Delta^2
    //              theta' = theta*decay - lr * (m'*inv_c1) / (sqrt(v'*inv_c2) + eps)
    const float delta = __fmul_rn(scale, sum);  // exact when scale == 1
    if (r.optimizer == KOPT_ADAM) {
        m_new = __fmaf_rn(r.b1, m, __fmul_rn(r.one_minus_b1, delta));
        v = __fmaf_rn(r.b2, v, __fmul_rn(r.one_minus_b2, __fmul_rn(delta, delta)));
        const float denom = __fadd_rn(__fsqrt_rn(__fmul_rn(v, r.inv_c2)), r.eps);
        const float step = __fdiv_rn(__fmul_rn(m_new, r.inv_c1), denom);
        theta_new = __fmaf_rn(-r.lr, step, __fmul_rn(theta, r.decay));
        return;
    }
    if (r.optimizer == KOPT_SGD) {
        m_new = m;
        theta_new = __fmaf_rn(-r.lr, delta, theta);
        return;
    }
    m_new = __fmaf_rn(r.mu, m, delta);
    const float g = r.optimizer == KOPT_NESTEROV ? __fmaf_rn(r.mu, m_new, delta) : m_new;
    theta_new = __fmaf_rn(-r.lr, g, theta);
}

template <typename T> struct PathIO;

template <> struct PathIO<float> {
    static __device__ __forceinline__ float load(const float *p) { return __ldcs(p); }
    static __device__ __forceinline__ void store(float *p, float v) { __stcs(p, v); }
};

template <> struct PathIO<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16 *p)
    {
        const unsigned short bits = __ldcs(reinterpret_cast<const unsigned short *>(p));
        return __uint_as_float(((unsigned)bits) << 16);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, float v)
    {
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        __stcs(reinterpret_cast<unsigned short *>(p), __bfloat16_as_ushort(h));
    }
};

// 16 bytes of path data <-> floats.  UE = elements per 16-byte unit.
template <typename T> struct Unit;

template <> struct Unit<float> {
    static constexpr int UE = 4;
    static __device__ __forceinline__ void widen(const uint4 &v, float *f)
    {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 narrow(const float *f)
    {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                          __float_as_uint(f[3]));
    }
};

template <> struct Unit<__nv_bfloat16> {
    static constexpr int UE = 8;
    static __device__ __forceinline__ void widen(const uint4 &v, float *f)
    {
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    static __device__ __forceinline__ unsigned pack(float lo, float hi)
    {
        const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);  // .x = lo (low half), .y = hi
        return *reinterpret_cast<const unsigned *>(&h);
    }
    static __device__ __forceinline__ uint4 narrow(const float *f)
    {
        return make_uint4(pack(f[0], f[1]), pack(f[2], f[3]), pack(f[4], f[5]), pack(f[6], f[7]));
    }
};

// ------------------------------------------------------------------------------------------
// Path data that is only element-aligned.  A thread's 16 bytes then straddle two aligned 16-byte
// units; both are loaded whole and the wanted bytes are cut out with funnel shifts.

// The 16 bytes that start s bytes into the 32 bytes (lo, hi); s even, 0 <= s < 16.  Branch free (a
// word-granular barrel shift by selects, then one funnel shift by 0 or 16 bits), so that the
// compiler can keep the loads of several contributors in flight across it.
__device__ __forceinline__ uint4 cut16(const uint4 &lo, const uint4 &hi, unsigned s)
{
    const bool by1 = (s & 4u) != 0, by2 = (s & 8u) != 0;
    const unsigned r = (s & 2u) * 8u;
    const unsigned w0 = lo.x, w1 = lo.y, w2 = lo.z, w3 = lo.w, w4 = hi.x, w5 = hi.y, w6 = hi.z, w7 = hi.w;
    const unsigned x0 = by1 ? w1 : w0, x1 = by1 ? w2 : w1, x2 = by1 ? w3 : w2, x3 = by1 ? w4 : w3,
                   x4 = by1 ? w5 : w4, x5 = by1 ? w6 : w5, x6 = by1 ? w7 : w6;
    const unsigned y0 = by2 ? x2 : x0, y1 = by2 ? x3 : x1, y2 = by2 ? x4 : x2, y3 = by2 ? x5 : x3,
                   y4 = by2 ? x6 : x4;
    return make_uint4(__funnelshift_r(y0, y1, r), __funnelshift_r(y1, y2, r), __funnelshift_r(y2, y3, r),
                      __funnelshift_r(y3, y4, r));
}

// UNITS * 16 bytes from an address that is only element-aligned: the aligned 16-byte units that
// contain them (one more than UNITS when the address lies inside a unit) and how far into the
// first unit the data starts.  Up to 15 bytes before and after the wanted range are read, inside
// the same aligned units.  Loading and cutting are separate so that a caller can issue the loads of
// several sources before it uses any of them.
template <int UNITS>
__device__ __forceinline__ unsigned load_around(const void *p, uint4 *raw)
{
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    const unsigned s = (unsigned)(a & 15u);
    const uint4 *base = reinterpret_cast<const uint4 *>(a - s);
#pragma unroll
    for (int u = 0; u < UNITS; ++u) raw[u] = __ldcs(base + u);
    raw[UNITS] = make_uint4(0u, 0u, 0u, 0u);
    if (s != 0) raw[UNITS] = __ldcs(base + UNITS);
    return s;
}

__device__ __forceinline__ uint4 shfl_down1(const uint4 &v)
{
    return make_uint4(__shfl_down_sync(0xffffffffu, v.x, 1), __shfl_down_sync(0xffffffffu, v.y, 1),
                      __shfl_down_sync(0xffffffffu, v.z, 1), __shfl_down_sync(0xffffffffu, v.w, 1));
}

__device__ __forceinline__ unsigned word_at(const uint4 &v, int i)
{
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

// Element i (of the 16-byte unit v) to *dst.
__device__ __forceinline__ void store_element(float *dst, const uint4 &v, int i)
{
    __stcs(reinterpret_cast<unsigned *>(dst), word_at(v, i));
}
__device__ __forceinline__ void store_element(__nv_bfloat16 *dst, const uint4 &v, int i)
{
    const unsigned w = word_at(v, i >> 1);
    __stcs(reinterpret_cast<unsigned short *>(dst), (unsigned short)((i & 1) ? (w >> 16) : (w & 0xffffu)));
}

// The bytes of a CTA's step that do not fill an aligned 16-byte unit of a shifted destination: the
// first `count` elements of the step's first thread (from_end = false) or the last `count` elements
// of its last thread (from_end = true).  `unit` is that thread's first, or last, 16 bytes.
template <typename PathT>
__device__ __forceinline__ void store_edge_elements(PathT *first_or_last, const uint4 &unit, int count,
                                                    bool from_end)
{
    constexpr int PER = 16 / (int)sizeof(PathT);  // elements per 16 bytes
#pragma unroll
    for (int i = 0; i < PER - 1; ++i) {
        if (i < count) {
            if (from_end) store_element(first_or_last - i, unit, PER - 1 - i);
            else store_element(first_or_last + i, unit, i);
        }
    }
}

// ------------------------------------------------------------------------------------------
// Direct kernels: every thread owns VEC consecutive elements and walks the contributors itself.

// SHIFTED (VEC = 8 only): theta, momentum, partial sums and second moment are 16-byte aligned at
// every thread's first element (the host cuts the range that way); the path buffers and the cast
// scratch may sit at any element alignment, each its own.  A thread loads the aligned 16-byte
// units around its data and cuts its bytes out; stores are put together into aligned units again
// across neighbouring threads.  Segments are whole CTA steps of 2048 elements.
template <typename PathT, int VEC, bool SHIFTED = false>
__global__ void __launch_bounds__(256, SHIFTED ? 2 : 0) sync_direct_kernel(LaunchParams p)
{
    static_assert(!SHIFTED || VEC == 8, "the shifted variant is the 8-element one");
    // a context whose error word is set (a bounded wait ran out earlier) does no further work
    // until the host has read the status
    if (*reinterpret_cast<volatile const int *>(p.error_word) != 0) return;
    const int seg_begin = p.cta_first[blockIdx.x];
    const int seg_end = p.cta_first[blockIdx.x + 1];
    for (int s = seg_begin; s < seg_end; ++s) {
        const SegmentDev seg = p.segs[s];
        const PassDev pass = p.passes[seg.pass];
        const ContribDev *contribs = p.contribs + pass.contrib_begin;
        void *const *members = p.members + pass.member_begin;
        float *theta = p.theta + pass.theta_off;
        float *momentum = p.momentum + pass.theta_off;
        float *partial = p.partial + pass.partial_off;
        const PathT *cast_src = static_cast<const PathT *>(p.cast_scratch) + pass.cast_off;

        for (long long k = seg.begin + (long long)threadIdx.x * VEC; k < seg.end;
             k += (long long)blockDim.x * VEC) {
            float th[VEC], acc[VEC];
            if constexpr (VEC == 1) {
                // widening the stored cast and narrowing it again reproduces its bits exactly
                th[0] = (pass.flags & KPASS_CAST_IN) ? PathIO<PathT>::load(cast_src + k) : theta[k];
                acc[0] = (pass.flags & KPASS_PARTIAL_IN) ? partial[k] : 0.0f;
                // loads of four contributors in flight, summation still in ascending order
                int j = 0;
                for (; j + 4 <= pass.contrib_count; j += 4) {
                    float x[4], cf[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const ContribDev c = contribs[j + u];
                        cf[u] = c.coeff;
                        x[u] = PathIO<PathT>::load(static_cast<const PathT *>(c.src) + k);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) acc[0] = sync_accumulate(acc[0], cf[u], th[0], x[u], p.input_kind);
                }
                for (; j < pass.contrib_count; ++j) {
                    const ContribDev c = contribs[j];
                    const float x = PathIO<PathT>::load(static_cast<const PathT *>(c.src) + k);
                    acc[0] = sync_accumulate(acc[0], c.coeff, th[0], x, p.input_kind);
                }
            } else {
                constexpr int UE = Unit<PathT>::UE;
                constexpr int UNITS = VEC / UE;  // 16-byte loads per contributor
                // contributors whose loads are issued together (the shifted variant loads one
                // more unit per contributor: 48 registers of path data in flight either way)
                constexpr int BATCH = SHIFTED ? (UNITS == 1 ? 6 : 3) : 8 / UNITS;
                if (pass.flags & KPASS_CAST_IN) {
                    if constexpr (SHIFTED) {
                        uint4 around[UNITS + 1];
                        const unsigned shift = load_around<UNITS>(cast_src + k, around);
#pragma unroll
                        for (int u = 0; u < UNITS; ++u)
                            Unit<PathT>::widen(cut16(around[u], around[u + 1], shift), th + u * UE);
                    } else {
                        const uint4 *src = reinterpret_cast<const uint4 *>(cast_src + k);
#pragma unroll
                        for (int u = 0; u < UNITS; ++u) Unit<PathT>::widen(__ldcs(src + u), th + u * UE);
                    }
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; v += 4) {
                        const float4 t = *reinterpret_cast<const float4 *>(theta + k + v);
                        th[v] = t.x; th[v + 1] = t.y; th[v + 2] = t.z; th[v + 3] = t.w;
                    }
                }
                if (pass.flags & KPASS_PARTIAL_IN) {
#pragma unroll
                    for (int v = 0; v < VEC; v += 4) {
                        const float4 t = *reinterpret_cast<const float4 *>(partial + k + v);
                        acc[v] = t.x; acc[v + 1] = t.y; acc[v + 2] = t.z; acc[v + 3] = t.w;
                    }
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) acc[v] = 0.0f;
                }
                for (int j0 = 0; j0 < pass.contrib_count; j0 += BATCH) {
                    uint4 raw[BATCH][UNITS + (SHIFTED ? 1 : 0)];
                    unsigned shift[BATCH];  // SHIFTED: how far into raw[b][0] the data starts
                    float coeff[BATCH];
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) {
                        shift[b] = 0;
                        if (j0 + b < pass.contrib_count) {
                            const ContribDev c = contribs[j0 + b];
                            coeff[b] = c.coeff;
                            if constexpr (SHIFTED) {
                                shift[b] = load_around<UNITS>(static_cast<const PathT *>(c.src) + k, raw[b]);
                            } else {
                                const uint4 *src = reinterpret_cast<const uint4 *>(
                                    static_cast<const PathT *>(c.src) + k);
#pragma unroll
                                for (int u = 0; u < UNITS; ++u) raw[b][u] = __ldcs(src + u);
                            }
                        }
                    }
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) {
                        if (j0 + b < pass.contrib_count) {
#pragma unroll
                            for (int u = 0; u < UNITS; ++u) {
                                float x[UE];
                                if constexpr (SHIFTED)
                                    Unit<PathT>::widen(cut16(raw[b][u], raw[b][u + 1], shift[b]), x);
                                else
                                    Unit<PathT>::widen(raw[b][u], x);
#pragma unroll
                                for (int i = 0; i < UE; ++i)
                                    acc[u * UE + i] =
                                        sync_accumulate(acc[u * UE + i], coeff[b], th[u * UE + i], x[i], p.input_kind);
                            }
                        }
                    }
                }
            }

            if (pass.flags & KPASS_PARTIAL_OUT) {
                if constexpr (VEC == 1) {
                    partial[k] = acc[0];
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; v += 4)
                        *reinterpret_cast<float4 *>(partial + k + v) =
                            make_float4(acc[v], acc[v + 1], acc[v + 2], acc[v + 3]);
                }
            }
            if (pass.flags & KPASS_UPDATE) {
                float mo[VEC];
                if constexpr (VEC == 1) {
                    mo[0] = momentum[k];
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; v += 4) {
                        const float4 t = *reinterpret_cast<const float4 *>(momentum + k + v);
                        mo[v] = t.x; mo[v + 1] = t.y; mo[v + 2] = t.z; mo[v + 3] = t.w;
                    }
                }
                const bool adam = p.rule.optimizer == KOPT_ADAM;
                float *second = p.second_moment + pass.theta_off;
                float sm[VEC];
#pragma unroll
                for (int v = 0; v < VEC; ++v) sm[v] = adam ? second[k + v] : 0.0f;
#pragma unroll
                for (int v = 0; v < VEC; ++v) {
                    float t1, m1;
                    sync_update(th[v], mo[v], sm[v], acc[v], pass.scale, p.rule, t1, m1);
                    th[v] = t1;
                    mo[v] = m1;
                }
                if (adam) {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) second[k + v] = sm[v];
                }
                if constexpr (VEC == 1) {
                    theta[k] = th[0];
                    momentum[k] = mo[0];
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; v += 4) {
                        *reinterpret_cast<float4 *>(theta + k + v) =
                            make_float4(th[v], th[v + 1], th[v + 2], th[v + 3]);
                        *reinterpret_cast<float4 *>(momentum + k + v) =
                            make_float4(mo[v], mo[v + 1], mo[v + 2], mo[v + 3]);
                    }
                }
            }
            if (pass.member_count > 0) {
                if constexpr (VEC == 1) {
                    for (int j = 0; j < pass.member_count; ++j)
                        PathIO<PathT>::store(static_cast<PathT *>(members[j]) + k, th[0]);
                } else {
                    constexpr int UE = Unit<PathT>::UE;
                    constexpr int UNITS = VEC / UE;
                    uint4 out[UNITS];
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) out[u] = Unit<PathT>::narrow(th + u * UE);
                    if constexpr (SHIFTED) {
                        // A destination that sits sh bytes into a 16-byte unit is written in
                        // aligned units all the same: the unit that straddles two threads takes
                        // its first sh bytes from the end of the earlier thread's data and the
                        // rest from the start of the next thread's (next lane by shuffle, next
                        // warp through shared memory).  That unit reaches into bytes that the
                        // next thread reads as input: inside a warp all lanes have their inputs
                        // by now, and the barrier makes it so across the warps of the CTA.  Only
                        // the two ends of the CTA's 2048 elements are left over and go out
                        // element by element.  The host sorts the members of a pass by their
                        // shift, so the realigned units are rebuilt once per shift.
                        __shared__ uint4 first_unit[8];
                        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
                        uint4 next_first = shfl_down1(out[0]);
                        if (lane == 0) first_unit[warp] = out[0];
                        __syncthreads();
                        if (lane == 31 && warp < 7) next_first = first_unit[warp + 1];
                        __syncthreads();
                        const bool last_thread = threadIdx.x == 255;
                        unsigned current = 0;
                        uint4 realigned[UNITS];
                        for (int j = 0; j < pass.member_count; ++j) {
                            PathT *dst = static_cast<PathT *>(members[j]) + k;
                            const uintptr_t a = reinterpret_cast<uintptr_t>(dst);
                            const unsigned sh = (unsigned)(a & 15u);
                            if (sh == 0) {
                                uint4 *d16 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
                                for (int u = 0; u < UNITS; ++u) __stcs(d16 + u, out[u]);
                                continue;
                            }
                            if (sh != current) {
                                current = sh;
#pragma unroll
                                for (int u = 0; u < UNITS; ++u)
                                    realigned[u] = cut16(out[u], u + 1 < UNITS ? out[u + 1] : next_first, 16u - sh);
                            }
                            uint4 *d16 = reinterpret_cast<uint4 *>(a + 16u - sh);
#pragma unroll
                            for (int u = 0; u + 1 < UNITS; ++u) __stcs(d16 + u, realigned[u]);
                            if (!last_thread) __stcs(d16 + UNITS - 1, realigned[UNITS - 1]);
                            if (threadIdx.x == 0)
                                store_edge_elements<PathT>(dst, out[0], (int)(16u - sh) / (int)sizeof(PathT), false);
                            if (last_thread)
                                store_edge_elements<PathT>(dst + VEC - 1, out[UNITS - 1], (int)sh / (int)sizeof(PathT), true);
                        }
                    } else {
                        for (int j = 0; j < pass.member_count; ++j) {
                            uint4 *dst = reinterpret_cast<uint4 *>(static_cast<PathT *>(members[j]) + k);
#pragma unroll
                            for (int u = 0; u < UNITS; ++u) __stcs(dst + u, out[u]);
                        }
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Bulk-copy (TMA) pipeline.

namespace ptx {

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// global -> shared bulk copy, completion signalled on an mbarrier (bytes: multiple of 16)
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, unsigned bytes,
                                          uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(smem_addr(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}
// shared -> global bulk copy, tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void bulk_store(void *dst_gmem, const void *src_smem, unsigned bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem),
                 "r"(smem_addr(src_smem)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all()
{
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

} // namespace ptx

constexpr int BULK_COMPUTE_WARPS = 8;
constexpr int BULK_COMPUTE_THREADS = BULK_COMPUTE_WARPS * 32;
constexpr int BULK_THREADS = BULK_COMPUTE_THREADS + 96;  // + load, store and scheduler warps
constexpr int BULK_SHIFTED_STORE_WARPS = 4;  // the variant for shifted path buffers stores with four warps
constexpr int BULK_SHIFTED_THREADS = BULK_THREADS + 32 * (BULK_SHIFTED_STORE_WARPS - 1);
constexpr int BULK_MAX_STAGES = 32;
constexpr int BULK_SCHED_DEPTH = 4;
constexpr int BULK_MAX_IO_SLOTS = 4;  // buffers of theta/momentum/partial/result tiles
constexpr unsigned long long BULK_WAIT_LIMIT_NS = 4000000000ull;  // every wait gives up after 4 s

// Bounded wait: returns false (and records the failure) if the phase does not complete in time.
__device__ __forceinline__ bool bounded_wait(uint64_t *bar, unsigned parity, int *error_word, int code,
                                             unsigned long long limit_ns = BULK_WAIT_LIMIT_NS)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = ptx::global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (ptx::mbar_try_wait(bar, parity)) return true;
        if (ptx::global_timer_ns() - t0 > limit_ns) {
            atomicCAS(error_word, 0, code);
            return false;
        }
    }
}

struct BulkShared {
    uint64_t full[BULK_MAX_STAGES];   // ring slot filled by a bulk load
    uint64_t empty[BULK_MAX_STAGES];  // ring slot released by the compute warps
    uint64_t io_full[BULK_MAX_IO_SLOTS];    // theta / momentum / partial tiles loaded
    uint64_t io_empty[BULK_MAX_IO_SLOTS];   // result tiles drained by the store warp
    uint64_t out_ready[BULK_MAX_IO_SLOTS];  // compute warps finished writing the result tiles
    uint64_t sched_full[BULK_SCHED_DEPTH];   // a work item was published by the scheduler warp
    uint64_t sched_empty[BULK_SCHED_DEPTH];  // all consumer warps (compute, load, store) have read it
    long long sched_begin[BULK_SCHED_DEPTH], sched_end[BULK_SCHED_DEPTH];
    int sched_pass[BULK_SCHED_DEPTH];        // -1 = no more work
    float slot_coeff[BULK_MAX_STAGES];
    unsigned slot_shift[BULK_MAX_STAGES];  // bytes from the start of a ring slot to the tile's data
    // store warps: the destinations that share the current shift (one list per warp)
    unsigned long long store_dst[BULK_SHIFTED_STORE_WARPS][32];
    const void *batch_src[32];
    float batch_coeff[32];
};

// Position in the shared-memory ring: slot index and the phase parity of its barriers.
struct RingPos {
    int slot = 0;
    unsigned phase = 0;
    unsigned used = 0;  // slots used so far
    __device__ __forceinline__ void advance(int stages)
    {
        ++used;
        if (++slot == stages) { slot = 0; phase ^= 1u; }
    }
    __device__ __forceinline__ void retreat(int stages)
    {
        --used;
        if (slot == 0) { slot = stages - 1; phase ^= 1u; } else { --slot; }
    }
};

// Work items are drawn from a global counter by the scheduler warp and published through a
// small shared-memory ring; the load, store and compute warps all walk the same item sequence.
struct ItemWalk {
    BulkShared *sh;
    int *error_word;
    long long tile;
    int lane;
    int slot = 0;
    unsigned phase = 0;
    int pass = -1;
    long long pos = 0, end = 0;
    __device__ ItemWalk(BulkShared *shared, int *err, long long tile_elems, int lane_id)
        : sh(shared), error_word(err), tile(tile_elems), lane(lane_id)
    {
    }
    // Next tile of this CTA: sets pass, its first element k0 and its element count n (a full tile,
    // or the partial last tile of a pass); false when the work is exhausted (ok stays true) or a
    // wait ran out (ok = false).  Must be called by all lanes of the warp together.
    __device__ bool next(long long &k0, unsigned &n, bool &ok)
    {
        if (pass >= 0) {
            pos += tile;
            if (pos < end) {
                k0 = pos;
                n = (unsigned)min(tile, end - pos);
                return true;
            }
        }
        ok = bounded_wait(&sh->sched_full[slot], phase, error_word, 7);
        if (!ok) return false;
        const int item_pass = sh->sched_pass[slot];
        const long long b = sh->sched_begin[slot], e = sh->sched_end[slot];
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh->sched_empty[slot]);
        if (++slot == BULK_SCHED_DEPTH) { slot = 0; phase ^= 1u; }
        if (item_pass < 0) return false;
        pass = item_pass; pos = b; end = e;
        k0 = pos;
        n = (unsigned)min(tile, end - pos);
        return true;
    }
};

// NU = 16-byte units of path data per compute thread and tile; tile = 256 * NU * UE elements.
// SHIFTED: the tiles of theta, momentum, partial sums, second moment and cast scratch are 16-byte
// aligned as always (the host cuts the range that way), but a path buffer may sit at any element
// alignment, each its own.  A contributor's tile is then loaded from the aligned address at or
// before it (16 bytes more) and the compute warps cut their bytes out of two neighbouring units;
// a member that is not aligned is written by the store warp itself, in aligned 16-byte units put
// together from the cast tile, instead of by a bulk store.
template <typename PathT, int NU, bool SHIFTED = false>
__global__ void __launch_bounds__(SHIFTED ? BULK_SHIFTED_THREADS : BULK_THREADS, 1)
sync_bulk_kernel(LaunchParams p, int stages, int io_arrays, int io_slots)
{
    // warps: 0..7 compute, 8 load, 9.. store (one, or four in the shifted variant), then the scheduler
    constexpr int STORE_WARPS = SHIFTED ? BULK_SHIFTED_STORE_WARPS : 1;
    constexpr int FIRST_STORE_WARP = BULK_COMPUTE_WARPS + 1;
    constexpr int SCHED_WARP = FIRST_STORE_WARP + STORE_WARPS;
    constexpr int ITEM_READERS = BULK_COMPUTE_WARPS + 1 + STORE_WARPS;  // warps that consume every work item
    constexpr int UE = Unit<PathT>::UE;
    constexpr int EPT = UE * NU;                         // elements per compute thread
    constexpr int TILE = BULK_COMPUTE_THREADS * EPT;     // elements per tile
    constexpr unsigned STAGE_BYTES = TILE * sizeof(PathT);
    constexpr unsigned STAGE_STRIDE = STAGE_BYTES + (SHIFTED ? 16u : 0u);  // ring slot size
    constexpr unsigned F32_TILE_BYTES = TILE * 4u;
    constexpr bool NEED_CAST_TILE = sizeof(PathT) != 4;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: ring | io[io_slots][io_arrays] fp32 tiles | cast tile[io_slots] (bf16 only) | BulkShared
    unsigned char *ring = smem_raw;
    unsigned char *io = ring + (size_t)stages * STAGE_STRIDE;
    unsigned char *cast_tiles = io + (size_t)io_slots * io_arrays * F32_TILE_BYTES;
    BulkShared *sh = reinterpret_cast<BulkShared *>(
        cast_tiles + (NEED_CAST_TILE ? (size_t)io_slots * STAGE_BYTES : (size_t)0));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(&sh->full[s], 1);
            ptx::mbar_init(&sh->empty[s], BULK_COMPUTE_WARPS);
        }
        for (int d = 0; d < BULK_SCHED_DEPTH; ++d) {
            ptx::mbar_init(&sh->sched_full[d], 1);
            ptx::mbar_init(&sh->sched_empty[d], ITEM_READERS);
        }
        for (int b = 0; b < io_slots; ++b) {
            ptx::mbar_init(&sh->io_full[b], 1);
            ptx::mbar_init(&sh->io_empty[b], STORE_WARPS);
            ptx::mbar_init(&sh->out_ready[b], BULK_COMPUTE_WARPS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto io_tile = [&](int b, int which) -> float * {
        return reinterpret_cast<float *>(io + ((size_t)b * io_arrays + which) * F32_TILE_BYTES);
    };
    // io tile roles: 0 = theta (becomes theta'), 1 = momentum (becomes m'), 2 = partial sum (chunked
    // contexts), v_index = second moment (Adam family)
    auto cast_tile = [&](int b) -> unsigned char * {
        return NEED_CAST_TILE ? cast_tiles + (size_t)b * STAGE_BYTES
                              : reinterpret_cast<unsigned char *>(io_tile(b, 0));
    };

    ItemWalk walk(sh, p.error_word, TILE, lane);
    long long k0;
    unsigned n;      // elements of the current tile (partial tiles: compute runs on the whole
                     // shared-memory tile, only the first n elements are loaded and stored)
    RingPos io_pos;  // theta/momentum/result buffer of the current tile (advances once per tile)
    RingPos q;       // ring position of this role

    if (warp == SCHED_WARP) {
        // ------------------------------------------------------------------ scheduler warp
        if (lane == 0) {
            int slot = 0;
            unsigned phase = 0;
            // A context whose error word is already set (a bounded wait ran out in an earlier
            // launch) does no further work until the host has read the status: this CTA publishes
            // its end-of-work marker at once and leaves the work counters alone.
            const bool poisoned = *reinterpret_cast<volatile const int *>(p.error_word) != 0;
            for (;;) {
                if (!bounded_wait(&sh->sched_empty[slot], phase ^ 1u, p.error_word, 8)) break;
                if (poisoned) {
                    sh->sched_pass[slot] = -1;
                    sh->sched_begin[slot] = 0;
                    sh->sched_end[slot] = 0;
                    ptx::mbar_arrive(&sh->sched_full[slot]);
                    break;
                }
                const int item = atomicAdd(p.work_counter, 1);
                int item_pass = -1;
                long long b = 0, e = 0;
                if (item < p.total_items) {
                    // last pass whose first item is <= item (passes without items sort before it)
                    int lo = 0, hi = p.num_passes - 1;
                    while (lo < hi) {
                        const int mid = (lo + hi + 1) >> 1;
                        if (p.passes[mid].item_first <= item) lo = mid; else hi = mid - 1;
                    }
                    const PassDev ps = p.passes[lo];
                    const long long first_tile = (long long)(item - ps.item_first) * ps.tiles_per_item;
                    const long long last_tile = min(first_tile + ps.tiles_per_item, ps.bulk_tiles);
                    item_pass = lo;
                    b = ps.bulk_begin + first_tile * TILE;
                    e = min(ps.bulk_begin + last_tile * TILE, ps.bulk_end);
                }
                sh->sched_pass[slot] = item_pass;
                sh->sched_begin[slot] = b;
                sh->sched_end[slot] = e;
                ptx::mbar_arrive(&sh->sched_full[slot]);
                if (item_pass < 0) {
                    // nobody draws after its own sentinel: the last CTA here re-arms the counters
                    if (atomicAdd(p.work_counter + 1, 1) == (int)gridDim.x - 1) {
                        p.work_counter[0] = 0;
                        p.work_counter[1] = 0;
                    }
                    break;
                }
                if (++slot == BULK_SCHED_DEPTH) { slot = 0; phase ^= 1u; }
            }
        }
    } else if (warp == BULK_COMPUTE_WARPS) {
        // ------------------------------------------------------------------ load warp
        bool ok = true;
        while (ok && walk.next(k0, n, ok)) {
            const PassDev pass = p.passes[walk.pass];
            const int b = io_pos.slot;
            if (lane == 0) {
                ok = bounded_wait(&sh->io_empty[b], io_pos.phase ^ 1u, p.error_word, 1);
                if (ok && (pass.flags & KPASS_CAST_IN)) {
                    // write-back only: the finished cast tile comes straight from the scratch
                    const unsigned path_bytes = n * (unsigned)sizeof(PathT);
                    ptx::mbar_arrive_expect_tx(&sh->io_full[b], path_bytes);
                    ptx::bulk_load(cast_tile(b),
                                   static_cast<const PathT *>(p.cast_scratch) + pass.cast_off + k0,
                                   path_bytes, &sh->io_full[b]);
                } else if (ok) {
                    const unsigned f32_bytes = n * 4u;
                    unsigned bytes = f32_bytes;
                    const bool adam = (pass.flags & KPASS_UPDATE) && p.rule.optimizer == KOPT_ADAM;
                    if (pass.flags & KPASS_UPDATE) bytes += f32_bytes;
                    if (adam) bytes += f32_bytes;
                    if (pass.flags & KPASS_PARTIAL_IN) bytes += f32_bytes;
                    ptx::mbar_arrive_expect_tx(&sh->io_full[b], bytes);
                    ptx::bulk_load(io_tile(b, 0), p.theta + pass.theta_off + k0, f32_bytes,
                                   &sh->io_full[b]);
                    if (pass.flags & KPASS_UPDATE)
                        ptx::bulk_load(io_tile(b, 1), p.momentum + pass.theta_off + k0, f32_bytes,
                                       &sh->io_full[b]);
                    if (pass.flags & KPASS_PARTIAL_IN)
                        ptx::bulk_load(io_tile(b, 2), p.partial + pass.partial_off + k0, f32_bytes,
                                       &sh->io_full[b]);
                    if (adam)
                        ptx::bulk_load(io_tile(b, p.v_index), p.second_moment + pass.theta_off + k0,
                                       f32_bytes, &sh->io_full[b]);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            for (int j0 = 0; ok && j0 < pass.contrib_count; j0 += 32) {
                const int cnt = min(32, pass.contrib_count - j0);
                if (lane < cnt) {
                    const ContribDev c = p.contribs[pass.contrib_begin + j0 + lane];
                    sh->batch_src[lane] = c.src;
                    sh->batch_coeff[lane] = c.coeff;
                }
                __syncwarp();
                if (lane == 0) {
                    for (int u = 0; u < cnt; ++u) {
                        const int s = q.slot;
                        ok = bounded_wait(&sh->empty[s], q.phase ^ 1u, p.error_word, 2);
                        if (!ok) break;
                        sh->slot_coeff[s] = sh->batch_coeff[u];
                        unsigned path_bytes = n * (unsigned)sizeof(PathT);
                        const PathT *from = static_cast<const PathT *>(sh->batch_src[u]) + k0;
                        if constexpr (SHIFTED) {
                            // start at the aligned address at or before the tile; the bytes in
                            // front of the data and the 16 more behind it lie in the same aligned
                            // units as the data
                            const unsigned shift = (unsigned)(reinterpret_cast<uintptr_t>(from) & 15u);
                            sh->slot_shift[s] = shift;
                            from = reinterpret_cast<const PathT *>(reinterpret_cast<const char *>(from) - shift);
                            if (shift) path_bytes += 16u;
                        }
                        ptx::mbar_arrive_expect_tx(&sh->full[s], path_bytes);
                        ptx::bulk_load(ring + (size_t)s * STAGE_STRIDE, from, path_bytes, &sh->full[s]);
                        q.advance(stages);
                    }
                }
                __syncwarp();
                ok = __shfl_sync(0xffffffffu, ok, 0);
            }
            io_pos.advance(io_slots);
        }
        // Leave only when every copy this warp started has landed: another CTA may get this
        // shared memory next.  Waits on already completed phases return at once.
        if (lane == 0) {
            for (int back = 0; back < stages && q.used > 0; ++back) {
                q.retreat(stages);
                bounded_wait(&sh->full[q.slot], q.phase, p.error_word, 3);
            }
            for (int back = 0; back < io_slots && io_pos.used > 0; ++back) {
                io_pos.retreat(io_slots);
                bounded_wait(&sh->io_full[io_pos.slot], io_pos.phase, p.error_word, 3);
            }
        }
    } else if (warp >= FIRST_STORE_WARP && warp < SCHED_WARP) {
        // ------------------------------------------------------------------ store warp(s)
        // The first store warp issues every bulk store; in the shifted variant all of them share
        // the members that are written with ordinary stores.
        const int rank = warp - FIRST_STORE_WARP;
        bool ok = true;
        while (ok && walk.next(k0, n, ok)) {
            const PassDev pass = p.passes[walk.pass];
            const int b = io_pos.slot;
            ok = bounded_wait(&sh->out_ready[b], io_pos.phase, p.error_word, 4);
            if (!ok) break;
            if (lane == 0 && rank == 0) {
                if (pass.flags & KPASS_UPDATE) {
                    ptx::bulk_store(p.theta + pass.theta_off + k0, io_tile(b, 0), n * 4u);
                    ptx::bulk_store(p.momentum + pass.theta_off + k0, io_tile(b, 1), n * 4u);
                    if (p.rule.optimizer == KOPT_ADAM)
                        ptx::bulk_store(p.second_moment + pass.theta_off + k0, io_tile(b, p.v_index),
                                        n * 4u);
                }
                if (pass.flags & KPASS_PARTIAL_OUT)
                    ptx::bulk_store(p.partial + pass.partial_off + k0, io_tile(b, 2), n * 4u);
            }
            const unsigned char *src = cast_tile(b);
            const int bulk_members = rank != 0 ? 0 : (SHIFTED ? pass.aligned_members : pass.member_count);
            for (int j = lane; j < bulk_members; j += 32) {
                PathT *dst = static_cast<PathT *>(p.members[pass.member_begin + j]) + k0;
                ptx::bulk_store(dst, src, n * (unsigned)sizeof(PathT));
            }
            if constexpr (SHIFTED) {
                // Members inside a 16-byte unit (the host puts them after the aligned ones, sorted
                // by their shift).  Thirty-two at a time, one per lane; for every shift among them
                // the store warps walk the tile once between them, build each aligned 16-byte unit
                // of output from two neighbouring units of the cast tile and store it to all
                // members with that shift.  The bytes in front of a member's first aligned unit
                // and behind its last one go out element by element (first store warp).
                const uint4 *tile16 = reinterpret_cast<const uint4 *>(src);
                const PathT *tile_el = reinterpret_cast<const PathT *>(src);
                const int units = (int)(n * (unsigned)sizeof(PathT) / 16u);
                constexpr int PER = 16 / (int)sizeof(PathT);
                for (int base = pass.aligned_members; base < pass.member_count; base += 32) {
                    const bool valid = base + lane < pass.member_count;
                    char *mine = valid ? reinterpret_cast<char *>(static_cast<PathT *>(
                                             p.members[pass.member_begin + base + lane]) + k0)
                                       : nullptr;
                    const unsigned my_shift = (unsigned)(reinterpret_cast<uintptr_t>(mine) & 15u);
                    unsigned todo = __ballot_sync(0xffffffffu, valid);
                    while (todo) {
                        const int leader = __ffs(todo) - 1;
                        const unsigned shift = __shfl_sync(0xffffffffu, my_shift, leader);
                        const unsigned group = __ballot_sync(0xffffffffu, valid && my_shift == shift) & todo;
                        todo &= ~group;
                        // the group's first aligned units, side by side in shared memory
                        __syncwarp();
                        if ((group >> lane) & 1u)
                            sh->store_dst[rank][__popc(group & ((1u << lane) - 1u))] =
                                (unsigned long long)reinterpret_cast<uintptr_t>(mine) + 16u - shift;
                        __syncwarp();
                        const int count = __popc(group);
                        // aligned unit i of the output holds tile bytes [16 i + 16 - shift, 16 i + 32 - shift)
                        for (int i = rank * 32 + lane; i + 1 < units; i += 32 * STORE_WARPS) {
                            const uint4 unit = cut16(tile16[i], tile16[i + 1], 16u - shift);
#pragma unroll 4
                            for (int m = 0; m < count; ++m)
                                __stcs(reinterpret_cast<uint4 *>(sh->store_dst[rank][m]) + i, unit);
                        }
                    }
                    // edges: each lane for its own member
                    if (valid && rank == 0) {
                        PathT *dst = reinterpret_cast<PathT *>(mine);
                        const int head = (int)(16u - my_shift) / (int)sizeof(PathT);
#pragma unroll
                        for (int e = 0; e < PER; ++e) {
                            const unsigned at = e < head ? (unsigned)e : n - (unsigned)PER + (unsigned)e;
                            dst[at] = tile_el[at];
                        }
                    }
                }
            }
            ptx::bulk_commit();
            ptx::bulk_wait_read_all();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sh->io_empty[b]);
            io_pos.advance(io_slots);
        }
        ptx::bulk_wait_all();
    } else {
        // ------------------------------------------------------------------ compute warps
        const int ct = threadIdx.x;  // 0 .. BULK_COMPUTE_THREADS-1
        bool ok = true;
        while (ok && walk.next(k0, n, ok)) {
            const PassDev pass = p.passes[walk.pass];
            const int b = io_pos.slot;
            ok = bounded_wait(&sh->io_full[b], io_pos.phase, p.error_word, 5);
            if (!ok) break;
            if (pass.flags & KPASS_CAST_IN) {
                // the cast tile arrived ready-made: hand it on to the store warp
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&sh->out_ready[b]);
                io_pos.advance(io_slots);
                continue;
            }
            float th[EPT], acc[EPT];
            float *th_tile = io_tile(b, 0);
#pragma unroll
            for (int u = 0; u < NU; ++u) {
                const int e0 = (u * BULK_COMPUTE_THREADS + ct) * UE;
#pragma unroll
                for (int v = 0; v < UE; v += 4) {
                    const float4 x = *reinterpret_cast<const float4 *>(th_tile + e0 + v);
                    th[u * UE + v] = x.x; th[u * UE + v + 1] = x.y;
                    th[u * UE + v + 2] = x.z; th[u * UE + v + 3] = x.w;
                }
            }
            if (pass.flags & KPASS_PARTIAL_IN) {
                const float *pt = io_tile(b, 2);
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    const int e0 = (u * BULK_COMPUTE_THREADS + ct) * UE;
#pragma unroll
                    for (int v = 0; v < UE; v += 4) {
                        const float4 x = *reinterpret_cast<const float4 *>(pt + e0 + v);
                        acc[u * UE + v] = x.x; acc[u * UE + v + 1] = x.y;
                        acc[u * UE + v + 2] = x.z; acc[u * UE + v + 3] = x.w;
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < EPT; ++i) acc[i] = 0.0f;
            }

            for (int j = 0; j < pass.contrib_count; ++j) {
                const int s = q.slot;
                ok = bounded_wait(&sh->full[s], q.phase, p.error_word, 6);
                if (!ok) break;
                const float c = sh->slot_coeff[s];
                const uint4 *slot = reinterpret_cast<const uint4 *>(ring + (size_t)s * STAGE_STRIDE);
                uint4 raw[NU];
#pragma unroll
                for (int u = 0; u < NU; ++u) raw[u] = slot[u * BULK_COMPUTE_THREADS + ct];
                if constexpr (SHIFTED) {
                    const unsigned shift = sh->slot_shift[s];
                    if (shift) {  // the same for the whole CTA
#pragma unroll
                        for (int u = 0; u < NU; ++u)
                            raw[u] = cut16(raw[u], slot[u * BULK_COMPUTE_THREADS + ct + 1], shift);
                    }
                }
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    float x[UE];
                    Unit<PathT>::widen(raw[u], x);
#pragma unroll
                    for (int i = 0; i < UE; ++i)
                        acc[u * UE + i] = sync_accumulate(acc[u * UE + i], c, th[u * UE + i], x[i], p.input_kind);
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&sh->empty[s]);
                q.advance(stages);
            }
            if (!ok) break;

            if (pass.flags & KPASS_PARTIAL_OUT) {
                float *pt = io_tile(b, 2);
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    const int e0 = (u * BULK_COMPUTE_THREADS + ct) * UE;
#pragma unroll
                    for (int v = 0; v < UE; v += 4)
                        *reinterpret_cast<float4 *>(pt + e0 + v) =
                            make_float4(acc[u * UE + v], acc[u * UE + v + 1], acc[u * UE + v + 2],
                                        acc[u * UE + v + 3]);
                }
            }
            if (pass.flags & KPASS_UPDATE) {
                float *mo_tile = io_tile(b, 1);
                const bool adam = p.rule.optimizer == KOPT_ADAM;
                float *v_tile = io_tile(b, adam ? p.v_index : 1);
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    const int e0 = (u * BULK_COMPUTE_THREADS + ct) * UE;
#pragma unroll
                    for (int v = 0; v < UE; v += 4) {
                        const float4 m4 = *reinterpret_cast<const float4 *>(mo_tile + e0 + v);
                        const float mo[4] = {m4.x, m4.y, m4.z, m4.w};
                        float sm[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                        if (adam) {
                            const float4 v4 = *reinterpret_cast<const float4 *>(v_tile + e0 + v);
                            sm[0] = v4.x; sm[1] = v4.y; sm[2] = v4.z; sm[3] = v4.w;
                        }
                        float m1[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            sync_update(th[u * UE + v + i], mo[i], sm[i], acc[u * UE + v + i], pass.scale,
                                        p.rule, th[u * UE + v + i], m1[i]);
                        if (adam)
                            *reinterpret_cast<float4 *>(v_tile + e0 + v) =
                                make_float4(sm[0], sm[1], sm[2], sm[3]);
                        *reinterpret_cast<float4 *>(mo_tile + e0 + v) =
                            make_float4(m1[0], m1[1], m1[2], m1[3]);
                        *reinterpret_cast<float4 *>(th_tile + e0 + v) =
                            make_float4(th[u * UE + v], th[u * UE + v + 1], th[u * UE + v + 2],
                                        th[u * UE + v + 3]);
                    }
                }
            }
            if (NEED_CAST_TILE && pass.member_count > 0) {
                uint4 *ct_tile = reinterpret_cast<uint4 *>(cast_tile(b));
#pragma unroll
                for (int u = 0; u < NU; ++u)
                    ct_tile[u * BULK_COMPUTE_THREADS + ct] = Unit<PathT>::narrow(th + u * UE);
            }
            ptx::fence_proxy_async();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sh->out_ready[b]);
            io_pos.advance(io_slots);
        }
    }
}

} // namespace dipaco
