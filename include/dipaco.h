/*
 * dipaco.h - C ABI of the module-wise outer synchronisation of DiPaCo on one CUDA device.
 *
 * The operation (DiPaCo, Algorithm 1, the outer-optimisation loop over levels and experts;
 * Sections 2.5-2.7).  A model is a grid of L levels with K_l modules per level (Section 2.2);
 * a path picks one module per level.  After the inner optimisation every path i holds its own
 * copy x_i of each module it passes through.  For every module (l,e):
 *
 *     Delta = sum_{i in R(l,e)} c_i * (theta - x_i)            outer gradient, Algorithm 1
 *     m'    = mu * m + Delta                                   Nesterov momentum (Section 2.5,
 *     theta'= theta - lr * (Delta + mu * m')                    lr/mu: supplementary details)
 *     x_i   = cast(theta')   for every path i through (l,e)    re-dispatch (Section 2.5)
 *
 * R(l,e) are the paths through (l,e) that reported this round (Section 2.6.2 trains subsets of
 * paths; Section 3.1 describes preempted workers); c_i = w_i / sum_{j in R} w_j with w the raw
 * per-path weights (shard sizes, Section 2.7 "Loss reweighing"; uniform when absent).  A module
 * with no reporting path, or zero total weight, keeps theta and m bit for bit; its copies are
 * still overwritten with cast(theta).  The reduction runs in ascending path id in fp32 with
 * fused multiply-adds, so results are bitwise reproducible and identical between the resident
 * and the chunked mode.
 *
 * Layouts.  theta and momentum: fp32, sum_l K_l*N_l elements ordered [level][module][element]
 * (N_l = |B_l|, the size of every module of level l).  A path copy: sum_l N_l elements, the
 * path's L modules concatenated in level order, fp32 or bf16 (round-to-nearest-even on write).
 *
 * Ownership.  The caller owns theta, momentum and all path buffers; they are updated in place.
 * A context owns small device tables and, in chunked mode, an fp32 partial-sum scratch.
 *
 * Errors.  Every function returns a status (0 = ok, negative = error) and never throws, aborts
 * or prints.  Arguments are validated before anything is launched: on a validation error the
 * caller's buffers are untouched.  Calls are asynchronous on the given stream unless noted; all
 * calls on one context must be ordered on one stream (or externally synchronised).
 */
#ifndef DIPACO_H
#define DIPACO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dipaco_ctx dipaco_ctx;

enum { DIPACO_F32 = 0, DIPACO_BF16 = 1 };

enum {
    DIPACO_OK = 0,
    DIPACO_EINVAL = -1,   /* bad argument (null, out of range, non-finite, wrong state value)   */
    DIPACO_ECUDA = -2,    /* a CUDA runtime call failed                                         */
    DIPACO_ENOMEM = -3,   /* host or device allocation failed                                   */
    DIPACO_ESTATE = -4,   /* call not allowed in the context's current state                    */
    DIPACO_ETIMEOUT = -5, /* a bounded wait inside a kernel ran out (reported by device_status) */
    DIPACO_ENODEV = -6,   /* the context was created without a device (plan only)               */
    DIPACO_ELIMIT = -7    /* a size exceeds a fixed limit of the entry point (static scratch)   */
};

/* outer optimisers for dipaco_set_optimizer */
enum {
    DIPACO_OPT_NESTEROV = 0, /* m' = mu*m + Delta; theta' = theta - lr*(Delta + mu*m')   (the paper's) */
    DIPACO_OPT_MOMENTUM = 1, /* m' = mu*m + Delta; theta' = theta - lr*m'                (heavy ball)  */
    DIPACO_OPT_SGD = 2,      /* theta' = theta - lr*Delta; momentum left as it is (lr = 1: averaging)   */
    DIPACO_OPT_ADAM = 3      /* Adam family, configured by dipaco_set_adam                              */
};

/* what the path buffers hold on entry, for dipaco_set_input_kind */
enum {
    DIPACO_INPUT_COPIES = 0,   /* each path's copy x_i of its modules: Delta = sum c_i (theta - x_i)  */
    DIPACO_INPUT_GRADIENTS = 1 /* each path's gradient g_i of its modules: Delta = sum c_i g_i         */
};

/* kernel selection for dipaco_set_kernel */
enum {
    DIPACO_KERNEL_AUTO = 0,   /* bulk-copy (TMA) pipeline, one element per thread for the few elements
                                 before and after its range                                            */
    DIPACO_KERNEL_VECTOR = 1, /* 128-bit register loads/stores on whole steps, one element per thread
                                 for the rest                                                         */
    DIPACO_KERNEL_SCALAR = 2  /* one element per thread everywhere                                    */
};
/*
 * Alignment.  Nothing has to be aligned beyond its element size.  Path copies may start at any
 * element boundary, each at its own, and level sizes may be odd (modules and slots then start
 * inside 16-byte units): the bulk-copy and the vector kernel each have a variant that loads the
 * aligned 16-byte units around the data and writes realigned units, at 0.91-0.95 of the speed of
 * fully aligned buffers (bulk-copy kernel).  They need theta, momentum (and the second moment) to
 * sit at the same place within a 16-byte unit, which holds whenever these arrays are allocated the
 * same way; otherwise the module falls back to one element per thread.
 */

/*
 * Build a context for one module grid (Algorithm 1, "Require" lines; Section 2.2 notation).
 *   num_levels         L >= 1
 *   modules_per_level  host [L], K_l >= 1
 *   level_numel        host [L], N_l >= 0
 *   num_paths          P >= 1; any set of paths, not only the full product (Section 2.6.2)
 *   path_to_module     host [P*L] row-major, entry (i,l) in [0,K_l); a module no path uses is
 *                      allowed and never touched (Section 2.6.1: any sharing pattern)
 *   path_weights       host [P] raw weights >= 0, finite (Section 2.7), or NULL = uniform
 *   outer_lr, outer_momentum   finite; the paper uses 0.7 and 0.9
 *   path_dtype         DIPACO_F32 or DIPACO_BF16
 *   chunk_paths        0 = all path copies are resident at once; c > 0 = copies are presented
 *                      in chunks of c consecutive path ids (Section 3.3, online averaging)
 *   device             CUDA device ordinal, or -1 for a plan-only context (no CUDA call is made;
 *                      only the dipaco_plan_* queries work, everything else returns ENODEV)
 * All host arrays are copied.  Synchronous.
 */
int dipaco_create(dipaco_ctx **out, int32_t num_levels, const int32_t *modules_per_level,
                  const int64_t *level_numel, int32_t num_paths, const int32_t *path_to_module,
                  const float *path_weights, float outer_lr, float outer_momentum,
                  int32_t path_dtype, int32_t chunk_paths, int32_t device);

/*
 * One outer synchronisation of every module, in place (Algorithm 1, outer loop, plus re-dispatch).
 *   theta, momentum  device, fp32, layout above; in/out
 *   path_ptrs        HOST array [P] of DEVICE pointers, one per path copy; in/out
 *   reported         HOST [P], nonzero = path i reported; NULL = all reported
 *   cuda_stream      a cudaStream_t (0 = default stream)
 * With chunk_paths = 0 this is one fused pass; otherwise the library walks the chunks in
 * ascending order over the same device pointers, one launch per chunk, carrying fp32 partial
 * sums; the launch that sees a module's last reporting path finishes the module and writes
 * cast(theta') into all of its paths.  A call with the same settings, buffers and mask as the
 * previous one on this context reuses that call's plan and device tables: it only launches
 * kernels (no upload, no allocation, no synchronisation), so it may be recorded in a CUDA graph
 * by stream capture once one ordinary call has planned it.  Replaying the graph is then the
 * cheapest way to repeat a small synchronisation (2x2 grid: 5.5 us per replayed call against
 * 8.2 us per launched call).  Any dipaco_set_* call, another mask or other buffers make the next
 * call plan and upload again, which must not happen during capture.
 */
int dipaco_outer_sync(dipaco_ctx *ctx, float *theta, float *momentum, void *const *path_ptrs,
                      const uint8_t *reported, void *cuda_stream);

/*
 * Incremental form of the same operation for callers that hold only one chunk of path copies
 * on the device at a time (Section 3.3, "Online Parameter Gradient Averaging": each checkpoint
 * is added to a partial sum as it arrives).  Requires chunk_paths > 0.  Chunk c covers path ids
 * [c*chunk_paths, min(P, (c+1)*chunk_paths)).
 *   begin      fixes theta, momentum, the mask and the stream for this round.
 *   accumulate chunk_index must be 0,1,2,... in order; chunk_ptrs is a HOST array of the
 *              chunk's DEVICE pointers.  Adds the chunk's reporting copies to the partial sums;
 *              a module whose last reporting path lies in this chunk is updated right away and
 *              written into this chunk's copies.
 *   writeback  after every chunk has been accumulated, any order: fills every slot of the
 *              chunk's copies with cast(theta') (the contents of chunk_ptrs are not read, so the
 *              buffers may be fresh).
 *   end        checks that every chunk was accumulated and returns the context to idle.
 * With bf16 copies the first begin on a context allocates a scratch of 2 bytes per module
 * parameter: the finishing passes store cast(theta') there and the write-back launches read it
 * instead of fp32 theta'.  If that allocation fails the write-back reads theta' (same results).
 */
int dipaco_sync_begin(dipaco_ctx *ctx, float *theta, float *momentum, const uint8_t *reported,
                      void *cuda_stream);
int dipaco_sync_accumulate(dipaco_ctx *ctx, int32_t chunk_index, void *const *chunk_ptrs);
int dipaco_sync_writeback(dipaco_ctx *ctx, int32_t chunk_index, void *const *chunk_ptrs);
int dipaco_sync_end(dipaco_ctx *ctx);

/*
 * The same synchronisation for state that lives in HOST memory (checkpoints that do not fit
 * on the device; Section 3.3: the executor loads checkpoints and averages them as they come):
 * theta, momentum [module params] and the P path copies are host buffers (pinned memory gives
 * full copy speed).  The work is streamed through the device slab by slab: an element range of
 * one module together with that range of every reporting copy is uploaded, reduced, updated and
 * cast in one fused pass, and the result is copied back into theta, momentum and the slot of
 * every path of the module while the next slab is already being uploaded.  Device staging is
 * bounded by the size of chunk_paths path copies (> 0 required) plus theta and momentum.  Paths
 * that did not report are not uploaded.  Path copies that lie equally spaced in host memory
 * (rows of one allocation) are moved with one strided copy per slab instead of one per path.
 * By default a pool of host threads fans each module's result out to its paths
 * (dipaco_set_host_threads).  Results are bitwise those of dipaco_outer_sync.  Synchronous: returns when all host buffers
 * hold the result, and on an error only after every copy it started has finished.
 */
int dipaco_outer_sync_host(dipaco_ctx *ctx, float *theta_host, float *momentum_host,
                           void *const *path_ptrs_host, const uint8_t *reported,
                           void *cuda_stream);

/* Replace the raw per-path weights (host [P], or NULL = uniform).  Section 2.7. */
int dipaco_set_weights(dipaco_ctx *ctx, const float *path_weights);

/*
 * Outer gradient norm rescaling (Section 2.7): the finished outer gradient of module (l,e) is
 * multiplied by module_scale[(l,e)] before the optimiser step, Delta <- s * Delta.  host
 * [sum_l K_l], level-major, finite; NULL = no rescaling.  The paper rescales by the square root
 * of the number of paths through the module; the factor itself (sqrt(P) or its inverse) is the
 * caller's to supply.  A factor of exactly 1 leaves the result bit-identical.
 */
int dipaco_set_module_scale(dipaco_ctx *ctx, const float *module_scale);

/*
 * Levels that take no part in the exchange (Section 4.2: in the models with path-specific
 * modules some blocks stay local to their path): host [L], 0 = theta, momentum and every copy
 * of the level's modules are left untouched; NULL = every level is synchronised.
 */
int dipaco_set_level_sync(dipaco_ctx *ctx, const uint8_t *level_sync);

/*
 * Outer optimiser (Section 2.5: Nesterov momentum is the paper's choice; other optimisers of the
 * federated family fit the same scheme).  DIPACO_OPT_*; the default is Nesterov.
 */
int dipaco_set_optimizer(dipaco_ctx *ctx, int32_t optimizer);

/*
 * Adam-family optimiser.  It covers the adaptive federated optimisers that Section 2.5 names as
 * alternatives (step = 0: no bias correction, eps plays the role of their adaptivity constant)
 * and the AdamW of the fully synchronous ablation of Section 4.5 (step = t >= 1: bias-corrected,
 * decoupled weight decay).  With Delta the module's outer gradient, the `momentum` argument of
 * the sync calls as first moment m and second_moment as v:
 *     m' = b1*m + (1-b1)*Delta        v' = b2*v + (1-b2)*Delta^2
 *     theta' = theta*(1 - lr*weight_decay) - lr * (m'/c1) / (sqrt(v'/c2) + eps)
 *     c1 = 1 - b1^step, c2 = 1 - b2^step   (both 1 when step = 0)
 * second_moment: device, fp32, same layout as theta, caller-owned, in/out.  0 <= b1, b2 < 1,
 * eps >= 0.  Selects DIPACO_OPT_ADAM; call again to advance `step`.  The outer_momentum given at
 * create is not used.  second_moment lives where theta lives: a device array for
 * dipaco_outer_sync and the chunk API, a host array for dipaco_outer_sync_host.
 */
int dipaco_set_adam(dipaco_ctx *ctx, float *second_moment, float beta1, float beta2, float eps,
                    float weight_decay, int32_t step);

/*
 * What the path buffers hold on entry (DIPACO_INPUT_*).  With gradients the reduction is the
 * module-by-module gradient aggregation of Section 4.5; the buffers are still overwritten with
 * cast(theta') on exit, so after the call every path holds the new parameters of its modules.
 */
int dipaco_set_input_kind(dipaco_ctx *ctx, int32_t input_kind);

/*
 * Sharded executor (Section 3.3, "Sharded Outer Optimization Executor": modules, and the
 * parameters inside a module, are independent, so the update can be split over executors with no
 * exchange between them).  This context then owns slab shard_index of shard_count of EVERY
 * module (equal element ranges cut at multiples of 8192 elements; the last shard takes the
 * remainder) and touches nothing else: theta, momentum and the path copies outside its slabs are
 * neither read nor written.  Pointers and layouts stay those of the whole problem, so S contexts
 * (one per GPU, each holding at least its slabs at the usual offsets) together perform exactly
 * the unsharded update, bit for bit.  Default: shard 0 of 1.
 */
int dipaco_set_shard(dipaco_ctx *ctx, int32_t shard_index, int32_t shard_count);

/*
 * The same partition for executors that hold ONLY their slab (Section 3.3: each executor of the
 * sharded outer optimiser owns a part of the parameters and the matching part of every
 * checkpoint).  Every module of level l has N_l elements, so shard s of S owns the same element
 * range [begin_l, end_l) of every module of that level; dipaco_plan_shard returns it (host only,
 * works on plan-only contexts).  Ranges are cut at multiples of 8192 elements, the last shard
 * takes the remainder; over s = 0..S-1 they tile [0, N_l) exactly once.
 */
int dipaco_plan_shard(const dipaco_ctx *ctx, int32_t shard_index, int32_t shard_count, int32_t level,
                      int64_t *begin, int64_t *end);

/*
 * A context for shard shard_index of shard_count of the problem that `whole` describes, in the
 * compact layout: the shard is itself a module grid with the same levels, modules, paths and
 * weights and with N_l replaced by end_l - begin_l.  Its theta, momentum (and second moment)
 * hold, module after module, elements [begin_l, end_l) of each module; its path copies hold,
 * level after level, elements [begin_l, end_l) of the path's slot: each executor allocates 1/S
 * of everything and no pointer to the rest is ever needed.  Every entry point works on it as on
 * any context, and the S results, put back side by side, are bit for bit the unsharded update:
 * no exchange between executors (elements are independent).  The new context copies the
 * weights, module scales, level flags, learning rate, momentum, optimiser, input kind, chunk
 * size, kernel choice and tuning of `whole` as they are at the time of the call (`whole` may be
 * plan-only and may be destroyed afterwards); the Adam family must be selected on the shard
 * itself with dipaco_set_adam, because it needs the shard's own second-moment array.
 * device: CUDA device of this executor, or -1 for plan only.
 */
int dipaco_create_shard(dipaco_ctx **out, const dipaco_ctx *whole, int32_t shard_index,
                        int32_t shard_count, int32_t device);

/* Choose the kernel family (DIPACO_KERNEL_*); all families give bitwise identical results. */
int dipaco_set_kernel(dipaco_ctx *ctx, int32_t kernel);

/*
 * Tuning of the bulk-copy kernel: persistent CTAs per SM (1..8), pipeline depth in tiles (2..32),
 * 16-byte units of path data per compute thread and tile (1, 2 or 4; the tile is
 * 256 threads * units * 16 bytes) and the number of theta/momentum/result tile buffers (2..4;
 * more of them help modules with few contributors).  0 keeps a value.  A depth that does not fit
 * the shared memory of the chosen layout is rejected with DIPACO_EINVAL and nothing changes;
 * result buffers beyond two are dropped at launch while they would leave the ring shallower than a
 * launch of that mix of modules needs (10 stages when most elements have 8 or more contributors,
 * 6 otherwise).  A launch that stages more fp32 tiles per buffer than the layout was accepted
 * for (the second moment of an Adam-family optimiser selected later) falls back to the next
 * smaller tile that fits; results do not depend on any of this.
 */
int dipaco_set_tuning(dipaco_ctx *ctx, int32_t ctas_per_sm, int32_t stages,
                      int32_t units_per_thread, int32_t io_slots);

/*
 * Tuning of the bulk-copy kernel's dynamic scheduling: a launch is cut into work items (runs of
 * tiles of one module) that the persistent CTAs draw from a counter.  An item moves at most
 * max_item_bytes of traffic (default 2 MiB) and a launch is cut into at least items_per_cta
 * items per CTA (default 64) so that the CTAs finish together.  0 keeps a value.  Results do not
 * depend on the cut.
 */
int dipaco_set_work_items(dipaco_ctx *ctx, int64_t max_item_bytes, int32_t items_per_cta);

/*
 * Tuning of dipaco_outer_sync_host: the most bytes of path data that one streamed unit stages
 * on the device in each direction (0 = the default, 512 MiB; always at least one tile of every
 * copy of the module, at most 1/6 of chunk_paths path copies).  The download of a unit cannot
 * start before the unit is uploaded and reduced, so a call takes about one unit's transfer time
 * longer than the PCIe transfer itself: smaller units shorten that, larger ones mean fewer and
 * larger copies.
 */
int dipaco_set_host_unit_bytes(dipaco_ctx *ctx, int64_t bytes);

/*
 * Host threads of dipaco_outer_sync_host.  Every path of a module receives the same
 * cast(theta'), so with threads > 0 each streamed piece of it is downloaded once, into a pinned
 * buffer of the library, and `threads` host threads copy it into the slot of every path while
 * later pieces are still being uploaded: PCIe carries one copy per module instead of one per
 * path.  The threads belong to the context (created by the first call that needs them, joined
 * by dipaco_destroy) and sleep between calls.  0 = no host threads: the device writes one copy
 * per path and all of them are downloaded.  -1 = the default (half the hardware threads, at
 * most 4: more of them compete with the uploads for host memory bandwidth).  Results are
 * identical either way.
 */
int dipaco_set_host_threads(dipaco_ctx *ctx, int32_t threads);

/*
 * Synchronise the context's last stream and report what the kernels recorded: DIPACO_OK, or
 * DIPACO_ETIMEOUT if a bounded wait gave up, or DIPACO_ECUDA.  Clears the recorded status.
 *
 * Every wait inside the kernels is bounded (4 s).  A kernel whose wait runs out records a code
 * in the context's error word and ends in an orderly way (copies in flight are waited for); the
 * results of that call are undefined.  The error is sticky on the device: every later launch on
 * the context sees the error word set and does nothing at all (buffers untouched, status of the
 * entry point still DIPACO_OK since launches are asynchronous) until this function has been
 * called; it returns DIPACO_ETIMEOUT once, re-arms the context (error word and work counters
 * back to zero) and from then on calls work again.
 */
int dipaco_device_status(dipaco_ctx *ctx);

/*
 * Diagnostic: make a bounded wait run out on purpose, harmlessly.  Launches one warp on the
 * given stream whose first thread waits at most limit_ns (1 .. 1e9) on a barrier that nothing
 * will complete; no copy is in flight and no buffer of the caller is involved.  When the wait
 * gives up the kernel leaves what a pipeline kernel that gave up leaves: a code in the error
 * word and a work counter that is not back at zero.  Afterwards the context behaves as after a
 * real time-out (see dipaco_device_status).  Lets an application or a test check its handling of
 * DIPACO_ETIMEOUT.  The paper has no counterpart.
 */
int dipaco_selftest_wait_expiry(dipaco_ctx *ctx, int64_t limit_ns, void *cuda_stream);

/* Number of kernels this context has launched so far. */
int64_t dipaco_launch_count(const dipaco_ctx *ctx);

/*
 * Plan queries (host only; work on plan-only contexts too).  They expose the host-side
 * decisions: the contributor set of a module under a mask and the normalised coefficients.
 *   members / contributors  out, capacity num_paths each; ascending path ids
 *   coeff                   out, capacity num_paths; c_i as the kernels use them (fp32)
 *   will_update             out; 0 when no path reports or the total weight is zero
 * Any out pointer may be NULL.
 */
int dipaco_plan_module(const dipaco_ctx *ctx, int32_t level, int32_t module,
                       const uint8_t *reported, int32_t *num_members, int32_t *members,
                       int32_t *num_contributors, int32_t *contributors, float *coeff,
                       int32_t *will_update);
/* Offsets (in elements) of module (level, module) in theta and of the level in a path copy. */
int dipaco_plan_offsets(const dipaco_ctx *ctx, int32_t level, int32_t module,
                        int64_t *theta_offset, int64_t *path_offset, int64_t *numel);
/* Number of chunks (1 when chunk_paths = 0) and fp32 elements of partial-sum scratch. */
int dipaco_plan_chunks(const dipaco_ctx *ctx, int32_t *num_chunks, int64_t *scratch_elems);

/*
 * Bytes that one dipaco_outer_sync on this context moves through device memory by
 * construction (every read and write of theta, momentum, partial sums and path copies, summed
 * over its launches), and the number of launches (tail launches not counted).  For a resident
 * context this is the algorithmic minimum; for a chunked one it includes the partial-sum traffic.
 */
int dipaco_plan_traffic(const dipaco_ctx *ctx, const uint8_t *reported, int64_t *bytes,
                        int32_t *launches);

/*
 * The split of the resident-mode launch over num_ctas persistent CTAs in tiles of `tile`
 * elements (all pointers assumed aligned): CTA b processes segments
 * [cta_first[b], cta_first[b+1]); segment s covers elements [seg_begin[s], seg_end[s]) of
 * module (seg_level[s], seg_module[s]).  Arrays have `capacity` entries (cta_first: num_ctas+1).
 * Returns the number of segments (>= 0), or a negative status (EINVAL also when capacity is
 * too small).
 */
int dipaco_plan_split(const dipaco_ctx *ctx, const uint8_t *reported, int32_t num_ctas, int64_t tile,
                      int32_t capacity, int32_t *seg_level, int32_t *seg_module, int64_t *seg_begin,
                      int64_t *seg_end, int32_t *cta_first);

int dipaco_destroy(dipaco_ctx *ctx);

/*
 * Synchronise ONE module without allocating anything.  (The paper has no counterpart for this
 * entry point; it exists for the sake of its callers.)
 *
 * Who needs it: code that is not allowed to touch the device allocator.  Examples are a process
 * that has handed all device memory to a pool of its own at start-up, so that a later cudaMalloc
 * simply fails, and a latency-critical loop that cannot accept the device-wide synchronisation
 * that cudaMalloc and cudaFree imply.  Such callers cannot use dipaco_create (it allocates
 * tables, and in chunked mode the partial-sum scratch).  This function takes everything as
 * arguments, passes the per-chunk tables inside the kernel arguments and keeps the partial sums
 * in a static device array that is part of the library image.  It calls no cudaMalloc, cudaFree,
 * cudaMallocHost or any other allocating routine, on the device or on the host heap.
 *
 * What it computes: the same result, bit for bit, as dipaco_outer_sync on a grid with a single
 * level and a single module shared by num_paths paths, walked in chunks of chunk_paths.
 *   theta, momentum   device, fp32 [numel]; in/out
 *   numel             0 <= numel <= DIPACO_STATIC_MAX_NUMEL (4 Mi parameters = 16 MiB of partial
 *                     sums); larger sizes are refused with DIPACO_ELIMIT and nothing is launched
 *   num_paths         >= 1
 *   copy_ptrs         HOST array [num_paths] of DEVICE pointers, each a copy of the module
 *                     ([numel] of path_dtype); in/out, every copy is overwritten with cast(theta')
 *   path_weights      HOST [num_paths] raw weights >= 0 or NULL = uniform
 *   reported          HOST [num_paths], nonzero = reported, or NULL = all
 *   chunk_paths       1..32 copies per chunk
 *   device            CUDA device that owns all the buffers; made current during the call
 *   cuda_stream       stream the kernels are launched on (asynchronous)
 *
 * The static array: 16 MiB per GPU.  It is part of the library's CUDA module, so the CUDA runtime
 * reserves it when it loads that module on a GPU: with lazy module loading (the default) that is
 * the first call of this function on the device, with eager loading the creation of the context.
 * From then on the GPU holds the 16 MiB until the process exits, whether or not this function is
 * called again.  The first call on a device (any numel >= 1) is therefore the set-up call: make
 * it while the device still has room for the module (a caller that gives all device memory to
 * its own pool makes it before that), and before any stream capture begins; if the module cannot
 * be loaded it returns DIPACO_ENOMEM (or DIPACO_ECUDA), launches nothing and leaves no CUDA error
 * pending.  Every call looks the array's device address up again (cudaGetSymbolAddress: no
 * allocation once the module is loaded).  All calls on one device share the array and it keeps
 * whatever the last call left in it: each call starts its sums from zero in the kernel, so stale
 * contents are never read, but two calls that overlap on the GPU (different streams, or
 * different host threads) race on it and must be serialised by the caller.
 */
#define DIPACO_STATIC_MAX_NUMEL (4 * 1024 * 1024)
int dipaco_module_sync_static(float *theta, float *momentum, int64_t numel, int32_t num_paths,
                              void *const *copy_ptrs, const float *path_weights,
                              const uint8_t *reported, float outer_lr, float outer_momentum,
                              int32_t path_dtype, int32_t chunk_paths, int32_t device,
                              void *cuda_stream);

const char *dipaco_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DIPACO_H */
