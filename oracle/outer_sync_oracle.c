/*
 * CPU oracle for DiPaCo's module-wise outer synchronisation.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or
 * constant with the CUDA path and must never be called from it.
 *
 * What it computes (DiPaCo, Algorithm 1, the "outer optimization" loop over
 * levels and experts, together with the re-dispatch of the updated module to
 * every path, Section 2.5 / 2.6; weights from Section 2.7 "Loss reweighing"):
 *
 * For every level l and module e, with
 *     S(l,e) = { paths i : path_to_module[i][l] == e }          (Section 2.6.1)
 *     R(l,e) = { i in S(l,e) : reported[i] }                    (Section 2.6.2)
 *   1. W = sum_{i in R} w_i   (w_i = 1 without weights).  If R is empty or
 *      W == 0 the module keeps theta and momentum unchanged; go to step 4.
 *   2. Delta[k] = sum_{i in R} (w_i / W) * (theta[k] - x_i[k])
 *      (Algorithm 1, outer-gradient line; shard-size weights, Section 2.7).
 *   3. Nesterov momentum, gradient evaluated at the current point
 *      (Section 2.5 names the optimiser; supplementary "Additional Details"
 *      gives lr 0.7 and momentum 0.9):
 *          m'[k]     = mu * m[k] + Delta[k]
 *          theta'[k] = theta[k] - lr * (Delta[k] + mu * m'[k])
 *   4. every path of S(l,e), reporting or not, receives cast(theta')
 *      (Section 2.5: the new global vector is re-dispatched to all workers).
 *
 * Options of Sections 2.5, 2.7, 4.2 and 4.5, off by default:
 *   - module_scale: the outer gradient of module (l,e) is multiplied by s(l,e) before the
 *     optimiser step, Delta <- s * Delta ("Outer Gradient Norm Rescaling": the paper rescales
 *     by the square root of the number of paths through the module; the caller supplies s, so
 *     whether that means sqrt(P) or 1/sqrt(P) is the caller's reading).
 *   - level_sync: a level flagged 0 takes no part in the exchange (Section 4.2 keeps some
 *     blocks of the path-specific models local to their path): theta, momentum and every copy
 *     of its modules are left untouched.
 *
 *   - optimizer: Section 2.5 notes that other outer optimisers of the federated family fit the
 *     same scheme.  Besides Nesterov (0, the paper's choice) the oracle defines heavy-ball
 *     momentum (1): m' = mu*m + Delta, theta' = theta - lr*m'; and plain SGD (2):
 *     theta' = theta - lr*Delta with the momentum buffer left as it is (lr = 1 is plain
 *     averaging of the copies); and the Adam family (3), which covers both the adaptive
 *     federated optimiser the paper points to in Section 2.5 and the AdamW of its fully
 *     synchronous ablation (Section 4.5):
 *         m' = b1*m + (1-b1)*Delta          v' = b2*v + (1-b2)*Delta^2
 *         theta' = theta*(1 - lr*wd) - lr * (m'/c1) / (sqrt(v'/c2) + eps)
 *     with c1 = c2 = 1 and wd = 0 for the federated form, c1 = 1-b1^t, c2 = 1-b2^t for the
 *     bias-corrected form at step t.  m is the momentum array, v a second array.
 *   - input_kind: 1 = the path buffers hold gradients g_i of the path's copy instead of the
 *     copy itself (the synchronous ablation aggregates gradients module by module every step):
 *     Delta = sum_i alpha_i * g_i; the buffers are still overwritten with cast(theta').
 *
 * Arithmetic: steps 1-3 in double, theta' and m' rounded once to float;
 * a bf16 path copy receives round-to-nearest-even of that float.
 * Loop order: module, element, contributor (ascending path id).
 *
 * Parity pins (tests/test_oracle_pins.py): closed forms (identical deltas,
 * lr=1/mu=0 weighted mean, single path, empty module, geometric momentum
 * series), a library Nesterov step, exact rational brute force on tiny grids
 * with the contributor sets the paper states for its 2x2 figure.  The
 * readings of the paper that no number in the paper fixes (the Nesterov form
 * and the treatment of non-reporting paths) are pinned only by those closed
 * forms.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

static double widen_bf16(uint16_t h)
{
    uint32_t bits = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* float -> bf16, round to nearest, ties to even; NaN stays a quiet NaN */
static uint16_t narrow_bf16(float f)
{
    uint32_t bits;
    memcpy(&bits, &f, sizeof bits);
    if ((bits & 0x7fffffffu) > 0x7f800000u)
        return (uint16_t)((bits >> 16) | 0x0040u);
    uint32_t lower = bits & 0xffffu;
    uint32_t upper = bits >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u)))
        upper += 1u;
    return (uint16_t)upper;
}

static double read_copy(const void *buf, int dtype, int64_t idx)
{
    if (dtype == ORACLE_BF16)
        return widen_bf16(((const uint16_t *)buf)[idx]);
    return (double)((const float *)buf)[idx];
}

static void write_copy(void *buf, int dtype, int64_t idx, float v)
{
    if (dtype == ORACLE_BF16)
        ((uint16_t *)buf)[idx] = narrow_bf16(v);
    else
        ((float *)buf)[idx] = v;
}

/*
 * One outer synchronisation, in place.
 *
 *  num_levels          L
 *  modules_per_level   K_l, [L]
 *  level_numel         |B_l|, [L]; every module of level l has this many parameters
 *  num_paths           P
 *  path_to_module      [P*L] row-major, entry (i,l) in [0, K_l)
 *  path_weights        [P] raw non-negative weights (shard sizes) or NULL = uniform
 *  reported            [P] 1 = the path reported this round, or NULL = all reported
 *  theta, momentum     float, [sum_l K_l*|B_l|], ordered level, module, element
 *  path_ptrs           [P] pointers; copy i holds its L modules concatenated in level order
 *  num_threads         OpenMP threads for the element loop (elements are independent)
 *
 *  module_scale        [sum_l K_l] factor on each module's outer gradient, level-major, or NULL = 1
 *  level_sync          [L] 0 = leave the level untouched, or NULL = every level is synchronised
 *  optimizer           0 = Nesterov momentum, 1 = heavy-ball momentum, 2 = plain SGD, 3 = Adam family
 *  second_moment       float, same shape as theta; in/out (Adam family only, else NULL)
 *  adam                {b1, b2, eps, weight decay, c1, c2} (Adam family only, else NULL)
 *  input_kind          0 = path buffers hold copies of the modules, 1 = they hold gradients
 *
 * Returns 0, or -1 on an invalid argument.
 */
int oracle_outer_sync_ex(int32_t num_levels, const int32_t *modules_per_level,
                         const int64_t *level_numel, int32_t num_paths,
                         const int32_t *path_to_module, const float *path_weights,
                         const uint8_t *reported, double outer_lr, double outer_momentum,
                         int32_t path_dtype, float *theta, float *momentum,
                         void *const *path_ptrs, int32_t num_threads,
                         const double *module_scale, const uint8_t *level_sync, int32_t optimizer,
                         float *second_moment, const double *adam, int32_t input_kind)
{
    if (optimizer < 0 || optimizer > 3 || input_kind < 0 || input_kind > 1)
        return -1;
    if (optimizer == 3 && (!second_moment || !adam))
        return -1;
    if (num_levels < 1 || num_paths < 1 || !modules_per_level || !level_numel ||
        !path_to_module || !theta || !momentum || !path_ptrs)
        return -1;
    if (path_dtype != ORACLE_F32 && path_dtype != ORACLE_BF16)
        return -1;
    for (int32_t i = 0; i < num_paths; ++i)
        for (int32_t l = 0; l < num_levels; ++l) {
            int32_t e = path_to_module[(int64_t)i * num_levels + l];
            if (e < 0 || e >= modules_per_level[l])
                return -1;
        }
    if (num_threads < 1)
        num_threads = 1;
    (void)num_threads;

    int32_t *members = (int32_t *)malloc(sizeof(int32_t) * (size_t)num_paths);
    int32_t *reporters = (int32_t *)malloc(sizeof(int32_t) * (size_t)num_paths);
    double *alpha = (double *)malloc(sizeof(double) * (size_t)num_paths);
    if (!members || !reporters || !alpha) {
        free(members); free(reporters); free(alpha);
        return -1;
    }

    int64_t module_base = 0;  /* offset of module (l,e) inside theta / momentum */
    int64_t level_base = 0;   /* offset of level l inside one path copy */
    int32_t module_index = 0; /* level-major index of module (l,e) */
    for (int32_t l = 0; l < num_levels; ++l) {
        const int64_t n = level_numel[l];
        if (level_sync && !level_sync[l]) {  /* level not communicated: nothing is touched */
            module_base += n * modules_per_level[l];
            module_index += modules_per_level[l];
            level_base += n;
            continue;
        }
        for (int32_t e = 0; e < modules_per_level[l]; ++e, ++module_index) {
            const double scale = module_scale ? module_scale[module_index] : 1.0;
            /* S(l,e) and R(l,e) by a linear scan of the table, ascending path id */
            int32_t n_members = 0, n_reporters = 0;
            double total_weight = 0.0;
            for (int32_t i = 0; i < num_paths; ++i) {
                if (path_to_module[(int64_t)i * num_levels + l] != e)
                    continue;
                members[n_members++] = i;
                if (reported && !reported[i])
                    continue;
                reporters[n_reporters++] = i;
                total_weight += path_weights ? (double)path_weights[i] : 1.0;
            }
            const int update = (n_reporters > 0 && total_weight > 0.0);
            if (update)
                for (int32_t r = 0; r < n_reporters; ++r) {
                    double w = path_weights ? (double)path_weights[reporters[r]] : 1.0;
                    alpha[r] = w / total_weight;
                }

            float *th = theta + module_base;
            float *mo = momentum + module_base;
            float *v2 = second_moment ? second_moment + module_base : NULL;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(num_threads) if (num_threads > 1)
#endif
            for (int64_t k = 0; k < n; ++k) {
                float new_theta = th[k];
                if (update) {
                    const double t0 = (double)th[k];
                    double delta = 0.0;
                    for (int32_t r = 0; r < n_reporters; ++r) {
                        double x = read_copy(path_ptrs[reporters[r]], path_dtype, level_base + k);
                        delta += alpha[r] * (input_kind == 1 ? x : t0 - x);
                    }
                    delta *= scale;
                    double m1, t1;
                    if (optimizer == 0) {          /* Nesterov momentum */
                        m1 = outer_momentum * (double)mo[k] + delta;
                        t1 = t0 - outer_lr * (delta + outer_momentum * m1);
                    } else if (optimizer == 1) {   /* heavy-ball momentum */
                        m1 = outer_momentum * (double)mo[k] + delta;
                        t1 = t0 - outer_lr * m1;
                    } else if (optimizer == 2) {   /* plain SGD, momentum buffer untouched */
                        m1 = (double)mo[k];
                        t1 = t0 - outer_lr * delta;
                    } else {                       /* Adam family */
                        const double b1 = adam[0], b2 = adam[1], eps = adam[2], wd = adam[3];
                        const double c1 = adam[4], c2 = adam[5];
                        m1 = b1 * (double)mo[k] + (1.0 - b1) * delta;
                        const double v1 = b2 * (double)v2[k] + (1.0 - b2) * delta * delta;
                        t1 = t0 * (1.0 - outer_lr * wd) - outer_lr * (m1 / c1) / (sqrt(v1 / c2) + eps);
                        v2[k] = (float)v1;
                    }
                    mo[k] = (float)m1;
                    new_theta = (float)t1;
                    th[k] = new_theta;
                }
                for (int32_t s = 0; s < n_members; ++s)
                    write_copy(path_ptrs[members[s]], path_dtype, level_base + k, new_theta);
            }
            module_base += n;
        }
        level_base += n;
    }
    free(members); free(reporters); free(alpha);
    return 0;
}

int oracle_outer_sync(int32_t num_levels, const int32_t *modules_per_level,
                      const int64_t *level_numel, int32_t num_paths,
                      const int32_t *path_to_module, const float *path_weights,
                      const uint8_t *reported, double outer_lr, double outer_momentum,
                      int32_t path_dtype, float *theta, float *momentum,
                      void *const *path_ptrs, int32_t num_threads)
{
    return oracle_outer_sync_ex(num_levels, modules_per_level, level_numel, num_paths,
                                path_to_module, path_weights, reported, outer_lr, outer_momentum,
                                path_dtype, theta, momentum, path_ptrs, num_threads, NULL, NULL, 0, NULL, NULL,
                                0);
}

/* number of OpenMP threads the element loop can use on this host (1 without OpenMP) */
int32_t oracle_max_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}
