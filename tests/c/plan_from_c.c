/* A C99 caller of the library: proves that include/dipaco.h compiles as C and that the ABI needs
 * nothing but plain pointers and sizes.  Uses a plan-only context (no device), so it runs anywhere. */
#include <stdio.h>
#include <string.h>

#include "dipaco.h"

int main(void)
{
    /* the 2x2 toy mixture: one shared module, then two levels of two modules each */
    const int32_t modules_per_level[3] = {1, 2, 2};
    const int64_t level_numel[3] = {16, 64, 64};
    const int32_t table[4 * 3] = {0, 0, 0, 0, 0, 1, 0, 1, 0, 0, 1, 1};
    const float weights[4] = {1.0f, 3.0f, 2.0f, 2.0f};
    const uint8_t reported[4] = {1, 1, 0, 1};
    dipaco_ctx *ctx = NULL;
    int rc = dipaco_create(&ctx, 3, modules_per_level, level_numel, 4, table, weights, 0.7f, 0.9f,
                           DIPACO_BF16, 2, -1);
    if (rc != DIPACO_OK || !ctx) { printf("create failed: %s\n", dipaco_strerror(rc)); return 1; }

    int32_t members[4], contributors[4], n_members = 0, n_contributors = 0, will_update = 0;
    float coeff[4];
    /* level 3, module b: paths 2 and 4 (ids 1 and 3); both reported, weights 3 and 2 */
    rc = dipaco_plan_module(ctx, 2, 1, reported, &n_members, members, &n_contributors, contributors,
                            coeff, &will_update);
    if (rc != DIPACO_OK || n_members != 2 || members[0] != 1 || members[1] != 3 ||
        n_contributors != 2 || !will_update || coeff[0] != 0.6f || coeff[1] != 0.4f) {
        printf("plan_module mismatch\n");
        return 1;
    }
    /* level 2, module b: paths 3 and 4 (ids 2 and 3); only id 3 reported */
    rc = dipaco_plan_module(ctx, 1, 1, reported, &n_members, members, &n_contributors, contributors,
                            coeff, &will_update);
    if (rc != DIPACO_OK || n_members != 2 || n_contributors != 1 || contributors[0] != 3 || coeff[0] != 1.0f) {
        printf("plan_module (masked) mismatch\n");
        return 1;
    }
    int64_t theta_off = 0, path_off = 0, numel = 0;
    rc = dipaco_plan_offsets(ctx, 2, 1, &theta_off, &path_off, &numel);
    if (rc != DIPACO_OK || theta_off != 16 + 128 + 64 || path_off != 80 || numel != 64) {
        printf("plan_offsets mismatch\n");
        return 1;
    }
    int32_t chunks = 0;
    int64_t scratch = 0;
    if (dipaco_plan_chunks(ctx, &chunks, &scratch) != DIPACO_OK || chunks != 2 || scratch != 16 + 2 * 64) {
        printf("plan_chunks mismatch\n");
        return 1;
    }
    /* compute entry points refuse a context without a device */
    float dummy = 0.0f;
    void *ptrs[4] = {&dummy, &dummy, &dummy, &dummy};
    if (dipaco_outer_sync(ctx, &dummy, &dummy, ptrs, NULL, NULL) != DIPACO_ENODEV) {
        printf("outer_sync should have refused\n");
        return 1;
    }
    /* two executors that each hold half of every module (Section 3.3): slab bounds and the
     * plan-only context of executor 1 of a grid large enough to be cut at the 8192 grain */
    {
        const int64_t big_numel[3] = {40000, 16384, 100};
        dipaco_ctx *whole = NULL, *half = NULL;
        int64_t a = -1, b = -1, n = -1;
        if (dipaco_create(&whole, 3, modules_per_level, big_numel, 4, table, weights, 0.7f, 0.9f,
                          DIPACO_BF16, 0, -1) != DIPACO_OK)
            return 1;
        if (dipaco_plan_shard(whole, 0, 2, 0, &a, &b) != DIPACO_OK || a != 0 || b != 16384 ||
            dipaco_plan_shard(whole, 1, 2, 0, &a, &b) != DIPACO_OK || a != 16384 || b != 40000 ||
            dipaco_plan_shard(whole, 1, 2, 2, &a, &b) != DIPACO_OK || a != 0 || b != 100 ||
            dipaco_plan_shard(whole, 2, 2, 0, &a, &b) != DIPACO_EINVAL) {
            printf("plan_shard mismatch\n");
            return 1;
        }
        if (dipaco_create_shard(&half, whole, 1, 2, -1) != DIPACO_OK || !half ||
            dipaco_plan_offsets(half, 0, 0, NULL, NULL, &n) != DIPACO_OK || n != 40000 - 16384 ||
            dipaco_plan_offsets(half, 1, 1, &theta_off, &path_off, &n) != DIPACO_OK || n != 8192 ||
            theta_off != (40000 - 16384) + 8192 || path_off != 40000 - 16384) {
            printf("create_shard mismatch\n");
            return 1;
        }
        if (dipaco_destroy(whole) != DIPACO_OK || dipaco_destroy(half) != DIPACO_OK) return 1;
    }
    if (strcmp(dipaco_strerror(DIPACO_ENODEV), "unknown status") == 0) return 1;
    if (dipaco_destroy(ctx) != DIPACO_OK) return 1;
    printf("ok\n");
    return 0;
}
