/* The library's C ABI used from plain C99 (no C++, no Python): the host controller on the
 * hand-derived case -- throughputs (1,2,4,8), B = 64, bounds (2,48), dead-band 10 % -- and the
 * shard ranges of a 1000-element bucket over three ranks.  Prints what the test compares. */
#include <stdio.h>

#include "omni.h"

int main(void)
{
    omni_config cfg;
    omni_ctx *ctx = NULL;
    const double T[4] = {1.0, 2.0, 4.0, 8.0};
    int32_t b[4], changed[4];
    int rc, step, k, rank;

    cfg.K = 4;
    cfg.global_batch = 64;
    cfg.b_min = 2;
    cfg.b_max = 48;
    cfg.deadband = 0.10;
    cfg.ewma_alpha = 1.0;
    cfg.mode = OMNI_BSP;
    cfg.flags = 0u;
    rc = omni_create(&cfg, &ctx);
    if (rc != OMNI_OK) {
        printf("create: %s\n", omni_strerror(rc));
        return 1;
    }
    for (step = 0; step < 4; ++step) {
        rc = omni_rebatch(ctx, T, b, changed);
        if (rc != OMNI_OK) {
            printf("rebatch: %s\n", omni_strerror(rc));
            return 1;
        }
        for (k = 0; k < 4; ++k) printf("%d%c", (int)b[k], k == 3 ? '\n' : ' ');
    }
    rc = omni_rebatch(ctx, NULL, b, changed);
    printf("%d %s\n", rc, omni_strerror(rc));
    omni_destroy(ctx);
    for (rank = 0; rank < 3; ++rank) {
        uint64_t begin, count;
        if (omni_shard_range(1000u, 3, rank, &begin, &count) != OMNI_OK) return 1;
        printf("%lu+%lu%c", (unsigned long)begin, (unsigned long)count, rank == 2 ? '\n' : ' ');
    }
    return 0;
}
