// Parameter-range sharding for one rank per GPU: which elements of a bucket a rank owns.
// Host arithmetic only; the step on the owned range is the ordinary fused kernel.
#include "../../include/omni.h"

extern "C" int omni_shard_range(uint64_t n, int32_t world, int32_t rank, uint64_t *begin, uint64_t *count)
{
    if (!begin || !count) return OMNI_ERR_NULL;
    if (world < 1 || rank < 0 || rank >= world) return OMNI_ERR_BAD_CONFIG;
    const uint64_t units = (n + OMNI_SHARD_UNIT - 1) / OMNI_SHARD_UNIT;
    // whole units dealt out contiguously; the first (units mod world) ranks take one more
    const uint64_t q = units / uint64_t(world), r = units % uint64_t(world), me = uint64_t(rank);
    const uint64_t first = me * q + (me < r ? me : r);
    const uint64_t mine = q + (me < r ? 1 : 0);
    uint64_t lo = first * OMNI_SHARD_UNIT, hi = (first + mine) * OMNI_SHARD_UNIT;
    if (lo > n) lo = n;
    if (hi > n) hi = n;
    *begin = lo;
    *count = hi - lo;
    return OMNI_OK;
}
