// Instantiations of the bulk-copy ring kernel for every K and both gradient types.
#include "dispatch.h"
#include "tma_kernels.cuh"

namespace omni {
namespace {

// Diagnostic: one thread waits, with a short limit, on an mbarrier that nothing will ever
// complete, then records the expiry in the status word exactly as the ring kernel does.  Lets a
// test (or an operator) see the bounded-wait path end to end without any kernel misbehaving.
__global__ void expire_wait_kernel(Workspace *ws, unsigned attempts)
{
    __shared__ __align__(8) unsigned long long never;
    if (threadIdx.x == 0) {
        mbar_init(&never, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        bool done = false;
        for (unsigned i = 0; i < attempts && !done; ++i) done = mbar_try_wait(&never, 0);
        if (!done) atomicExch(&ws->status, kStatusTimeout);
    }
}


__global__ void __launch_bounds__(32) sqnorm_finalize_kernel(const Workspace *ws, int slots, double *out)
{
    const double s = ordered_partial_sum(ws->partials, slots);
    if (threadIdx.x == 0) *out = s;
}

template <typename G, int K> KernelInfo bulk_info()
{
    constexpr TmaShape sh = tma_shape<G>(K);
    return {reinterpret_cast<KernelFn>(&bsp_tma_kernel<G, K, sh.tile, sh.stages, sh.consumer_warps>),
            (sh.consumer_warps + 1) * 32, 1, (unsigned long long)sh.tile, tma_smem_bytes<G>(K), true};
}

template <typename G> KernelInfo bulk_for(int K)
{
    switch (K) {
#define OMNI_CASE(k) case k: return bulk_info<G, k>();
        OMNI_FOR_EACH_K(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

// the same kernel in the shape for short launches (the very same instantiation where the shapes agree)
template <typename G, int K> KernelInfo bulk_short_info()
{
    constexpr TmaShape sh = tma_short_shape<G>(K);
    return {reinterpret_cast<KernelFn>(&bsp_tma_kernel<G, K, sh.tile, sh.stages, sh.consumer_warps>),
            (sh.consumer_warps + 1) * 32, 1, (unsigned long long)sh.tile, tma_ring_bytes(sh, K, int(sizeof(G))), true};
}

template <typename G> KernelInfo bulk_short_for(int K)
{
    switch (K) {
#define OMNI_CASE(k) case k: return bulk_short_info<G, k>();
        OMNI_FOR_EACH_K(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

template <typename G, int M> KernelInfo bulk_seq_info()
{
    constexpr TmaShape sh = tma_seq_shape<G>(M);
    return {reinterpret_cast<KernelFn>(&bsp_tma_kernel<G, M, sh.tile, sh.stages, sh.consumer_warps, true>),
            (sh.consumer_warps + 1) * 32, 1, (unsigned long long)sh.tile, tma_ring_bytes(sh, M, int(sizeof(G))), true};
}

template <typename G> KernelInfo bulk_seq_for(int M)
{
    switch (M) {
#define OMNI_CASE(k) case k: return bulk_seq_info<G, k>();
        OMNI_FOR_EACH_QUEUE(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

template <typename G> KernelInfo bulk_overwrite_info()
{
    constexpr TmaShape sh = tma_seq_shape<G>(1);
    return {reinterpret_cast<KernelFn>(&bsp_tma_kernel<G, 1, sh.tile, sh.stages, sh.consumer_warps, true, false, true>),
            (sh.consumer_warps + 1) * 32, 1, (unsigned long long)sh.tile, tma_ring_bytes(sh, 1, int(sizeof(G))), true};
}

}  // namespace

KernelInfo bulk_overwrite_kernel(int dtype)
{
    return dtype == OMNI_BF16 ? bulk_overwrite_info<__nv_bfloat16>() : bulk_overwrite_info<float>();
}

KernelInfo bulk_kernel(int dtype, int K) { return dtype == OMNI_BF16 ? bulk_for<__nv_bfloat16>(K) : bulk_for<float>(K); }
KernelInfo bulk_short_kernel(int dtype, int K)
{
    return dtype == OMNI_BF16 ? bulk_short_for<__nv_bfloat16>(K) : bulk_short_for<float>(K);
}
int short_launch_tiles_per_cta() { return kShortLaunchTilesPerCta; }
KernelInfo bulk_seq_kernel(int dtype, int M) { return dtype == OMNI_BF16 ? bulk_seq_for<__nv_bfloat16>(M) : bulk_seq_for<float>(M); }

int launch_sqnorm_finalize(void *workspace, int slots, double *out, void *stream)
{
    sqnorm_finalize_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const Workspace *>(workspace), slots, out);
    return int(cudaGetLastError());
}

int launch_expire_wait(void *workspace, unsigned attempts, void *stream)
{
    expire_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<Workspace *>(workspace), attempts);
    return int(cudaGetLastError());
}

bool bulk_preferred(int dtype, int streams)
{
    const TmaShape sh = dtype == OMNI_BF16 ? tma_shape<__nv_bfloat16>(streams) : tma_shape<float>(streams);
    return sh.tile * (dtype == OMNI_BF16 ? 2 : 4) >= 2048;
}

}  // namespace omni
