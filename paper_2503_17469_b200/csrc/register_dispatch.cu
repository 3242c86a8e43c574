// Instantiations of the register-staged kernels for every worker count, queue length, gradient
// type and vector width, with the launch geometry that goes with each.
#include "dispatch.h"
#include "kernels.cuh"

namespace omni {
namespace {

template <typename G, int K, bool WIDE> KernelInfo bsp_info()
{
    constexpr Shape sh = bsp_shape<G>(K);
    return {reinterpret_cast<KernelFn>(&bsp_fused_kernel<G, K, sh.threads, sh.chunks, WIDE>), sh.threads,
            sh.ctas_per_sm, (unsigned long long)sh.threads * Geo<G, WIDE>::E * sh.chunks};
}
template <typename G, bool WIDE> KernelInfo bsp_kernel_for(int K)
{
    switch (K) {
#define OMNI_CASE(k) case k: return bsp_info<G, k, WIDE>();
        OMNI_FOR_EACH_K(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

// Batched asynchronous apply, M = arrivals in the batch; launch shape as the synchronous kernel with K = M.
template <typename G, int M, bool WIDE> KernelInfo seq_info()
{
    constexpr Shape sh = bsp_shape<G>(M);
    return {reinterpret_cast<KernelFn>(&asp_batch_kernel<G, M, sh.threads, sh.chunks, WIDE>), sh.threads,
            sh.ctas_per_sm, (unsigned long long)sh.threads * Geo<G, WIDE>::E * sh.chunks};
}
template <typename G, bool WIDE> KernelInfo seq_kernel_for(int M)
{
    switch (M) {
#define OMNI_CASE(k) case k: return seq_info<G, k, WIDE>();
        OMNI_FOR_EACH_QUEUE(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

template <typename G, bool WIDE> KernelInfo overwrite_info()
{
    return {reinterpret_cast<KernelFn>(&asp_overwrite_kernel<G, kAspThreads, kAspChunks, WIDE>), kAspThreads,
            asp_ctas_per_sm(false), (unsigned long long)kAspThreads * Geo<G, WIDE>::E * kAspChunks};
}

template <typename G, bool WIDE> KernelInfo asp_info(bool momentum)
{
    return {reinterpret_cast<KernelFn>(&asp_apply_kernel<G, kAspThreads, kAspChunks, WIDE>), kAspThreads,
            asp_ctas_per_sm(momentum), (unsigned long long)kAspThreads * Geo<G, WIDE>::E * kAspChunks};
}

}  // namespace

KernelInfo bsp_kernel(int dtype, int K, bool wide)
{
    if (dtype == OMNI_BF16) return wide ? bsp_kernel_for<__nv_bfloat16, true>(K) : bsp_kernel_for<__nv_bfloat16, false>(K);
    return wide ? bsp_kernel_for<float, true>(K) : bsp_kernel_for<float, false>(K);
}

KernelInfo seq_kernel(int dtype, int M, bool wide)
{
    if (dtype == OMNI_BF16) return wide ? seq_kernel_for<__nv_bfloat16, true>(M) : seq_kernel_for<__nv_bfloat16, false>(M);
    return wide ? seq_kernel_for<float, true>(M) : seq_kernel_for<float, false>(M);
}

KernelInfo overwrite_kernel(int dtype, bool wide)
{
    if (dtype == OMNI_BF16) return wide ? overwrite_info<__nv_bfloat16, true>() : overwrite_info<__nv_bfloat16, false>();
    return wide ? overwrite_info<float, true>() : overwrite_info<float, false>();
}

KernelInfo asp_kernel(int dtype, bool wide, bool momentum)
{
    if (dtype == OMNI_BF16) return wide ? asp_info<__nv_bfloat16, true>(momentum) : asp_info<__nv_bfloat16, false>(momentum);
    return wide ? asp_info<float, true>(momentum) : asp_info<float, false>(momentum);
}

}  // namespace omni
