// Kernel selection shared by the translation units of the library (internal).
#pragma once

namespace omni {

using KernelFn = const void *;

// A kernel instantiation with the launch geometry that goes with it.
struct KernelInfo {
    KernelFn fn = nullptr;
    int threads = 0;
    int ctas_per_sm = 0;          // wanted CTAs per SM (capped by what fits)
    unsigned long long tile = 0;  // elements per tile
    unsigned smem = 0;            // dynamic shared memory per CTA, bytes
};

// Bulk-copy ring variant of the synchronous step (bulk_dispatch.cu).
KernelInfo bulk_kernel(int dtype, int K);

}  // namespace omni
