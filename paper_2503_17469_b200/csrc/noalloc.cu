// omni_aggregate_bsp_noalloc: the synchronous fused step for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they run a step: code
// that runs inside another framework's memory-pool callback or while that framework holds its
// allocator lock, services that start with the whole device memory already handed out to a
// pool, and real-time loops that forbid anything that may synchronise the device (cudaMalloc
// and cudaFree may).  The regular entry point allocates a small workspace the first time a
// context launches a kernel; this one never allocates.  The kernel's scratch -- one squared-norm
// partial per CTA -- lives in a fixed array in device memory that is part of the library image,
// so every GPU that loads the library carries these ~19 KB until the process exits.
//
// Consequences the caller has to know (also stated in omni.h):
//   - the array is shared by every call on that device and keeps the last call's contents;
//     nothing in it has to start at zero (a launch overwrites every cell that is read after
//     it), but two calls whose kernels overlap on the GPU (different streams) race on it;
//   - the first call on each device looks up the array's device address; make that first call
//     outside any stream capture;
//   - sizes are bounded (OMNI_NOALLOC_MAX_BUCKETS, OMNI_NOALLOC_MAX_ELEMENTS).
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>

#include "dispatch.h"
#include "kernels.cuh"

namespace omni {
namespace {

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is
// not a device address and must never be passed to a kernel as is.
static __device__ __align__(256) unsigned long long noalloc_scratch[(sizeof(Workspace) + 7) / 8];

constexpr int kMaxDevices = 64;
Workspace *g_scratch_addr[kMaxDevices] = {};  // device address of noalloc_scratch, per device
int g_sm_count[kMaxDevices] = {};
int g_grid[kMaxDevices][2][2][OMNI_MAX_K + 1] = {};  // [device][dtype][256-bit][K]: persistent grid, 0 = not asked yet

// Once per device, with that device current: resolve the device address of the scratch array.
cudaError_t scratch_for_current_device(Workspace **out, int *sms)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, noalloc_scratch);
        if (e != cudaSuccess) return e;
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        g_sm_count[dev] = n;
        g_scratch_addr[dev] = static_cast<Workspace *>(ptr);
    }
    *out = g_scratch_addr[dev];
    *sms = g_sm_count[dev];
    return cudaSuccess;
}

bool is_aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace
}  // namespace omni

using namespace omni;

extern "C" int omni_aggregate_bsp_noalloc(int32_t K, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                                          const int32_t *b, uint32_t flags, float lr, float momentum,
                                          float weight_decay, double *grad_sqnorm_dev, void *stream)
{
    if (K < 1 || K > OMNI_MAX_K) return OMNI_ERR_BAD_K;
    if (!b || (n_buckets > 0 && !buckets)) return OMNI_ERR_NULL;
    if (n_buckets < 0 || (grad_dtype != OMNI_F32 && grad_dtype != OMNI_BF16) || !std::isfinite(momentum))
        return OMNI_ERR_BAD_CONFIG;
    if (flags & ~uint32_t(OMNI_UNSCALED_MEAN)) return OMNI_ERR_BAD_CONFIG;   // no other flag means anything here
    int64_t total_b = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] < 1) return OMNI_ERR_BAD_BATCH;
        total_b += b[k];
    }
    int live = 0;
    unsigned long long elems = 0;
    bool wide = true;
    for (int i = 0; i < n_buckets; ++i) {
        const omni_bucket &bk = buckets[i];
        if (bk.n == 0) continue;
        if (!bk.param || !bk.grads) return OMNI_ERR_NULL;
        if (momentum != 0.0f && !bk.momentum) return OMNI_ERR_BAD_CONFIG;
        if (!is_aligned(bk.param, 16) || !is_aligned(bk.momentum, 16) || !is_aligned(bk.param_lp, 16)) return OMNI_ERR_ALIGN;
        wide = wide && is_aligned(bk.param, 32) && is_aligned(bk.momentum, 32) && is_aligned(bk.param_lp, 32);
        for (int k = 0; k < K; ++k) {
            if (!bk.grads[k]) return OMNI_ERR_NULL;
            if (!is_aligned(bk.grads[k], 16)) return OMNI_ERR_ALIGN;
            wide = wide && is_aligned(bk.grads[k], 32);
        }
        if (bk.n > OMNI_NOALLOC_MAX_ELEMENTS || elems + bk.n > OMNI_NOALLOC_MAX_ELEMENTS) return OMNI_ERR_TOO_LARGE;
        elems += bk.n;
        if (++live > OMNI_NOALLOC_MAX_BUCKETS) return OMNI_ERR_TOO_LARGE;
    }
    if (grad_sqnorm_dev && !is_aligned(grad_sqnorm_dev, 8)) return OMNI_ERR_ALIGN;

    Workspace *ws = nullptr;
    int sms = 0;
    if (scratch_for_current_device(&ws, &sms) != cudaSuccess) return OMNI_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    const KernelInfo pk = bsp_kernel(grad_dtype, K, wide);   // the register-staged synchronous kernel
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return OMNI_ERR_CUDA;
    // persistent grid of this kernel on this device, asked of the runtime once and kept
    int &cached = g_grid[dev][grad_dtype][wide ? 1 : 0][K];
    if (cached == 0) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pk.fn, pk.threads, 0) != cudaSuccess) return OMNI_ERR_CUDA;
        if (per_sm < 1) per_sm = 1;
        if (pk.ctas_per_sm > 0 && per_sm > pk.ctas_per_sm) per_sm = pk.ctas_per_sm;
        cached = sms * per_sm > kMaxGrid ? kMaxGrid : sms * per_sm;
    }
    int grid = cached;

    BspParams p;
    std::memset(&p, 0, sizeof p);
    unsigned long long tiles = 0;
    int nb = 0;
    for (int i = 0; i < n_buckets; ++i) {
        const omni_bucket &bk = buckets[i];
        if (bk.n == 0) continue;
        p.bk[nb] = {static_cast<float *>(bk.param), static_cast<float *>(bk.momentum),
                    static_cast<__nv_bfloat16 *>(bk.param_lp), bk.n, tiles};
        for (int k = 0; k < K; ++k) p.g[nb][k] = bk.grads[k];
        tiles += (bk.n + pk.tile - 1) / pk.tile;
        ++nb;
    }
    for (int k = 0; k < K; ++k)
        p.lam[k] = float((flags & OMNI_UNSCALED_MEAN) ? 1.0 / double(K) : double(b[k]) / double(total_b));
    p.lr = lr; p.mu = momentum; p.wd = weight_decay;
    p.nb = nb;
    p.accumulate = 0;
    p.tiles = tiles;
    p.ws = ws;
    if (tiles < (unsigned long long)grid) grid = tiles < 1 ? 1 : int(tiles);

    // The array keeps whatever the previous call left.  Nothing in it has to start at zero: every
    // CTA of this launch overwrites its own partial-sum slot (p.accumulate == 0), and the sum
    // below reads exactly the slots this launch wrote.
    void *args[] = {&p};
    if (cudaLaunchKernel(pk.fn, dim3(grid), dim3(pk.threads), args, 0, s) != cudaSuccess) return OMNI_ERR_CUDA;
    if (grad_sqnorm_dev && launch_sqnorm_finalize(ws, grid, grad_sqnorm_dev, stream) != 0) return OMNI_ERR_CUDA;
    return OMNI_OK;
}
