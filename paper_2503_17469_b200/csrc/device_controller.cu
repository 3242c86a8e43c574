// The proportional batch-size controller as a one-warp kernel (getBsz of Algorithm 1 for all K
// workers + the global-batch rule, Eq. 6a/6b/7/8), and the ring-kernel instantiations that read
// the weights it leaves in device memory.
//
// Lane k owns worker k.  Every floating-point step is a single correctly rounded IEEE double
// operation written as an intrinsic (__dadd_rn, __dmul_rn, __ddiv_rn: never contracted into a
// multiply-add), and the one sum that depends on order (the mean compute time) is taken by
// every lane in ascending k, so the integers that come out are the host controller's, bit for
// bit.  After the single rounding step everything is integer arithmetic on warp votes and
// shuffles.
#include <cuda_runtime.h>

#include "device_controller.h"
#include "dispatch.h"
#include "tma_kernels.cuh"

namespace omni {
namespace {

struct CtlConst {
    int K, B, b_min, b_max, mode;
    unsigned flags;
    double deadband, alpha;
};

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ long long warp_sum(long long x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(kFull, x, o);
    return x;
}
__device__ __forceinline__ long long warp_min(long long x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long y = __shfl_xor_sync(kFull, x, o);
        x = y < x ? y : x;
    }
    return x;
}

// Sum of one value per worker in ascending worker order, the same in every lane.
__device__ __forceinline__ double ordered_worker_sum(double x, int K)
{
    double total = 0.0;
#pragma unroll
    for (int j = 0; j < OMNI_MAX_K; ++j) {
        const double xj = __shfl_sync(kFull, x, j);
        if (j < K) total = __dadd_rn(total, xj);
    }
    return total;
}

// getBsz without the rounding step: Eq. 6b, dead-band (Eq. 7), bounds.
__device__ __forceinline__ double get_bsz_real(double bd, double s, double tbar, const CtlConst &cc)
{
    const double lo = double(cc.b_min), hi = double(cc.b_max);
    const double throughput = __ddiv_rn(bd, s);
    const double error = __dsub_rn(s, tbar);
    const double target = __dsub_rn(bd, __dmul_rn(throughput, error));
    const double rel = fabs(__ddiv_rn(__dsub_rn(target, bd), target));
    double chosen = bd;
    if (rel >= cc.deadband) chosen = target < lo ? lo : target > hi ? hi : target;
    return chosen;
}

// The one rounding step: half up, kept inside the bounds.
__device__ __forceinline__ int32_t to_integer_batch(double chosen, const CtlConst &cc)
{
    const double lo = double(cc.b_min), hi = double(cc.b_max);
    double r = floor(__dadd_rn(chosen, 0.5));
    r = r < lo ? lo : r;
    r = hi < r ? hi : r;
    return int32_t(r);
}

// EWMA of the compute time; the first sample seeds it.
__device__ __forceinline__ double smoothed(double t, double prev, int32_t seen, const CtlConst &cc)
{
    if (!seen) return t;
    return __dadd_rn(__dmul_rn(cc.alpha, t), __dmul_rn(__dsub_rn(1.0, cc.alpha), prev));
}

__global__ void __launch_bounds__(32) rebatch_kernel(DeviceCtl *c, const CtlConst cc, const double *measured, int32_t *new_b)
{
    const int k = threadIdx.x;
    const bool on = k < cc.K;

    // Launched with programmatic stream serialization: the step that follows may take its SMs and
    // set up while this warp works, and nothing is read here before the previous launch (a step
    // that read the weights, or whatever produced the measurements) has finished.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // a measurement that is not a positive finite number fails the call; nothing changes
    // all of this lane's state is fetched at once (one memory latency instead of three in a row)
    const double m = on ? measured[k] : 1.0;
    const int32_t b = on ? c->batch[k] : 1;
    const int32_t seen = on ? c->seen[k] : 0;
    const double prev = on ? c->time[k] : 0.0;
    if (__any_sync(kFull, on && !(isfinite(m) && m > 0.0))) {
        if (k == 0) atomicCAS(&c->status, 0, int(OMNI_ERR_BAD_MEASUREMENT));
        return;
    }
    const double bd = double(b);

    // Eq. 6a read backwards (t = b / T), then the EWMA of the compute time
    const double t = (cc.flags & OMNI_INPUT_IS_TIME) ? m : __ddiv_rn(bd, m);
    const double s = smoothed(t, prev, seen, cc);

    // mean compute time, summed in ascending k by every lane
    const double tbar = __ddiv_rn(ordered_worker_sum(s, cc.K), double(cc.K));

    // getBsz: Eq. 6b, dead-band (Eq. 7), bounds, one rounding to an integer (half up)
    int32_t n = 0;
    double chosen = on ? get_bsz_real(bd, s, tbar, cc) : 0.0;
    if (cc.mode == OMNI_BSP && (cc.flags & OMNI_CONSERVE_MULTIPLICATIVE)) {
        // the other reading of the sentence after Eq. 8: renormalise the real-valued results to the
        // global batch before rounding (their sum in ascending k by every lane, as on the host)
        const double csum = ordered_worker_sum(chosen, cc.K);
        if (on) chosen = __ddiv_rn(__dmul_rn(chosen, double(cc.B)), csum);
    }
    if (on) n = to_integer_batch(chosen, cc);

    // Eq. 8 on integers with bounds: whole rounds of one unit per movable worker, then the last
    // partial round to the largest batches (lowest index first among equals)
    if (cc.mode == OMNI_BSP) {
        long long gap = (long long)cc.B - warp_sum(on ? n : 0);
        for (int pass = 0; gap != 0; ++pass) {
            const int dir = gap > 0 ? 1 : -1;
            const int wall = dir > 0 ? cc.b_max : cc.b_min;
            const long long room_k = on ? (long long)(wall - n) * dir : 0;   // units until worker k is pinned
            const bool movable = room_k > 0;
            const unsigned members = __ballot_sync(kFull, movable);
            const int count = __popc(members);
            if (count == 0 || pass > 2 * OMNI_MAX_K + 2) {
                if (k == 0) atomicCAS(&c->status, 0, int(OMNI_ERR_INFEASIBLE));
                return;
            }
            const long long room = warp_min(movable ? room_k : (long long)0x7fffffffffffffffLL);
            const long long need = gap * dir;
            const long long per = need / count;
            const long long rounds = room < per ? room : per;
            if (rounds > 0) {
                if (movable) n += int32_t(dir * rounds);
                gap -= dir * rounds * count;
                continue;
            }
            int rank = 0;   // movable workers that come before this one: larger batch, or equal batch and lower index
            for (int j = 0; j < 32; ++j) {
                const int32_t nj = __shfl_sync(kFull, n, j);
                if (((members >> j) & 1u) && (nj > n || (nj == n && j < k))) ++rank;
            }
            if (movable && rank < need) n += dir;
            gap = 0;
        }
    }

    // commit, then the weights of Eq. 4b for the step that follows
    const long long sum_b = warp_sum(on ? n : 0);
    if (on) {
        c->batch[k] = n;
        c->time[k] = s;
        c->seen[k] = 1;
        if (new_b) new_b[k] = n;
        const float lam = __double2float_rn((cc.flags & OMNI_UNSCALED_MEAN) ? __ddiv_rn(1.0, double(cc.K))
                                                                  : __ddiv_rn(double(n), double(sum_b)));
        c->lam[k] = lam;
    }
    if (k == 0) c->rebatches += 1u;     // (the sum of the weights is taken on the host when the state is read back)
}

// evalBsz of Algorithm 2 on the device copy: one worker reports the batch it ran and its
// measurement (a device value); the server stores both and, once every worker has an entry,
// re-evaluates getBsz for all K entries against their mean time (no global-batch rule).  Same
// operations in the same order as the host controller's report.
__global__ void __launch_bounds__(32) report_kernel(DeviceCtl *c, const CtlConst cc, int worker, int32_t b_used,
                                                    const double *measured, int32_t *new_b_k)
{
    const int k = threadIdx.x;
    const bool on = k < cc.K;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const double m = *measured;
    int32_t b = on ? c->batch[k] : 1;
    int32_t seen = on ? c->seen[k] : 1;
    double s = on ? c->time[k] : 0.0;
    if (!(isfinite(m) && m > 0.0)) {      // the same value in every lane: the whole warp leaves, nothing changes
        if (k == 0) atomicCAS(&c->status, 0, int(OMNI_ERR_BAD_MEASUREMENT));
        return;
    }
    if (k == worker) {                    // wrkB[k] = b, wrkTime[k] = smoothed compute time
        const double t = (cc.flags & OMNI_INPUT_IS_TIME) ? m : __ddiv_rn(double(b_used), m);
        s = smoothed(t, s, seen, cc);
        seen = 1;
        b = b_used;
    }
    const bool all = __all_sync(kFull, seen != 0);
    int32_t n = b;
    if (all) {
        const double tbar = __ddiv_rn(ordered_worker_sum(s, cc.K), double(cc.K));
        if (on) n = to_integer_batch(get_bsz_real(double(b), s, tbar, cc), cc);
    }
    if (on) {
        c->batch[k] = n;
        c->time[k] = s;
        c->seen[k] = seen;
    }
    if (k == worker && new_b_k) *new_b_k = all ? n : b_used;
}

template <typename G, int K> KernelInfo devlam_info()
{
    constexpr TmaShape sh = tma_shape<G>(K);
    return {reinterpret_cast<KernelFn>(&bsp_tma_kernel<G, K, sh.tile, sh.stages, sh.consumer_warps, false, true>),
            (sh.consumer_warps + 1) * 32, 1, (unsigned long long)sh.tile, tma_smem_bytes<G>(K), true};
}

template <typename G, int K> KernelInfo devlam_short_info()
{
    constexpr TmaShape sh = tma_short_shape<G>(K);
    return {reinterpret_cast<KernelFn>(&bsp_tma_kernel<G, K, sh.tile, sh.stages, sh.consumer_warps, false, true>),
            (sh.consumer_warps + 1) * 32, 1, (unsigned long long)sh.tile, tma_ring_bytes(sh, K, int(sizeof(G))), true};
}

template <typename G> KernelInfo devlam_short_for(int K)
{
    switch (K) {
#define OMNI_CASE(k) case k: return devlam_short_info<G, k>();
        OMNI_FOR_EACH_K(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

template <typename G> KernelInfo devlam_for(int K)
{
    switch (K) {
#define OMNI_CASE(k) case k: return devlam_info<G, k>();
        OMNI_FOR_EACH_K(OMNI_CASE)
#undef OMNI_CASE
    }
    return {};
}

}  // namespace

KernelInfo bulk_devlam_kernel(int dtype, int K)
{
    return dtype == OMNI_BF16 ? devlam_for<__nv_bfloat16>(K) : devlam_for<float>(K);
}

KernelInfo bulk_devlam_short_kernel(int dtype, int K)
{
    return dtype == OMNI_BF16 ? devlam_short_for<__nv_bfloat16>(K) : devlam_short_for<float>(K);
}

int launch_device_report(DeviceCtl *ctl, const omni_config &cfg, int32_t worker, int32_t b_used, const double *measured_dev,
                         int32_t *new_b_dev, void *stream)
{
    const CtlConst cc{cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.mode, cfg.flags, cfg.deadband, cfg.ewma_alpha};
    cudaLaunchConfig_t cfgl = {};
    cfgl.gridDim = dim3(1);
    cfgl.blockDim = dim3(32);
    cfgl.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfgl.attrs = attr;
    cfgl.numAttrs = 1;
    return int(cudaLaunchKernelEx(&cfgl, report_kernel, ctl, cc, int(worker), b_used, measured_dev, new_b_dev));
}

int launch_device_rebatch(DeviceCtl *ctl, const omni_config &cfg, const double *measured_dev, int32_t *new_b_dev,
                          void *stream)
{
    const CtlConst cc{cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.mode, cfg.flags, cfg.deadband, cfg.ewma_alpha};
    cudaLaunchConfig_t cfgl = {};
    cfgl.gridDim = dim3(1);
    cfgl.blockDim = dim3(32);
    cfgl.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfgl.attrs = attr;
    cfgl.numAttrs = 1;
    return int(cudaLaunchKernelEx(&cfgl, rebatch_kernel, ctl, cc, measured_dev, new_b_dev));
}

}  // namespace omni
