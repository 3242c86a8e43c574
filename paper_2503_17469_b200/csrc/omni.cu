// C ABI of the library: context, argument validation, weights, kernel launches.
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <new>

#include "controller.h"
#include "device_controller.h"
#include "dispatch.h"
#include "kernels.cuh"

namespace omni {

struct LaunchShape { int grid = 0; int block = 0; };  // grid == 0: not yet sized for this device

}  // namespace omni

struct omni_ctx {
    explicit omni_ctx(const omni_config &c) : ctl(c) {}
    omni::BatchController ctl;
    omni_stats tally{};
    omni::Workspace *ws = nullptr;   // device
    double *host_cell = nullptr;     // pinned, receives the squared norm
    int device = -1;
    int sm_count = 0;
    int last_cuda = 0;
    uint64_t launches = 0;
    unsigned sweep = 0;              // calls that walked the parameters so far (parity = sweep direction)
    int sq_slots = 0;                // per-CTA norm partials the last synchronous step left in the workspace
    omni::DeviceCtl *dctl = nullptr; // device copy of the controller (omni_ctl_to_device), or null
    omni::DeviceCtl dctl_stage{};    // host staging for its uploads and downloads
    omni::LaunchShape bsp_shape[2][2][OMNI_MAX_K + 1];  // [dtype][wide][K]
    omni::LaunchShape bulk_shape[2][OMNI_MAX_K + 1];    // [dtype][K], bulk-copy ring kernel
    omni::LaunchShape bulk_short_shape[2][OMNI_MAX_K + 1];  // [dtype][K], the same in its shape for short launches
    omni::LaunchShape bulk_seq_shape[2][OMNI_MAX_ASP_BATCH + 1];  // [dtype][M]
    omni::LaunchShape bulk_devlam_shape[2][OMNI_MAX_K + 1];       // [dtype][K], ring kernel with device-resident weights
    omni::LaunchShape bulk_devlam_short_shape[2][OMNI_MAX_K + 1]; // [dtype][K], the same in the short-launch shape
    omni::LaunchShape asp_shape[2][2][2];               // [dtype][wide][momentum]
    omni::LaunchShape overwrite_shape[2][2];            // [dtype][wide]
    omni::LaunchShape bulk_overwrite_shape[2];          // [dtype], ring kernel as push with overwrite
    omni::LaunchShape seq_shape[2][2][OMNI_MAX_ASP_BATCH + 1];  // [dtype][wide][M]
};

namespace omni {
namespace {

#define OMNI_CUDA(ctx, call)                         \
    do {                                             \
        const cudaError_t e_ = (call);               \
        if (e_ != cudaSuccess) {                     \
            (ctx)->last_cuda = int(e_);              \
            return OMNI_ERR_CUDA;                    \
        }                                            \
    } while (0)

// First kernel-launching call of a context: bind to the current device, allocate the workspace.
int ensure_device(omni_ctx *ctx)
{
    if (ctx->ws) {
        int cur = -1;
        OMNI_CUDA(ctx, cudaGetDevice(&cur));
        if (cur != ctx->device) return OMNI_ERR_BAD_CONFIG;
        return OMNI_OK;
    }
    int dev = -1;
    OMNI_CUDA(ctx, cudaGetDevice(&dev));
    OMNI_CUDA(ctx, cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dev));
    Workspace *ws = nullptr;
    OMNI_CUDA(ctx, cudaMalloc(&ws, sizeof(Workspace)));
    cudaError_t e = cudaMemset(ws, 0, sizeof(Workspace));
    if (e == cudaSuccess) e = cudaMallocHost(&ctx->host_cell, 2 * sizeof(double));
    if (e != cudaSuccess) {
        cudaFree(ws);
        ctx->last_cuda = int(e);
        return OMNI_ERR_CUDA;
    }
    *ctx->host_cell = 0.0;
    ctx->ws = ws;
    ctx->device = dev;
    return OMNI_OK;
}

// Persistent grid = SM count x CTAs per SM (the kernel's tuned figure, capped by what is resident
// at once and by the partial-sum slots).
int shape_for(omni_ctx *ctx, const KernelInfo &ki, LaunchShape &s)
{
    if (s.grid > 0) return OMNI_OK;
    int per_sm = 0;
    if (ki.smem > 0)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(ki.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, int(ki.smem)));
    OMNI_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ki.fn, ki.threads, ki.smem));
    if (per_sm < 1) per_sm = 1;
    if (ki.ctas_per_sm > 0 && per_sm > ki.ctas_per_sm) per_sm = ki.ctas_per_sm;
    int grid = ctx->sm_count * per_sm;
    if (grid > kMaxGrid) grid = kMaxGrid / ctx->sm_count * ctx->sm_count;
    s.grid = grid;
    s.block = ki.threads;
    return OMNI_OK;
}

// Kernel family for a call with this many gradient streams: the flags force one, otherwise the
// bulk-copy ring runs wherever its copies are large enough.
bool use_bulk(const omni_ctx *ctx, int dtype, int streams)
{
    const uint32_t f = ctx->ctl.config().flags;
    if (f & OMNI_NO_BULK_COPY) return false;
    if (f & OMNI_BULK_COPY) return true;
    return bulk_preferred(dtype, streams);
}

// Asynchronous applies take the same decision with the number of queued arrivals as stream count.
bool use_bulk_seq(const omni_ctx *ctx, int dtype, int m, bool /*momentum*/) { return use_bulk(ctx, dtype, m); }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned32(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// The 256-bit kernels need every buffer of every non-empty bucket on a 32-byte boundary.
bool all_aligned32(const omni_bucket *buckets, int32_t n_buckets, int k0, int k1)
{
    for (int i = 0; i < n_buckets; ++i) {
        const omni_bucket &b = buckets[i];
        if (b.n == 0) continue;
        if (!aligned32(b.param) || !aligned32(b.momentum) || !aligned32(b.param_lp)) return false;
        for (int k = k0; k < k1; ++k)
            if (!aligned32(b.grads[k])) return false;
    }
    return true;
}

// Checks shared by the synchronous and asynchronous entry points.  worker < 0: all K gradients.
int check_buckets(const omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t dtype, int worker,
                  float momentum)
{
    if (n_buckets < 0 || (dtype != OMNI_F32 && dtype != OMNI_BF16)) return OMNI_ERR_BAD_CONFIG;
    if (n_buckets > 0 && !buckets) return OMNI_ERR_NULL;
    if (!std::isfinite(momentum)) return OMNI_ERR_BAD_CONFIG;
    const int K = ctx->ctl.K();
    for (int i = 0; i < n_buckets; ++i) {
        const omni_bucket &b = buckets[i];
        if (b.n == 0) continue;
        if (!b.param || !b.grads) return OMNI_ERR_NULL;
        if (momentum != 0.0f && !b.momentum) return OMNI_ERR_BAD_CONFIG;
        if (!aligned16(b.param) || !aligned16(b.momentum) || !aligned16(b.param_lp)) return OMNI_ERR_ALIGN;
        for (int k = (worker < 0 ? 0 : worker); k < (worker < 0 ? K : worker + 1); ++k) {
            if (!b.grads[k]) return OMNI_ERR_NULL;
            if (!aligned16(b.grads[k])) return OMNI_ERR_ALIGN;
        }
    }
    return OMNI_OK;
}

int launch(omni_ctx *ctx, const KernelInfo &ki, int grid, void *params, cudaStream_t stream)
{
    void *args[] = {params};
    if (ki.dependent_launch) {
        // the ring kernels order themselves after the previous launch (see tma_kernels.cuh)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(ki.threads);
        cfg.dynamicSmemBytes = ki.smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        OMNI_CUDA(ctx, cudaLaunchKernelExC(&cfg, ki.fn, args));
        ctx->launches += 1;
        return OMNI_OK;
    }
    OMNI_CUDA(ctx, cudaLaunchKernel(ki.fn, dim3(grid), dim3(ki.threads), args, ki.smem, stream));
    ctx->launches += 1;
    return OMNI_OK;
}

// The squared norm of the last synchronous step: add its per-CTA partials up on the device.
int finalize_sqnorm(omni_ctx *ctx, cudaStream_t stream)
{
    if (ctx->sq_slots == 0) return OMNI_OK;
    const int e = launch_sqnorm_finalize(ctx->ws, ctx->sq_slots, &ctx->ws->sqnorm, stream);
    if (e != 0) {
        ctx->last_cuda = e;
        return OMNI_ERR_CUDA;
    }
    ctx->launches += 1;
    return OMNI_OK;
}

// Staleness bookkeeping of one asynchronous arrival (the paper defines no staleness-dependent
// factor, so tau is only tallied): histogram with an overflow bin, maximum, sum.
void tally_arrival(omni_ctx *ctx, int32_t tau)
{
    ctx->tally.arrivals += 1;
    ctx->tally.tau_hist[tau < OMNI_TAU_BINS - 1 ? tau : OMNI_TAU_BINS - 1] += 1;
    if (tau > ctx->tally.tau_max) ctx->tally.tau_max = tau;
    ctx->tally.tau_sum += uint64_t(tau);
}

// Eq. 4b: lambda_k = b_k / sum b, evaluated in double and rounded once to float.
double fill_weights(const omni_ctx *ctx, const int32_t *b, float *lam)
{
    const int K = ctx->ctl.K();
    int64_t total = 0;
    for (int k = 0; k < K; ++k) total += b[k];
    double wsum = 0.0;
    for (int k = 0; k < K; ++k) {
        const double l = (ctx->ctl.config().flags & OMNI_UNSCALED_MEAN) ? 1.0 / double(K) : double(b[k]) / double(total);
        lam[k] = float(l);
        wsum += double(lam[k]);
    }
    return wsum;
}

// lam: the K weights on the host (they travel as kernel parameters), or null with lam_dev: the
// weights in device memory, which only the ring kernel built for that reads.
int enqueue_bsp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t dtype, const float *lam,
                const float *lam_dev, float lr, float mu, float wd, cudaStream_t stream)
{
    const int K = ctx->ctl.K();
    const bool bulk = lam_dev || use_bulk(ctx, dtype, K);
    const bool wide = all_aligned32(buckets, n_buckets, 0, K);
    KernelInfo ki = lam_dev ? bulk_devlam_kernel(dtype, K) : bulk ? bulk_kernel(dtype, K) : bsp_kernel(dtype, K, wide);
    LaunchShape *shape_slot = lam_dev ? &ctx->bulk_devlam_shape[dtype][K]
                              : bulk  ? &ctx->bulk_shape[dtype][K]
                                      : &ctx->bsp_shape[dtype][wide][K];
    if (bulk) {
        // a launch of a few rounds per CTA takes the short-launch shape, as long as that still
        // gives every SM a tile
        const KernelInfo ks = lam_dev ? bulk_devlam_short_kernel(dtype, K) : bulk_short_kernel(dtype, K);
        unsigned long long regular_tiles = 0, short_tiles = 0;
        for (int i = 0; i < n_buckets; ++i) {
            regular_tiles += (buckets[i].n + ki.tile - 1) / ki.tile;
            short_tiles += (buckets[i].n + ks.tile - 1) / ks.tile;
        }
        // ... which pays when the larger tiles halve the number of fill-consume rounds exactly
        const unsigned long long sms = (unsigned long long)ctx->sm_count;
        const unsigned long long rounds = (regular_tiles + sms - 1) / sms, short_rounds = (short_tiles + sms - 1) / sms;
        if (ks.fn != ki.fn && short_tiles >= sms && rounds <= (unsigned long long)short_launch_tiles_per_cta() &&
            2 * short_rounds == rounds) {
            ki = ks;
            shape_slot = lam_dev ? &ctx->bulk_devlam_short_shape[dtype][K] : &ctx->bulk_short_shape[dtype][K];
        }
    }
    LaunchShape &shape = *shape_slot;
    int rc = shape_for(ctx, ki, shape);
    if (rc != OMNI_OK) return rc;
    const unsigned long long tile = ki.tile;

    BspParams p;
    int launched = 0, i = 0, slots = 0;
    while (i < n_buckets || launched == 0) {
        std::memset(&p, 0, sizeof p);
        unsigned long long tiles = 0;
        int nb = 0;
        for (; i < n_buckets && nb < kMaxBucketsPerLaunch; ++i) {
            const omni_bucket &b = buckets[i];
            if (b.n == 0) continue;
            p.bk[nb] = {static_cast<float *>(b.param), static_cast<float *>(b.momentum),
                        static_cast<__nv_bfloat16 *>(b.param_lp), b.n, tiles};
            for (int k = 0; k < K; ++k) p.g[nb][k] = b.grads[k];
            tiles += (b.n + tile - 1) / tile;
            ++nb;
        }
        // an empty call still runs one (empty) launch so that the squared norm reads 0
        for (int k = 0; k < K && lam; ++k) p.lam[k] = lam[k];
        p.lam_dev = lam_dev;
        p.lr = lr; p.mu = mu; p.wd = wd;
        p.nb = nb;
        p.accumulate = slots;
        p.reverse = int(ctx->sweep & 1u);
        p.tiles = tiles;
        p.ws = ctx->ws;
        const unsigned long long want = tiles < 1 ? 1 : tiles;
        const int grid = want < (unsigned long long)shape.grid ? int(want) : shape.grid;
        rc = launch(ctx, ki, grid, &p, stream);
        if (rc != OMNI_OK) return rc;
        if (grid > slots) slots = grid;
        ++launched;
    }
    ctx->sq_slots = slots;
    // Alternate the sweep direction from call to call: the parameters and momentum touched last
    // are the ones still in L2 (loaded and stored with evict-last priority), so the next call
    // starts where this one ended and finds part of them there instead of in DRAM.
    ctx->sweep += 1;
    return OMNI_OK;
}

}  // namespace
}  // namespace omni

using namespace omni;

extern "C" {

const char *omni_strerror(int s)
{
    switch (s) {
        case OMNI_OK: return "ok";
        case OMNI_ERR_NULL: return "a required pointer is NULL";
        case OMNI_ERR_BAD_K: return "K outside 1..32";
        case OMNI_ERR_BAD_WORKER: return "worker index out of range";
        case OMNI_ERR_BAD_BATCH: return "batch size < 1 or batch sizes do not sum to the global batch";
        case OMNI_ERR_INFEASIBLE: return "bounds cannot hold the global batch";
        case OMNI_ERR_BAD_MEASUREMENT: return "measurement not finite or not positive";
        case OMNI_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case OMNI_ERR_BAD_TAU: return "negative staleness";
        case OMNI_ERR_CUDA: return "CUDA call failed (see omni_last_cuda_error)";
        case OMNI_ERR_TIMEOUT: return "device-side wait ran out";
        case OMNI_ERR_BAD_CONFIG: return "invalid configuration or argument";
        case OMNI_ERR_TOO_LARGE: return "size beyond the stated maximum";
        case OMNI_ERR_NO_MEMORY: return "host memory allocation failed";
    }
    return "unknown status";
}

int omni_create(const omni_config *cfg, omni_ctx **out)
{
    if (!cfg || !out) return OMNI_ERR_NULL;
    const int rc = BatchController::validate(*cfg);
    if (rc != OMNI_OK) return rc;
    omni_ctx *ctx = new (std::nothrow) omni_ctx(*cfg);
    if (!ctx) return OMNI_ERR_NO_MEMORY;
    ctx->tally.tau_max = 0;
    *out = ctx;
    return OMNI_OK;
}

void omni_destroy(omni_ctx *ctx)
{
    if (!ctx) return;
    if (ctx->ws) cudaFree(ctx->ws);
    if (ctx->dctl) cudaFree(ctx->dctl);
    if (ctx->host_cell) cudaFreeHost(ctx->host_cell);
    delete ctx;
}

int omni_get_batches(const omni_ctx *ctx, int32_t *b)
{
    if (!ctx || !b) return OMNI_ERR_NULL;
    std::memcpy(b, ctx->ctl.batches(), sizeof(int32_t) * ctx->ctl.K());
    return OMNI_OK;
}

int omni_set_batches(omni_ctx *ctx, const int32_t *b)
{
    if (!ctx || !b) return OMNI_ERR_NULL;
    return ctx->ctl.set_batches(b);
}

// Controller state as a flat record for checkpoints: what re-batching needs to continue where it
// stopped (the paper's re-batching goes through a checkpoint of the training job).
namespace {
struct CtlRecord {
    uint32_t magic, version;
    int32_t K, global_batch;
    int32_t batch[OMNI_MAX_K];
    int32_t seen[OMNI_MAX_K];
    double time[OMNI_MAX_K];
};
constexpr uint32_t kCtlMagic = 0x4c544d4fu;   // "OMTL"
}  // namespace

int omni_ctl_export(const omni_ctx *ctx, void *record, uint64_t *size)
{
    if (!ctx || !size) return OMNI_ERR_NULL;
    const uint64_t have = *size;
    *size = sizeof(CtlRecord);
    if (!record) return OMNI_OK;                       // size query
    if (have < sizeof(CtlRecord)) return OMNI_ERR_TOO_LARGE;
    CtlRecord r{};
    r.magic = kCtlMagic;
    r.version = 1;
    r.K = ctx->ctl.K();
    r.global_batch = ctx->ctl.B();
    ctx->ctl.export_state(r.batch, r.time, r.seen);
    std::memcpy(record, &r, sizeof r);
    return OMNI_OK;
}

int omni_ctl_import(omni_ctx *ctx, const void *record, uint64_t size)
{
    if (!ctx || !record) return OMNI_ERR_NULL;
    if (size < sizeof(CtlRecord)) return OMNI_ERR_BAD_CONFIG;
    CtlRecord r;
    std::memcpy(&r, record, sizeof r);
    if (r.magic != kCtlMagic || r.version != 1 || r.K != ctx->ctl.K() || r.global_batch != ctx->ctl.B())
        return OMNI_ERR_BAD_CONFIG;
    for (int k = 0; k < r.K; ++k)
        if (r.seen[k] && !(std::isfinite(r.time[k]) && r.time[k] > 0.0)) return OMNI_ERR_BAD_MEASUREMENT;
    const int rc = ctx->ctl.set_batches(r.batch);      // validates b_k >= 1 and, in BSP mode, the sum
    if (rc != OMNI_OK) return rc;
    ctx->ctl.import_state(r.batch, r.time, r.seen);
    return OMNI_OK;
}

int omni_rebatch(omni_ctx *ctx, const double *measured, int32_t *new_b, int32_t *changed)
{
    if (!ctx || !measured || !new_b) return OMNI_ERR_NULL;
    return ctx->ctl.rebatch(measured, new_b, changed);
}

int omni_asp_report(omni_ctx *ctx, int32_t worker, int32_t b_used, double measured, int32_t *new_b_k)
{
    if (!ctx || !new_b_k) return OMNI_ERR_NULL;
    return ctx->ctl.report(worker, b_used, measured, new_b_k);
}

int omni_rebatch_static(omni_ctx *ctx, const double *capacity, int32_t *new_b)
{
    if (!ctx || !capacity || !new_b) return OMNI_ERR_NULL;
    return ctx->ctl.rebatch_static(capacity, new_b);
}

static int check_bsp_batches(const omni_ctx *ctx, const int32_t *b)
{
    int64_t total = 0;
    for (int k = 0; k < ctx->ctl.K(); ++k) {
        if (b[k] < 1) return OMNI_ERR_BAD_BATCH;
        total += b[k];
    }
    if (ctx->ctl.config().mode == OMNI_BSP && total != ctx->ctl.B()) return OMNI_ERR_BAD_BATCH;
    return OMNI_OK;
}

// m queued arrivals applied in one pass (m = 1: a single arrival), bulk-copy ring or registers.
static int enqueue_seq(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t dtype, int32_t m,
                       const int32_t *workers, const int32_t *b_used, float lr, float momentum, float weight_decay,
                       cudaStream_t stream)
{
    const bool bulk = use_bulk_seq(ctx, dtype, m, momentum != 0.0f);
    bool wide = true;
    for (int i = 0; i < m; ++i) wide = wide && all_aligned32(buckets, n_buckets, workers[i], workers[i] + 1);
    const KernelInfo ki = bulk ? bulk_seq_kernel(dtype, m) : seq_kernel(dtype, m, wide);
    LaunchShape &shape = bulk ? ctx->bulk_seq_shape[dtype][m] : ctx->seq_shape[dtype][wide][m];
    int rc = shape_for(ctx, ki, shape);
    if (rc != OMNI_OK) return rc;

    BspParams p;
    int i = 0;
    while (i < n_buckets) {
        std::memset(&p, 0, sizeof p);
        unsigned long long tiles = 0;
        int nb = 0;
        for (; i < n_buckets && nb < kMaxBucketsPerLaunch; ++i) {
            const omni_bucket &bk = buckets[i];
            if (bk.n == 0) continue;
            p.bk[nb] = {static_cast<float *>(bk.param), static_cast<float *>(bk.momentum),
                        static_cast<__nv_bfloat16 *>(bk.param_lp), bk.n, tiles};
            for (int a = 0; a < m; ++a) p.g[nb][a] = bk.grads[workers[a]];
            tiles += (bk.n + ki.tile - 1) / ki.tile;
            ++nb;
        }
        if (nb == 0) break;
        // Eq. 5b per arrival: eta = lr * b_used / B, in double, rounded once to float
        for (int a = 0; a < m; ++a)
            p.lam[a] = float((ctx->ctl.config().flags & OMNI_ASP_NO_LR_SCALE)
                                 ? double(lr)
                                 : double(lr) * double(b_used[a]) / double(ctx->ctl.B()));
        p.mu = momentum; p.wd = weight_decay;
        p.nb = nb;
        p.reverse = int(ctx->sweep & 1u);
        p.tiles = tiles;
        p.ws = ctx->ws;
        const int grid = tiles < (unsigned long long)shape.grid ? int(tiles) : shape.grid;
        rc = launch(ctx, ki, grid, &p, stream);
        if (rc != OMNI_OK) return rc;
    }
    ctx->sweep += 1;
    return OMNI_OK;
}

int omni_aggregate_bsp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                       const int32_t *b, float lr, float momentum, float weight_decay, void *stream)
{
    if (!ctx || !b) return OMNI_ERR_NULL;
    int rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, -1, momentum);
    if (rc != OMNI_OK) return rc;
    rc = check_bsp_batches(ctx, b);
    if (rc != OMNI_OK) return rc;
    rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    float lam[OMNI_MAX_K];
    const double wsum = fill_weights(ctx, b, lam);
    rc = enqueue_bsp(ctx, buckets, n_buckets, grad_dtype, lam, nullptr, lr, momentum, weight_decay,
                     static_cast<cudaStream_t>(stream));
    if (rc != OMNI_OK) return rc;
    ctx->tally.weight_sum = wsum;
    ctx->tally.steps += 1;
    return OMNI_OK;
}

int omni_step_bsp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                  const double *measured, float lr, float momentum, float weight_decay, int32_t *next_b,
                  int32_t *changed, void *stream)
{
    if (!ctx || !measured || !next_b) return OMNI_ERR_NULL;
    int rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, -1, momentum);
    if (rc != OMNI_OK) return rc;
    // the weights of this step come from the batches the gradients were computed with
    int32_t used[OMNI_MAX_K];
    std::memcpy(used, ctx->ctl.batches(), sizeof(int32_t) * ctx->ctl.K());
    // Re-batch first: it is host arithmetic, and a refused measurement leaves the controller as it
    // was, so nothing has been enqueued yet if it fails.  Keep what is needed to undo it should
    // the launch fail afterwards.
    int32_t old_b[OMNI_MAX_K], old_seen[OMNI_MAX_K];
    double old_t[OMNI_MAX_K];
    ctx->ctl.export_state(old_b, old_t, old_seen);
    rc = ctx->ctl.rebatch(measured, next_b, changed);
    if (rc != OMNI_OK) return rc;
    float lam[OMNI_MAX_K];
    const double wsum = fill_weights(ctx, used, lam);
    rc = ensure_device(ctx);
    if (rc == OMNI_OK)
        rc = enqueue_bsp(ctx, buckets, n_buckets, grad_dtype, lam, nullptr, lr, momentum, weight_decay,
                         static_cast<cudaStream_t>(stream));
    if (rc != OMNI_OK) {
        ctx->ctl.import_state(old_b, old_t, old_seen);   // undo the re-batch
        return rc;
    }
    ctx->tally.weight_sum = wsum;
    ctx->tally.steps += 1;
    return OMNI_OK;
}

int omni_aggregate_bsp_host(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                            const void *const *host_grads, const int32_t *b, float lr, float momentum,
                            float weight_decay, void *stream, double *grad_sqnorm)
{
    if (!ctx || !b || (n_buckets > 0 && !host_grads)) return OMNI_ERR_NULL;
    int rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, -1, momentum);
    if (rc != OMNI_OK) return rc;
    rc = check_bsp_batches(ctx, b);
    if (rc != OMNI_OK) return rc;
    const int K = ctx->ctl.K();
    for (int i = 0; i < n_buckets; ++i)
        for (int k = 0; k < K && buckets[i].n; ++k)
            if (!host_grads[size_t(i) * K + k]) return OMNI_ERR_NULL;
    rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esz = grad_dtype == OMNI_BF16 ? 2 : 4;
    for (int i = 0; i < n_buckets; ++i)
        for (int k = 0; k < K && buckets[i].n; ++k)
            OMNI_CUDA(ctx, cudaMemcpyAsync(const_cast<void *>(buckets[i].grads[k]), host_grads[size_t(i) * K + k],
                                           buckets[i].n * esz, cudaMemcpyHostToDevice, s));
    float lam[OMNI_MAX_K];
    const double wsum = fill_weights(ctx, b, lam);
    rc = enqueue_bsp(ctx, buckets, n_buckets, grad_dtype, lam, nullptr, lr, momentum, weight_decay, s);
    if (rc != OMNI_OK) return rc;
    ctx->tally.weight_sum = wsum;
    ctx->tally.steps += 1;
    rc = finalize_sqnorm(ctx, s);
    if (rc != OMNI_OK) return rc;
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->host_cell, &ctx->ws->sqnorm, sizeof(double), cudaMemcpyDeviceToHost, s));
    OMNI_CUDA(ctx, cudaStreamSynchronize(s));
    if (grad_sqnorm) *grad_sqnorm = *ctx->host_cell;
    return OMNI_OK;
}

int omni_apply_asp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                   int32_t worker, int32_t b_used, int32_t tau, float lr, float momentum, float weight_decay,
                   void *stream)
{
    if (!ctx) return OMNI_ERR_NULL;
    const int K = ctx->ctl.K();
    if (worker < 0 || worker >= K) return OMNI_ERR_BAD_WORKER;
    if (b_used < 1) return OMNI_ERR_BAD_BATCH;
    if (tau < 0) return OMNI_ERR_BAD_TAU;
    int rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, worker, momentum);
    if (rc != OMNI_OK) return rc;
    rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;

    // Eq. 5b: eta_k = eta * b_k / B, in double, rounded once to float
    const double eta_k = (ctx->ctl.config().flags & OMNI_ASP_NO_LR_SCALE)
                             ? double(lr)
                             : double(lr) * double(b_used) / double(ctx->ctl.B());
    if (use_bulk_seq(ctx, grad_dtype, 1, momentum != 0.0f)) {
        // the ring kernel in sequential mode with one arrival
        rc = enqueue_seq(ctx, buckets, n_buckets, grad_dtype, 1, &worker, &b_used, lr, momentum, weight_decay,
                         static_cast<cudaStream_t>(stream));
        if (rc != OMNI_OK) return rc;
        tally_arrival(ctx, tau);
        return OMNI_OK;
    }
    const bool wide = all_aligned32(buckets, n_buckets, worker, worker + 1);
    const KernelInfo ki = asp_kernel(grad_dtype, wide, momentum != 0.0f);
    LaunchShape &shape = ctx->asp_shape[grad_dtype][wide][momentum != 0.0f];
    rc = shape_for(ctx, ki, shape);
    if (rc != OMNI_OK) return rc;
    const unsigned long long tile = ki.tile;

    AspParams p;
    int i = 0;
    while (i < n_buckets) {
        std::memset(&p, 0, sizeof p);
        unsigned long long tiles = 0;
        int nb = 0;
        for (; i < n_buckets && nb < kMaxBucketsPerLaunch; ++i) {
            const omni_bucket &bk = buckets[i];
            if (bk.n == 0) continue;
            p.bk[nb] = {static_cast<float *>(bk.param), static_cast<float *>(bk.momentum),
                        static_cast<__nv_bfloat16 *>(bk.param_lp), bk.n, tiles};
            p.g[nb] = bk.grads[worker];
            tiles += (bk.n + tile - 1) / tile;
            ++nb;
        }
        if (nb == 0) break;
        p.eta = float(eta_k); p.mu = momentum; p.wd = weight_decay;
        p.nb = nb;
        p.tiles = tiles;
        const int grid = tiles < (unsigned long long)shape.grid ? int(tiles) : shape.grid;
        rc = launch(ctx, ki, grid, &p, static_cast<cudaStream_t>(stream));
        if (rc != OMNI_OK) return rc;
    }
    tally_arrival(ctx, tau);
    return OMNI_OK;
}

int omni_apply_asp_batch(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype, int32_t m,
                         const int32_t *workers, const int32_t *b_used, const int32_t *tau, float lr, float momentum,
                         float weight_decay, void *stream)
{
    if (!ctx || !workers || !b_used || !tau) return OMNI_ERR_NULL;
    if (m < 1 || m > OMNI_MAX_ASP_BATCH) return OMNI_ERR_TOO_LARGE;
    const int K = ctx->ctl.K();
    for (int i = 0; i < m; ++i) {
        if (workers[i] < 0 || workers[i] >= K) return OMNI_ERR_BAD_WORKER;
        if (b_used[i] < 1) return OMNI_ERR_BAD_BATCH;
        if (tau[i] < 0) return OMNI_ERR_BAD_TAU;
    }
    int rc = OMNI_OK;
    for (int i = 0; i < m && rc == OMNI_OK; ++i) rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, workers[i], momentum);
    if (rc != OMNI_OK) return rc;
    rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;

    rc = enqueue_seq(ctx, buckets, n_buckets, grad_dtype, m, workers, b_used, lr, momentum, weight_decay,
                     static_cast<cudaStream_t>(stream));
    if (rc != OMNI_OK) return rc;
    for (int a = 0; a < m; ++a) {
        tally_arrival(ctx, tau[a]);
    }
    return OMNI_OK;
}

int omni_asp_pull(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, void *const *snapshots, void *stream)
{
    if (!ctx || (n_buckets > 0 && (!buckets || !snapshots))) return OMNI_ERR_NULL;
    if (n_buckets < 0) return OMNI_ERR_BAD_CONFIG;
    for (int i = 0; i < n_buckets; ++i) {
        if (buckets[i].n == 0) continue;
        if (!buckets[i].param || !snapshots[i]) return OMNI_ERR_NULL;
        if (!aligned16(buckets[i].param) || !aligned16(snapshots[i])) return OMNI_ERR_ALIGN;
    }
    for (int i = 0; i < n_buckets; ++i)
        if (buckets[i].n)
            OMNI_CUDA(ctx, cudaMemcpyAsync(snapshots[i], buckets[i].param, buckets[i].n * sizeof(float),
                                           cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    return OMNI_OK;
}

// Algorithm 2's worker step + pushToPS (and, with write_back, the pullFromPS that follows it) in
// one launch: ring kernel by default, register kernel on a context that forces that family.
static int push_overwrite(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                          int32_t worker, int32_t b_used, int32_t tau, void *const *snapshots, bool write_back,
                          float lr, float weight_decay, void *stream)
{
    if (!ctx) return OMNI_ERR_NULL;
    const int K = ctx->ctl.K();
    if (worker < 0 || worker >= K) return OMNI_ERR_BAD_WORKER;
    if (b_used < 1) return OMNI_ERR_BAD_BATCH;
    if (tau < 0) return OMNI_ERR_BAD_TAU;
    if (n_buckets > 0 && !snapshots) return OMNI_ERR_NULL;
    int rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, worker, 0.0f);
    if (rc != OMNI_OK) return rc;
    bool wide = all_aligned32(buckets, n_buckets, worker, worker + 1);
    for (int i = 0; i < n_buckets; ++i) {
        if (buckets[i].n == 0) continue;
        if (!snapshots[i]) return OMNI_ERR_NULL;
        if (!aligned16(snapshots[i])) return OMNI_ERR_ALIGN;
        wide = wide && aligned32(snapshots[i]);
    }
    rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    const double eta_k = (ctx->ctl.config().flags & OMNI_ASP_NO_LR_SCALE)
                             ? double(lr)
                             : double(lr) * double(b_used) / double(ctx->ctl.B());
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (use_bulk(ctx, grad_dtype, 1)) {
        const KernelInfo ki = bulk_overwrite_kernel(grad_dtype);
        LaunchShape &shape = ctx->bulk_overwrite_shape[grad_dtype];
        rc = shape_for(ctx, ki, shape);
        if (rc != OMNI_OK) return rc;
        BspParams p;
        int i = 0;
        while (i < n_buckets) {
            std::memset(&p, 0, sizeof p);
            unsigned long long tiles = 0;
            int nb = 0;
            for (; i < n_buckets && nb < kMaxBucketsPerLaunch; ++i) {
                const omni_bucket &bk = buckets[i];
                if (bk.n == 0) continue;
                p.bk[nb] = {static_cast<float *>(bk.param), nullptr, static_cast<__nv_bfloat16 *>(bk.param_lp), bk.n, tiles};
                p.g[nb][0] = bk.grads[worker];
                p.src[nb] = static_cast<const float *>(snapshots[i]);
                p.copy[nb] = write_back ? static_cast<float *>(snapshots[i]) : nullptr;
                tiles += (bk.n + ki.tile - 1) / ki.tile;
                ++nb;
            }
            if (nb == 0) break;
            p.lam[0] = float(eta_k);
            p.wd = weight_decay;
            p.nb = nb;
            p.reverse = int(ctx->sweep & 1u);
            p.tiles = tiles;
            p.ws = ctx->ws;
            const int grid = tiles < (unsigned long long)shape.grid ? int(tiles) : shape.grid;
            rc = launch(ctx, ki, grid, &p, s);
            if (rc != OMNI_OK) return rc;
        }
        ctx->sweep += 1;
    } else {
        const KernelInfo ki = overwrite_kernel(grad_dtype, wide);
        LaunchShape &shape = ctx->overwrite_shape[grad_dtype][wide];
        rc = shape_for(ctx, ki, shape);
        if (rc != OMNI_OK) return rc;
        OverwriteParams p;
        int i = 0;
        while (i < n_buckets) {
            std::memset(&p, 0, sizeof p);
            unsigned long long tiles = 0;
            int nb = 0;
            for (; i < n_buckets && nb < kMaxBucketsPerLaunch; ++i) {
                const omni_bucket &bk = buckets[i];
                if (bk.n == 0) continue;
                p.bk[nb] = {static_cast<float *>(bk.param), nullptr, static_cast<__nv_bfloat16 *>(bk.param_lp), bk.n, tiles};
                p.g[nb] = bk.grads[worker];
                p.snap[nb] = static_cast<const float *>(snapshots[i]);
                tiles += (bk.n + ki.tile - 1) / ki.tile;
                ++nb;
            }
            if (nb == 0) break;
            p.eta = float(eta_k); p.wd = weight_decay;
            p.nb = nb;
            p.tiles = tiles;
            const int grid = tiles < (unsigned long long)shape.grid ? int(tiles) : shape.grid;
            rc = launch(ctx, ki, grid, &p, s);
            if (rc != OMNI_OK) return rc;
        }
        if (write_back)   // the register family pulls with plain device copies
            for (int j = 0; j < n_buckets; ++j)
                if (buckets[j].n)
                    OMNI_CUDA(ctx, cudaMemcpyAsync(snapshots[j], buckets[j].param, buckets[j].n * sizeof(float),
                                                   cudaMemcpyDeviceToDevice, s));
    }
    tally_arrival(ctx, tau);
    return OMNI_OK;
}

int omni_asp_push_overwrite(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                            int32_t worker, int32_t b_used, int32_t tau, const void *const *snapshots, float lr,
                            float weight_decay, void *stream)
{
    return push_overwrite(ctx, buckets, n_buckets, grad_dtype, worker, b_used, tau,
                          const_cast<void *const *>(snapshots), false, lr, weight_decay, stream);
}

int omni_asp_push_pull(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                       int32_t worker, int32_t b_used, int32_t tau, void *const *snapshots, float lr,
                       float weight_decay, void *stream)
{
    return push_overwrite(ctx, buckets, n_buckets, grad_dtype, worker, b_used, tau, snapshots, true, lr, weight_decay,
                          stream);
}

// ---- device-resident controller ----------------------------------------------------------------

int omni_ctl_to_device(omni_ctx *ctx, void *stream)
{
    if (!ctx) return OMNI_ERR_NULL;
    int rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    if (!ctx->dctl) OMNI_CUDA(ctx, cudaMalloc(&ctx->dctl, sizeof(DeviceCtl)));
    DeviceCtl &st = ctx->dctl_stage;
    std::memset(&st, 0, sizeof st);
    ctx->ctl.export_state(st.batch, st.time, st.seen);
    st.weight_sum = fill_weights(ctx, st.batch, st.lam);
    // pageable source: the runtime stages it before the call returns, so `st` may be reused
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->dctl, &st, sizeof st, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream)));
    return OMNI_OK;
}

int omni_ctl_from_device(omni_ctx *ctx, void *stream)
{
    if (!ctx) return OMNI_ERR_NULL;
    if (!ctx->dctl) return OMNI_ERR_BAD_CONFIG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DeviceCtl &st = ctx->dctl_stage;
    OMNI_CUDA(ctx, cudaMemcpyAsync(&st, ctx->dctl, sizeof st, cudaMemcpyDeviceToHost, s));
    OMNI_CUDA(ctx, cudaStreamSynchronize(s));
    ctx->ctl.import_state(st.batch, st.time, st.seen);
    st.weight_sum = 0.0;
    for (int k = 0; k < ctx->ctl.K(); ++k) st.weight_sum += double(st.lam[k]);
    ctx->tally.weight_sum = st.weight_sum;
    if (st.status != 0) {
        // a device re-batch refused its input since the last read: report it once and clear it
        OMNI_CUDA(ctx, cudaMemsetAsync(&ctx->dctl->status, 0, sizeof(int32_t), s));
        return st.status;
    }
    return OMNI_OK;
}

int omni_rebatch_device(omni_ctx *ctx, const double *measured_dev, int32_t *new_b_dev, void *stream)
{
    if (!ctx || !measured_dev) return OMNI_ERR_NULL;
    if (!ctx->dctl) return OMNI_ERR_BAD_CONFIG;
    if ((reinterpret_cast<uintptr_t>(measured_dev) & 7u) || (reinterpret_cast<uintptr_t>(new_b_dev) & 3u)) return OMNI_ERR_ALIGN;
    int rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    const int e = launch_device_rebatch(ctx->dctl, ctx->ctl.config(), measured_dev, new_b_dev, stream);
    if (e != 0) {
        ctx->last_cuda = e;
        return OMNI_ERR_CUDA;
    }
    ctx->launches += 1;
    return OMNI_OK;
}

int omni_asp_report_device(omni_ctx *ctx, int32_t worker, int32_t b_used, const double *measured_dev,
                           int32_t *new_b_dev, void *stream)
{
    if (!ctx || !measured_dev) return OMNI_ERR_NULL;
    if (worker < 0 || worker >= ctx->ctl.K()) return OMNI_ERR_BAD_WORKER;
    if (b_used < 1) return OMNI_ERR_BAD_BATCH;
    if (!ctx->dctl) return OMNI_ERR_BAD_CONFIG;
    if ((reinterpret_cast<uintptr_t>(measured_dev) & 7u) || (reinterpret_cast<uintptr_t>(new_b_dev) & 3u)) return OMNI_ERR_ALIGN;
    int rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    const int e = launch_device_report(ctx->dctl, ctx->ctl.config(), worker, b_used, measured_dev, new_b_dev, stream);
    if (e != 0) {
        ctx->last_cuda = e;
        return OMNI_ERR_CUDA;
    }
    ctx->launches += 1;
    return OMNI_OK;
}

int omni_aggregate_bsp_device_batches(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                                      float lr, float momentum, float weight_decay, void *stream)
{
    if (!ctx) return OMNI_ERR_NULL;
    if (!ctx->dctl) return OMNI_ERR_BAD_CONFIG;
    int rc = check_buckets(ctx, buckets, n_buckets, grad_dtype, -1, momentum);
    if (rc != OMNI_OK) return rc;
    rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    rc = enqueue_bsp(ctx, buckets, n_buckets, grad_dtype, nullptr, ctx->dctl->lam, lr, momentum, weight_decay,
                     static_cast<cudaStream_t>(stream));
    if (rc != OMNI_OK) return rc;
    ctx->tally.steps += 1;
    return OMNI_OK;
}

int omni_get_stats(omni_ctx *ctx, omni_stats *out, void *stream)
{
    if (!ctx || !out) return OMNI_ERR_NULL;
    if (ctx->ws) {
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        const int rc = finalize_sqnorm(ctx, s);
        if (rc != OMNI_OK) return rc;
        OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->host_cell, &ctx->ws->sqnorm, 2 * sizeof(double), cudaMemcpyDeviceToHost, s));
        OMNI_CUDA(ctx, cudaStreamSynchronize(s));
        ctx->tally.grad_sqnorm = ctx->host_cell[0];
        unsigned int words[2];
        std::memcpy(words, &ctx->host_cell[1], sizeof words);   // reserved, status
        if (words[1] != 0) {
            // a bounded device-side wait ran out in some earlier launch: report once and clear
            OMNI_CUDA(ctx, cudaMemsetAsync(&ctx->ws->status, 0, sizeof(unsigned int), s));
            *out = ctx->tally;
            return OMNI_ERR_TIMEOUT;
        }
    }
    *out = ctx->tally;
    return OMNI_OK;
}

int omni_selftest_wait_expiry(omni_ctx *ctx, void *stream)
{
    if (!ctx) return OMNI_ERR_NULL;
    int rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    const int e = launch_expire_wait(ctx->ws, 2048u, stream);
    if (e != 0) {
        ctx->last_cuda = e;
        return OMNI_ERR_CUDA;
    }
    ctx->launches += 1;
    return OMNI_OK;
}

int omni_last_cuda_error(const omni_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }

int omni_query_launch(omni_ctx *ctx, int32_t K, int32_t grad_dtype, int32_t *grid, int32_t *block)
{
    if (!ctx || !grid || !block) return OMNI_ERR_NULL;
    if (K < 1 || K > OMNI_MAX_K) return OMNI_ERR_BAD_K;
    if (grad_dtype != OMNI_F32 && grad_dtype != OMNI_BF16) return OMNI_ERR_BAD_CONFIG;
    int rc = ensure_device(ctx);
    if (rc != OMNI_OK) return rc;
    const bool bulk = use_bulk(ctx, grad_dtype, K);
    LaunchShape &shape = bulk ? ctx->bulk_shape[grad_dtype][K] : ctx->bsp_shape[grad_dtype][1][K];
    rc = shape_for(ctx, bulk ? bulk_kernel(grad_dtype, K) : bsp_kernel(grad_dtype, K, true), shape);
    if (rc != OMNI_OK) return rc;
    *grid = shape.grid;
    *block = shape.block;
    return OMNI_OK;
}

uint64_t omni_kernel_launches(const omni_ctx *ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
