/*
 * omni.h -- C ABI of the OmniLearn data-parallel hot path on one GPU.
 *
 * The library implements, for K workers whose gradients sit in K device buffers:
 *   - the proportional batch-size controller (paper Eq. 6a/6b, dead-band Eq. 7, batch bounds,
 *     global-batch rule Eq. 8; procedures getBsz of Algorithm 1 and evalBsz of Algorithm 2),
 *   - the batch-size-weighted aggregation of the K gradients fused with the parameter update
 *     (Eq. 4b, Eq. 4c; Algorithm 1 "AllReduce(lambda_k g)" and "theta - eta gbar"),
 *   - the asynchronous per-arrival update with the batch-scaled learning rate
 *     (Eq. 5b; Algorithm 2 "eta_k = eta b / B", "theta - eta_k g").
 *
 * Conventions
 *   - Every function returns 0 (OMNI_OK) or a negative omni_status.  Nothing throws, aborts or
 *     traps.  Arguments are validated before any state changes or any kernel is enqueued: a
 *     failed call leaves the context and all buffers as they were.
 *   - "device pointer" = memory of the CUDA device that is current when the call is made;
 *     "host pointer" = ordinary host memory.  Parameter-sized buffers are owned by the caller
 *     and must stay alive until the stream has executed the call.
 *   - Kernels are enqueued on the caller's stream (a cudaStream_t passed as void*, NULL = the
 *     default stream) and the call returns without synchronising, unless stated otherwise.
 *   - A context is not thread-safe.  It owns a small device workspace (per-block partial sums
 *     and the gradient-norm cell, a few tens of KB) that is allocated by the first call that
 *     launches a kernel and freed by omni_destroy; calls on different streams that share a
 *     context and overlap on the GPU race on it.  The synchronous step leaves one partial sum of
 *     the squared gradient norm per thread block there; they are added up, in a fixed order, by
 *     a one-warp kernel that omni_get_stats and omni_aggregate_bsp_host enqueue, so a step that
 *     nobody asks the norm of pays nothing for it.
 *   - OMNI_MAX_K = 32 workers.
 */
#ifndef OMNI_H_
#define OMNI_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OMNI_MAX_K 32
#define OMNI_TAU_BINS 33 /* staleness 0..31 and one overflow bin */

typedef enum {
    OMNI_OK = 0,
    OMNI_ERR_NULL = -1,            /* a required pointer is NULL */
    OMNI_ERR_BAD_K = -2,           /* K outside 1..OMNI_MAX_K */
    OMNI_ERR_BAD_WORKER = -3,      /* worker index outside 0..K-1 */
    OMNI_ERR_BAD_BATCH = -4,       /* some b_k < 1, or sum b_k != B in synchronous mode */
    OMNI_ERR_INFEASIBLE = -5,      /* K*b_min > B or K*b_max < B in synchronous mode */
    OMNI_ERR_BAD_MEASUREMENT = -6, /* throughput/time not finite or <= 0 */
    OMNI_ERR_ALIGN = -7,           /* a device pointer is not 16-byte aligned */
    OMNI_ERR_BAD_TAU = -8,         /* negative staleness */
    OMNI_ERR_CUDA = -9,            /* a CUDA call failed; see omni_last_cuda_error */
    OMNI_ERR_TIMEOUT = -10,        /* a bounded device-side wait ran out */
    OMNI_ERR_BAD_CONFIG = -11,     /* invalid omni_config field or call argument */
    OMNI_ERR_TOO_LARGE = -12,      /* size beyond a stated maximum */
    OMNI_ERR_NO_MEMORY = -13       /* a host allocation failed */
} omni_status;

typedef enum { OMNI_BSP = 0, OMNI_ASP = 1 } omni_mode;
typedef enum { OMNI_F32 = 0, OMNI_BF16 = 1 } omni_dtype;

/* omni_config.flags */
#define OMNI_UNSCALED_MEAN 1u   /* lambda_k = 1/K: the unweighted arm of the paper's "weighted aggregation" table */
#define OMNI_ASP_NO_LR_SCALE 2u /* eta_k = eta: the "w/o LR scaling" arm of the paper's ASP table */
#define OMNI_INPUT_IS_TIME 4u   /* measurements are compute times t_k instead of throughputs T_k */
/* Global-batch rule, second reading.  Eq. 8 subtracts the same Delta B / K from every worker
 * (the default); the sentence after it (Sec. III-B, "Control Stability") speaks of reducing the
 * adjusted batches "proportionately".  With this flag the synchronous re-batch renormalises the
 * real-valued getBsz results c_k of all workers, c_k <- c_k * B / sum_i c_i, before the rounding
 * step, and the unit steps of the default rule only close what rounding and the bounds leave.
 * From equal batches without dead-band and bounds this gives B * T_k / sum(T) in one step
 * (Eq. 4a with the throughputs as capacities).  Ignored in asynchronous mode. */
#define OMNI_CONSERVE_MULTIPLICATIVE 32u
/* Kernel family.  By default the device calls stage their inputs through shared memory with
 * bulk (TMA) copies and an mbarrier ring; register-staged 128/256-bit-load kernels exist for
 * every call as well (and serve omni_aggregate_bsp_noalloc).  The ring
 * kernels also alternate the direction in which successive calls walk the parameters and keep
 * theta and v in L2 with evict-last priority, so that a call finds the part its predecessor
 * touched last still in cache, and are launched with programmatic stream serialization (they
 * wait for the previous launch themselves, after their set-up).  The two flags force
 * one family; results are the same bit for bit.  A bounded wait of the ring that runs out
 * surfaces as OMNI_ERR_TIMEOUT from omni_get_stats.
 * Contract for the caller's own kernels on the same stream: the ring kernels (and the one-warp
 * kernels of the device-resident controller) signal "dependents may launch" (griddepcontrol.launch_dependents) as soon as
 * their set-up is done, long before their last store.  A kernel enqueued after a library call
 * in the ordinary way is not affected: the stream still runs it after the library's kernel has
 * finished.  A kernel that the caller launches WITH the programmatic-stream-serialization
 * attribute, however, may start while the library's kernel is still writing: it must execute
 * griddepcontrol.wait (cudaGridDependencySynchronize) before it touches theta, v, the bf16
 * copy, the batches or any other buffer of the call.  Contexts created with OMNI_NO_BULK_COPY
 * launch only ordinary kernels and never signal early. */
#define OMNI_BULK_COPY 8u
#define OMNI_NO_BULK_COPY 16u
/* omni_create refuses flag bits it does not know and both kernel-family flags together (BAD_CONFIG). */

/* The "Input:" line of Algorithm 1 / Algorithm 2 (K, B, Delta b_k, b_min, b_max) plus the EWMA weight. */
typedef struct {
    int32_t K;            /* workers, 1..OMNI_MAX_K */
    int32_t global_batch; /* B; initial b_k = B / K (first B mod K workers take one more) */
    int32_t b_min, b_max; /* batch-size bounds, 1 <= b_min <= b_max */
    double deadband;      /* Delta b_k of Eq. 7 as a fraction, >= 0 */
    double ewma_alpha;    /* weight of the newest compute-time sample, (0, 1]; 1 = no smoothing */
    int32_t mode;         /* OMNI_BSP: Eq. 8 keeps sum b_k = B.  OMNI_ASP: no such rule. */
    uint32_t flags;
} omni_config;

/* One bucket = contiguous storage holding one or more whole tensors.  A flat model is one bucket. */
typedef struct {
    void *param;              /* device, float[n], 16-byte aligned, read and written: master parameters theta */
    void *momentum;           /* device, float[n], 16-byte aligned, read and written: v.  May be NULL iff momentum == 0 */
    void *param_lp;           /* device, bfloat16[n], 16-byte aligned, written: rounded copy of the new theta; or NULL */
    const void *const *grads; /* HOST array of K device pointers (float[n] or bfloat16[n], 16-byte aligned, read only) */
    uint64_t n;               /* elements; 0 is allowed (the bucket is skipped) */
} omni_bucket;

typedef struct {
    double grad_sqnorm;  /* sum_j gbar_j^2 of the aggregated gradient of the last omni_aggregate_bsp call */
    double weight_sum;   /* sum_k lambda_k (as rounded to float) of that call */
    uint64_t steps;      /* synchronous steps enqueued */
    uint64_t arrivals;   /* asynchronous arrivals enqueued */
    uint64_t tau_hist[OMNI_TAU_BINS]; /* arrivals by staleness 0..31, last bin: 32 and more */
    int32_t tau_max;
    uint64_t tau_sum;    /* sum of the staleness of all arrivals (mean = tau_sum / arrivals) */
} omni_stats;

typedef struct omni_ctx omni_ctx;

const char *omni_strerror(int status);

/* Create a controller context with b_k = B / K (Algorithm 1, first line of Train).  Needs no GPU.
 * Errors: NULL, BAD_K, BAD_CONFIG, INFEASIBLE, NO_MEMORY. */
int omni_create(const omni_config *cfg, omni_ctx **out);
void omni_destroy(omni_ctx *ctx);

/* Current batch sizes, b[K] host array (BSP: the controller's b_k; ASP: the server's wrkB map). */
int omni_get_batches(const omni_ctx *ctx, int32_t *b);
/* Overwrite them.  BAD_BATCH if some b_k < 1 or, in BSP mode, sum != B. */
int omni_set_batches(omni_ctx *ctx, const int32_t *b);

/* Controller state for checkpoints (the paper notes that a batch re-adjustment goes through a
 * checkpoint of the job, Sec. III-B): the batches, the smoothed compute times and which workers
 * have one yet, as one flat record.  omni_ctl_export: *size (host, in/out) holds the capacity of
 * `record` (host) and receives the record's size; record == NULL only queries the size.
 * omni_ctl_import restores a record into a context created with the same K and global batch;
 * batch sizes and times are validated and a failed import changes nothing.  Parameter buffers,
 * momentum and the device copy of the controller are the caller's to save.
 * Errors: NULL, TOO_LARGE (capacity below the record's size), BAD_CONFIG (not a record, or made
 * for another K or global batch), BAD_BATCH, BAD_MEASUREMENT. */
int omni_ctl_export(const omni_ctx *ctx, void *record, uint64_t *size);
int omni_ctl_import(omni_ctx *ctx, const void *record, uint64_t size);

/* Synchronous re-batch: getAvgComputeTime + getBsz for every worker (Algorithm 1) + Eq. 8.
 * measured[K] (host): throughput T_k in samples per time unit seen with the current b_k, or the
 * compute time t_k if OMNI_INPUT_IS_TIME.  Steps, all in IEEE double, sums in ascending k:
 *   t_k = b_k / T_k;  s_k = EWMA(t_k);  tbar = (sum s_k) / K;                      (Eq. 6a)
 *   b*_k = b_k - (b_k / s_k) (s_k - tbar);                                          (Eq. 6b)
 *   if |(b*_k - b_k) / b*_k| >= deadband: b*_k clamped to [b_min, b_max], else b_k;  (Eq. 7)
 *   round half up to an integer; BSP: shift all workers not pinned at a bound, one unit at a
 *   time, until sum = B; leftover units go to the largest batches, lowest index first.  (Eq. 8)
 * new_b[K] (host, out) receives the batches; changed[K] (host, out, may be NULL) 0/1 flags.
 * Errors: NULL, BAD_MEASUREMENT, INFEASIBLE. */
int omni_rebatch(omni_ctx *ctx, const double *measured, int32_t *new_b, int32_t *changed);

/* Asynchronous re-batch: evalBsz of Algorithm 2.  Worker `worker` reports the batch it ran and
 * its measurement; both are stored.  Until every worker has reported once, *new_b_k = b_used.
 * Afterwards getBsz is re-evaluated for all K stored entries against their mean time (no Eq. 8)
 * and *new_b_k is the caller's entry.  Errors: NULL, BAD_WORKER, BAD_BATCH, BAD_MEASUREMENT. */
int omni_asp_report(omni_ctx *ctx, int32_t worker, int32_t b_used, double measured, int32_t *new_b_k);

/* Static variable batching, Eq. 4a: b_k = c_k / sum(c) * B from worker capacities c_k (host,
 * K positive values, e.g. core counts), rounded to integers within the bounds with sum = B in
 * BSP mode.  Stores and returns the batches.  Errors: NULL, BAD_MEASUREMENT, INFEASIBLE. */
int omni_rebatch_static(omni_ctx *ctx, const double *capacity, int32_t *new_b);

/* One synchronous step over all buckets: Eq. 4b/4c fused with the optimiser update.  Per element j:
 *   lambda_k = float(b_k / sum_i b_i)          (1/K with OMNI_UNSCALED_MEAN)
 *   gbar = fma(lambda_{K-1}, g_{K-1,j}, ... fma(lambda_0, g_{0,j}, 0))   ascending k, single precision
 *   d = weight_decay ? fma(weight_decay, theta_j, gbar) : gbar
 *   v_j = momentum ? fma(momentum, v_j, d) : d          (stored when the momentum buffer is given)
 *   theta_j = fma(-lr, v_j, theta_j);  param_lp_j = bfloat16(theta_j) round-to-nearest-even
 * and the squared norm of gbar over all buckets is left in the context (omni_get_stats).
 * buckets: host array of n_buckets descriptors; b: host int32[K], the batches these gradients
 * were computed with (each >= 1; in BSP mode sum must equal B).  grad_dtype selects float or
 * bfloat16 gradients (bfloat16 is widened exactly).  Enqueues on `stream`, does not synchronise.
 * Errors: NULL, BAD_BATCH, ALIGN, BAD_CONFIG (n_buckets < 0, bad dtype, momentum != 0 with a
 * NULL momentum buffer), CUDA. */
int omni_aggregate_bsp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                       const int32_t *b, float lr, float momentum, float weight_decay, void *stream);

/* One iteration of Algorithm 1's training loop in a single call: the aggregate + update of
 * omni_aggregate_bsp with the controller's CURRENT batches (the ones the workers computed these
 * gradients with: lambda_k = b_k / B), followed by omni_rebatch from `measured` (host, K values
 * observed during this iteration), whose result applies to the next iteration's gradients.
 * next_b[K] (host, out) receives the new batches, changed[K] (host, out, may be NULL) the 0/1 flags.
 * Same arithmetic and the same kernels as the two calls made one after the other; it exists so
 * that a step costs one trip through the binding instead of two, which matters for models small
 * enough to be bound by the host's launch rate.  All arguments, the measurements included, are
 * validated before the kernel is enqueued or the controller changes.
 * Errors: those of omni_aggregate_bsp and omni_rebatch. */
int omni_step_bsp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                  const double *measured, float lr, float momentum, float weight_decay, int32_t *next_b,
                  int32_t *changed, void *stream);

/* One asynchronous arrival: worker `worker`'s gradient (buckets[i].grads[worker]), computed on
 * b_used samples, is applied to the server parameters with eta_k = float(lr * b_used / B)
 * (Eq. 5b; eta_k = lr with OMNI_ASP_NO_LR_SCALE):
 *   d = weight_decay ? fma(weight_decay, theta_j, g_j) : g_j;  v_j = momentum ? fma(momentum, v_j, d) : d;
 *   theta_j = fma(-eta_k, v_j, theta_j)
 * tau = server updates since this worker last read the parameters; the paper defines no
 * staleness-dependent factor, so tau is only tallied (omni_stats.tau_hist, tau_max).
 * Errors: NULL, BAD_WORKER, BAD_BATCH (b_used < 1), BAD_TAU, ALIGN, BAD_CONFIG, CUDA. */
int omni_apply_asp(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                   int32_t worker, int32_t b_used, int32_t tau, float lr, float momentum, float weight_decay,
                   void *stream);

/* A batch of m queued asynchronous arrivals applied in one pass over the parameters, in the order
 * given: exactly the result of m successive omni_apply_asp calls (the element goes through the
 * m updates of Eq. 5b one after the other, theta and v staying in registers), but theta and v
 * are read and written once, so the traffic is 4m+8 (+8 with momentum) bytes per parameter
 * instead of 12m (20m).  workers[m], b_used[m], tau[m]: host arrays; a worker may appear more
 * than once (its buffer is then applied again).  1 <= m <= OMNI_MAX_ASP_BATCH.
 * Errors: as omni_apply_asp, plus TOO_LARGE for m out of range. */
#define OMNI_MAX_ASP_BATCH 16
int omni_apply_asp_batch(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype, int32_t m,
                         const int32_t *workers, const int32_t *b_used, const int32_t *tau, float lr, float momentum,
                         float weight_decay, void *stream);

/* Algorithm 2 taken literally (pull / local update / push with overwrite), for callers that want
 * the paper's parameter-server semantics instead of "apply to the current copy".
 * omni_asp_pull: pullFromPS -- snapshots[i] (HOST array of n_buckets device pointers, float[n]
 * each, 16-byte aligned, caller-owned, one set per worker) <- buckets[i].param, by device copies
 * enqueued on `stream`.
 * omni_asp_push_overwrite: the worker's local step and pushToPS in one launch --
 *   theta_j <- fma(-eta_k, d, s_j),  d = weight_decay ? fma(weight_decay, s_j, g_j) : g_j,
 * with s the snapshot that worker pulled, g = buckets[i].grads[worker], eta_k as in omni_apply_asp.
 * The server copy is OVERWRITTEN: whatever other workers pushed since this worker's pull is lost
 * (the paper's "overridden" updates), so here the staleness tau changes the result, although it
 * still enters no formula; it is tallied as in omni_apply_asp.  Plain SGD as in Algorithm 2 (no
 * momentum buffer is read or written).  With tau = 0 the result equals omni_apply_asp's.
 * omni_asp_push_pull: the push above followed at once by the same worker's next pull, as in the
 * worker loop of Algorithm 2 (pushToPS at the end of one iteration, pullFromPS at the start of the
 * next), in the same launch: the server copy AND the worker's snapshot receive the new
 * parameters (snapshots are read and written).  Same result as omni_asp_push_overwrite followed
 * by omni_asp_pull of that worker, at 16 instead of 20 bytes per parameter.
 * Errors: NULL, BAD_WORKER, BAD_BATCH, BAD_TAU, ALIGN, BAD_CONFIG, CUDA. */
int omni_asp_pull(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, void *const *snapshots, void *stream);
int omni_asp_push_overwrite(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                            int32_t worker, int32_t b_used, int32_t tau, const void *const *snapshots, float lr,
                            float weight_decay, void *stream);
int omni_asp_push_pull(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                       int32_t worker, int32_t b_used, int32_t tau, void *const *snapshots, float lr,
                       float weight_decay, void *stream);

/* Device-resident controller: the synchronous re-batch (getBsz of Algorithm 1 for every worker,
 * Eq. 6a/6b, dead-band Eq. 7, bounds, Eq. 8) as a one-warp kernel on a device copy of the
 * controller state, so that a whole step -- re-batch from measurements that are already on the
 * GPU, then aggregate + update with the new weights -- is enqueued (or captured in a CUDA graph)
 * without a host round trip.  Arithmetic and results are those of omni_rebatch, bit for bit:
 * single correctly rounded double operations in the same order, then integers.
 *
 * omni_ctl_to_device: copies the host controller state (b_k, smoothed times) and the weights
 *   lambda_k = float(b_k / sum b) to the device copy, allocating it on a context's first call
 *   (make that call outside stream capture).  Enqueued on `stream`.
 * omni_rebatch_device: measured_dev = DEVICE double[K] (throughputs, or times with
 *   OMNI_INPUT_IS_TIME), 8-byte aligned; new_b_dev = DEVICE int32[K] out, or NULL.  Updates the
 *   device copy's batches, smoothed times and weights.  A measurement that is not finite or not
 *   positive leaves the device copy untouched and records OMNI_ERR_BAD_MEASUREMENT, which the
 *   next omni_ctl_from_device returns (once).  The host controller is not touched: host calls
 *   (omni_rebatch, omni_get_batches, ...) keep seeing the state of the last
 *   omni_ctl_from_device.
 * omni_asp_report_device: evalBsz of Algorithm 2 (omni_asp_report) on the device copy: worker and
 *   b_used are host values, measured_dev = DEVICE double[1] (8-byte aligned), new_b_k_dev = DEVICE
 *   int32[1] out or NULL.  Stores the worker's batch and smoothed time in the device copy and,
 *   once every worker has an entry, re-evaluates all K entries (no Eq. 8); a bad measurement is
 *   recorded as for omni_rebatch_device.  Same integers as omni_asp_report, bit for bit.
 * omni_aggregate_bsp_device_batches: omni_aggregate_bsp with the weights the device copy holds
 *   (no `b` argument; nothing is checked against B on the host).  Always the bulk-copy ring kernel.
 * omni_ctl_from_device: synchronises `stream`, copies the device copy back into the host
 *   controller and omni_stats.weight_sum; returns a recorded device re-batch failure, if any.
 * omni_ctl_to_device and omni_ctl_from_device copy between pageable host memory and the device and
 * are not meant to be captured; omni_rebatch_device and omni_aggregate_bsp_device_batches are
 * plain kernel launches.
 * Errors: NULL, BAD_CONFIG (no device copy yet; or as omni_aggregate_bsp), ALIGN, CUDA;
 * omni_asp_report_device also BAD_WORKER, BAD_BATCH. */
int omni_ctl_to_device(omni_ctx *ctx, void *stream);
int omni_ctl_from_device(omni_ctx *ctx, void *stream);
int omni_rebatch_device(omni_ctx *ctx, const double *measured_dev, int32_t *new_b_dev, void *stream);
int omni_asp_report_device(omni_ctx *ctx, int32_t worker, int32_t b_used, const double *measured_dev,
                           int32_t *new_b_k_dev, void *stream);
int omni_aggregate_bsp_device_batches(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                                      float lr, float momentum, float weight_decay, void *stream);

/* Parameter-range sharding for one rank per GPU (no counterpart in the paper, whose workers
 * all-reduce whole gradients; this is the reduce-scatter form of the same sum).  Every element of
 * the step is independent of every other, so the AllReduce of Algorithm 1 followed by the update
 * can run as: rank r owns the elements [begin, begin + count) of each bucket, reads that range of
 * all K workers' gradients (its own locally, the others through peer-mapped pointers placed in
 * omni_bucket.grads), runs omni_aggregate_bsp on the sub-range, and the ranks then exchange the
 * updated ranges (all-gather) and add their squared norms.  This call only computes the range:
 * n elements are cut into units of OMNI_SHARD_UNIT elements (so that every range starts on a
 * 256-byte boundary of a float buffer and a 128-byte boundary of a bfloat16 buffer) and the
 * units are dealt out contiguously, rank counts differing by at most one unit; the ranges of
 * ranks 0..world-1 tile [0, n) in order.  count may be 0 when n is small.
 * Errors: NULL, BAD_CONFIG (world < 1, rank outside 0..world-1). */
#define OMNI_SHARD_UNIT 64
int omni_shard_range(uint64_t n, int32_t world, int32_t rank, uint64_t *begin, uint64_t *count);

/* Same step as omni_aggregate_bsp for gradients that arrive in HOST memory (pinned memory gives
 * asynchronous copies).  host_grads: host array of n_buckets*K host pointers, entry [i*K + k] =
 * worker k's gradient for bucket i.  buckets[i].grads must point at K device staging buffers of
 * n elements each, owned by the caller; the call copies every host gradient into its staging
 * buffer on `stream`, runs the fused step, copies the squared gradient norm back, synchronises
 * the stream and stores it in *grad_sqnorm (host, may be NULL).
 * Errors: as omni_aggregate_bsp.  Unlike the other calls, a CUDA failure part-way (a copy or the
 * launch refused by the runtime) can leave the staging buffers holding some of the new
 * gradients; theta and v are only ever changed by the fused step itself. */
int omni_aggregate_bsp_host(omni_ctx *ctx, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                            const void *const *host_grads, const int32_t *b, float lr, float momentum,
                            float weight_decay, void *stream, double *grad_sqnorm);

/* The same fused step as omni_aggregate_bsp for callers that are not allowed to allocate device
 * memory when they run a step.  (The paper has no counterpart: this is a deployment variant of
 * the call above, not part of the method.)
 *
 * Who needs it: code that runs inside another framework's allocator callback or under its
 * allocator lock, processes whose device memory has all been handed to a pool at start-up, and
 * latency-critical loops that ban calls which may synchronise the device, as cudaMalloc and
 * cudaFree may.  omni_aggregate_bsp allocates a small workspace on a context's first launch;
 * this function calls no cudaMalloc, cudaFree or other allocating routine (see "Warm-up" below
 * for what the CUDA runtime does on its own the first time a kernel is used).  Its kernel's
 * scratch (one partial sum of the squared norm per CTA, about 19 KB) is a fixed
 * array inside the library's device image: every GPU that loads the library holds it until the
 * process exits.
 *
 * It takes no context: K, the batches and the flags (OMNI_UNSCALED_MEAN) come as arguments and
 * lambda_k = b_k / sum b.  Arithmetic, layouts and alignment rules are those of
 * omni_aggregate_bsp.  grad_sqnorm_dev (DEVICE pointer, 8-byte aligned, may be NULL) receives
 * the squared norm of the aggregate from a one-warp kernel enqueued after the step (it adds the
 * partial sums in a fixed order; with NULL it is not launched).  Enqueues on `stream`, does not
 * synchronise.
 *
 * Limits: at most OMNI_NOALLOC_MAX_BUCKETS non-empty buckets and OMNI_NOALLOC_MAX_ELEMENTS
 * elements in total; more returns OMNI_ERR_TOO_LARGE and does nothing.
 * Sharing: all calls on one device use the same array, which keeps the previous call's
 * contents; no cell has to start at zero (each launch overwrites every cell it later reads).  Calls
 * whose kernels overlap on the GPU (issued on different streams without ordering) race on it
 * and give wrong norms: keep them on one stream or order them with events.
 * First call: the first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) with that device current; make that call before any stream capture.
 * It is not thread-safe against another first call on the same device.
 * Warm-up: "never allocates" is what this function does itself.  The CUDA runtime loads a
 * kernel's code, and whatever device memory that code needs, the first time the kernel is
 * launched, and the first call for a combination of (device, gradient type, K, all buffers
 * 32-byte aligned or not) also asks the runtime once for that kernel's occupancy.  A caller
 * whose restriction covers the runtime's own lazy loading should therefore make one call per
 * combination it will use (tiny buffers will do) before it enters the restricted region; every
 * later call is one kernel launch and, with grad_sqnorm_dev, a second one-warp launch, both
 * asynchronous.
 * flags: OMNI_UNSCALED_MEAN or 0; any other bit returns OMNI_ERR_BAD_CONFIG.
 * Errors: BAD_K, NULL, BAD_CONFIG, BAD_BATCH (some b_k < 1), ALIGN, TOO_LARGE, CUDA. */
#define OMNI_NOALLOC_MAX_BUCKETS 8
#define OMNI_NOALLOC_MAX_ELEMENTS (1ull << 31)
int omni_aggregate_bsp_noalloc(int32_t K, const omni_bucket *buckets, int32_t n_buckets, int32_t grad_dtype,
                               const int32_t *b, uint32_t flags, float lr, float momentum, float weight_decay,
                               double *grad_sqnorm_dev, void *stream);

/* Synchronises `stream` and fills *out (host).  The squared norm of the last synchronous step is
 * summed here, by a one-warp kernel enqueued on `stream`: pass the stream that step was enqueued
 * on, or one that has been ordered after it. */
int omni_get_stats(omni_ctx *ctx, omni_stats *out, void *stream);

/* Failure-path self-test (no counterpart in the paper).  Every device-side wait of the library is
 * bounded; when one runs out the kernel records it and the next omni_get_stats returns
 * OMNI_ERR_TIMEOUT once, then clears the record.  This call enqueues a one-warp kernel that waits,
 * with a short limit, on a barrier nothing completes, so that the path can be observed without
 * any kernel misbehaving: afterwards omni_get_stats must return OMNI_ERR_TIMEOUT, the context
 * stays usable, and the following omni_get_stats returns OMNI_OK.  Errors: NULL, CUDA. */
int omni_selftest_wait_expiry(omni_ctx *ctx, void *stream);

/* The cudaError_t of the last failed CUDA call made through this context (0 if none). */
int omni_last_cuda_error(const omni_ctx *ctx);

/* Persistent-grid size and block size the synchronous kernel for this K and dtype is launched
 * with on the current device for a launch of ordinary length (32-byte aligned buffers assumed;
 * block = 224 means the bulk-copy ring: 6 consumer warps + 1 producer warp; very short launches
 * may use a ring of 288 threads), and the number of kernels enqueued so far. */
int omni_query_launch(omni_ctx *ctx, int32_t K, int32_t grad_dtype, int32_t *grid, int32_t *block);
uint64_t omni_kernel_launches(const omni_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* OMNI_H_ */
