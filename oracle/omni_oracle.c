/*
 * omni_oracle.c -- plain, single-threaded CPU statement of the OmniLearn data-parallel rules.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the yardstick the CUDA library is compared with and
 * the CPU baseline that the benchmark times.  The product never calls it, links it or includes
 * it, and it includes nothing of the product: every struct and constant is declared here.
 *
 * What it states (paper = "OmniLearn", arXiv 2503.17469):
 *   - weighted aggregation lambda_k = b_k / sum(b), gbar = sum_k lambda_k g_k      (Eq. 4b, 4c; Alg. 1)
 *   - the parameter update theta <- theta - eta * gbar, with the heavy-ball momentum and
 *     weight-decay form of the optimiser the paper trains with                     (Eq. 4c; Sec. IV-A)
 *   - the asynchronous per-arrival update with eta_k = eta * b_k / B               (Eq. 5b; Alg. 2)
 *   - the proportional batch-size controller: throughput T = b/t, error t - tbar,
 *     b* = b - T (t - tbar), dead-band, (b_min, b_max) bounds, global-batch rule   (Eq. 6, 7, 8; getBsz)
 *   - the parameter-server bookkeeping of evalBsz                                  (Alg. 2)
 *
 * Two arithmetic modes exist for the element-wise rules:
 *   *_f64 : every operation in IEEE double on double state.  This is the definition.
 *   *_f32 : the paper trains in single precision; this mode keeps theta and v in float and does
 *           one correctly rounded fused multiply-add per term, workers in ascending order.
 * The controller is IEEE double, round-to-nearest, sums in ascending worker order, compiled with
 * -ffp-contract=off so no multiply-add is fused; after one rounding step it is integer only.
 *
 * Readings of points the paper leaves open are marked "reading:" where they are taken.
 * Parity pins: tests check these functions against hand-derived cases, closed forms (b* = T tbar),
 * brute force on tiny inputs and a library optimiser; see tests/test_oracle_*.py.
 * Parity unpinned against the paper: the paper prints no controller trace and no aggregated
 * tensor, so the steps it leaves open -- rounding to integers, the order dead-band / bounds /
 * global-batch rule, Eq. 8 next to the bounds, and the multiplicative variant of that rule behind
 * ORACLE_FLAG_CONSERVE_MULTIPLICATIVE (oracle_rebatch, oracle_asp_report,
 * oracle_rebatch_static from the rounding step on) -- are pinned to this file's stated readings
 * through hand-derived cases, an exhaustive-search restatement of Eq. 8 and invariants, not to
 * numbers of the paper.  The element-wise rules (oracle_bsp_step_*, oracle_asp_apply_*,
 * oracle_asp_push_overwrite_*) are pinned to plain means, dyadic hand cases and a library optimiser.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAX_K 32

enum { ORACLE_MODE_BSP = 0, ORACLE_MODE_ASP = 1 };
enum {
    ORACLE_FLAG_UNSCALED_MEAN = 1u,   /* ablation: lambda_k = 1/K (Table "weighted aggregation") */
    ORACLE_FLAG_ASP_NO_LR_SCALE = 2u, /* ablation: eta_k = eta (Table "LR scaling in ASP")       */
    ORACLE_FLAG_INPUT_IS_TIME = 4u,   /* measurements are compute times, not throughputs         */
    ORACLE_FLAG_CONSERVE_MULTIPLICATIVE = 8u /* other reading of the sentence after Eq. 8, see oracle_rebatch */
};
enum {
    ORACLE_OK = 0,
    ORACLE_ERR_ARG = -1,
    ORACLE_ERR_INFEASIBLE = -2,
    ORACLE_ERR_MEASUREMENT = -3
};

/* Controller state: the inputs of Alg. 1 / Alg. 2 plus per-worker b_k and smoothed compute time. */
typedef struct {
    int32_t K;
    int32_t B;        /* global batch, sum of b_k in BSP */
    int32_t b_min, b_max;
    double deadband;  /* Delta b_k of Eq. 7, a fraction */
    double alpha;     /* EWMA weight of the newest sample, (0, 1]; 1 = no smoothing */
    int32_t mode;
    uint32_t flags;
    int32_t b[ORACLE_MAX_K];       /* current batch sizes (BSP), wrkB map (ASP) */
    double s[ORACLE_MAX_K];        /* smoothed compute time, wrkTime map (ASP) */
    int32_t seen[ORACLE_MAX_K];    /* has worker k ever reported a measurement */
} oracle_ctl;

/* ------------------------------------------------------------------------------------------- */
/* Controller                                                                                  */
/* ------------------------------------------------------------------------------------------- */

/* Alg. 1 / Alg. 2: every worker starts at B / K.
 * reading: when K does not divide B the first (B mod K) workers take one more sample. */
int oracle_ctl_init(oracle_ctl *c, int32_t K, int32_t B, int32_t b_min, int32_t b_max,
                    double deadband, double alpha, int32_t mode, uint32_t flags)
{
    if (!c || K < 1 || K > ORACLE_MAX_K || B < K || b_min < 1 || b_max < b_min) return ORACLE_ERR_ARG;
    if (!(deadband >= 0.0) || !(alpha > 0.0 && alpha <= 1.0)) return ORACLE_ERR_ARG;
    if (mode == ORACLE_MODE_BSP) {
        if ((int64_t)K * b_min > B || (int64_t)K * b_max < B) return ORACLE_ERR_INFEASIBLE;
    }
    memset(c, 0, sizeof *c);
    c->K = K; c->B = B; c->b_min = b_min; c->b_max = b_max;
    c->deadband = deadband; c->alpha = alpha; c->mode = mode; c->flags = flags;
    for (int k = 0; k < K; ++k) c->b[k] = B / K + (k < B % K ? 1 : 0);
    return ORACLE_OK;
}

int oracle_ctl_set_batches(oracle_ctl *c, const int32_t *b)
{
    int64_t sum = 0;
    for (int k = 0; k < c->K; ++k) {
        if (b[k] < 1) return ORACLE_ERR_ARG;
        sum += b[k];
    }
    if (c->mode == ORACLE_MODE_BSP && sum != c->B) return ORACLE_ERR_ARG;
    for (int k = 0; k < c->K; ++k) c->b[k] = b[k];
    return ORACLE_OK;
}

void oracle_ctl_get_batches(const oracle_ctl *c, int32_t *b)
{
    for (int k = 0; k < c->K; ++k) b[k] = c->b[k];
}

/* Compute time of one iteration from a measurement: Eq. 6a gives T = b / t, so t = b / T. */
static double measured_time(const oracle_ctl *c, int32_t b, double measured)
{
    if (c->flags & ORACLE_FLAG_INPUT_IS_TIME) return measured;
    return (double)b / measured;
}

/* EWMA of the compute time (Alg. 1 "EWMA(time() - t_init)").
 * reading: the first sample initialises the average; alpha weighs the newest sample. */
static void smooth(oracle_ctl *c, int k, double x)
{
    if (!c->seen[k]) { c->s[k] = x; c->seen[k] = 1; }
    else c->s[k] = c->alpha * x + (1.0 - c->alpha) * c->s[k];
}

/* getBsz of Alg. 1 for one worker, real-valued:
 *   T  = b / t                                   (Eq. 6a)
 *   b* = b - T (t - tbar)                        (Eq. 6b)
 *   if |(b* - b) / b*| >= deadband: clamp b* to [b_min, b_max], else keep b     (Eq. 7, bounds) */
static double get_bsz_real(const oracle_ctl *c, int32_t b, double t, double tbar, double *bstar_out)
{
    double T = (double)b / t;
    double err = t - tbar;
    double bstar = (double)b - T * err;
    double cand;
    if (bstar_out) *bstar_out = bstar;
    if (fabs((bstar - (double)b) / bstar) >= c->deadband) {
        if (bstar < (double)c->b_min) cand = (double)c->b_min;
        else if (bstar > (double)c->b_max) cand = (double)c->b_max;
        else cand = bstar;
    } else {
        cand = (double)b;
    }
    return cand;
}

/* The one rounding step to an integer.
 * reading: integer batch = floor(x + 1/2), clamped again so that rounding cannot leave the bounds. */
static int32_t to_integer_batch(const oracle_ctl *c, double cand)
{
    double r = floor(cand + 0.5);
    if (r < (double)c->b_min) r = (double)c->b_min;
    if (r > (double)c->b_max) r = (double)c->b_max;
    return (int32_t)r;
}

/* getBsz followed by the rounding step */
static int32_t get_bsz(const oracle_ctl *c, int32_t b, double t, double tbar, double *bstar_out)
{
    return to_integer_batch(c, get_bsz_real(c, b, t, tbar, bstar_out));
}

/* Eq. 8: keep sum(b) = B by taking Delta B / K off every worker.
 * reading: on integers with bounds, the shift is taken one unit at a time from every worker that
 * is not pinned at the bound in the direction of the shift; when fewer units remain than there
 * are such workers, the workers with the largest batches move (ties: lowest index). */
static int conserve_global_batch(const oracle_ctl *c, int32_t *n)
{
    int64_t D = c->B;
    for (int k = 0; k < c->K; ++k) D -= n[k];
    while (D != 0) {
        int dir = D > 0 ? 1 : -1;
        int movable[ORACLE_MAX_K], m = 0;
        for (int k = 0; k < c->K; ++k) {
            if (dir > 0 ? n[k] < c->b_max : n[k] > c->b_min) movable[m++] = k;
        }
        if (m == 0) return ORACLE_ERR_INFEASIBLE;
        int64_t need = D > 0 ? D : -D;
        if (need >= m) {
            for (int i = 0; i < m; ++i) n[movable[i]] += dir;
            D -= (int64_t)dir * m;
        } else {
            /* pick the `need` largest batches among movable, ties to the lowest index */
            int taken[ORACLE_MAX_K] = {0};
            for (int64_t u = 0; u < need; ++u) {
                int best = -1;
                for (int i = 0; i < m; ++i) {
                    int k = movable[i];
                    if (taken[k]) continue;
                    if (best < 0 || n[k] > n[best]) best = k;
                }
                taken[best] = 1;
            }
            for (int k = 0; k < c->K; ++k) if (taken[k]) n[k] += dir;
            D = 0;
        }
    }
    return ORACLE_OK;
}

/* One synchronous re-batch: getAvgComputeTime + getBsz for every worker + Eq. 8 (Alg. 1).
 * measured[k]: throughput of worker k in samples per time unit (or its compute time when the
 * INPUT_IS_TIME flag is set) observed while it ran batch b[k].
 * bstar_out (nullable) receives the real-valued b* of Eq. 6b, changed (nullable) 0/1 flags,
 * scaled_out (nullable) the real-valued batches after the multiplicative renormalisation below
 * (the getBsz values themselves without the flag).
 * A failed call leaves the state untouched.
 *
 * The sentence after Eq. 8 (Sec. III-B, "Control Stability") says the adjusted batches are
 * reduced "proportionately", while Eq. 8 itself subtracts the same Delta B / K from every worker.
 * reading (default): the equation.  reading (CONSERVE_MULTIPLICATIVE, synchronous mode only): the
 * real-valued getBsz results c_k of all workers are renormalised, c_k <- c_k * B / sum_i c_i,
 * before the rounding step; whatever rounding and the bounds then leave of the gap to B is closed
 * by the unit steps of the default reading.  From equal batches without dead-band and bounds this
 * lands on B * T_k / sum(T) in one step, i.e. Eq. 4a with the throughputs as capacities. */
int oracle_rebatch(oracle_ctl *c, const double *measured, int32_t *new_b, int32_t *changed,
                   double *bstar_out, double *scaled_out)
{
    oracle_ctl w = *c;
    int32_t n[ORACLE_MAX_K];
    for (int k = 0; k < w.K; ++k) {
        if (!isfinite(measured[k]) || !(measured[k] > 0.0)) return ORACLE_ERR_MEASUREMENT;
        smooth(&w, k, measured_time(&w, w.b[k], measured[k]));
    }
    double tsum = 0.0;
    for (int k = 0; k < w.K; ++k) tsum += w.s[k];
    double tbar = tsum / (double)w.K;
    if (w.mode == ORACLE_MODE_BSP && (w.flags & ORACLE_FLAG_CONSERVE_MULTIPLICATIVE)) {
        double cand[ORACLE_MAX_K], csum = 0.0;
        for (int k = 0; k < w.K; ++k)
            cand[k] = get_bsz_real(&w, w.b[k], w.s[k], tbar, bstar_out ? &bstar_out[k] : NULL);
        for (int k = 0; k < w.K; ++k) csum += cand[k];
        for (int k = 0; k < w.K; ++k) {
            double scaled = cand[k] * (double)w.B / csum;
            if (scaled_out) scaled_out[k] = scaled;
            n[k] = to_integer_batch(&w, scaled);
        }
    } else {
        for (int k = 0; k < w.K; ++k) {
            double cand = get_bsz_real(&w, w.b[k], w.s[k], tbar, bstar_out ? &bstar_out[k] : NULL);
            if (scaled_out) scaled_out[k] = cand;
            n[k] = to_integer_batch(&w, cand);
        }
    }
    if (w.mode == ORACLE_MODE_BSP) {
        int rc = conserve_global_batch(&w, n);
        if (rc != ORACLE_OK) return rc;
    }
    for (int k = 0; k < w.K; ++k) {
        if (changed) changed[k] = n[k] != c->b[k];
        w.b[k] = n[k];
        new_b[k] = n[k];
    }
    *c = w;
    return ORACLE_OK;
}

/* Static variable batching, Eq. 4a: b_k = c_k / sum_i c_i * K b, with K b the global batch B and
 * c_k the compute capacity of worker k (cores, FLOPs).
 * reading: the real-valued shares become integers the same way as in the dynamic controller
 * (clamp to the bounds, round half up, then the global-batch rule in synchronous mode). */
int oracle_rebatch_static(oracle_ctl *c, const double *capacity, int32_t *new_b)
{
    double csum = 0.0;
    int32_t n[ORACLE_MAX_K];
    for (int k = 0; k < c->K; ++k) {
        if (!isfinite(capacity[k]) || !(capacity[k] > 0.0)) return ORACLE_ERR_MEASUREMENT;
        csum += capacity[k];
    }
    for (int k = 0; k < c->K; ++k) {
        double x = capacity[k] / csum * (double)c->B;
        double r = floor(x + 0.5);
        if (r < (double)c->b_min) r = (double)c->b_min;
        if (r > (double)c->b_max) r = (double)c->b_max;
        n[k] = (int32_t)r;
    }
    if (c->mode == ORACLE_MODE_BSP) {
        int rc = conserve_global_batch(c, n);
        if (rc != ORACLE_OK) return rc;
    }
    for (int k = 0; k < c->K; ++k) { c->b[k] = n[k]; new_b[k] = n[k]; }
    return ORACLE_OK;
}

/* evalBsz of Alg. 2: worker k reports the batch it ran and its measurement; the server stores
 * both, and once every worker has an entry it re-evaluates getBsz for all K entries against the
 * mean stored time and returns the caller's entry.  No global-batch rule (Sec. IV-D, ASP).
 * reading: before all K have reported, the caller keeps its batch; entries are never cleared. */
int oracle_asp_report(oracle_ctl *c, int32_t worker, int32_t b_used, double measured,
                      int32_t *new_b)
{
    if (worker < 0 || worker >= c->K || b_used < 1) return ORACLE_ERR_ARG;
    if (!isfinite(measured) || !(measured > 0.0)) return ORACLE_ERR_MEASUREMENT;
    c->b[worker] = b_used;
    smooth(c, worker, measured_time(c, b_used, measured));
    int all = 1;
    for (int k = 0; k < c->K; ++k) all = all && c->seen[k];
    if (!all) { *new_b = b_used; return ORACLE_OK; }
    double tsum = 0.0;
    for (int k = 0; k < c->K; ++k) tsum += c->s[k];
    double tbar = tsum / (double)c->K;
    int32_t n[ORACLE_MAX_K];
    for (int k = 0; k < c->K; ++k) n[k] = get_bsz(c, c->b[k], c->s[k], tbar, NULL);
    for (int k = 0; k < c->K; ++k) c->b[k] = n[k];
    *new_b = c->b[worker];
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------- */
/* Weights                                                                                     */
/* ------------------------------------------------------------------------------------------- */

/* lambda_k = b_k / sum_i b_i (Eq. 4b); with the UNSCALED_MEAN ablation, 1 / K. */
static double lambda_of(int K, const int32_t *b, uint32_t flags, int k)
{
    if (flags & ORACLE_FLAG_UNSCALED_MEAN) return 1.0 / (double)K;
    int64_t B = 0;
    for (int i = 0; i < K; ++i) B += b[i];
    return (double)b[k] / (double)B;
}

void oracle_bsp_weights(int32_t K, const int32_t *b, uint32_t flags, double *lambda64, float *lambda32)
{
    for (int k = 0; k < K; ++k) {
        double l = lambda_of(K, b, flags, k);
        if (lambda64) lambda64[k] = l;
        if (lambda32) lambda32[k] = (float)l;
    }
}

/* eta_k = eta * b_k / B with B the configured global batch (Alg. 2, "eta_k = eta b / B"). */
double oracle_asp_lr(double lr, int32_t b_used, int32_t B, uint32_t flags)
{
    if (flags & ORACLE_FLAG_ASP_NO_LR_SCALE) return lr;
    return lr * (double)b_used / (double)B;
}

/* ------------------------------------------------------------------------------------------- */
/* bfloat16 (1 sign, 8 exponent, 7 mantissa bits: the upper half of an IEEE float)             */
/* ------------------------------------------------------------------------------------------- */

static float bf16_to_float(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round to nearest, ties to even; NaN stays a quiet NaN */
static uint16_t float_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

void oracle_float_to_bf16(const float *x, uint16_t *y, uint64_t n)
{
    for (uint64_t j = 0; j < n; ++j) y[j] = float_to_bf16(x[j]);
}

void oracle_bf16_to_float(const uint16_t *x, float *y, uint64_t n)
{
    for (uint64_t j = 0; j < n; ++j) y[j] = bf16_to_float(x[j]);
}

static double grad_at(const void *const *g, int dtype_bf16, int k, uint64_t j)
{
    if (dtype_bf16) return (double)bf16_to_float(((const uint16_t *)g[k])[j]);
    return (double)((const float *)g[k])[j];
}

/* ------------------------------------------------------------------------------------------- */
/* Synchronous step: weighted aggregation + update                                             */
/* ------------------------------------------------------------------------------------------- */

/* One BSP step in double (the definition).  Per element j:
 *   gbar = sum_{k ascending} lambda_k g_k[j]               (Eq. 4b/4c, Alg. 1 AllReduce of lambda g)
 *   d    = gbar + wd * theta[j]                            weight decay (Sec. IV-A)
 *   v[j] = mu * v[j] + d                                   momentum, dampening 0, no Nesterov
 *   theta[j] = theta[j] - lr * v[j]                        (Eq. 4c when mu = wd = 0, v = gbar)
 * reading: the paper's equations are plain SGD and name momentum/weight decay only as training
 * hyper-parameters; the heavy-ball form above is that of the optimiser it used.
 * v may be NULL only when mu == 0.  *sqnorm (nullable) = sum_j gbar^2.
 * g: K pointers to float (dtype_bf16 = 0) or bfloat16 bit patterns (dtype_bf16 = 1). */
void oracle_bsp_step_f64(int32_t K, uint64_t n, const void *const *g, int dtype_bf16,
                         const int32_t *b, uint32_t flags, double *theta, double *v,
                         double lr, double mu, double wd, double *sqnorm)
{
    double lam[ORACLE_MAX_K];
    for (int k = 0; k < K; ++k) lam[k] = lambda_of(K, b, flags, k);
    double sq = 0.0;
    for (uint64_t j = 0; j < n; ++j) {
        double gbar = 0.0;
        for (int k = 0; k < K; ++k) gbar += lam[k] * grad_at(g, dtype_bf16, k, j);
        double d = gbar + wd * theta[j];
        double vn = d;
        if (v) { vn = mu * v[j] + d; v[j] = vn; }
        theta[j] = theta[j] - lr * vn;
        sq += gbar * gbar;
    }
    if (sqnorm) *sqnorm = sq;
}

/* The same step in the paper's precision: float state, lambda rounded once to float, one
 * correctly rounded fused multiply-add per term, workers ascending.  theta_lp (nullable)
 * receives the updated parameter rounded to bfloat16.  sqnorm accumulates in double. */
void oracle_bsp_step_f32(int32_t K, uint64_t n, const void *const *g, int dtype_bf16,
                         const int32_t *b, uint32_t flags, float *theta, float *v,
                         uint16_t *theta_lp, float lr, float mu, float wd, double *sqnorm)
{
    float lam[ORACLE_MAX_K];
    for (int k = 0; k < K; ++k) lam[k] = (float)lambda_of(K, b, flags, k);
    double sq = 0.0;
    for (uint64_t j = 0; j < n; ++j) {
        float acc = 0.0f;
        for (int k = 0; k < K; ++k) acc = fmaf(lam[k], (float)grad_at(g, dtype_bf16, k, j), acc);
        float d = wd != 0.0f ? fmaf(wd, theta[j], acc) : acc;
        float vn = d;
        if (mu != 0.0f) vn = fmaf(mu, v[j], d);
        if (v) v[j] = vn;
        theta[j] = fmaf(-lr, vn, theta[j]);
        if (theta_lp) theta_lp[j] = float_to_bf16(theta[j]);
        sq += (double)acc * (double)acc;
    }
    if (sqnorm) *sqnorm = sq;
}

/* ------------------------------------------------------------------------------------------- */
/* Asynchronous arrival                                                                        */
/* ------------------------------------------------------------------------------------------- */

/* One arrival of worker k's gradient g (computed on b_used samples) applied to the server's
 * parameters with eta_k = eta * b_used / B (Eq. 5b; Alg. 2 "theta - eta_k g").
 * reading: the server applies the gradient to its current parameters; this equals the
 * pull / local-update / push-overwrite of Alg. 2 whenever nothing arrived in between.
 * reading: momentum, when used, is one server-side buffer; Alg. 2 itself is mu = 0. */
void oracle_asp_apply_f64(uint64_t n, const void *g, int dtype_bf16, int32_t b_used, int32_t B,
                          uint32_t flags, double *theta, double *v, double lr, double mu, double wd)
{
    double eta_k = oracle_asp_lr(lr, b_used, B, flags);
    const void *gp[1] = { g };
    for (uint64_t j = 0; j < n; ++j) {
        double d = grad_at(gp, dtype_bf16, 0, j) + wd * theta[j];
        double vn = d;
        if (v) { vn = mu * v[j] + d; v[j] = vn; }
        theta[j] = theta[j] - eta_k * vn;
    }
}

void oracle_asp_apply_f32(uint64_t n, const void *g, int dtype_bf16, int32_t b_used, int32_t B,
                          uint32_t flags, float *theta, float *v, uint16_t *theta_lp,
                          float lr, float mu, float wd)
{
    float eta_k = (float)oracle_asp_lr((double)lr, b_used, B, flags);
    const void *gp[1] = { g };
    for (uint64_t j = 0; j < n; ++j) {
        float gj = (float)grad_at(gp, dtype_bf16, 0, j);
        float d = wd != 0.0f ? fmaf(wd, theta[j], gj) : gj;
        float vn = d;
        if (mu != 0.0f) vn = fmaf(mu, v[j], d);
        if (v) v[j] = vn;
        theta[j] = fmaf(-eta_k, vn, theta[j]);
        if (theta_lp) theta_lp[j] = float_to_bf16(theta[j]);
    }
}

/* Algorithm 2 taken literally: the worker pulled the server parameters some updates ago (its
 * snapshot), computes theta_k = snapshot - eta_k g on its replica and pushes theta_k, and the
 * server OVERWRITES its parameters with it, so whatever other workers pushed since the pull is
 * lost.  theta (out) never enters the arithmetic.  Plain SGD as in Algorithm 2; the optional
 * weight-decay term acts on the replica: d = g + wd * snapshot. */
void oracle_asp_push_overwrite_f64(uint64_t n, const void *g, int dtype_bf16, int32_t b_used, int32_t B,
                                   uint32_t flags, double *theta, const double *snapshot, double lr, double wd)
{
    double eta_k = oracle_asp_lr(lr, b_used, B, flags);
    const void *gp[1] = { g };
    for (uint64_t j = 0; j < n; ++j) {
        double d = grad_at(gp, dtype_bf16, 0, j) + wd * snapshot[j];
        theta[j] = snapshot[j] - eta_k * d;
    }
}

void oracle_asp_push_overwrite_f32(uint64_t n, const void *g, int dtype_bf16, int32_t b_used, int32_t B,
                                   uint32_t flags, float *theta, const float *snapshot, uint16_t *theta_lp,
                                   float lr, float wd)
{
    float eta_k = (float)oracle_asp_lr((double)lr, b_used, B, flags);
    const void *gp[1] = { g };
    for (uint64_t j = 0; j < n; ++j) {
        float gj = (float)grad_at(gp, dtype_bf16, 0, j);
        float d = wd != 0.0f ? fmaf(wd, snapshot[j], gj) : gj;
        theta[j] = fmaf(-eta_k, d, snapshot[j]);
        if (theta_lp) theta_lp[j] = float_to_bf16(theta[j]);
    }
}

/* Staleness bookkeeping of the arrival stream: tau = server updates since the worker's last
 * read.  The paper defines no staleness-dependent factor, so tau is tallied, never multiplied in.
 * hist has 33 bins: 0..31 and one overflow bin. */
void oracle_tau_record(uint64_t *hist, int32_t *tau_max, int32_t tau)
{
    hist[tau < 32 ? tau : 32] += 1;
    if (tau > *tau_max) *tau_max = tau;
}

size_t oracle_ctl_sizeof(void) { return sizeof(oracle_ctl); }
