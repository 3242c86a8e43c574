// Proportional batch-size controller on the host.  K <= 32 scalars per call: microseconds.
//
// Floating point is IEEE double with one operation per statement where the order matters, sums
// in ascending worker order, and this file is compiled without multiply-add contraction, so
// the integer batch sizes are reproducible bit for bit.  After the single rounding step
// (to_integer) everything is integer arithmetic.
#include "controller.h"

#include <algorithm>
#include <cmath>
#include <numeric>

namespace omni {

int BatchController::validate(const omni_config &c)
{
    if (c.K < 1 || c.K > OMNI_MAX_K) return OMNI_ERR_BAD_K;
    if (c.global_batch < c.K || c.b_min < 1 || c.b_max < c.b_min) return OMNI_ERR_BAD_CONFIG;
    if (!(c.deadband >= 0.0) || !std::isfinite(c.deadband)) return OMNI_ERR_BAD_CONFIG;
    if (!(c.ewma_alpha > 0.0) || !(c.ewma_alpha <= 1.0)) return OMNI_ERR_BAD_CONFIG;
    if (c.mode != OMNI_BSP && c.mode != OMNI_ASP) return OMNI_ERR_BAD_CONFIG;
    constexpr uint32_t known = OMNI_UNSCALED_MEAN | OMNI_ASP_NO_LR_SCALE | OMNI_INPUT_IS_TIME | OMNI_BULK_COPY |
                               OMNI_NO_BULK_COPY | OMNI_CONSERVE_MULTIPLICATIVE;
    if (c.flags & ~known) return OMNI_ERR_BAD_CONFIG;
    if ((c.flags & OMNI_BULK_COPY) && (c.flags & OMNI_NO_BULK_COPY)) return OMNI_ERR_BAD_CONFIG;
    if (c.mode == OMNI_BSP) {
        const int64_t lo = int64_t(c.K) * c.b_min, hi = int64_t(c.K) * c.b_max;
        if (lo > c.global_batch || hi < c.global_batch) return OMNI_ERR_INFEASIBLE;
    }
    return OMNI_OK;
}

BatchController::BatchController(const omni_config &cfg) : cfg_(cfg)
{
    // Algorithm 1 / 2: b = B / K; a remainder is spread over the first workers.
    const int q = cfg.global_batch / cfg.K, r = cfg.global_batch % cfg.K;
    for (int k = 0; k < cfg.K; ++k) batch_[k] = q + (k < r);
}

int BatchController::set_batches(const int32_t *b)
{
    int64_t total = 0;
    for (int k = 0; k < cfg_.K; ++k) {
        if (b[k] < 1) return OMNI_ERR_BAD_BATCH;
        total += b[k];
    }
    if (cfg_.mode == OMNI_BSP && total != cfg_.global_batch) return OMNI_ERR_BAD_BATCH;
    std::copy(b, b + cfg_.K, batch_.begin());
    return OMNI_OK;
}

// Eq. 6a read backwards: a throughput T observed at batch b means a compute time t = b / T.
double BatchController::to_time(int32_t b, double measured) const
{
    if (cfg_.flags & OMNI_INPUT_IS_TIME) return measured;
    const double bd = double(b);
    return bd / measured;
}

// EWMA of the compute time (Algorithm 1, "EWMA(time() - t_init)"); the first sample seeds it.
double BatchController::smoothed(int k, double t, const std::array<double, OMNI_MAX_K> &cur,
                                 const std::array<bool, OMNI_MAX_K> &seen) const
{
    if (!seen[k]) return t;
    const double fresh = cfg_.ewma_alpha * t;
    const double keep = 1.0 - cfg_.ewma_alpha;
    const double old = keep * cur[k];
    return fresh + old;
}

int32_t BatchController::to_integer(double x) const
{
    double r = std::floor(x + 0.5);
    r = std::max(r, double(cfg_.b_min));
    r = std::min(r, double(cfg_.b_max));
    return int32_t(r);
}

// getBsz: throughput, proportional correction (Eq. 6b), dead-band (Eq. 7), bounds.
BatchController::Proposal BatchController::propose(int32_t b, double t, double tbar) const
{
    const double bd = double(b);
    const double throughput = bd / t;
    const double error = t - tbar;
    const double correction = throughput * error;
    const double target = bd - correction;
    const double rel = std::fabs((target - bd) / target);
    double chosen = bd;
    if (rel >= cfg_.deadband)
        chosen = target < double(cfg_.b_min) ? double(cfg_.b_min)
               : target > double(cfg_.b_max) ? double(cfg_.b_max) : target;
    return {target, chosen, to_integer(chosen)};
}

// Eq. 8 on integers with bounds.  The uniform shift Delta B / K is applied in blocks of whole
// rounds: all workers that can still move take `rounds` units each, where `rounds` stops at the
// first worker reaching its bound or when the gap no longer covers a full round.  The last
// partial round goes to the largest batches (lowest index first among equals).
int BatchController::close_gap(std::array<int32_t, OMNI_MAX_K> &n) const
{
    const int K = cfg_.K;
    int64_t gap = cfg_.global_batch - std::accumulate(n.begin(), n.begin() + K, int64_t(0));
    while (gap != 0) {
        const int dir = gap > 0 ? +1 : -1;
        const int32_t wall = dir > 0 ? cfg_.b_max : cfg_.b_min;
        int idx[OMNI_MAX_K], m = 0;
        int64_t room = INT64_MAX;
        for (int k = 0; k < K; ++k) {
            const int64_t r = int64_t(wall - n[k]) * dir;   // units until worker k is pinned
            if (r > 0) { idx[m++] = k; room = std::min(room, r); }
        }
        if (m == 0) return OMNI_ERR_INFEASIBLE;
        const int64_t need = gap * dir;
        const int64_t rounds = std::min(room, need / m);
        if (rounds > 0) {
            for (int i = 0; i < m; ++i) n[idx[i]] += int32_t(dir * rounds);
            gap -= dir * rounds * m;
            continue;
        }
        // fewer units than movable workers: largest batches first, ties by index
        std::stable_sort(idx, idx + m, [&](int a, int b) { return n[a] > n[b]; });
        for (int64_t i = 0; i < need; ++i) n[idx[i]] += dir;
        gap = 0;
    }
    return OMNI_OK;
}

int BatchController::rebatch(const double *measured, int32_t *new_b, int32_t *changed)
{
    const int K = cfg_.K;
    for (int k = 0; k < K; ++k)
        if (!std::isfinite(measured[k]) || !(measured[k] > 0.0)) return OMNI_ERR_BAD_MEASUREMENT;

    std::array<double, OMNI_MAX_K> t = time_;
    for (int k = 0; k < K; ++k) t[k] = smoothed(k, to_time(batch_[k], measured[k]), time_, seen_);
    double total = 0.0;
    for (int k = 0; k < K; ++k) total += t[k];
    const double tbar = total / double(K);

    std::array<int32_t, OMNI_MAX_K> n{};
    if (cfg_.mode == OMNI_BSP && (cfg_.flags & OMNI_CONSERVE_MULTIPLICATIVE)) {
        // the other reading of the sentence after Eq. 8: renormalise the real-valued getBsz
        // results to the global batch before the rounding step
        std::array<double, OMNI_MAX_K> c{};
        double csum = 0.0;
        for (int k = 0; k < K; ++k) c[k] = propose(batch_[k], t[k], tbar).chosen;
        for (int k = 0; k < K; ++k) csum += c[k];
        for (int k = 0; k < K; ++k) {
            const double scaled_up = c[k] * double(cfg_.global_batch);
            n[k] = to_integer(scaled_up / csum);
        }
    } else {
        for (int k = 0; k < K; ++k) n[k] = propose(batch_[k], t[k], tbar).rounded;
    }
    if (cfg_.mode == OMNI_BSP) {
        const int rc = close_gap(n);
        if (rc != OMNI_OK) return rc;
    }
    for (int k = 0; k < K; ++k) {
        if (changed) changed[k] = n[k] != batch_[k];
        new_b[k] = n[k];
        batch_[k] = n[k];
        time_[k] = t[k];
        seen_[k] = true;
    }
    return OMNI_OK;
}

int BatchController::report(int32_t worker, int32_t b_used, double measured, int32_t *new_b_k)
{
    const int K = cfg_.K;
    if (worker < 0 || worker >= K) return OMNI_ERR_BAD_WORKER;
    if (b_used < 1) return OMNI_ERR_BAD_BATCH;
    if (!std::isfinite(measured) || !(measured > 0.0)) return OMNI_ERR_BAD_MEASUREMENT;

    // evalBsz: wrkB[k] = b, wrkTime[k] = smoothed compute time
    time_[worker] = smoothed(worker, to_time(b_used, measured), time_, seen_);
    seen_[worker] = true;
    batch_[worker] = b_used;
    if (!std::all_of(seen_.begin(), seen_.begin() + K, [](bool s) { return s; })) {
        *new_b_k = b_used;
        return OMNI_OK;
    }
    double total = 0.0;
    for (int k = 0; k < K; ++k) total += time_[k];
    const double tbar = total / double(K);
    std::array<int32_t, OMNI_MAX_K> n{};
    for (int k = 0; k < K; ++k) n[k] = propose(batch_[k], time_[k], tbar).rounded;
    std::copy(n.begin(), n.begin() + K, batch_.begin());
    *new_b_k = batch_[worker];
    return OMNI_OK;
}

void BatchController::export_state(int32_t *b, double *time, int32_t *seen) const
{
    for (int k = 0; k < OMNI_MAX_K; ++k) {
        b[k] = batch_[k];
        time[k] = time_[k];
        seen[k] = seen_[k] ? 1 : 0;
    }
}

void BatchController::import_state(const int32_t *b, const double *time, const int32_t *seen)
{
    for (int k = 0; k < cfg_.K; ++k) {
        batch_[k] = b[k];
        time_[k] = time[k];
        seen_[k] = seen[k] != 0;
    }
}

// Eq. 4a: b_k = c_k / sum(c) * (K b) with K b = B.
int BatchController::rebatch_static(const double *capacity, int32_t *new_b)
{
    const int K = cfg_.K;
    double total = 0.0;
    for (int k = 0; k < K; ++k) {
        if (!std::isfinite(capacity[k]) || !(capacity[k] > 0.0)) return OMNI_ERR_BAD_MEASUREMENT;
        total += capacity[k];
    }
    std::array<int32_t, OMNI_MAX_K> n{};
    for (int k = 0; k < K; ++k) {
        const double share = capacity[k] / total;
        n[k] = to_integer(share * double(cfg_.global_batch));
    }
    if (cfg_.mode == OMNI_BSP) {
        const int rc = close_gap(n);
        if (rc != OMNI_OK) return rc;
    }
    std::copy(n.begin(), n.begin() + K, batch_.begin());
    std::copy(n.begin(), n.begin() + K, new_b);
    return OMNI_OK;
}

}  // namespace omni
