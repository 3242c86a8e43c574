// Host-side proportional batch-size controller (paper Eq. 6-8; getBsz / evalBsz).
// Internal to the library; the public face is include/omni.h.
#pragma once
#include <array>
#include <cstdint>

#include "../../include/omni.h"

namespace omni {

class BatchController {
public:
    // Validates the configuration; returns an omni_status.
    static int validate(const omni_config &cfg);
    explicit BatchController(const omni_config &cfg);

    int K() const { return cfg_.K; }
    int B() const { return cfg_.global_batch; }
    const omni_config &config() const { return cfg_; }
    const int32_t *batches() const { return batch_.data(); }

    int set_batches(const int32_t *b);
    // Algorithm 1: all K measurements at once, then Eq. 8 in synchronous mode.
    int rebatch(const double *measured, int32_t *new_b, int32_t *changed);
    // Algorithm 2, evalBsz: one worker reports.
    int report(int32_t worker, int32_t b_used, double measured, int32_t *new_b_k);
    // Eq. 4a: open-loop split of B by capacity.
    int rebatch_static(const double *capacity, int32_t *new_b);
    // Whole state (batches, smoothed times, which workers have a time yet), for the copy of the
    // controller that lives on the device.  Arrays of OMNI_MAX_K entries.
    void export_state(int32_t *b, double *time, int32_t *seen) const;
    void import_state(const int32_t *b, const double *time, const int32_t *seen);

private:
    struct Proposal { double real; double chosen; int32_t rounded; };   // b* of Eq. 6b; after dead-band and bounds; as an integer
    double to_time(int32_t b, double measured) const;
    double smoothed(int k, double t, const std::array<double, OMNI_MAX_K> &cur,
                    const std::array<bool, OMNI_MAX_K> &seen) const;
    Proposal propose(int32_t b, double t, double tbar) const;
    int32_t to_integer(double x) const;
    int close_gap(std::array<int32_t, OMNI_MAX_K> &n) const;

    omni_config cfg_;
    std::array<int32_t, OMNI_MAX_K> batch_{};
    std::array<double, OMNI_MAX_K> time_{};
    std::array<bool, OMNI_MAX_K> seen_{};
};

}  // namespace omni
