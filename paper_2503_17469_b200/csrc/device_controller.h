// Device-resident copy of the batch-size controller (internal to the library).
//
// The host controller (controller.cpp) is the default: K <= 32 scalars, microseconds.  When the
// per-worker measurements are produced on the GPU, or when a whole synchronous step (re-batch +
// aggregate + update) is to be enqueued or captured in a CUDA graph without a host round trip,
// the same procedure runs as a one-warp kernel on this state and leaves the weights lambda_k of
// Eq. 4b in device memory, where the fused step reads them.
#pragma once
#include <cstdint>

#include "../../include/omni.h"

namespace omni {

struct DeviceCtl {
    double time[OMNI_MAX_K];     // smoothed compute time per worker (EWMA of Algorithm 1)
    int32_t batch[OMNI_MAX_K];   // b_k
    int32_t seen[OMNI_MAX_K];    // 0 until the worker's first measurement has seeded the EWMA
    float lam[OMNI_MAX_K];       // lambda_k = float(b_k / sum b)  (1/K with OMNI_UNSCALED_MEAN)
    double weight_sum;           // sum of lam as doubles, ascending k (filled on the host side of a download)
    int32_t status;              // 0, or the omni_status of the first device re-batch that failed since the last read
    uint32_t rebatches;          // device re-batches that completed
};

// Enqueues the one-warp asynchronous report kernel (evalBsz); returns the cudaError_t as int.
int launch_device_report(DeviceCtl *ctl, const omni_config &cfg, int32_t worker, int32_t b_used, const double *measured_dev,
                         int32_t *new_b_dev, void *stream);

// Enqueues the one-warp re-batch kernel (device_controller.cu); returns the cudaError_t as int.
int launch_device_rebatch(DeviceCtl *ctl, const omni_config &cfg, const double *measured_dev, int32_t *new_b_dev,
                          void *stream);

}  // namespace omni
