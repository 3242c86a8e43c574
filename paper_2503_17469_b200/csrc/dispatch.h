// Kernel selection shared by the translation units of the library (internal).
#pragma once
#include "../../include/omni.h"

namespace omni {

using KernelFn = const void *;

// A kernel instantiation with the launch geometry that goes with it.
struct KernelInfo {
    KernelFn fn = nullptr;
    int threads = 0;
    int ctas_per_sm = 0;          // wanted CTAs per SM (capped by what fits)
    unsigned long long tile = 0;  // elements per tile
    unsigned smem = 0;            // dynamic shared memory per CTA, bytes
    bool dependent_launch = false;  // the kernel waits for its predecessor itself (griddepcontrol.wait): launch it
                                    // with programmatic stream serialization so that its set-up overlaps that tail
};

// Kernels are templates on the worker count (the ordered FMA chain is unrolled at compile time), so
// every selection by a run-time count is a switch over all of them.  The case lists live here,
// once: X(k) for every worker count / every length of a queue of asynchronous arrivals.
#define OMNI_FOR_EACH_K(X)                                                                                  \
    X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12) X(13) X(14) X(15) X(16)                  \
    X(17) X(18) X(19) X(20) X(21) X(22) X(23) X(24) X(25) X(26) X(27) X(28) X(29) X(30) X(31) X(32)
#define OMNI_FOR_EACH_QUEUE(X) \
    X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12) X(13) X(14) X(15) X(16)
static_assert(OMNI_MAX_K == 32 && OMNI_MAX_ASP_BATCH == 16, "the case lists above cover 1..32 and 1..16");

// Register-staged kernels (register_dispatch.cu): the synchronous step for K workers, the
// asynchronous apply of one arrival and of M queued arrivals, the push with overwrite.
// wide = every buffer is 32-byte aligned (256-bit loads and stores), else 128-bit.
KernelInfo bsp_kernel(int dtype, int K, bool wide);
KernelInfo seq_kernel(int dtype, int M, bool wide);
KernelInfo asp_kernel(int dtype, bool wide, bool momentum);
KernelInfo overwrite_kernel(int dtype, bool wide);

// Bulk-copy ring kernels (bulk_dispatch.cu): the synchronous step for K workers, and the
// asynchronous apply of M queued arrivals (M = 1: a single arrival; M <= OMNI_MAX_ASP_BATCH).
KernelInfo bulk_kernel(int dtype, int K);
KernelInfo bulk_seq_kernel(int dtype, int M);
// The synchronous ring kernel in its shape for short launches (larger tiles, two stages; the same
// kernel as bulk_kernel where no such shape fits), chosen when the regular shape would give a CTA
// at most short_launch_tiles_per_cta() tiles (rounded up), the larger tiles exactly half as many,
// and the larger tiles still number one per SM or more.
KernelInfo bulk_short_kernel(int dtype, int K);
int short_launch_tiles_per_cta();
// The synchronous ring kernel that reads its K weights from device memory (BspParams::lam_dev),
// where the device-side controller leaves them (device_controller.cu).
KernelInfo bulk_devlam_kernel(int dtype, int K);
KernelInfo bulk_devlam_short_kernel(int dtype, int K);   // the same in the short-launch shape
// The ring kernel as push with overwrite (Algorithm 2): one gradient stream, the snapshot in
// place of theta (BspParams::src), optional copy of the result back to the snapshot (::copy).
KernelInfo bulk_overwrite_kernel(int dtype);
// Whether the ring is the better choice for this many streams: its bulk copies must be at least
// 2 KB each (true for every K up to OMNI_MAX_K with the current ring geometry; 1 KB copies halve
// the bandwidth).
bool bulk_preferred(int dtype, int streams);

// Enqueues the one-warp kernel that adds the first `slots` per-CTA partials of the workspace in
// index order and stores the sum in *out (a device address: the workspace's own cell, or the
// caller's); returns the cudaError_t as int.
int launch_sqnorm_finalize(void *workspace, int slots, double *out, void *stream);

// Launches the bounded-wait diagnostic kernel (bulk_dispatch.cu); returns the cudaError_t as int.
int launch_expire_wait(void *workspace, unsigned attempts, void *stream);

}  // namespace omni
