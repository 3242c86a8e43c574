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
    bool dependent_launch = false;  // the kernel waits for its predecessor itself (griddepcontrol.wait): launch it
                                    // with programmatic stream serialization so that its set-up overlaps that tail
};

// Bulk-copy ring kernels (bulk_dispatch.cu): the synchronous step for K workers, and the
// asynchronous apply of M queued arrivals (M = 1: a single arrival; M <= OMNI_MAX_ASP_BATCH).
KernelInfo bulk_kernel(int dtype, int K);
KernelInfo bulk_seq_kernel(int dtype, int M);
// The synchronous ring kernel that reads its K weights from device memory (BspParams::lam_dev),
// where the device-side controller leaves them (device_controller.cu).
KernelInfo bulk_devlam_kernel(int dtype, int K);
// The ring kernel as push with overwrite (Algorithm 2): one gradient stream, the snapshot in
// place of theta (BspParams::src), optional copy of the result back to the snapshot (::copy).
KernelInfo bulk_overwrite_kernel(int dtype);
// Whether the ring is the better choice for this many streams: its bulk copies must be at least
// 2 KB each (true for every K up to OMNI_MAX_K with the current ring geometry; 1 KB copies halve
// the bandwidth).
bool bulk_preferred(int dtype, int streams);

// Launches the bounded-wait diagnostic kernel (bulk_dispatch.cu); returns the cudaError_t as int.
int launch_expire_wait(void *workspace, unsigned attempts, void *stream);

}  // namespace omni
