// Streaming kernels of the weighted aggregate + update path (sm_100a).
//
// The work is HBM-bound: per parameter a synchronous step reads K gradient values plus theta and
// v and writes theta and v (4K+16 bytes in float, 2K+16 with bfloat16 gradients); an
// asynchronous arrival moves 12 or 20 bytes.  There is no data reuse and no contraction, so the
// design goal is bytes in flight and DRAM-friendly request shapes:
//   - every thread issues all of its loads (K gradient streams, theta, v) before the first
//     dependent FMA;
//   - loads and stores are 256 bits wide (ld/st.global.v8.b32, new with sm_100) whenever all
//     buffers are 32-byte aligned, so one warp instruction covers 1 KB of one stream; a 128-bit
//     variant serves buffers that are only 16-byte aligned;
//   - nothing is read twice, so gradient loads go through the non-coherent path without L1
//     allocation and everything is marked evict-first in L2;
//   - the grid is persistent (SM count x resident CTAs) and walks tiles with a grid stride, so
//     that at any moment the whole GPU sweeps one narrow window of each stream.
//
// Arithmetic is the ordered single-precision FMA chain documented in omni.h; the worker loop is
// unrolled at compile time (K is a template argument) so the chain order is fixed in the code.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/omni.h"

namespace omni {

constexpr int kMaxBucketsPerLaunch = 8;  // bucket descriptors carried in the kernel parameters
constexpr int kMaxGrid = 148 * 16;       // upper bound of the persistent grid = partial-sum slots

struct BucketDesc {
    float *theta;
    float *v;
    __nv_bfloat16 *lp;
    unsigned long long n;      // elements
    unsigned long long tile0;  // index of the bucket's first tile in this launch
};

// Device workspace of one context.
struct Workspace {
    double partials[kMaxGrid];  // one squared-norm partial per CTA of the last synchronous step
    double sqnorm;              // their sum, written by sqnorm_finalize_kernel when the host asks for it
    unsigned int reserved;
    unsigned int status;        // set non-zero by a kernel whose bounded wait ran out
};

struct BspParams {
    BucketDesc bk[kMaxBucketsPerLaunch];
    const void *g[kMaxBucketsPerLaunch][OMNI_MAX_K];
    float lam[OMNI_MAX_K];
    float lr, mu, wd;
    int nb;
    int accumulate;  // partial-sum slots that earlier launches of the same call have written (a CTA below that
                     // index adds to its slot, the others overwrite theirs); 0 in a call's first launch
    int reverse;     // walk the tiles from the last to the first (see omni.cu: alternating sweeps)
    unsigned long long tiles;
    Workspace *ws;
    const float *lam_dev;  // device copy of the K weights (device-side controller), read instead of lam by the kernels built for it
    // push with overwrite on the ring (Algorithm 2): per bucket the snapshot the worker pulled
    // (read in place of theta) and, if the worker pulls again at once, where the result is copied
    const float *src[kMaxBucketsPerLaunch];
    float *copy[kMaxBucketsPerLaunch];
};

struct AspParams {
    BucketDesc bk[kMaxBucketsPerLaunch];
    const void *g[kMaxBucketsPerLaunch];
    float eta, mu, wd;
    int nb;
    unsigned long long tiles;
};

// ---------------------------------------------------------------------------------------------
// Launch shape per (gradient type, K): threads per CTA, gradient vectors per thread and stream,
// and CTAs per SM of the persistent grid.  Taken from timing scans on B200 over
// threads x vectors x CTAs/SM: bandwidth peaks at a moderate number of resident threads
// (about 500-770 thread-vectors per SM) and falls on both sides -- too few leave HBM latency
// uncovered, too many widen the window of DRAM pages open at once.
// ---------------------------------------------------------------------------------------------
struct Shape { int threads, chunks, ctas_per_sm; };

template <typename G> __host__ __device__ constexpr Shape bsp_shape(int K)
{
    if (sizeof(G) == 4) {
        if (K >= 20) return {256, 1, 3};
        if (K >= 11) return {192, 1, 3};
        if (K >= 7) return {128, 2, 2};
        if (K >= 3) return {128, 2, 3};
        if (K == 2) return {128, 4, 1};
        return {256, 2, 1};
    }
    if (K >= 12) return {192, 1, 3};
    if (K >= 5) return {128, 2, 1};
    return {192, 1, 3};
}
constexpr int kAspThreads = 256;
constexpr int kAspChunks = 2;
__host__ __device__ constexpr int asp_ctas_per_sm(bool momentum) { return momentum ? 1 : 2; }

// ---------------------------------------------------------------------------------------------
// 128- and 256-bit global memory access with streaming hints
// ---------------------------------------------------------------------------------------------
template <int WORDS> struct Raw { unsigned w[WORDS]; };

// read-only stream (gradients): non-coherent path
template <int WORDS> __device__ __forceinline__ Raw<WORDS> ld_ro(const void *p)
{
    Raw<WORDS> r;
    if constexpr (WORDS == 8)
        asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]), "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                     : "l"(p));
    else {
        const uint4 x = __ldcs(reinterpret_cast<const uint4 *>(p));
        r.w[0] = x.x; r.w[1] = x.y; r.w[2] = x.z; r.w[3] = x.w;
    }
    return r;
}
// buffers this kernel also writes (theta, v): coherent path
template <int WORDS> __device__ __forceinline__ Raw<WORDS> ld_rw(const void *p)
{
    Raw<WORDS> r;
    if constexpr (WORDS == 8)
        asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]), "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                     : "l"(p) : "memory");
    else {
        const uint4 x = __ldcs(reinterpret_cast<const uint4 *>(p));
        r.w[0] = x.x; r.w[1] = x.y; r.w[2] = x.z; r.w[3] = x.w;
    }
    return r;
}
template <int WORDS> __device__ __forceinline__ void st_words(void *p, const unsigned *w)
{
    if constexpr (WORDS == 8)
        asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                     :: "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "l"(p) : "memory");
    else if constexpr (WORDS == 4)
        __stcs(reinterpret_cast<uint4 *>(p), make_uint4(w[0], w[1], w[2], w[3]));
    else
        __stcs(reinterpret_cast<uint2 *>(p), make_uint2(w[0], w[1]));
}

// Vector geometry: one gradient vector is VB bytes = E elements; theta/v need E floats.
template <typename G, bool WIDE> struct Geo {
    static constexpr int VB = WIDE ? 32 : 16;
    static constexpr int GW = VB / 4;               // 32-bit words per gradient vector
    static constexpr int E = VB / int(sizeof(G));   // elements per vector
    static constexpr int FW = GW;                   // words per theta/v access (same width)
    static constexpr int FN = E / FW;               // theta/v accesses per vector (1 for float, 2 for bfloat16)
    static constexpr int LW = E / 2;                // words of the bfloat16 copy per vector
};

template <typename G, int GW> __device__ __forceinline__ void widen(const Raw<GW> &r, float *o)
{
    if constexpr (sizeof(G) == 4) {
#pragma unroll
        for (int i = 0; i < GW; ++i) o[i] = __uint_as_float(r.w[i]);
    } else {
#pragma unroll
        for (int i = 0; i < GW; ++i) {
            o[2 * i] = __uint_as_float(r.w[i] << 16);
            o[2 * i + 1] = __uint_as_float(r.w[i] & 0xffff0000u);
        }
    }
}
template <typename G> __device__ __forceinline__ float widen1(const G *p, unsigned long long j)
{
    if constexpr (sizeof(G) == 4) return __ldcs(reinterpret_cast<const float *>(p) + j);
    else return __uint_as_float((unsigned)__ldcs(reinterpret_cast<const unsigned short *>(p) + j) << 16);
}

template <int FW, int FN> __device__ __forceinline__ void load_floats(const float *p, float *o)
{
#pragma unroll
    for (int i = 0; i < FN; ++i) {
        const Raw<FW> r = ld_rw<FW>(p + FW * i);
#pragma unroll
        for (int j = 0; j < FW; ++j) o[FW * i + j] = __uint_as_float(r.w[j]);
    }
}
template <int FW, int FN> __device__ __forceinline__ void store_floats(float *p, const float *o)
{
#pragma unroll
    for (int i = 0; i < FN; ++i) {
        unsigned w[FW];
#pragma unroll
        for (int j = 0; j < FW; ++j) w[j] = __float_as_uint(o[FW * i + j]);
        st_words<FW>(p + FW * i, w);
    }
}
__device__ __forceinline__ unsigned pack_bf16(float a, float b)
{
    const unsigned lo = __bfloat16_as_ushort(__float2bfloat16_rn(a));
    const unsigned hi = __bfloat16_as_ushort(__float2bfloat16_rn(b));
    return lo | (hi << 16);
}
template <int LW> __device__ __forceinline__ void store_lp(__nv_bfloat16 *p, const float *o)
{
    unsigned w[LW];
#pragma unroll
    for (int i = 0; i < LW; ++i) w[i] = pack_bf16(o[2 * i], o[2 * i + 1]);
    st_words<LW>(p, w);
}

// The update of one element after gbar is known.  Returns the new theta, writes the new v.
__device__ __forceinline__ float update_one(float gbar, float theta, float &v, float lr, float mu, float wd)
{
    const float d = wd != 0.0f ? __fmaf_rn(wd, theta, gbar) : gbar;
    const float vn = mu != 0.0f ? __fmaf_rn(mu, v, d) : d;
    v = vn;
    return __fmaf_rn(-lr, vn, theta);
}

template <int NB> __device__ __forceinline__ int find_bucket(const BucketDesc *bk, int nb, unsigned long long tile)
{
    int bi = 0;
#pragma unroll
    for (int i = 1; i < NB; ++i)
        if (i < nb && tile >= bk[i].tile0) bi = i;
    return bi;
}

// Squared-norm epilogue: warp tree, CTA sum in warp order, one partial per CTA.  Nothing else
// happens inside the step: no fence, no atomic, no last-CTA pass (together they cost 2.7 us at the
// end of every launch, 40 % of a step on a cache-resident model).  The partials are added up in
// index order by sqnorm_finalize_kernel, which the host enqueues only when the norm is asked for;
// the result depends only on the grid sizes of the call's launches.
template <int THREADS> __device__ __forceinline__ void finish_sqnorm(double sq, Workspace *ws, int accumulate)
{
    __shared__ double wsum[THREADS / 32];
    const int tid = threadIdx.x;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
    if ((tid & 31) == 0) wsum[tid >> 5] = sq;
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) s += wsum[w];
        double *slot = &ws->partials[blockIdx.x];
        *slot = int(blockIdx.x) < accumulate ? *slot + s : s;
    }
}

// Sum of the first n per-CTA partials in a fixed order (lane-strided, then a shuffle tree): one warp.
__device__ __forceinline__ double ordered_partial_sum(const double *partials, int n)
{
    double s = 0.0;
    for (int i = threadIdx.x; i < n; i += 32) s += __ldcg(partials + i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    return s;
}

// ---------------------------------------------------------------------------------------------
// Synchronous step: K-way weighted sum + update + squared norm of the aggregate
// ---------------------------------------------------------------------------------------------
template <typename G, int K, int THREADS, int C, bool WIDE>
__global__ void __launch_bounds__(THREADS) bsp_fused_kernel(const __grid_constant__ BspParams p)
{
    using Ge = Geo<G, WIDE>;
    constexpr int E = Ge::E;
    constexpr unsigned long long TILE = (unsigned long long)THREADS * E * C;
    const int tid = threadIdx.x;
    const float lr = p.lr, mu = p.mu, wd = p.wd;
    double sq = 0.0;

    for (unsigned long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
        const BucketDesc bd = p.bk[bi];
        const unsigned long long base = (tile - bd.tile0) * TILE;
        const bool has_v = bd.v != nullptr, has_lp = bd.lp != nullptr;

        if (base + TILE <= bd.n) {
            // full tile: every load of this thread is issued before the first FMA
            Raw<Ge::GW> raw[C][K];
            float th[C][E], vv[C][E];
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
#pragma unroll
                for (int k = 0; k < K; ++k) raw[c][k] = ld_ro<Ge::GW>(static_cast<const G *>(p.g[bi][k]) + off);
                load_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (mu != 0.0f) load_floats<Ge::FW, Ge::FN>(bd.v + off, vv[c]);
            }
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                float acc[E];
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = 0.0f;
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    float gk[E];
                    widen<G, Ge::GW>(raw[c][k], gk);
                    const float lam = p.lam[k];
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[e] = __fmaf_rn(lam, gk[e], acc[e]);
                }
                float part = 0.0f;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    part = __fmaf_rn(acc[e], acc[e], part);
                    th[c][e] = update_one(acc[e], th[c][e], vv[c][e], lr, mu, wd);
                }
                sq += (double)part;
                store_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (has_v) store_floats<Ge::FW, Ge::FN>(bd.v + off, vv[c]);
                if (has_lp) store_lp<Ge::LW>(bd.lp + off, th[c]);
            }
        } else {
            // ragged last tile of a bucket: whole vectors as above (one chunk at a time), then the
            // last partial vector element by element; same arithmetic
#pragma unroll 1
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                if (off + E <= bd.n) {
                    Raw<Ge::GW> raw[K];
                    float th[E], vv[E], acc[E];
#pragma unroll
                    for (int k = 0; k < K; ++k) raw[k] = ld_ro<Ge::GW>(static_cast<const G *>(p.g[bi][k]) + off);
                    load_floats<Ge::FW, Ge::FN>(bd.theta + off, th);
                    if (mu != 0.0f) load_floats<Ge::FW, Ge::FN>(bd.v + off, vv);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[e] = 0.0f;
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        float gk[E];
                        widen<G, Ge::GW>(raw[k], gk);
                        const float lam = p.lam[k];
#pragma unroll
                        for (int e = 0; e < E; ++e) acc[e] = __fmaf_rn(lam, gk[e], acc[e]);
                    }
                    float part = 0.0f;
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        part = __fmaf_rn(acc[e], acc[e], part);
                        th[e] = update_one(acc[e], th[e], vv[e], lr, mu, wd);
                    }
                    sq += (double)part;
                    store_floats<Ge::FW, Ge::FN>(bd.theta + off, th);
                    if (has_v) store_floats<Ge::FW, Ge::FN>(bd.v + off, vv);
                    if (has_lp) store_lp<Ge::LW>(bd.lp + off, th);
                } else {
                    for (unsigned long long j = off; j < bd.n; ++j) {
                        float acc = 0.0f;
#pragma unroll
                        for (int k = 0; k < K; ++k)
                            acc = __fmaf_rn(p.lam[k], widen1<G>(static_cast<const G *>(p.g[bi][k]), j), acc);
                        float vj = mu != 0.0f ? __ldcs(bd.v + j) : 0.0f;
                        const float t = update_one(acc, __ldcs(bd.theta + j), vj, lr, mu, wd);
                        sq += (double)(acc * acc);
                        bd.theta[j] = t;
                        if (has_v) bd.v[j] = vj;
                        if (has_lp) bd.lp[j] = __float2bfloat16_rn(t);
                    }
                }
            }
        }
    }
    finish_sqnorm<THREADS>(sq, p.ws, p.accumulate);
}

// ---------------------------------------------------------------------------------------------
// Asynchronous arrival: one gradient stream applied with eta_k
// ---------------------------------------------------------------------------------------------
template <typename G, int THREADS, int C, bool WIDE>
__global__ void __launch_bounds__(THREADS) asp_apply_kernel(const __grid_constant__ AspParams p)
{
    using Ge = Geo<G, WIDE>;
    constexpr int E = Ge::E;
    constexpr unsigned long long TILE = (unsigned long long)THREADS * E * C;
    const int tid = threadIdx.x;
    const float eta = p.eta, mu = p.mu, wd = p.wd;

    for (unsigned long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
        const BucketDesc bd = p.bk[bi];
        const G *g = static_cast<const G *>(p.g[bi]);
        const unsigned long long base = (tile - bd.tile0) * TILE;
        const bool has_v = bd.v != nullptr, has_lp = bd.lp != nullptr;

        if (base + TILE <= bd.n) {
            Raw<Ge::GW> raw[C];
            float th[C][E], vv[C][E];
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                raw[c] = ld_ro<Ge::GW>(g + off);
                load_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (mu != 0.0f) load_floats<Ge::FW, Ge::FN>(bd.v + off, vv[c]);
            }
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                float gk[E];
                widen<G, Ge::GW>(raw[c], gk);
#pragma unroll
                for (int e = 0; e < E; ++e) th[c][e] = update_one(gk[e], th[c][e], vv[c][e], eta, mu, wd);
                store_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (has_v) store_floats<Ge::FW, Ge::FN>(bd.v + off, vv[c]);
                if (has_lp) store_lp<Ge::LW>(bd.lp + off, th[c]);
            }
        } else {
            // ragged last tile: whole vectors one chunk at a time, then the partial vector
#pragma unroll 1
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                if (off + E <= bd.n) {
                    float th[E], vv[E], gk[E];
                    const Raw<Ge::GW> raw = ld_ro<Ge::GW>(g + off);
                    load_floats<Ge::FW, Ge::FN>(bd.theta + off, th);
                    if (mu != 0.0f) load_floats<Ge::FW, Ge::FN>(bd.v + off, vv);
                    widen<G, Ge::GW>(raw, gk);
#pragma unroll
                    for (int e = 0; e < E; ++e) th[e] = update_one(gk[e], th[e], vv[e], eta, mu, wd);
                    store_floats<Ge::FW, Ge::FN>(bd.theta + off, th);
                    if (has_v) store_floats<Ge::FW, Ge::FN>(bd.v + off, vv);
                    if (has_lp) store_lp<Ge::LW>(bd.lp + off, th);
                } else {
                    for (unsigned long long j = off; j < bd.n; ++j) {
                        float vj = mu != 0.0f ? __ldcs(bd.v + j) : 0.0f;
                        const float t = update_one(widen1<G>(g, j), __ldcs(bd.theta + j), vj, eta, mu, wd);
                        bd.theta[j] = t;
                        if (has_v) bd.v[j] = vj;
                        if (has_lp) bd.lp[j] = __float2bfloat16_rn(t);
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Batched asynchronous apply: M queued arrivals in one pass.  Same streaming skeleton as the
// synchronous kernel (M gradient streams + theta + v), but instead of one weighted sum followed
// by one update, each element goes through the M per-arrival updates in order with theta and v
// held in registers: bit-identical to M single-arrival launches at 4M+8 (+8 with momentum)
// bytes per parameter instead of 12M (20M).  p.lam[k] carries eta_k.  No norm is produced.
// ---------------------------------------------------------------------------------------------
template <typename G, int M, int THREADS, int C, bool WIDE>
__global__ void __launch_bounds__(THREADS) asp_batch_kernel(const __grid_constant__ BspParams p)
{
    using Ge = Geo<G, WIDE>;
    constexpr int E = Ge::E;
    constexpr unsigned long long TILE = (unsigned long long)THREADS * E * C;
    const int tid = threadIdx.x;
    const float mu = p.mu, wd = p.wd;

    for (unsigned long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
        const BucketDesc bd = p.bk[bi];
        const unsigned long long base = (tile - bd.tile0) * TILE;
        const bool has_v = bd.v != nullptr, has_lp = bd.lp != nullptr;

        if (base + TILE <= bd.n) {
            Raw<Ge::GW> raw[C][M];
            float th[C][E], vv[C][E];
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
#pragma unroll
                for (int k = 0; k < M; ++k) raw[c][k] = ld_ro<Ge::GW>(static_cast<const G *>(p.g[bi][k]) + off);
                load_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (mu != 0.0f) load_floats<Ge::FW, Ge::FN>(bd.v + off, vv[c]);
            }
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
#pragma unroll
                for (int k = 0; k < M; ++k) {
                    float gk[E];
                    widen<G, Ge::GW>(raw[c][k], gk);
                    const float eta = p.lam[k];
#pragma unroll
                    for (int e = 0; e < E; ++e) th[c][e] = update_one(gk[e], th[c][e], vv[c][e], eta, mu, wd);
                }
                store_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (has_v) store_floats<Ge::FW, Ge::FN>(bd.v + off, vv[c]);
                if (has_lp) store_lp<Ge::LW>(bd.lp + off, th[c]);
            }
        } else {
            // ragged last tile: whole vectors one chunk at a time, then the partial vector
#pragma unroll 1
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                if (off + E <= bd.n) {
                    Raw<Ge::GW> raw[M];
                    float th[E], vv[E];
#pragma unroll
                    for (int k = 0; k < M; ++k) raw[k] = ld_ro<Ge::GW>(static_cast<const G *>(p.g[bi][k]) + off);
                    load_floats<Ge::FW, Ge::FN>(bd.theta + off, th);
                    if (mu != 0.0f) load_floats<Ge::FW, Ge::FN>(bd.v + off, vv);
#pragma unroll
                    for (int k = 0; k < M; ++k) {
                        float gk[E];
                        widen<G, Ge::GW>(raw[k], gk);
                        const float eta = p.lam[k];
#pragma unroll
                        for (int e = 0; e < E; ++e) th[e] = update_one(gk[e], th[e], vv[e], eta, mu, wd);
                    }
                    store_floats<Ge::FW, Ge::FN>(bd.theta + off, th);
                    if (has_v) store_floats<Ge::FW, Ge::FN>(bd.v + off, vv);
                    if (has_lp) store_lp<Ge::LW>(bd.lp + off, th);
                } else {
                    for (unsigned long long j = off; j < bd.n; ++j) {
                        float vj = mu != 0.0f ? __ldcs(bd.v + j) : 0.0f;
                        float t = __ldcs(bd.theta + j);
#pragma unroll
                        for (int k = 0; k < M; ++k)
                            t = update_one(widen1<G>(static_cast<const G *>(p.g[bi][k]), j), t, vj, p.lam[k], mu, wd);
                        bd.theta[j] = t;
                        if (has_v) bd.v[j] = vj;
                        if (has_lp) bd.lp[j] = __float2bfloat16_rn(t);
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Asynchronous push with overwrite (Algorithm 2 taken literally): the server copy is replaced by
// snapshot - eta_k * (g + wd * snapshot), where snapshot is what the worker pulled earlier.
// Reads snapshot and g, writes theta (and the bf16 copy): 12 bytes per parameter.
// ---------------------------------------------------------------------------------------------
struct OverwriteParams {
    BucketDesc bk[kMaxBucketsPerLaunch];      // theta = destination; v unused
    const void *g[kMaxBucketsPerLaunch];
    const float *snap[kMaxBucketsPerLaunch];
    float eta, wd;
    int nb;
    unsigned long long tiles;
};

template <typename G, int THREADS, int C, bool WIDE>
__global__ void __launch_bounds__(THREADS) asp_overwrite_kernel(const __grid_constant__ OverwriteParams p)
{
    using Ge = Geo<G, WIDE>;
    constexpr int E = Ge::E;
    constexpr unsigned long long TILE = (unsigned long long)THREADS * E * C;
    const int tid = threadIdx.x;
    const float eta = p.eta, wd = p.wd;

    for (unsigned long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
        const BucketDesc bd = p.bk[bi];
        const G *g = static_cast<const G *>(p.g[bi]);
        const float *snap = p.snap[bi];
        const unsigned long long base = (tile - bd.tile0) * TILE;
        const bool has_lp = bd.lp != nullptr;

        if (base + TILE <= bd.n) {
            Raw<Ge::GW> raw[C];
            float th[C][E];
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                raw[c] = ld_ro<Ge::GW>(g + off);
                load_floats<Ge::FW, Ge::FN>(snap + off, th[c]);
            }
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                float gk[E], unused;
                widen<G, Ge::GW>(raw[c], gk);
#pragma unroll
                for (int e = 0; e < E; ++e) th[c][e] = update_one(gk[e], th[c][e], unused, eta, 0.0f, wd);
                store_floats<Ge::FW, Ge::FN>(bd.theta + off, th[c]);
                if (has_lp) store_lp<Ge::LW>(bd.lp + off, th[c]);
            }
        } else {
#pragma unroll 1
            for (int c = 0; c < C; ++c) {
                const unsigned long long off = base + (unsigned long long)(c * THREADS + tid) * E;
                for (unsigned long long j = off; j < bd.n && j < off + E; ++j) {
                    float unused;
                    const float t = update_one(widen1<G>(g, j), __ldcs(snap + j), unused, eta, 0.0f, wd);
                    bd.theta[j] = t;
                    if (has_lp) bd.lp[j] = __float2bfloat16_rn(t);
                }
            }
        }
    }
}

}  // namespace omni
