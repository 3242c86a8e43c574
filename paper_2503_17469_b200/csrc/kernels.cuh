// Streaming kernels of the weighted aggregate + update path (sm_100a).
//
// The work is HBM-bound: per parameter a synchronous step reads K gradient values plus theta and
// v and writes theta and v (4K+16 bytes in float, 2K+16 with bfloat16 gradients); an
// asynchronous arrival moves 12 or 20 bytes.  There is no data reuse and no contraction, so the
// design goal is bytes in flight: every thread issues all of its 128-bit loads (K gradient
// streams, theta, v) before the first dependent FMA, the grid is persistent (a multiple of the
// SM count) and walks tiles with a grid stride so that neighbouring CTAs touch neighbouring
// DRAM pages, and loads/stores carry streaming cache hints because nothing is read twice.
//
// Arithmetic is the ordered single-precision FMA chain documented in omni.h; the worker loop is
// unrolled at compile time (K is a template argument) so the chain order is fixed in the code.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/omni.h"

namespace omni {

constexpr int kThreads = 256;            // threads per CTA
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
    double partials[kMaxGrid];  // one squared-norm partial per CTA
    double sqnorm;              // result cell
    unsigned int ticket;        // CTAs finished in the current launch; reset by the last one
    unsigned int pad;
};

struct BspParams {
    BucketDesc bk[kMaxBucketsPerLaunch];
    const void *g[kMaxBucketsPerLaunch][OMNI_MAX_K];
    float lam[OMNI_MAX_K];
    float lr, mu, wd;
    int nb;
    int accumulate;  // 0: sqnorm = sum of this launch; 1: sqnorm += sum (later launch of one call)
    unsigned long long tiles;
    Workspace *ws;
};

struct AspParams {
    BucketDesc bk[kMaxBucketsPerLaunch];
    const void *g[kMaxBucketsPerLaunch];
    float eta, mu, wd;
    int nb;
    unsigned long long tiles;
};

// Elements one thread handles per 128-bit gradient load.
template <typename G> struct Vec { static constexpr int n = 16 / sizeof(G); };

// How many 128-bit vectors per stream a thread keeps in flight: small K gets more so that the
// bytes in flight per SM stay high.
__host__ __device__ constexpr int bsp_unroll(int K) { return K <= 2 ? 4 : K <= 5 ? 3 : K <= 10 ? 2 : 1; }
constexpr int kAspUnroll = 4;

template <typename G> __host__ __device__ constexpr unsigned long long bsp_tile(int K)
{
    return (unsigned long long)kThreads * Vec<G>::n * bsp_unroll(K);
}
template <typename G> __host__ __device__ constexpr unsigned long long asp_tile()
{
    return (unsigned long long)kThreads * Vec<G>::n * kAspUnroll;
}

// ---------------------------------------------------------------------------------------------
// loads / stores with streaming hints
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const void *p) { return __ldcs(reinterpret_cast<const uint4 *>(p)); }
__device__ __forceinline__ void st_stream(void *p, uint4 x) { __stcs(reinterpret_cast<uint4 *>(p), x); }
__device__ __forceinline__ void st_stream(void *p, uint2 x) { __stcs(reinterpret_cast<uint2 *>(p), x); }

__device__ __forceinline__ float bf16_lo(unsigned w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(unsigned w) { return __uint_as_float(w & 0xffff0000u); }

// One 128-bit gradient vector -> Vec<G>::n floats.
template <typename G> __device__ __forceinline__ void widen(const uint4 &r, float *out);
template <> __device__ __forceinline__ void widen<float>(const uint4 &r, float *o)
{
    o[0] = __uint_as_float(r.x); o[1] = __uint_as_float(r.y);
    o[2] = __uint_as_float(r.z); o[3] = __uint_as_float(r.w);
}
template <> __device__ __forceinline__ void widen<__nv_bfloat16>(const uint4 &r, float *o)
{
    o[0] = bf16_lo(r.x); o[1] = bf16_hi(r.x); o[2] = bf16_lo(r.y); o[3] = bf16_hi(r.y);
    o[4] = bf16_lo(r.z); o[5] = bf16_hi(r.z); o[6] = bf16_lo(r.w); o[7] = bf16_hi(r.w);
}
template <typename G> __device__ __forceinline__ float widen1(const G *p, unsigned long long j);
template <> __device__ __forceinline__ float widen1<float>(const float *p, unsigned long long j) { return __ldcs(p + j); }
template <> __device__ __forceinline__ float widen1<__nv_bfloat16>(const __nv_bfloat16 *p, unsigned long long j)
{
    return __uint_as_float((unsigned)__ldcs(reinterpret_cast<const unsigned short *>(p) + j) << 16);
}

__device__ __forceinline__ unsigned pack_bf16(float a, float b)
{
    const unsigned lo = __bfloat16_as_ushort(__float2bfloat16_rn(a));
    const unsigned hi = __bfloat16_as_ushort(__float2bfloat16_rn(b));
    return lo | (hi << 16);
}

// The update of one element after gbar is known.  Returns the new theta, writes the new v.
__device__ __forceinline__ float update_one(float gbar, float theta, float &v, float lr, float mu, float wd)
{
    const float d = wd != 0.0f ? __fmaf_rn(wd, theta, gbar) : gbar;
    const float vn = mu != 0.0f ? __fmaf_rn(mu, v, d) : d;
    v = vn;
    return __fmaf_rn(-lr, vn, theta);
}

template <int N> __device__ __forceinline__ void load_f32(const float *p, float *o)
{
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
        const uint4 r = ld_stream(p + 4 * i);
        o[4 * i] = __uint_as_float(r.x); o[4 * i + 1] = __uint_as_float(r.y);
        o[4 * i + 2] = __uint_as_float(r.z); o[4 * i + 3] = __uint_as_float(r.w);
    }
}
template <int N> __device__ __forceinline__ void store_f32(float *p, const float *o)
{
#pragma unroll
    for (int i = 0; i < N / 4; ++i)
        st_stream(p + 4 * i, make_uint4(__float_as_uint(o[4 * i]), __float_as_uint(o[4 * i + 1]),
                                        __float_as_uint(o[4 * i + 2]), __float_as_uint(o[4 * i + 3])));
}
template <int N> __device__ __forceinline__ void store_lp(__nv_bfloat16 *p, const float *o)
{
    if constexpr (N == 8)
        st_stream(p, make_uint4(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3]), pack_bf16(o[4], o[5]), pack_bf16(o[6], o[7])));
    else
        st_stream(p, make_uint2(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3])));
}

template <int NB> __device__ __forceinline__ int find_bucket(const BucketDesc *bk, int nb, unsigned long long tile)
{
    int bi = 0;
#pragma unroll
    for (int i = 1; i < NB; ++i)
        if (i < nb && tile >= bk[i].tile0) bi = i;
    return bi;
}

// ---------------------------------------------------------------------------------------------
// Synchronous step: K-way weighted sum + update + squared norm of the aggregate
// ---------------------------------------------------------------------------------------------
template <typename G, int K>
__global__ void __launch_bounds__(kThreads) bsp_fused_kernel(const __grid_constant__ BspParams p)
{
    constexpr int V = Vec<G>::n;
    constexpr int U = bsp_unroll(K);
    constexpr unsigned long long TILE = bsp_tile<G>(K);
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
            uint4 raw[U][K];
            float th[U][V], vv[U][V];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned long long off = base + (unsigned long long)(u * kThreads + tid) * V;
#pragma unroll
                for (int k = 0; k < K; ++k) raw[u][k] = ld_stream(static_cast<const G *>(p.g[bi][k]) + off);
                load_f32<V>(bd.theta + off, th[u]);
                if (mu != 0.0f) load_f32<V>(bd.v + off, vv[u]);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned long long off = base + (unsigned long long)(u * kThreads + tid) * V;
                float acc[V];
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = 0.0f;
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    float gk[V];
                    widen<G>(raw[u][k], gk);
                    const float lam = p.lam[k];
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[e] = __fmaf_rn(lam, gk[e], acc[e]);
                }
                float part = 0.0f;
#pragma unroll
                for (int e = 0; e < V; ++e) {
                    part = __fmaf_rn(acc[e], acc[e], part);
                    th[u][e] = update_one(acc[e], th[u][e], vv[u][e], lr, mu, wd);
                }
                sq += (double)part;
                store_f32<V>(bd.theta + off, th[u]);
                if (has_v) store_f32<V>(bd.v + off, vv[u]);
                if (has_lp) store_lp<V>(bd.lp + off, th[u]);
            }
        } else {
            // ragged last tile of a bucket: element by element, same arithmetic
            for (unsigned long long j = base + tid; j < bd.n; j += kThreads) {
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

    // squared norm: warp tree, CTA sum in warp order, one partial per CTA; the CTA that takes the
    // last ticket adds the partials in index order, so the result depends only on the grid size.
    __shared__ double wsum[kThreads / 32];
    __shared__ bool is_last;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
    if ((tid & 31) == 0) wsum[tid >> 5] = sq;
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) s += wsum[w];
        p.ws->partials[blockIdx.x] = s;
        __threadfence();
        const unsigned t = atomicAdd(&p.ws->ticket, 1u);
        is_last = t == gridDim.x - 1;
    }
    __syncthreads();
    if (is_last && tid < 32) {
        __threadfence();
        double s = 0.0;
        for (unsigned i = tid; i < gridDim.x; i += 32) s += __ldcg(&p.ws->partials[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
        if (tid == 0) {
            p.ws->sqnorm = p.accumulate ? p.ws->sqnorm + s : s;
            p.ws->ticket = 0u;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Asynchronous arrival: one gradient stream applied with eta_k
// ---------------------------------------------------------------------------------------------
template <typename G>
__global__ void __launch_bounds__(kThreads) asp_apply_kernel(const __grid_constant__ AspParams p)
{
    constexpr int V = Vec<G>::n;
    constexpr int U = kAspUnroll;
    constexpr unsigned long long TILE = asp_tile<G>();
    const int tid = threadIdx.x;
    const float eta = p.eta, mu = p.mu, wd = p.wd;

    for (unsigned long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
        const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
        const BucketDesc bd = p.bk[bi];
        const G *g = static_cast<const G *>(p.g[bi]);
        const unsigned long long base = (tile - bd.tile0) * TILE;
        const bool has_v = bd.v != nullptr, has_lp = bd.lp != nullptr;

        if (base + TILE <= bd.n) {
            uint4 raw[U];
            float th[U][V], vv[U][V];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned long long off = base + (unsigned long long)(u * kThreads + tid) * V;
                raw[u] = ld_stream(g + off);
                load_f32<V>(bd.theta + off, th[u]);
                if (mu != 0.0f) load_f32<V>(bd.v + off, vv[u]);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned long long off = base + (unsigned long long)(u * kThreads + tid) * V;
                float gk[V];
                widen<G>(raw[u], gk);
#pragma unroll
                for (int e = 0; e < V; ++e) th[u][e] = update_one(gk[e], th[u][e], vv[u][e], eta, mu, wd);
                store_f32<V>(bd.theta + off, th[u]);
                if (has_v) store_f32<V>(bd.v + off, vv[u]);
                if (has_lp) store_lp<V>(bd.lp + off, th[u]);
            }
        } else {
            for (unsigned long long j = base + tid; j < bd.n; j += kThreads) {
                float vj = mu != 0.0f ? __ldcs(bd.v + j) : 0.0f;
                const float t = update_one(widen1<G>(g, j), __ldcs(bd.theta + j), vj, eta, mu, wd);
                bd.theta[j] = t;
                if (has_v) bd.v[j] = vj;
                if (has_lp) bd.lp[j] = __float2bfloat16_rn(t);
            }
        }
    }
}

}  // namespace omni
