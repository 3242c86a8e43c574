// Bulk-copy (TMA) variant of the synchronous fused step.
//
// One producer warp streams tiles of all K gradient buffers plus theta and v into a ring of
// shared-memory stages with 1-D bulk copies (cp.async.bulk, completion counted on an mbarrier);
// consumer warps take full stages, run the ordered FMA chain and the update out of shared
// memory and write theta / v / the bf16 copy straight to global memory.  The amount of data in
// flight per SM is fixed by the ring (stages x stage bytes), not by how the compiler schedules
// loads, and every request to DRAM is a contiguous burst of 2-8 KB of one stream.
//
// SEQ = true is the asynchronous apply on the same ring: the K streams are K queued arrivals
// (K = 1: a single arrival), lam[k] carries eta_k, and each element goes through the K
// per-arrival updates in order instead of one weighted sum and one update; no norm is produced.
//
// OVW = true (with SEQ, one stream, no momentum) is the push with overwrite of Algorithm 2 on the
// same ring: the "theta" slot of a stage is filled from the worker's snapshot (p.src) instead of
// the server copy, the result replaces the server copy, and where p.copy is set it is also
// written there (the worker's pull that follows its push, fused into the same pass).
//
// Every wait on an mbarrier is bounded: when the limit is hit the thread records it in the
// workspace status word and leaves the kernel; the host reports OMNI_ERR_TIMEOUT.
// Bulk copies need 16-byte aligned addresses and sizes, which the library's alignment contract
// gives for full tiles; the ragged last tile of a bucket is read with ordinary loads.
#pragma once
#include "kernels.cuh"

namespace omni {

constexpr unsigned kTmaWaitLimit = 1u << 22;  // try_wait attempts before giving up (seconds, far beyond any real wait)
constexpr unsigned kStatusTimeout = 1u;

__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long *b, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *b, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *b)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *b, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_addr(b)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; false = gave up.
__device__ __forceinline__ bool mbar_wait(unsigned long long *b, unsigned parity)
{
    for (unsigned i = 0; i < kTmaWaitLimit; ++i)
        if (mbar_try_wait(b, parity)) return true;
    return false;
}
// L2 eviction policies: gradients are read once (evict first); theta and v come back in the
// next launch (evict last), see the alternating sweeps in omni.cu.
__device__ __forceinline__ unsigned long long policy_evict_first()
{
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ unsigned long long policy_evict_last()
{
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gmem_src, unsigned bytes, unsigned long long *bar,
                                          unsigned long long policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy) : "memory");
}
// 16-byte stores of floats with an L2 policy
template <int N> __device__ __forceinline__ void store_floats_policy(float *p, const float *o, unsigned long long policy)
{
#pragma unroll
    for (int i = 0; i < N / 4; ++i)
        asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1,%2,%3,%4}, %5;"
                     ::"l"(p + 4 * i), "r"(__float_as_uint(o[4 * i])), "r"(__float_as_uint(o[4 * i + 1])),
                       "r"(__float_as_uint(o[4 * i + 2])), "r"(__float_as_uint(o[4 * i + 3])), "l"(policy) : "memory");
}

struct TmaShape { int tile, stages, consumer_warps; };

// Ring geometry per (gradient type, K).  Timing scans on B200: what matters is the size of each
// bulk copy (4 KB or more per gradient stream is as fast as the register kernel, 2 KB costs
// 2-3 %, 1 KB halves the bandwidth) and about 150 KB in flight per SM; more stages do not help.
// So: the largest tile whose stage stays within 80 KB, and as many stages as make ~150 KB
// (halving the stage size or a 110 KB ring cost 3-5 % in back-to-back runs; with 4 KB copies a
// larger ring loses 1-4 %).  Where that rule leaves copies of 2 KB (float K > 18, bfloat16
// K > 16), a tile of one and a half times the size -- 3 KB copies, two stages of up to 108 KB --
// wins 2-4 % (float K = 24: 7.10 vs 6.95 TB/s, K = 32: 6.93 vs 6.68; bfloat16 K = 32: 6.85 vs
// 6.63), while 4 KB copies in a 213 KB ring lose again (float K = 24: 6.88).  Six consumer
// warps.  Scan of 4 / 6 / 8 warps on 25.6 M parameters (us per step, back to back; cold = L2
// flushed before every step): bfloat16 K = 8 106.6 / 106.3 / 109.1 (cold 122.9 / 122.9 / 124.9),
// bfloat16 K = 16 167.0 / 167.1 / 168.2 (cold 185.3 / 184.4 / 187.3), bfloat16 K = 32 295.6 /
// 291.1 / 293.7, bfloat16 K = 4 81.4 / 82.1 / 82.4, float K = 8 165.9 / 166.4 / 166.9, float
// K = 24 402.3 / 399.2 / 400.0, float K = 1, 4, 16 within 0.5 %; four warps lose 2.7 % at float
// K = 2 (83.3 / 81.3 / 81.1) and sixteen were slower on bfloat16.  Six is never behind eight by
// more than 0.4 % and ahead by up to 2.6 %: fewer resident warps spinning on barriers under the
// power cap.  (The short-launch shape below keeps eight: 4.41 us against 4.67 with six.)
template <typename G> __host__ __device__ constexpr TmaShape tma_shape(int K)
{
    const int per_elem = K * int(sizeof(G)) + 8;
    int tile = 4096;
    while (tile > 256 && tile * per_elem > 80 * 1024) tile /= 2;
    if (tile * int(sizeof(G)) < 4096 && 2 * (tile * 3 / 2) * per_elem <= 216 * 1024) tile = tile * 3 / 2;
    const int stage = tile * per_elem;
    int stages = (152 * 1024 + stage / 2) / stage;
    // float K = 12, 13: three 56-60 KB stages (168-180 KB) lose 3 % to two (7.03 vs 7.22, 6.98 vs 7.23 TB/s)
    if (sizeof(G) == 4 && tile == 1024 && stages * stage > 160 * 1024) stages = 2;
    if (stages < 2) stages = 2;
    if (stages > 8) stages = 8;
    return {tile, stages, 6};
}
// Short launches.  A launch that gives every CTA only a handful of tiles never reaches the ring's
// steady state: its time is a few rounds of "fill a stage, consume it", and what counts is how
// much each round moves.  Where two stages of twice the regular tile still fit in shared memory
// (float K = 4; bfloat16 K = 7, 8 -- smaller K already use 4096-element tiles, larger K do not
// fit), that shape is used for such launches: on the cache-resident 2^20-parameter K = 4 model,
// captured in a CUDA graph, 4096 x 2 runs a step in 4.40 us against 4.85 us for 2048 x 3 (and
// 4.55 us for 2048 x 4, 5.2-5.4 us for 2048 x 2 and 1536 x 4; tiles of 1024 and 512 elements, which
// balance the last wave better, were slower still: 8.0 and 11.4 us against 6.7 us before the norm's
// final sum left the kernel).  A short launch costs about a fixed part plus its number of
// fill-consume rounds (tiles per CTA, rounded up) times a cost per round that is 1.6 times higher
// for the large tiles, so the large tiles pay when they halve the number of rounds exactly and
// lose when the regular count is odd: 2^19 parameters (2 regular rounds, fewer large tiles than
// SMs) tie at 3.1 us, 2^18 (1 round) 2.4 vs 2.9 us, bfloat16 K = 8 on 3 * 2^18 parameters (3 rounds
// against 2 large ones) 4.50 vs 4.79 us, on 2^20 (4 against 2) 5.25 vs 4.89 us (K = 7: 5.03 vs 4.73),
// and from 2^21 parameters on (7 regular rounds) the regular shape's extra stage wins again (6.7 vs
// 7.1 us, 13.3 vs 13.7, 27.5 vs 28.4).  So the short shape is chosen when the regular shape would
// run at most kShortLaunchTilesPerCta rounds, the large tiles run exactly half as many, and they
// still number at least one per SM.
constexpr int kShortLaunchTilesPerCta = 4;
template <typename G> __host__ __device__ constexpr TmaShape tma_short_shape(int K)
{
    const TmaShape s = tma_shape<G>(K);
    const int per_elem = K * int(sizeof(G)) + 8;
    if (s.tile < 4096 && 2 * (2 * s.tile) * per_elem <= 200 * 1024) return {2 * s.tile, 2, 8};
    return s;
}

// The asynchronous apply of M queued arrivals uses the same geometry with M streams, except for
// the shortest queues: with most of theta coming from L2 (see the alternating sweeps in omni.cu)
// they are no longer DRAM-bound, and a deeper ring with more consumer warps gains 2-6 %
// (float M = 1: 8.20 vs 7.96 TB/s algorithmic with sixteen warps, another 1.4 % with twelve;
// M = 2: 8.70 vs 8.24; M = 3: 8.55 vs 8.38; bfloat16 M = 1: 8.73 vs 8.59, twelve warps 8.48;
// from M = 4 on nothing changed, six warps or eight).
template <typename G> __host__ __device__ constexpr TmaShape tma_seq_shape(int M)
{
    if (sizeof(G) == 4) {
        if (M == 1) return {4096, 4, 12};   // 12 warps: 33.8 us per arrival; 16: 34.3; 10, 14: 36.6, 37.9; 8: 36.6
        if (M == 2) return {4096, 3, 16};
        if (M == 3) return {2048, 4, 16};
    } else if (M == 1) {
        return {4096, 4, 16};
    }
    TmaShape s = tma_shape<G>(M);
    s.consumer_warps = 8;   // the queues were tuned with eight
    return s;
}
__host__ __device__ constexpr unsigned tma_ring_bytes(TmaShape s, int streams, int gsize)
{
    return unsigned(s.stages) * unsigned(s.tile) * unsigned(streams * gsize + 8);
}
template <typename G> __host__ __device__ constexpr unsigned tma_smem_bytes(int K)
{
    return tma_ring_bytes(tma_shape<G>(K), K, int(sizeof(G)));
}

template <typename G, int K, int TILE, int STAGES, int NCW, bool SEQ = false, bool DEVLAM = false, bool OVW = false>
__global__ void __launch_bounds__((NCW + 1) * 32) bsp_tma_kernel(const __grid_constant__ BspParams p)
{
    constexpr int THREADS = (NCW + 1) * 32;
    constexpr int NCT = NCW * 32;                       // consumer threads
    constexpr int V = 16 / int(sizeof(G));              // elements per 16-byte gradient vector
    constexpr int NV = 1;                               // gradient vectors per work item
    constexpr int E = V * NV;                           // elements per work item
    constexpr unsigned GB = TILE * sizeof(G);           // bytes of one gradient tile
    constexpr unsigned FB = TILE * 4;                   // bytes of a theta or v tile
    constexpr unsigned SB = K * GB + 2 * FB;            // bytes of one stage
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long full[STAGES], empty[STAGES];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const float lr = p.lr, mu = p.mu, wd = p.wd;
    const bool with_v = mu != 0.0f;
    const unsigned long long first = blockIdx.x, stride = gridDim.x;
    const unsigned long long pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
    const unsigned long long mine = first < p.tiles ? (p.tiles - first + stride - 1) / stride : 0;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NCW); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch (the host launches this kernel with stream serialization
    // relaxed): let the next launch of the stream take this SM as soon as this CTA leaves it, and
    // do not touch global memory before the previous launch has finished and its writes are
    // visible.  Everything above is set-up that may overlap the predecessor's tail.  Without
    // the launch attribute both instructions do nothing.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    double sq = 0.0;
    if (warp == NCW) {
        // ---------------- producer warp: lane 0 issues the copies ----------------
        if (lane == 0) {
            unsigned long long armed = 0;          // stages armed so far (= issue index of the next one)
            for (unsigned long long i = 0; i < mine; ++i) {
                const int s = int(i % STAGES);
                const unsigned long long t = first + i * stride;
                const unsigned long long tile = p.reverse ? p.tiles - 1 - t : t;
                const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
                const BucketDesc bd = p.bk[bi];
                const unsigned long long base = (tile - bd.tile0) * TILE;
                if (i >= STAGES && !mbar_wait(&empty[s], unsigned((i / STAGES - 1) & 1))) {
                    atomicExch(&p.ws->status, kStatusTimeout);
                    break;
                }
                armed = i + 1;
                if (base + TILE > bd.n) {          // ragged tile: consumers read it from global memory
                    mbar_arrive(&full[s]);
                    continue;
                }
                unsigned char *st = ring + size_t(s) * SB;
                mbar_expect_tx(&full[s], K * GB + FB + (with_v ? FB : 0u));
#pragma unroll
                for (int k = 0; k < K; ++k) bulk_load(st + k * GB, static_cast<const G *>(p.g[bi][k]) + base, GB, &full[s], pol_stream);
                if constexpr (OVW) bulk_load(st + K * GB, p.src[bi] + base, FB, &full[s], pol_stream);
                else bulk_load(st + K * GB, bd.theta + base, FB, &full[s], pol_keep);
                if (with_v) bulk_load(st + K * GB + FB, bd.v + base, FB, &full[s], pol_keep);
            }
            // Leave no copy in flight when this CTA gives its shared memory back: the stages armed
            // last must have landed.  After a normal run the consumers have already seen them
            // land, so this returns at once; it matters when a wait above or below gave up.
            for (unsigned long long j = armed > STAGES ? armed - STAGES : 0; j < armed; ++j)
                if (!mbar_wait(&full[j % STAGES], unsigned((j / STAGES) & 1))) {
                    atomicExch(&p.ws->status, kStatusTimeout);
                    break;
                }
        }
    } else {
        // ---------------- consumer warps ----------------
        // DEVLAM: the weights come from device memory (written by the device-side controller)
        // instead of the kernel parameters.
        float lamr[DEVLAM ? K : 1];
        if constexpr (DEVLAM) {
#pragma unroll
            for (int k = 0; k < K; ++k) lamr[k] = __ldcg(p.lam_dev + k);
        }
        auto weight = [&](int k) -> float {
            if constexpr (DEVLAM) return lamr[k];
            else return p.lam[k];
        };
        for (unsigned long long i = 0; i < mine; ++i) {
            const int s = int(i % STAGES);
            const unsigned long long t = first + i * stride;
            const unsigned long long tile = p.reverse ? p.tiles - 1 - t : t;
            const int bi = find_bucket<kMaxBucketsPerLaunch>(p.bk, p.nb, tile);
            const BucketDesc bd = p.bk[bi];
            const unsigned long long base = (tile - bd.tile0) * TILE;
            const bool has_v = bd.v != nullptr, has_lp = bd.lp != nullptr;
            const float *tsrc = bd.theta;      // where the ragged path reads the "theta" operand
            float *cpy = nullptr;              // second destination of the result (OVW: the snapshot)
            if constexpr (OVW) { tsrc = p.src[bi]; cpy = p.copy[bi]; }
            if (!mbar_wait(&full[s], unsigned((i / STAGES) & 1))) {
                atomicExch(&p.ws->status, kStatusTimeout);
                break;
            }
            if (base + TILE <= bd.n) {
                const unsigned char *st = ring + size_t(s) * SB;
                const float *sth = reinterpret_cast<const float *>(st + K * GB);
                const float *sv = reinterpret_cast<const float *>(st + K * GB + FB);
#pragma unroll 1
                for (int j = tid; j < TILE / E; j += NCT) {
                    float th[E], vv[E];
#pragma unroll
                    for (int q = 0; q < E / 4; ++q) {
                        const float4 t4 = *reinterpret_cast<const float4 *>(sth + j * E + 4 * q);
                        th[4 * q] = t4.x; th[4 * q + 1] = t4.y; th[4 * q + 2] = t4.z; th[4 * q + 3] = t4.w;
                        if (with_v) {
                            const float4 v4 = *reinterpret_cast<const float4 *>(sv + j * E + 4 * q);
                            vv[4 * q] = v4.x; vv[4 * q + 1] = v4.y; vv[4 * q + 2] = v4.z; vv[4 * q + 3] = v4.w;
                        }
                    }
                    if constexpr (SEQ) {
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            const float eta = weight(k);
#pragma unroll
                            for (int h = 0; h < NV; ++h) {
                                const uint4 r = *reinterpret_cast<const uint4 *>(st + k * GB + size_t(j * NV + h) * 16);
                                Raw<4> raw; raw.w[0] = r.x; raw.w[1] = r.y; raw.w[2] = r.z; raw.w[3] = r.w;
                                float gk[V];
                                widen<G, 4>(raw, gk);
#pragma unroll
                                for (int e = 0; e < V; ++e)
                                    th[h * V + e] = update_one(gk[e], th[h * V + e], vv[h * V + e], eta, mu, wd);
                            }
                        }
                    } else {
                        float acc[E];
#pragma unroll
                        for (int e = 0; e < E; ++e) acc[e] = 0.0f;
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            const float lam = weight(k);
#pragma unroll
                            for (int h = 0; h < NV; ++h) {
                                const uint4 r = *reinterpret_cast<const uint4 *>(st + k * GB + size_t(j * NV + h) * 16);
                                Raw<4> raw; raw.w[0] = r.x; raw.w[1] = r.y; raw.w[2] = r.z; raw.w[3] = r.w;
                                float gk[V];
                                widen<G, 4>(raw, gk);
#pragma unroll
                                for (int e = 0; e < V; ++e) acc[h * V + e] = __fmaf_rn(lam, gk[e], acc[h * V + e]);
                            }
                        }
#pragma unroll
                        for (int h = 0; h < NV; ++h) {
                            float part = 0.0f;
#pragma unroll
                            for (int e = 0; e < V; ++e) {
                                part = __fmaf_rn(acc[h * V + e], acc[h * V + e], part);
                                th[h * V + e] = update_one(acc[h * V + e], th[h * V + e], vv[h * V + e], lr, mu, wd);
                            }
                            sq += (double)part;
                        }
                    }
                    const unsigned long long off = base + (unsigned long long)j * E;
                    store_floats_policy<E>(bd.theta + off, th, pol_keep);
                    if (has_v) store_floats_policy<E>(bd.v + off, vv, pol_keep);
                    if (has_lp) store_lp<E / 2>(bd.lp + off, th);
                    if constexpr (OVW) { if (cpy) store_floats<4, E / 4>(cpy + off, th); }
                }
            } else {
                // ragged tile from global memory: whole 16-byte vectors, then single elements
                for (unsigned long long off = base + (unsigned long long)tid * V; off < bd.n; off += (unsigned long long)NCT * V) {
                    if (off + V <= bd.n) {
                        float th[V], vv[V];
                        Raw<4> raw[K];
#pragma unroll
                        for (int k = 0; k < K; ++k) raw[k] = ld_ro<4>(static_cast<const G *>(p.g[bi][k]) + off);
                        load_floats<4, V / 4>(tsrc + off, th);
                        if (with_v) load_floats<4, V / 4>(bd.v + off, vv);
                        if constexpr (SEQ) {
#pragma unroll
                            for (int k = 0; k < K; ++k) {
                                float gk[V];
                                widen<G, 4>(raw[k], gk);
#pragma unroll
                                for (int e = 0; e < V; ++e) th[e] = update_one(gk[e], th[e], vv[e], weight(k), mu, wd);
                            }
                        } else {
                            float acc[V];
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[e] = 0.0f;
#pragma unroll
                            for (int k = 0; k < K; ++k) {
                                float gk[V];
                                widen<G, 4>(raw[k], gk);
                                const float lam = weight(k);
#pragma unroll
                                for (int e = 0; e < V; ++e) acc[e] = __fmaf_rn(lam, gk[e], acc[e]);
                            }
                            float part = 0.0f;
#pragma unroll
                            for (int e = 0; e < V; ++e) {
                                part = __fmaf_rn(acc[e], acc[e], part);
                                th[e] = update_one(acc[e], th[e], vv[e], lr, mu, wd);
                            }
                            sq += (double)part;
                        }
                        store_floats<4, V / 4>(bd.theta + off, th);
                        if (has_v) store_floats<4, V / 4>(bd.v + off, vv);
                        if (has_lp) store_lp<V / 2>(bd.lp + off, th);
                        if constexpr (OVW) { if (cpy) store_floats<4, V / 4>(cpy + off, th); }
                    } else {
                        for (unsigned long long j = off; j < bd.n; ++j) {
                            float vj = with_v ? __ldcs(bd.v + j) : 0.0f;
                            float t = __ldcs(tsrc + j);
                            if constexpr (SEQ) {
#pragma unroll
                                for (int k = 0; k < K; ++k)
                                    t = update_one(widen1<G>(static_cast<const G *>(p.g[bi][k]), j), t, vj, weight(k), mu, wd);
                            } else {
                                float acc = 0.0f;
#pragma unroll
                                for (int k = 0; k < K; ++k)
                                    acc = __fmaf_rn(weight(k), widen1<G>(static_cast<const G *>(p.g[bi][k]), j), acc);
                                t = update_one(acc, t, vj, lr, mu, wd);
                                sq += (double)(acc * acc);
                            }
                            bd.theta[j] = t;
                            if (has_v) bd.v[j] = vj;
                            if (has_lp) bd.lp[j] = __float2bfloat16_rn(t);
                            if constexpr (OVW) { if (cpy) cpy[j] = t; }
                        }
                    }
                }
            }
            // this warp is done with the stage
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
    }
    if constexpr (!SEQ) finish_sqnorm<THREADS>(sq, p.ws, p.accumulate);
}

}  // namespace omni
