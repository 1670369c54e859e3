// The step after the path in the paper's dataflow: per-sample absmax quantisation of float
// activations to int8 (paper, Section 3.1 "Activations", Eq. 6-7, and the activation figure of
// the pseudocode appendix):
//     gamma_i = max |X[i][...]|,  scale_i = 127 / max(gamma_i, eps),
//     X-hat[i][...] = clip(round(X[i][...] * scale_i), -128, 127)
// with round = ties to even and eps = 1e-5 guarding the division as in the figure.  The
// quotient and the product are single correctly rounded binary32 operations (__fdiv_rn,
// __fmul_rn: no contraction, no approximate division), the precision the paper's framework
// computes in, so the codes do not depend on how the work is split.
//
// Two routes.  Fused: a thread-block cluster per sample; every CTA copies its slice of the
// sample into shared memory once (bulk copies), the CTAs exchange their maxima through
// distributed shared memory, and the slice is quantised from shared memory: each float is read
// from HBM once (5 bytes per element).  Two-pass: one kernel takes the maxima with atomicMax
// on the bit pattern, a second one quantises (9 bytes per element; for samples whose slice
// does not fit shared memory or whose size is not a multiple of 4).
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"
#include "ptx.cuh"

namespace prom { namespace actq {

namespace cg = cooperative_groups;

constexpr int kThreads = 512;
constexpr int kMaxCluster = 8;
constexpr unsigned long long kWaitLimitNs = 100000000ull;
constexpr uint32_t kCopyBytes = 32768;          // one bulk copy
constexpr int kMaxChunks = 8;                   // 8 x 32 KB >= the shared memory of an SM

// round(x * sc) as an integer, ties to even: adding 1.5 * 2^23 rounds the sum to a whole number
// in one correctly rounded binary32 addition, and the whole number sits in the low mantissa
// bits.  Exact for |x * sc| < 2^22; |x| <= gamma keeps the product at 127 (plus rounding).
__device__ __forceinline__ int round_scaled(float x, float sc)
{
    const float r = __fadd_rn(__fmul_rn(x, sc), 12582912.0f);
    return __float_as_int(r) - 0x4B400000;
}

__device__ __forceinline__ int8_t quantise_one(float x, float sc)
{
    int r = round_scaled(x, sc);
    r = r > 127 ? 127 : (r < -128 ? -128 : r);
    return (int8_t)r;
}

// four codes in one word: saturating packs clip to [-128, 127]
__device__ __forceinline__ uint32_t quantise_four(const float4 v, float sc)
{
    uint32_t w;
    asm("{\n\t.reg .b32 t;\n\t"
        "cvt.pack.sat.s8.s32.b32 t, %4, %3, 0;\n\t"
        "cvt.pack.sat.s8.s32.b32 %0, %2, %1, t;\n\t}"
        : "=r"(w)
        : "r"(round_scaled(v.x, sc)), "r"(round_scaled(v.y, sc)), "r"(round_scaled(v.z, sc)),
          "r"(round_scaled(v.w, sc)));
    return w;
}

__device__ __forceinline__ float scale_of(float gamma, float eps)
{
    return __fdiv_rn(127.0f, gamma < eps ? eps : gamma);
}

// max |x| over a block; every thread gets the result.  NaNs are skipped (a > m is false).
__device__ __forceinline__ float block_absmax(float m, float *part)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const float o = __shfl_xor_sync(0xFFFFFFFFu, m, d);
        m = o > m ? o : m;
    }
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
    __syncthreads();
    float r = 0.0f;
    for (int i = 0; i < kThreads / 32; ++i) r = part[i] > r ? part[i] : r;
    __syncthreads();
    return r;
}

// Fused route.  The grid is as many clusters as the GPU holds at once; cluster k takes samples
// k, k + clusters, ...  CTA r of a cluster owns floats [r * slice, min(per, (r + 1) * slice)) of
// each of them; slice is a multiple of 16 and slice * 4 bytes fit the dynamic shared memory.
// The slice arrives in chunks of kCopyBytes, one mbarrier each: the maximum of a chunk is taken
// while later chunks are on their way, and as soon as a chunk has been quantised its place is
// filled with the same chunk of the cluster's next sample, so the copies never stop.
__global__ void __launch_bounds__(kThreads, 1)
act_quant_cluster_kernel(const float *__restrict__ x, int batch, long long per, int slice, float eps,
                         int8_t *__restrict__ q, float *__restrict__ gamma, float *__restrict__ scale)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    float *buf = reinterpret_cast<float *>(smem_raw);
    __shared__ float part[kThreads / 32];
    __shared__ float peer_max[2][kMaxCluster];
    __shared__ __align__(8) uint64_t bar[kMaxChunks];
    __shared__ int failed;

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank(), csize = cluster.num_blocks();
    const int cid = blockIdx.x / csize, nclusters = gridDim.x / csize;
    const long long first = (long long)rank * slice;
    long long count = per - first;
    count = count < 0 ? 0 : (count > slice ? slice : count);        // floats of this CTA
    const uint32_t bytes = (uint32_t)count * 4u;
    const int nchunks = (int)((bytes + kCopyBytes - 1) / kCopyBytes);
    const uint32_t bar_addr = ptx::smem_u32(&bar[0]);
    const uint32_t buf_addr = ptx::smem_u32(buf);
    const float4 *b4 = reinterpret_cast<const float4 *>(buf);
    // every CTA of the cluster must be running before another one writes into its shared
    // memory: arrive now, wait just before the first exchange
    cluster.barrier_arrive();

    auto load_chunk = [&](int sample, int c) {      // thread 0 only
        const uint8_t *src = reinterpret_cast<const uint8_t *>(x + (long long)sample * per + first);
        const uint32_t off = (uint32_t)c * kCopyBytes;
        const uint32_t len = bytes - off < kCopyBytes ? bytes - off : kCopyBytes;
        ptx::mbar_expect_tx(bar_addr + 8 * c, len);
        ptx::bulk_load(buf_addr + off, src + off, len, bar_addr + 8 * c);
    };
    if (threadIdx.x == 0) {
        failed = 0;
        for (int c = 0; c < nchunks; ++c) ptx::mbar_init(bar_addr + 8 * c, 1);
        ptx::mbar_init_fence();
        if (cid < batch)
            for (int c = 0; c < nchunks; ++c) load_chunk(cid, c);
    }
    __syncthreads();

    bool ok = true;
    bool first_exchange = true;
    uint32_t parity = 0;
    for (int sample = cid, it = 0; sample < batch; sample += nclusters, ++it, parity ^= 1u) {
        // ---- this CTA's maximum, chunk by chunk as the copies land (bounded waits) --------
        float m = 0.0f;
        for (int c = 0; c < nchunks && ok; ++c) {
            unsigned long long t0 = 0;
            for (uint32_t i = 1; !ptx::mbar_try_wait(bar_addr + 8 * c, parity); ++i) {
                if ((i & 255u) == 0) {
                    const unsigned long long now = ptx::globaltimer();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kWaitLimitNs) { ok = false; break; }
                }
            }
            if (!ok) break;
            const int lo = c * (int)(kCopyBytes / 16);
            const int hi = min((int)(count >> 2), lo + (int)(kCopyBytes / 16));
            for (int i = lo + threadIdx.x; i < hi; i += kThreads) {
                const float4 v = b4[i];
                float a = fabsf(v.x); m = a > m ? a : m;
                a = fabsf(v.y); m = a > m ? a : m;
                a = fabsf(v.z); m = a > m ? a : m;
                a = fabsf(v.w); m = a > m ? a : m;
            }
        }
        if (!ok && !failed) {
            failed = 1;                   // any thread that gave up marks the CTA; the cluster
            raise_status(PROM_ERR_TIMEOUT);   // barriers below are still taken, so nobody hangs
        }
        m = block_absmax(m, part);        // two block-wide syncs inside
        ok = failed == 0;

        // ---- every CTA's maximum to every CTA ---------------------------------------------
        if (first_exchange) { cluster.barrier_wait(); first_exchange = false; }
        if (threadIdx.x < csize) *cluster.map_shared_rank(&peer_max[it & 1][rank], threadIdx.x) = m;
        cluster.sync();
        float g = 0.0f;
        for (unsigned r = 0; r < csize; ++r) g = peer_max[it & 1][r] > g ? peer_max[it & 1][r] : g;
        const float sc = scale_of(g, eps);
        if (rank == 0 && threadIdx.x == 0) {
            gamma[sample] = g;
            scale[sample] = sc;
        }

        // ---- quantise from shared memory, 16 codes per store; refill each chunk at once ----
        int8_t *dst = q + (long long)sample * per + first;
        const int next = sample + nclusters;
        for (int c = 0; c < nchunks; ++c) {
            if (ok) {
                const int lo = c * (int)(kCopyBytes / 64);
                const int hi = min((int)(count >> 4), lo + (int)(kCopyBytes / 64));
                for (int i = lo + threadIdx.x; i < hi; i += kThreads) {
                    uint32_t w[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) w[j] = quantise_four(b4[4 * i + j], sc);
                    *reinterpret_cast<uint4 *>(dst + 16 * (size_t)i) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            __syncthreads();              // the chunk has been read by everyone
            if (threadIdx.x == 0 && ok && next < batch) load_chunk(next, c);
        }
    }
    if (first_exchange) cluster.barrier_wait();     // a cluster without a sample still pairs its arrive
}

// Fused route without staging: the same clusters and slices, but a CTA reads its slice from
// global memory twice, first for the maximum, then (from L2, where the slice of a few hundred
// kilobytes still sits) to quantise it.  No shared-memory limit on the slice, several CTAs per SM.
__global__ void __launch_bounds__(kThreads)
act_quant_reread_kernel(const float *__restrict__ x, int batch, long long per, long long slice, float eps,
                        int8_t *__restrict__ q, float *__restrict__ gamma, float *__restrict__ scale)
{
    __shared__ float part[kThreads / 32];
    __shared__ float peer_max[2][kMaxCluster];
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank(), csize = cluster.num_blocks();
    const int cid = blockIdx.x / csize, nclusters = gridDim.x / csize;
    const long long first = (long long)rank * slice;
    long long count = per - first;
    count = count < 0 ? 0 : (count > slice ? slice : count);
    const int n4 = (int)(count >> 2), n16 = (int)(count >> 4);
    cluster.barrier_arrive();
    bool first_exchange = true;
    for (int sample = cid, it = 0; sample < batch; sample += nclusters, ++it) {
        const float4 *src = reinterpret_cast<const float4 *>(x + (long long)sample * per + first);
        float m = 0.0f;
        int i = threadIdx.x;
        for (; i + 3 * kThreads < n4; i += 4 * kThreads) {
            const float4 v0 = src[i], v1 = src[i + kThreads], v2 = src[i + 2 * kThreads], v3 = src[i + 3 * kThreads];
            float a;
            a = fmaxf(fmaxf(fabsf(v0.x), fabsf(v0.y)), fmaxf(fabsf(v0.z), fabsf(v0.w))); m = a > m ? a : m;
            a = fmaxf(fmaxf(fabsf(v1.x), fabsf(v1.y)), fmaxf(fabsf(v1.z), fabsf(v1.w))); m = a > m ? a : m;
            a = fmaxf(fmaxf(fabsf(v2.x), fabsf(v2.y)), fmaxf(fabsf(v2.z), fabsf(v2.w))); m = a > m ? a : m;
            a = fmaxf(fmaxf(fabsf(v3.x), fabsf(v3.y)), fmaxf(fabsf(v3.z), fabsf(v3.w))); m = a > m ? a : m;
        }
        for (; i < n4; i += kThreads) {
            const float4 v = src[i];
            const float a = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
            m = a > m ? a : m;
        }
        m = block_absmax(m, part);
        if (first_exchange) { cluster.barrier_wait(); first_exchange = false; }
        if (threadIdx.x < csize) *cluster.map_shared_rank(&peer_max[it & 1][rank], threadIdx.x) = m;
        cluster.sync();
        float g = 0.0f;
        for (unsigned r = 0; r < csize; ++r) g = peer_max[it & 1][r] > g ? peer_max[it & 1][r] : g;
        const float sc = scale_of(g, eps);
        if (rank == 0 && threadIdx.x == 0) {
            gamma[sample] = g;
            scale[sample] = sc;
        }
        int8_t *dst = q + (long long)sample * per + first;
        for (int j = threadIdx.x; j < n16; j += kThreads) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w[e] = quantise_four(src[4 * j + e], sc);
            *reinterpret_cast<uint4 *>(dst + 16 * (size_t)j) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    if (first_exchange) cluster.barrier_wait();
}

// Two-pass route, pass 1: gamma (zeroed beforehand) takes the maxima; |x| >= 0, so the order of
// the bit patterns is the order of the values.
__global__ void __launch_bounds__(kThreads)
act_absmax_kernel(const float *__restrict__ x, long long per, float *__restrict__ gamma)
{
    __shared__ float part[kThreads / 32];
    const long long sample = blockIdx.y;
    const float *src = x + sample * per;
    float m = 0.0f;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < per; i += (long long)gridDim.x * kThreads) {
        const float a = fabsf(src[i]);
        m = a > m ? a : m;
    }
    m = block_absmax(m, part);
    if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned int *>(gamma + sample), __float_as_uint(m));
}

// Two-pass route, pass 2.
__global__ void __launch_bounds__(kThreads)
act_quant_kernel(const float *__restrict__ x, long long per, float eps, const float *__restrict__ gamma,
                 int8_t *__restrict__ q, float *__restrict__ scale)
{
    const long long sample = blockIdx.y;
    const float sc = scale_of(gamma[sample], eps);
    if (blockIdx.x == 0 && threadIdx.x == 0) scale[sample] = sc;
    const float *src = x + sample * per;
    int8_t *dst = q + sample * per;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < per; i += (long long)gridDim.x * kThreads)
        dst[i] = quantise_one(src[i], sc);
}

}}  // namespace prom::actq
