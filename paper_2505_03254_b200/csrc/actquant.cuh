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

__device__ __forceinline__ int8_t quantise_one(float x, float sc)
{
    float r = rintf(__fmul_rn(x, sc));                      // ties to even
    r = r > 127.0f ? 127.0f : (r < -128.0f ? -128.0f : r);
    return (int8_t)(int)r;
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

// Fused route.  grid = batch * cluster CTAs, cluster dimension = `cluster`; CTA r of sample i
// owns floats [r * slice, min(per, (r + 1) * slice)) of the sample; slice is a multiple of 4 and
// slice * 4 bytes fit the dynamic shared memory.
__global__ void __launch_bounds__(kThreads, 1)
act_quant_cluster_kernel(const float *__restrict__ x, long long per, int slice, float eps,
                         int8_t *__restrict__ q, float *__restrict__ gamma, float *__restrict__ scale)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    float *buf = reinterpret_cast<float *>(smem_raw);
    __shared__ float part[kThreads / 32];
    __shared__ float peer_max[kMaxCluster];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int failed;

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank(), csize = cluster.num_blocks();
    const long long sample = blockIdx.x / csize;
    const long long first = (long long)rank * slice;
    long long count = per - first;
    count = count < 0 ? 0 : (count > slice ? slice : count);        // floats of this CTA
    const float *src = x + sample * per + first;
    const uint32_t bar_addr = ptx::smem_u32(&bar);
    // every CTA of the cluster must be running before another one writes into its shared
    // memory: arrive now, wait just before the exchange
    cluster.barrier_arrive();

    if (threadIdx.x == 0) {
        failed = 0;
        ptx::mbar_init(bar_addr, 1);
        ptx::mbar_init_fence();
        const uint32_t bytes = (uint32_t)count * 4u;
        if (bytes) {
            ptx::mbar_expect_tx(bar_addr, bytes);
            for (uint32_t off = 0; off < bytes; off += kCopyBytes)
                ptx::bulk_load(ptx::smem_u32(buf) + off, reinterpret_cast<const uint8_t *>(src) + off,
                               bytes - off < kCopyBytes ? bytes - off : kCopyBytes, bar_addr);
        } else {
            ptx::mbar_arrive(bar_addr);
        }
        // bounded wait for the copies
        const unsigned long long t0 = ptx::globaltimer();
        while (!ptx::mbar_try_wait(bar_addr, 0)) {
            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                failed = 1;
                raise_status(PROM_ERR_TIMEOUT);
                break;
            }
        }
    }
    __syncthreads();
    const bool ok = failed == 0;

    // this CTA's maximum, then every CTA's maximum to every CTA
    float m = 0.0f;
    if (ok) {
        const float4 *b4 = reinterpret_cast<const float4 *>(buf);
        for (int i = threadIdx.x; i < (int)(count >> 2); i += kThreads) {
            const float4 v = b4[i];
            float a = fabsf(v.x); m = a > m ? a : m;
            a = fabsf(v.y); m = a > m ? a : m;
            a = fabsf(v.z); m = a > m ? a : m;
            a = fabsf(v.w); m = a > m ? a : m;
        }
    }
    m = block_absmax(m, part);
    cluster.barrier_wait();
    if (threadIdx.x < csize) *cluster.map_shared_rank(&peer_max[rank], threadIdx.x) = m;
    cluster.sync();
    float g = 0.0f;
    for (unsigned r = 0; r < csize; ++r) g = peer_max[r] > g ? peer_max[r] : g;
    const float sc = scale_of(g, eps);
    if (rank == 0 && threadIdx.x == 0) {
        gamma[sample] = g;
        scale[sample] = sc;
    }

    // quantise from shared memory, 16 codes per store
    if (ok) {
        int8_t *dst = q + sample * per + first;
        const float4 *b4 = reinterpret_cast<const float4 *>(buf);
        const int n16 = (int)(count >> 4);
        for (int i = threadIdx.x; i < n16; i += kThreads) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float4 v = b4[4 * i + j];
                w[j] = (uint32_t)(uint8_t)quantise_one(v.x, sc) | ((uint32_t)(uint8_t)quantise_one(v.y, sc) << 8) |
                       ((uint32_t)(uint8_t)quantise_one(v.z, sc) << 16) |
                       ((uint32_t)(uint8_t)quantise_one(v.w, sc) << 24);
            }
            *reinterpret_cast<uint4 *>(dst + 16 * (size_t)i) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        for (int i = n16 * 16 + threadIdx.x; i < (int)count; i += kThreads) dst[i] = quantise_one(buf[i], sc);
    }
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
