// Rate probes behind the roofline figures: what one SM's tensor pipe sustains on
// tcgen05.mma.kind::i8 with both operands fixed in shared memory, and what its integer
// pipes sustain on the 32-bit high multiply of the requantising epilogue.  Both count SM
// clock cycles inside the kernel (clock64), so that the rates come out per clock; the host
// times the launch with events for the figure in operations per second.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace prom { namespace peak {

constexpr int kMmaThreads = 128;
constexpr int kMmaM = 128, kMmaN = 256, kMmaRowBytes = 128;      // one K chunk = 4 steps of K = 32
constexpr int kMmaSmem = (kMmaM + kMmaN) * kMmaRowBytes + 1024 + 64;
constexpr unsigned long long kDrainLimitNs = 2000000000ull;

// One CTA per SM.  A [128 x 128 B] and B [256 x 128 B] sit in shared memory in the K-major
// 128-byte-swizzled layout (the layout is a permutation of 16-byte pieces inside 1 KB atoms,
// so any byte pattern is a valid operand); one thread issues `iters` rounds of four
// 128x256x32 MMAs, alternating between two 256-column accumulators, then one commit and a
// bounded wait.  cycles[blockIdx.x] = SM clocks from the first issue to the drain.
__global__ void __launch_bounds__(kMmaThreads, 1) i8_mma_rate_kernel(int iters, long long *cycles)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const uint32_t a_addr = ptx::smem_u32(smem), b_addr = a_addr + kMmaM * kMmaRowBytes;
    // operands: small signed values from a hash of the byte index (sums stay far from overflow)
    for (int i = threadIdx.x; i < (kMmaM + kMmaN) * kMmaRowBytes / 4; i += kMmaThreads) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        uint32_t w = 0;
        for (int e = 0; e < 4; ++e) {
            const int v = (int)((h >> (8 * e)) & 7u) - 3;          // -3 .. 4
            w |= ((uint32_t)v & 0xFFu) << (8 * e);
        }
        reinterpret_cast<uint32_t *>(smem)[i] = w;
    }
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        ptx::mbar_init_fence();
    }
    if (threadIdx.x < 32) ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512u);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    if (threadIdx.x == 0) {
        // descriptor: start address, LBO = 1, SBO = 1024 bytes (8 rows of 128), 128-byte swizzle
        const uint64_t hi = (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
        const uint64_t a0 = hi | (uint64_t)((a_addr >> 4) & 0x3FFFu), b0 = hi | (uint64_t)((b_addr >> 4) & 0x3FFFu);
        // s8 x s8 -> s32, both K-major, M = 128, N = 256
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kMmaN >> 3) << 17) | ((128u >> 4) << 24);
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t d = tmem + (uint32_t)(it & 1) * kMmaN;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) ptx::mma_i8(d, a0 + 2 * ks, b0 + 2 * ks, idesc, (it > 1 || ks > 0) ? 1u : 0u);
        }
        ptx::mma_commit(ptx::smem_u32(&bar));
        const unsigned long long g0 = ptx::globaltimer();
        bool done = false;
        while (!(done = ptx::mbar_try_wait(ptx::smem_u32(&bar), 0u)) && ptx::globaltimer() - g0 < kDrainLimitNs) {}
        if (!done) raise_status(PROM_ERR_TIMEOUT);
        cycles[blockIdx.x] = clock64() - t0;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512u);
    }
}

// 8 independent chains of mul.hi.s32 per thread, `iters` rounds of 8 x 8 multiplies.
// cycles[blockIdx.x] = SM clocks of the loop (thread 0 of the block).
constexpr int kAluThreads = 512;
constexpr int kAluPerIter = 64;
template <int OP>   // 0: mul.hi.s32, 1: mad.lo.s32, 2: fma.rn.f32
__global__ void __launch_bounds__(kAluThreads, 2) alu_rate_kernel(int iters, int seed, int *sink, long long *cycles)
{
    int r[8];
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        r[j] = seed + (int)threadIdx.x * 8 + j + 0x40000000;
        f[j] = 1.0f + (float)(threadIdx.x * 8 + j) * 1e-6f;
    }
    const int mult = 0x7FFFFFF1 - (int)(threadIdx.x & 7);
    const float fm = 0.999f, fa = 1e-3f;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (OP == 0) asm volatile("mul.hi.s32 %0, %0, %1;" : "+r"(r[j]) : "r"(mult));
                else if (OP == 1) asm volatile("mad.lo.s32 %0, %0, %1, %1;" : "+r"(r[j]) : "r"(mult));
                else asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[j]) : "f"(fm), "f"(fa));
            }
        }
    }
    const long long t1 = clock64();
    int acc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc ^= r[j] ^ __float_as_int(f[j]);
    if (acc == 0x12345678) *sink = acc;          // keeps the chains alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}}  // namespace prom::peak
