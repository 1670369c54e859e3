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
// 0: mul.hi.s32, 1: mad.lo.s32, 2: fma.rn.f32, 3: mad.wide.s32 (the high word feeds the next one),
// 4: cvt.pack.sat.u8.s32, 5: shr.s32, 6: fma.rn.f64
template <int OP>
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
    double d[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) d[j] = 1.0 + (double)(threadIdx.x * 8 + j) * 1e-9;
    const double dm = 0.999, da = 1e-3;
    const long long add64 = (long long)seed << 33;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (OP == 0) asm volatile("mul.hi.s32 %0, %0, %1;" : "+r"(r[j]) : "r"(mult));
                else if (OP == 1) asm volatile("mad.lo.s32 %0, %0, %1, %1;" : "+r"(r[j]) : "r"(mult));
                else if (OP == 2) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[j]) : "f"(fm), "f"(fa));
                else if (OP == 3)
                    asm volatile("{\n\t.reg .b64 t;\n\t.reg .b32 lo;\n\t"
                                 "mad.wide.s32 t, %0, %1, %2;\n\t"
                                 "mov.b64 {lo, %0}, t;\n\t}"
                                 : "+r"(r[j]) : "r"(mult), "l"(add64));
                else if (OP == 4) asm volatile("cvt.pack.sat.u8.s32.b32 %0, %0, %1, %0;" : "+r"(r[j]) : "r"(mult));
                else if (OP == 5) asm volatile("shr.s32 %0, %0, %1;" : "+r"(r[j]) : "r"(seed));
                else asm volatile("fma.rn.f64 %0, %0, %1, %2;" : "+d"(d[j]) : "d"(dm), "d"(da));
            }
        }
    }
    const long long t1 = clock64();
    int acc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc ^= r[j] ^ __float_as_int(f[j]) ^ __double2hiint(d[j]);
    if (acc == 0x12345678) *sink = acc;          // keeps the chains alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// How often an SM accepts a tcgen05.mma: `nwarps` threads (lane 0 of warps 0..nwarps-1) each issue
// `iters` rounds of four 128 x n x 32 MMAs on fixed shared-memory operands into two accumulators
// of their own (tensor-memory columns [w * 2 * stride, (w + 1) * 2 * stride), stride = max(n, 64);
// the host checks that nwarps * 2 * stride <= 512), then commit and wait (bounded).
// cycles[4 * blockIdx.x + w] = SM clocks of warp w from its first issue to its drain.
__global__ void __launch_bounds__(kMmaThreads, 1) mma_issue_rate_kernel(int iters, int n, int nwarps, long long *cycles)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ uint64_t bar[4];
    __shared__ uint32_t tmem_slot;
    for (int i = threadIdx.x; i < (kMmaM + kMmaN) * kMmaRowBytes / 4; i += kMmaThreads)
        reinterpret_cast<uint32_t *>(smem)[i] = 0x01010101u * (uint32_t)(i & 3);
    if (threadIdx.x < 4) {
        ptx::mbar_init(ptx::smem_u32(&bar[threadIdx.x]), 1);
        ptx::mbar_init_fence();
    }
    if (threadIdx.x < 32) ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512u);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0 && warp < nwarps) {
        const uint32_t a_addr = ptx::smem_u32(smem), b_addr = a_addr + kMmaM * kMmaRowBytes;
        const uint64_t hi = (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
        const uint64_t a0 = hi | (uint64_t)((a_addr >> 4) & 0x3FFFu), b0 = hi | (uint64_t)((b_addr >> 4) & 0x3FFFu);
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t stride = n > 64 ? (uint32_t)n : 64u;
        const uint32_t bar_addr = ptx::smem_u32(&bar[warp]);
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t d = tmem + (uint32_t)warp * 2u * stride + (uint32_t)(it & 1) * stride;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) ptx::mma_i8(d, a0 + 2 * ks, b0 + 2 * ks, idesc, 1u);
        }
        ptx::mma_commit(bar_addr);
        const unsigned long long g0 = ptx::globaltimer();
        bool done = false;
        while (!(done = ptx::mbar_try_wait(bar_addr, 0u)) && ptx::globaltimer() - g0 < kDrainLimitNs) {}
        if (!done) raise_status(PROM_ERR_TIMEOUT);
        cycles[4 * blockIdx.x + warp] = clock64() - t0;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512u);
    }
}

// What an SM can pull out of L2: one thread per CTA (one CTA per SM) keeps `stages` bulk copies
// of 16 KB in flight from a region of global memory that fits L2 (every CTA starts at another
// offset and wraps around), `iters` copies in all; all waits bounded.
// cycles[blockIdx.x] = SM clocks from the first copy to the last arrival.
constexpr uint32_t kCopyBytes = 16384;
constexpr int kCopyMaxStages = 8;
__global__ void __launch_bounds__(32, 1)
l2_copy_rate_kernel(const uint8_t *src, unsigned long long region, int iters, int stages, long long *cycles)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((128u - (ptx::smem_u32(smem_raw) & 127u)) & 127u);
    __shared__ uint64_t bar[kCopyMaxStages];
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) ptx::mbar_init(ptx::smem_u32(&bar[i]), 1);
        ptx::mbar_init_fence();
        const unsigned long long nchunks = region / kCopyBytes;
        unsigned long long c = ((unsigned long long)blockIdx.x * 7ull) % nchunks;
        bool ok = true;
        const long long t0 = clock64();
        // ring position and phase advance by additions (a division per copy would be what is measured)
        int s = 0;
        uint32_t ph = 1;                            // parity of the stage's previous use; no wait in the first pass over the ring
        const uint32_t bar0 = ptx::smem_u32(&bar[0]), dst0 = ptx::smem_u32(smem);
        for (int it = 0; it < iters + stages && ok; ++it) {
            const uint32_t b = bar0 + 8u * (uint32_t)s;
            if (it >= stages) {
                const unsigned long long g0 = ptx::globaltimer();
                while (!ptx::mbar_try_wait(b, ph))
                    if (ptx::globaltimer() - g0 > kDrainLimitNs) { ok = false; break; }
            }
            if (it < iters && ok) {
                ptx::mbar_expect_tx(b, kCopyBytes);
                ptx::bulk_load(dst0 + (uint32_t)s * kCopyBytes, src + c * kCopyBytes, kCopyBytes, b);
                if (++c == nchunks) c = 0;
            }
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (!ok) {
            raise_status(PROM_ERR_TIMEOUT);
            const unsigned long long g0 = ptx::globaltimer();        // let what is in flight land
            while (ptx::globaltimer() - g0 < 100000ull) {}
        }
        cycles[blockIdx.x] = clock64() - t0;
    }
}

// Two things that share an SM with the MMAs.
// MODE 0: warp 0 issues `iters` rounds of four 128 x 128 x 32 MMAs (fixed operands, accumulator
// columns 384..511) while lane 0 of warp 1 keeps `stages` (0 = no copies, else 1..3) bulk copies
// of 16 KB in flight from `src` into a ring of its own until the MMAs are done.
// MODE 1: warps 0..nwarps-1 (4, 8 or 16) each read `iters` times 32 lanes x 32 columns out of the
// accumulator columns 0..383 with tcgen05.ld 32x32b.x32, wait and fold the registers, while (if
// `stages` != 0) lane 0 of warp 16 issues MMAs into columns 384..511 until the readers are done.
// out[8 * cta + 0] = SM clocks of the measured loop (the slowest reader in mode 1), [1] = MMAs
// issued, [2] = SM clocks of the MMA loop, [3] = copies issued.  All loops and waits are bounded.
constexpr int kBesideThreads = 32 * 17;
constexpr uint32_t kBesideOperands = (kMmaM + 128) * kMmaRowBytes;            // A and B: 32 KB
constexpr int kBesideSmem = (int)kBesideOperands + 3 * (int)kCopyBytes + 1024 + 64;
template <int MODE>
__global__ void __launch_bounds__(kBesideThreads, 1)
beside_mma_kernel(int iters, int nwarps, int stages, const uint8_t *src, unsigned long long region, long long *out)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ uint64_t bar_mma, bar_ld[3];
    __shared__ uint32_t tmem_slot;
    __shared__ int done;                                   // readers (mode 1) or the MMA thread (mode 0) finished
    __shared__ long long reader_max;
    for (int i = threadIdx.x; i < (int)kBesideOperands / 4; i += kBesideThreads)
        reinterpret_cast<uint32_t *>(smem)[i] = 0x01010101u * (uint32_t)(i & 3);
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar_mma), 1);
        for (int i = 0; i < 3; ++i) ptx::mbar_init(ptx::smem_u32(&bar_ld[i]), 1);
        ptx::mbar_init_fence();
        done = 0;
        reader_max = 0;
    }
    if (threadIdx.x < 32) ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512u);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *vdone = &done;
    const int mma_warp = MODE == 0 ? 0 : 16;
    if (warp == mma_warp && lane == 0 && (MODE == 0 || stages != 0)) {
        const uint32_t a_addr = ptx::smem_u32(smem), b_addr = a_addr + kMmaM * kMmaRowBytes;
        const uint64_t hi = (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
        const uint64_t a0 = hi | (uint64_t)((a_addr >> 4) & 0x3FFFu), b0 = hi | (uint64_t)((b_addr >> 4) & 0x3FFFu);
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
        const int rounds = MODE == 0 ? iters : (1 << 22);  // mode 1: until the readers are done
        long long n = 0;
        const long long t0 = clock64();
        for (int it = 0; it < rounds && (MODE == 0 || *vdone < nwarps); ++it) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) ptx::mma_i8(tmem + 384u, a0 + 2 * ks, b0 + 2 * ks, idesc, 1u);
            n += 4;
        }
        const long long t1 = clock64();
        ptx::mma_commit(ptx::smem_u32(&bar_mma));
        const unsigned long long g0 = ptx::globaltimer();
        bool ok = false;
        while (!(ok = ptx::mbar_try_wait(ptx::smem_u32(&bar_mma), 0u)) && ptx::globaltimer() - g0 < kDrainLimitNs) {}
        if (!ok) raise_status(PROM_ERR_TIMEOUT);
        out[8 * blockIdx.x + 1] = n;
        out[8 * blockIdx.x + 2] = t1 - t0;
        if (MODE == 0) {
            out[8 * blockIdx.x + 0] = clock64() - t0;
            *vdone = 1;
        }
    } else if (MODE == 0 && warp == 1 && lane == 0 && stages != 0) {
        const uint32_t ring = ptx::smem_u32(smem) + kBesideOperands;
        const unsigned long long nchunks = region / kCopyBytes;
        unsigned long long c = ((unsigned long long)blockIdx.x * 7ull) % nchunks;
        long long copies = 0;
        int s = 0;
        uint32_t ph = 1;
        bool ok = true;
        for (int it = 0; it < (1 << 22) && ok && !*vdone; ++it) {
            const uint32_t b = ptx::smem_u32(&bar_ld[s]);
            if (it >= stages) {
                const unsigned long long g0 = ptx::globaltimer();
                while (!ptx::mbar_try_wait(b, ph))
                    if (ptx::globaltimer() - g0 > kDrainLimitNs) { ok = false; break; }
            }
            if (!ok) break;
            ptx::mbar_expect_tx(b, kCopyBytes);
            ptx::bulk_load(ring + (uint32_t)s * kCopyBytes, src + c * kCopyBytes, kCopyBytes, b);
            if (++c == nchunks) c = 0;
            ++copies;
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (!ok) raise_status(PROM_ERR_TIMEOUT);
        const unsigned long long g0 = ptx::globaltimer();        // let what is in flight land
        while (ptx::globaltimer() - g0 < 100000ull) {}
        out[8 * blockIdx.x + 3] = copies;
    } else if (MODE == 1 && warp < nwarps) {
        // a warp reads its own lane quarter; the warps of a quarter start 96 columns apart
        const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t acc = 0, col = (uint32_t)(warp >> 2) * 96u;
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            uint32_t v[32];
            ptx::tmem_ld_x32(t_lane + col, v);             // columns col .. col + 31 <= 383
            ptx::tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) acc ^= v[j];
            col += 32u;
            if (col > 352u) col = 0u;
        }
        const long long t1 = clock64();
        if (acc == 0x12345678u) out[8 * blockIdx.x + 7] = 1;                   // keeps the loads alive
        if (lane == 0) {
            atomicMax(reinterpret_cast<unsigned long long *>(&reader_max), (unsigned long long)(t1 - t0));
            __threadfence_block();
            atomicAdd(&done, 1);
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (MODE == 1 && threadIdx.x == 0) out[8 * blockIdx.x + 0] = reader_max;
    if (threadIdx.x < 32) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512u);
    }
}

}}  // namespace prom::peak
