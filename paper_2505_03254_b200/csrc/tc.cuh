// The tensor-core variant: TMA-staged int8 activation tiles, ternary weights
// expanded from their 2-bit form into shared memory once per CTA, tcgen05
// int8 MMAs accumulating in tensor memory, and a fused requantising epilogue.
//
// Work decomposition
//   tile      = `tm` consecutive output rows (<= 128; one MMA M block)
//   subtile   = `nt` consecutive output channels (<= 256; one accumulator)
//   K chunk   = 128 bytes of a row (one TMA box, one swizzle-128B atom wide)
// A CTA keeps the expanded weights of its subtiles resident for its whole
// life and walks over tiles; warp 0 issues TMA loads, warp 1 issues MMAs,
// warps 2..5 drain the accumulators (one TMEM lane quarter each).
//
// Row folding: when cin or cout is not a multiple of 16 the matrices are
// viewed as X'[M/2][2*cin], Y'[M/2][2*cout] and the weights as the block
// diagonal [[W,0],[0,W]]; Y' is then byte-for-byte the same memory as Y.
//
// Fast epilogue (clamp [0,127], shifts of the CTA's channels within 4 of one
// another, no overflow): channel c's weights are expanded as
// +-2^(2+shmax-shift[c]), so that TMEM holds acc*2^(2+shmax-shift[c]) and
//     v1 = (hi32((tmem + bias') * mult) + 2^shmax) >> shmax
// equals floor(t*mult / 2^(30+shift)) + 1 exactly; the result is
// sat_u8(v1) >> 1.  Everything else takes the 64-bit definition.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace prom { namespace tc {

constexpr int kThreads = 192;
constexpr int kEpiWarps = 4;
constexpr int kStageBytes = 128 * 128;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr int kMaxStages = 8;

struct Params {
    long long m_rows;   // rows of the folded problem
    int k0, n0;         // layer cin, cout
    int fold;           // 1 or 2
    int kf, nf;         // folded cin, cout
    int tm;             // rows per tile
    int n_mtiles;
    int nt, nt_pad;     // subtile width, MMA N
    int n_sub, groups, subs_per_cta;
    int kc;             // K chunks per tile
    int ksteps_last;    // 32-wide MMA steps in the last chunk (1..4)
    int stages, acc_bufs, tmem_cols;
    int out_pitch;      // staging row pitch in bytes
    int mode_b;         // 1: nt % 16 == 8, linear staging
    int x3d, box_r;     // 3-D activation map (strided input); rows of dim 2 per tile
    uint32_t tx_bytes;
    uint32_t inv_cpr;   // ceil(2^20 / (nt/16))
    uint32_t off_w, off_out, off_consts, off_shift, off_wmag, off_bars;
    const uint8_t *w_packed;
    const int32_t *bias, *mult;
    const int8_t *shift;
    int act_min, act_max;
    int8_t *y;
    int pdl;            // launched with programmatic dependent launch
};

struct Ctx {
    volatile int *abort_flag;
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = ptx::globaltimer();
    for (uint32_t i = 1;; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 0) {
            if (*abort_flag) return false;
            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                raise_status(PROM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// K-major, 128-byte swizzle: 8-row atoms of 1024 bytes, stride 1024 between atoms.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}

// 4 two-bit codes (one byte) -> 4 int8 lanes of magnitude `mag` / (256 - mag).
__device__ __forceinline__ uint32_t expand4(uint32_t byte, uint32_t mag, uint32_t negmag,
                                            uint32_t &invalid)
{
    uint32_t x = (byte | (byte << 6) | (byte << 12) | (byte << 18)) & 0x03030303u;
    uint32_t b0 = x & 0x01010101u, b1 = (x >> 1) & 0x01010101u;
    invalid |= b1 & ~b0;
    return (b0 & ~b1) * mag + (b0 & b1) * negmag;
}

template <int NC>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&v)[NC])
{
    if constexpr (NC == 32) ptx::tmem_ld_x32(taddr, v);
    else if constexpr (NC == 16) ptx::tmem_ld_x16(taddr, v);
    else ptx::tmem_ld_x8(taddr, v);
}

// Drain NC accumulator columns of this thread's row, requantise, and write the
// packed bytes to the staging row.
template <int NC, bool FAST>
__device__ __forceinline__ void epi_cols(uint32_t taddr, const int2 *__restrict__ cb,
                                         const int *__restrict__ csh, int shmax, int lo, int hi,
                                         uint8_t *dst, bool mode_b)
{
    uint32_t v[NC];
    tmem_ld<NC>(taddr, v);
    ptx::tmem_wait_ld();
    uint32_t out[NC / 4];
    const int r = 1 << shmax;
#pragma unroll
    for (int c = 0; c < NC; c += 4) {
        int q[4];
#pragma unroll
        for (int e = 0; e < 4; e += 2) {
            int4 bm = *reinterpret_cast<const int4 *>(cb + c + e);   // two channels
            if constexpr (FAST) {
                q[e] = ptx::mad_hi((int)v[c + e] + bm.x, bm.y, r) >> shmax;
                q[e + 1] = ptx::mad_hi((int)v[c + e + 1] + bm.z, bm.w, r) >> shmax;
            } else {
                q[e] = requant_exact((int)v[c + e] + bm.x, bm.y, csh[c + e], lo, hi);
                q[e + 1] = requant_exact((int)v[c + e + 1] + bm.z, bm.w, csh[c + e + 1], lo, hi);
            }
        }
        if constexpr (FAST) {
            uint32_t w = ptx::pack_sat_u8(q[3], q[2], 0u);
            w = ptx::pack_sat_u8(q[1], q[0], w);
            out[c / 4] = (w >> 1) & 0x7F7F7F7Fu;
        } else {
            out[c / 4] = ((uint32_t)q[0] & 0xFFu) | (((uint32_t)q[1] & 0xFFu) << 8) |
                         (((uint32_t)q[2] & 0xFFu) << 16) | (((uint32_t)q[3] & 0xFFu) << 24);
        }
    }
    if (!mode_b) {
        if constexpr (NC >= 16) {
#pragma unroll
            for (int i = 0; i < NC / 16; ++i)
                *reinterpret_cast<uint4 *>(dst + 16 * i) =
                    make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < NC / 8; ++i)
            *reinterpret_cast<uint2 *>(dst + 8 * i) = make_uint2(out[2 * i], out[2 * i + 1]);
    }
}

template <bool FAST>
__device__ __forceinline__ void epi_subtile(const Params &p, uint32_t taddr, const int2 *cb,
                                            const int *csh, int shmax, uint8_t *dst_row)
{
    int c = 0;
    for (; c + 32 <= p.nt; c += 32)
        epi_cols<32, FAST>(taddr + c, cb + c, csh + c, shmax, p.act_min, p.act_max, dst_row + c,
                           p.mode_b);
    if (c + 16 <= p.nt) {
        epi_cols<16, FAST>(taddr + c, cb + c, csh + c, shmax, p.act_min, p.act_max, dst_row + c,
                           p.mode_b);
        c += 16;
    }
    if (c + 8 <= p.nt)
        epi_cols<8, FAST>(taddr + c, cb + c, csh + c, shmax, p.act_min, p.act_max, dst_row + c,
                          true);
}

__global__ void __launch_bounds__(kThreads, 1)
tc_conv_kernel(const __grid_constant__ CUtensorMap xmap, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint8_t *w_smem = smem + p.off_w;
    int2 *cb = reinterpret_cast<int2 *>(smem + p.off_consts);       // {bias', mult} per column
    int *csh = reinterpret_cast<int *>(smem + p.off_shift);         // shift per column
    uint8_t *cwmag = smem + p.off_wmag;                             // log2 weight magnitude
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + p.off_bars);
    // barrier slots: full[stages], empty[stages], tfull[2], tempty[2], drain
    const uint32_t bar_full = ptx::smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * kMaxStages;
    const uint32_t bar_tfull = bar_empty + 8 * kMaxStages;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kMaxStages + 5);
    volatile int *flags = reinterpret_cast<volatile int *>(bars + 2 * kMaxStages + 6);
    // flags[0] abort, flags[1] shmin, flags[2] shmax, flags[3] bad constants, flags[4] slow path

    const int g = blockIdx.x % p.groups;
    const int worker = blockIdx.x / p.groups;
    const int nworkers = gridDim.x / p.groups;
    const int ncols_res = p.subs_per_cta * p.nt_pad;

    // ---- prologue: independent of the previous kernel's output ----------------
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(bar_full + 8 * s, 1);
            ptx::mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar_tfull + 8 * b, 1);
            ptx::mbar_init(bar_tempty + 8 * b, kEpiWarps);
        }
        ptx::mbar_init(bar_drain, 1);
        ptx::mbar_init_fence();
        flags[0] = 0; flags[1] = 31; flags[2] = 0; flags[3] = 0; flags[4] = 0;
        ptx::tma_prefetch_desc(&xmap);
    }
    __syncthreads();
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32((const void *)tmem_slot), (uint32_t)p.tmem_cols);

    // constants of the resident channels: range check, shift span
    {
        int mn = 31, mx = 0, bad = 0;
        for (int i = threadIdx.x; i < ncols_res; i += kThreads) {
            int ls = i / p.nt_pad, c = i - ls * p.nt_pad;
            int sub = g + ls * p.groups;
            int nfold = sub * p.nt + c;
            if (c < p.nt && nfold < p.nf) {
                int n = nfold % p.n0;
                int b = p.bias[n], mu = p.mult[n], sh = p.shift[n];
                if (!requant_ok(b, mu, sh)) bad = 1;
                mn = min(mn, sh); mx = max(mx, sh);
            }
        }
        if (bad) flags[3] = 1;
        atomicMin((int *)&flags[1], mn);
        atomicMax((int *)&flags[2], mx);
    }
    __syncthreads();
    const int shmax = flags[2];
    const bool bad_consts = flags[3] != 0;
    {
        const bool span_ok = (p.act_min == 0 && p.act_max == 127) && (shmax - flags[1] <= 4);
        int slow = span_ok ? 0 : 1;
        for (int i = threadIdx.x; i < ncols_res; i += kThreads) {
            int ls = i / p.nt_pad, c = i - ls * p.nt_pad;
            int sub = g + ls * p.groups;
            int nfold = sub * p.nt + c;
            int b = 0, mu = 0, sh = 0;
            if (c < p.nt && nfold < p.nf && !bad_consts) {
                int n = nfold % p.n0;
                b = p.bias[n]; mu = p.mult[n]; sh = p.shift[n];
            }
            int lg = span_ok ? 2 + shmax - sh : 0;
            // |acc + bias| * 2^lg must stay below 2^31
            long long worst = ((long long)128 * p.k0 + (b < 0 ? -(long long)b : b)) << lg;
            if (worst >= (1ll << 31)) slow = 1;
            cwmag[i] = (uint8_t)lg;
            csh[i] = sh;
            cb[i] = make_int2(b, mu);      // bias is rescaled below once the path is known
        }
        if (slow) flags[4] = 1;
    }
    __syncthreads();
    const bool fast = flags[4] == 0;
    for (int i = threadIdx.x; i < ncols_res; i += kThreads) {
        if (fast) cb[i].x = cb[i].x << cwmag[i];
        else cwmag[i] = 0;
    }
    __syncthreads();

    // expand the resident weights into the K-major swizzle-128B operand layout
    {
        const int rowb = (p.k0 + 3) >> 2;
        const int pieces = p.subs_per_cta * p.kc * p.nt_pad * 8;
        const bool quick = (p.fold == 1) && ((p.k0 & 15) == 0);
        uint32_t invalid = 0;
        for (int i = threadIdx.x; i < pieces; i += kThreads) {
            int j = i & 7;
            int n = (i >> 3) % p.nt_pad;
            int blk = (i >> 3) / p.nt_pad;          // ls * kc + chunk
            int ls = blk / p.kc, chunk = blk - ls * p.kc;
            int kbase = chunk * 128 + j * 16;
            if (chunk == p.kc - 1 && j * 16 >= p.ksteps_last * 32) continue;   // never read
            int sub = g + ls * p.groups;
            int nfold = sub * p.nt + n;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (n < p.nt && nfold < p.nf && kbase < p.kf) {
                uint32_t mag = 1u << cwmag[ls * p.nt_pad + n];
                uint32_t negmag = 256u - mag;
                if (quick) {
                    uint32_t word = *reinterpret_cast<const uint32_t *>(
                        p.w_packed + (size_t)nfold * rowb + (kbase >> 2));
                    val.x = expand4(word & 0xFFu, mag, negmag, invalid);
                    val.y = expand4((word >> 8) & 0xFFu, mag, negmag, invalid);
                    val.z = expand4((word >> 16) & 0xFFu, mag, negmag, invalid);
                    val.w = expand4(word >> 24, mag, negmag, invalid);
                } else {
                    int pn = nfold / p.n0, n_ch = nfold - pn * p.n0;
                    uint32_t wd[4] = {0, 0, 0, 0};
                    for (int e = 0; e < 16; ++e) {
                        int kk = kbase + e;
                        if (kk >= p.kf) break;
                        int pk = kk / p.k0, k = kk - pk * p.k0;
                        if (pk != pn) continue;
                        int wv = weight_at(p.w_packed, rowb, n_ch, k);
                        if (wv == -2) { invalid = 1; wv = 0; }
                        uint32_t byte = wv == 0 ? 0u : (wv > 0 ? mag : negmag);
                        wd[e >> 2] |= byte << (8 * (e & 3));
                    }
                    val = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                }
            }
            *reinterpret_cast<uint4 *>(w_smem + ((size_t)blk * p.nt_pad + n) * 128 +
                                       ((j ^ (n & 7)) << 4)) = val;
        }
        if (invalid) raise_status(PROM_ERR_BAD_WEIGHT);
        if (bad_consts && threadIdx.x == 0) raise_status(PROM_ERR_BAD_REQUANT);
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (p.pdl) {
        ptx::grid_dep_launch();
        ptx::grid_dep_wait();
    }

    // instruction descriptor: s8 x s8 -> s32, both K-major, M = 128, N = nt_pad
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.nt_pad >> 3) << 17) |
                           ((128u >> 4) << 24);

    if (!bad_consts) {
        if (warp == 0) {
            // ---- TMA producer ----------------------------------------------------
            if (lane == 0) {
                uint32_t it = 0;
                bool ok = true;
                for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers)
                    for (int ls = 0; ls < p.subs_per_cta && ok; ++ls)
                        for (int chunk = 0; chunk < p.kc; ++chunk, ++it) {
                            uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                            if (!wait_bar(bar_empty + 8 * s, ph ^ 1u, flags)) { ok = false; break; }
                            ptx::mbar_expect_tx(bar_full + 8 * s, p.tx_bytes);
                            uint32_t dst = smem_base + s * kStageBytes;
                            if (p.x3d)
                                ptx::tma_load_3d(dst, &xmap, chunk * 128, 0, mt * p.box_r,
                                                 bar_full + 8 * s);
                            else
                                ptx::tma_load_2d(dst, &xmap, chunk * 128, mt * p.tm,
                                                 bar_full + 8 * s);
                        }
                if (!ok) {
                    // let the copies already issued land before the CTA goes away
                    uint32_t first = it > (uint32_t)p.stages ? it - p.stages : 0;
                    for (uint32_t j = first; j < it; ++j) {
                        unsigned long long t0 = ptx::globaltimer();
                        while (!ptx::mbar_try_wait(bar_full + 8 * (j % p.stages),
                                                   (j / p.stages) & 1u) &&
                               ptx::globaltimer() - t0 < kWaitLimitNs) {}
                    }
                }
            }
        } else if (warp == 1) {
            // ---- MMA issuer ---------------------------------------------------------
            if (lane == 0) {
                uint32_t it = 0, tile_it = 0;
                bool ok = true;
                const uint32_t w_addr = ptx::smem_u32(w_smem);
                for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers)
                    for (int ls = 0; ls < p.subs_per_cta && ok; ++ls, ++tile_it) {
                        uint32_t b = tile_it % p.acc_bufs, tph = (tile_it / p.acc_bufs) & 1u;
                        if (!wait_bar(bar_tempty + 8 * b, tph ^ 1u, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t d_tmem = tmem_base + b * p.nt_pad;
                        for (int chunk = 0; chunk < p.kc; ++chunk, ++it) {
                            uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                            if (!wait_bar(bar_full + 8 * s, ph, flags)) { ok = false; break; }
                            ptx::tc_fence_after_sync();
                            const uint32_t a_addr = smem_base + s * kStageBytes;
                            const uint32_t b_addr =
                                w_addr + (uint32_t)((ls * p.kc + chunk) * p.nt_pad) * 128u;
                            const int nks = (chunk == p.kc - 1) ? p.ksteps_last : 4;
                            for (int ks = 0; ks < nks; ++ks)
                                ptx::mma_i8(d_tmem, smem_desc(a_addr + 32 * ks),
                                            smem_desc(b_addr + 32 * ks), idesc,
                                            (chunk | ks) != 0 ? 1u : 0u);
                            ptx::mma_commit(bar_empty + 8 * s);
                        }
                        if (ok) ptx::mma_commit(bar_tfull + 8 * b);
                    }
                // every MMA has finished before tensor memory is released
                ptx::mma_commit(bar_drain);
                unsigned long long t0 = ptx::globaltimer();
                while (!ptx::mbar_try_wait(bar_drain, 0) &&
                       ptx::globaltimer() - t0 < kWaitLimitNs) {}
            }
        } else {
            // ---- epilogue ---------------------------------------------------------------
            const int q = warp & 3;                     // TMEM lane quarter of this warp
            uint8_t *stage = smem + p.off_out + (size_t)(warp - 2) * 32 * p.out_pitch;
            uint8_t *my_row = stage + lane * p.out_pitch;
            uint32_t tile_it = 0;
            bool ok = true;
            for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers)
                for (int ls = 0; ls < p.subs_per_cta && ok; ++ls, ++tile_it) {
                    uint32_t b = tile_it % p.acc_bufs, tph = (tile_it / p.acc_bufs) & 1u;
                    if (!wait_bar(bar_tfull + 8 * b, tph, flags)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + b * p.nt_pad;
                    const int2 *cbs = cb + ls * p.nt_pad;
                    const int *cshs = csh + ls * p.nt_pad;
                    if (fast) epi_subtile<true>(p, taddr, cbs, cshs, shmax, my_row);
                    else epi_subtile<false>(p, taddr, cbs, cshs, shmax, my_row);
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar_tempty + 8 * b);

                    // copy this warp's 32 staged rows out, coalesced
                    const long long row0 = (long long)mt * p.tm + q * 32;
                    long long lim = p.m_rows - row0;
                    int rows_valid = p.tm - q * 32;
                    if (lim < rows_valid) rows_valid = (int)lim;
                    if (rows_valid > 32) rows_valid = 32;
                    const int sub = g + ls * p.groups;
                    if (rows_valid > 0) {
                        if (!p.mode_b) {
                            const int cpr = p.nt >> 4;
                            const int total = rows_valid * cpr;
                            int8_t *ybase = p.y + row0 * p.nf + (long long)sub * p.nt;
                            for (int idx = lane; idx < total; idx += 32) {
                                int r = (int)(((uint32_t)idx * p.inv_cpr) >> 20);
                                int ch = idx - r * cpr;
                                uint4 vv = *reinterpret_cast<const uint4 *>(stage + r * p.out_pitch +
                                                                            ch * 16);
                                *reinterpret_cast<uint4 *>(ybase + (long long)r * p.nf + ch * 16) = vv;
                            }
                        } else {
                            const int valid = rows_valid * p.nt;
                            int8_t *ybase = p.y + row0 * p.nt;
                            for (int off = lane * 16; off < valid; off += 512) {
                                if (off + 16 <= valid)
                                    *reinterpret_cast<uint4 *>(ybase + off) =
                                        *reinterpret_cast<const uint4 *>(stage + off);
                                else
                                    *reinterpret_cast<uint2 *>(ybase + off) =
                                        *reinterpret_cast<const uint2 *>(stage + off);
                            }
                        }
                    }
                    __syncwarp();
                }
        }
    }

    // ---- teardown -------------------------------------------------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

}}  // namespace prom::tc
