// The int8 depthwise 3x3 convolution (stride 1) on TMA and the tensor cores.
//
// Channels do not mix in a depthwise convolution, so there is no contraction over channels;
// the contraction is over the nine taps.  For a slice of 16 channels and a tile of 16 x 8 output
// pixels, one TMA load brings the 18 x 10 x 16-byte halo patch into shared memory (pixels
// outside the image arrive as zeros).  Stored pixel after pixel, eight consecutive pixels of a
// patch row are exactly one 8 x 16-byte core matrix of the unswizzled K-major operand layout,
// and the next eight output rows of the MMA (the next image row of the tile) sit 160 bytes
// further on.  A tap (di, dj) is then nothing but a start address inside the patch: the A
// descriptor of an MMA points at the patch shifted by the first of two taps, its K-direction
// offset reaches the second, and B is a 16 x 32 block whose row n holds the two taps' weights
// of channel n at bytes n and 16 + n and zeros elsewhere.  Five tcgen05.mma.kind::i8 of shape
// 128 x 16 x 32 (the last with one tap) leave the 128 x 16 int32 sums of the slice in tensor
// memory; 15/16 of the multiplies meet zeros, which the tensor cores have to spare.  What is
// left per output is the requantiser.
//
// A CTA owns a group of up to four slices (their B blocks and constants stay in shared memory)
// and walks over the image tiles; warp 0 issues the TMA loads (a 5-D map whose fourth dimension
// is the slice, so that one load brings the group's patches one after the other), warp 1 the
// MMAs, warps 2..9 are two epilogue groups that take tiles alternately and store 16 bytes per
// pixel and slice straight from registers.
#pragma once

#include "tc.cuh"

namespace prom { namespace dwtc {

constexpr int kThreads = 320;
constexpr int kTileH = 16, kTileW = 8;                    // output pixels of a tile: 128 = one MMA M block
constexpr int kPatchH = kTileH + 2, kPatchW = kTileW + 2;
constexpr uint32_t kPatchBytes = kPatchH * kPatchW * 16;  // one slice: 2880
constexpr int kMaxSlices = 4;                             // slices (of 16 channels) per CTA
constexpr int kStages = 4;
constexpr uint32_t kStageBytes = kMaxSlices * kPatchBytes;          // 11520
constexpr uint32_t kBBytes = kMaxSlices * 5 * 512;                  // weights blocks: 10240
constexpr uint32_t kOffB = kStages * kStageBytes;
constexpr uint32_t kOffConst = kOffB + kBBytes;                     // bias*4, mult, shift per channel
constexpr uint32_t kOffBars = kOffConst + kMaxSlices * 16 * 12;
constexpr uint32_t kSmemBytes = kOffBars + 8 * (2 * kStages + 4 + 1) + 64 + 128;

struct Params {
    int batch, h, w, c;
    int ns;                 // slices per CTA group
    int groups;             // channel groups = c / (16 * ns)
    int tiles_y, tiles_x;   // tiles per image
    long long tiles;        // batch * tiles_y * tiles_x
    const int8_t *wt;       // [c][3][3]
    const int32_t *bias, *mult;
    const int8_t *shift;
    int lo, hi;
    int8_t *y;
    int pdl;                // launched with programmatic dependent launch behind the kernel that writes x
    int pdl_next;           // the next kernel of the stream is launched that way
};

// Unswizzled K-major operand: core matrices of 8 rows x 16 bytes; `k_off` bytes from a core
// matrix to the next along K, `mn_off` bytes to the next eight rows.
__device__ __forceinline__ uint64_t desc_plain(uint32_t addr, uint32_t k_off, uint32_t mn_off)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((k_off >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((mn_off >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

__global__ void __launch_bounds__(kThreads, 2) dw3x3_tc_kernel(const __grid_constant__ CUtensorMap xmap, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((128u - (ptx::smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kOffBars);
    const uint32_t bar_full = ptx::smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * kStages;
    const uint32_t bar_tfull = bar_empty + 8 * kStages;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kStages + 5);
    volatile int *flags = reinterpret_cast<volatile int *>(bars + 2 * kStages + 5) + 2;   // [0] abort

    const int g = blockIdx.x % p.groups;                  // channel group of this CTA
    const int worker = blockIdx.x / p.groups;
    const int nworkers = gridDim.x / p.groups;
    const int ch0 = g * p.ns * 16;                        // its first channel
    const int nch = p.ns * 16;

    if (p.pdl_next) ptx::grid_dep_launch();

    // ---- prologue (nothing here reads the previous kernel's output) -------------------------
    if (warp == 0) {
        if (lane < kStages) {
            ptx::mbar_init(bar_full + 8 * lane, 1);
            ptx::mbar_init(bar_empty + 8 * lane, 1);
        } else if (lane < kStages + 2) {
            const int b = lane - kStages;
            ptx::mbar_init(bar_tfull + 8 * b, 1);
            ptx::mbar_init(bar_tempty + 8 * b, 4);
        } else if (lane == 31) {
            ptx::mbar_init(bar_drain, 1);
            flags[0] = 0;
            ptx::tma_prefetch_desc(&xmap);
        }
        ptx::mbar_init_fence();
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32((const void *)tmem_slot), 128u);
    // weights blocks: slice s, tap pair t: 16 rows (channel n) x 32 bytes, as four core matrices
    // {k half, n half}; row n holds tap 2t at byte n and tap 2t+1 at byte 16 + n
    for (int i = threadIdx.x; i < p.ns * 5 * 32; i += kThreads) {
        const int blk = i >> 5, part = i & 31;            // part: (k half, n half, row in core matrix)
        const int s = blk / 5, t = blk - s * 5;
        const int khalf = part >> 4, n = part & 15;
        const int tap = 2 * t + khalf;
        uint32_t w4[4] = {0u, 0u, 0u, 0u};
        if (tap < 9) {
            const uint32_t v = (uint32_t)(uint8_t)p.wt[(size_t)(ch0 + s * 16 + n) * 9 + tap];
            w4[n >> 2] = v << (8 * (n & 3));
        }
        uint8_t *dst = smem + kOffB + (size_t)blk * 512 + (khalf * 2 + (n >> 3)) * 128 + (n & 7) * 16;
        *reinterpret_cast<uint4 *>(dst) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
    }
    // constants of the group's channels: {4 * bias, mult, shift}
    int *cst = reinterpret_cast<int *>(smem + kOffConst);
    for (int i = threadIdx.x; i < nch; i += kThreads) {
        int b = __ldg(p.bias + ch0 + i), mu = __ldg(p.mult + ch0 + i), sh = __ldg(p.shift + ch0 + i);
        if (!requant_ok(b, mu, sh)) { raise_status(PROM_ERR_BAD_REQUANT); b = 0; mu = 0; sh = 0; }
        cst[i] = b; cst[64 + i] = mu; cst[128 + i] = sh;
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tx_bytes = (uint32_t)p.ns * kPatchBytes;
    const int tiles_img = p.tiles_y * p.tiles_x;

    if (warp == 0) {
        // ---- TMA producer -------------------------------------------------------------------
        if (lane == 0) {
            uint32_t slot = 0, ph = 0, issued = 0;
            bool ok = true;
            if (p.pdl) ptx::grid_dep_wait();      // the loads are the only reads of x
            for (long long t = worker; t < p.tiles && ok; t += nworkers) {
                const int b = (int)(t / tiles_img), r = (int)(t - (long long)b * tiles_img);
                const int ty = r / p.tiles_x, tx = r - ty * p.tiles_x;
                if (!tc::wait_bar(bar_empty + 8 * slot, ph ^ 1u, flags)) { ok = false; break; }
                const uint32_t bfull = bar_full + 8 * slot;
                ptx::mbar_expect_tx(bfull, tx_bytes);
                // {channel in slice, x, y, slice, image}; the halo starts one pixel up and left
                ptx::tma_load_5d(smem_base + slot * kStageBytes, &xmap, 0, tx * kTileW - 1, ty * kTileH - 1,
                                 g * p.ns, b, bfull);
                ++issued;
                if (++slot == kStages) { slot = 0; ph ^= 1u; }
            }
            if (!ok) {
                for (uint32_t j = issued > (uint32_t)kStages ? issued - kStages : 0; j < issued; ++j) {
                    const unsigned long long g0 = ptx::globaltimer();
                    while (!ptx::mbar_try_wait(bar_full + 8 * (j % kStages), (j / kStages) & 1u) &&
                           ptx::globaltimer() - g0 < tc::kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -----------------------------------------------------------------------
        if (lane == 0) {
            // s8 x s8 -> s32, both K-major, M = 128, N = 16
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
            // tap pairs: start of the first tap inside the patch, offset to the second
            const uint32_t a_start[5] = {0u, 32u, 176u, 320u, 352u};
            const uint32_t a_koff[5] = {16u, 128u, 16u, 16u, 16u};
            uint32_t slot = 0, ph = 0, u = 0;
            bool ok = true;
            for (long long t = worker; t < p.tiles && ok; t += nworkers, ++u) {
                const uint32_t b = u & 1u;
                if (!tc::wait_bar(bar_tempty + 8 * b, ((u >> 1) & 1u) ^ 1u, flags)) { ok = false; break; }
                if (!tc::wait_bar(bar_full + 8 * slot, ph, flags)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t patch = smem_base + slot * kStageBytes;
                for (int s = 0; s < p.ns; ++s) {
                    const uint32_t d = tmem_base + b * 64u + (uint32_t)s * 16u;
#pragma unroll
                    for (int tp = 0; tp < 5; ++tp)
                        ptx::mma_i8(d, desc_plain(patch + (uint32_t)s * kPatchBytes + a_start[tp], a_koff[tp], kPatchW * 16u),
                                    desc_plain(smem_base + kOffB + (uint32_t)(s * 5 + tp) * 512u, 256u, 128u), idesc,
                                    tp > 0 ? 1u : 0u);
                }
                ptx::mma_commit(bar_empty + 8 * slot);
                ptx::mma_commit(bar_tfull + 8 * b);
                if (++slot == kStages) { slot = 0; ph ^= 1u; }
            }
            ptx::mma_commit(bar_drain);
            const unsigned long long g0 = ptx::globaltimer();
            while (!ptx::mbar_try_wait(bar_drain, 0) && ptx::globaltimer() - g0 < tc::kWaitLimitNs) {}
        }
    } else {
        // ---- epilogue -----------------------------------------------------------------------------
        const int q = warp & 3, grp = (warp - 2) >> 2;
        const int m = q * 32 + lane;                       // this thread's pixel of the tile
        const int py = m >> 3, px = m & 7;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)grp * 64u;
        const bool relu127 = p.lo == 0 && p.hi == 127;
        const uint32_t bar_rel = bar_tempty + 8 * grp;
        bool ok = true;
        uint32_t u = 0;
        for (long long t = worker; t < p.tiles && ok; t += nworkers, ++u) {
            if ((int)(u & 1u) != grp) continue;
            const int b = (int)(t / tiles_img), r = (int)(t - (long long)b * tiles_img);
            const int ty = r / p.tiles_x, tx = r - ty * p.tiles_x;
            const int oy = ty * kTileH + py, ox = tx * kTileW + px;
            const bool inside = oy < p.h && ox < p.w;
            int8_t *yp = p.y + (((size_t)b * p.h + oy) * p.w + ox) * (size_t)p.c + ch0;
            if (!tc::wait_bar<true>(bar_tfull + 8 * grp, (u >> 1) & 1u, flags)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            for (int s = 0; s < p.ns; ++s) {
                uint32_t v[16];
                ptx::tmem_ld_x16(t_lane + (uint32_t)s * 16u, v);
                ptx::tmem_wait_ld();
                if (s == p.ns - 1) tc::release_acc(bar_rel);
                const int *cb = cst + s * 16, *cm = cst + 64 + s * 16, *cs = cst + 128 + s * 16;
                uint32_t out[4];
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    int qv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int k = c4 * 4 + e;
                        const int acc = (int)v[k];
                        if (relu127) qv[e] = (__mulhi(acc * 4 + cb[k] * 4, cm[k]) >> cs[k]) + 1;
                        else {
                            const int tt = acc + cb[k];
                            qv[e] = p.lo >= 0 ? requant_floor(tt, cm[k], cs[k], p.lo, p.hi)
                                              : requant_exact(tt, cm[k], cs[k], p.lo, p.hi);
                        }
                    }
                    if (relu127) {
                        uint32_t wv = ptx::pack_sat_u8(qv[3], qv[2], 0u);
                        wv = ptx::pack_sat_u8(qv[1], qv[0], wv);
                        out[c4] = (wv >> 1) & 0x7F7F7F7Fu;
                    } else {
                        out[c4] = ptx::pack_sat_s8(qv[1], qv[0], ptx::pack_sat_s8(qv[3], qv[2], 0u));
                    }
                }
                if (inside) *reinterpret_cast<uint4 *>(yp + s * 16) = make_uint4(out[0], out[1], out[2], out[3]);
            }
        }
    }

    // ---- teardown -------------------------------------------------------------------------------
    // every CTA waits for the previous kernel before it ends, also one whose loader had no tile
    if (p.pdl && threadIdx.x == 32) ptx::grid_dep_wait();
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 128u);
    }
}

}}  // namespace prom::dwtc
