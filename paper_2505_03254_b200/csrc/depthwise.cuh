// The int8 depthwise 3x3 convolution between a block's expand and project convolutions
// (paper, Section 2; its weights are 8-bit, Section 3.1, Eq. 4-5): per channel
//     acc[b][i][j][c] = sum_{di,dj} x[b][i*s + di - 1][j*s + dj - 1][c] * w[c][di][dj]
// with one pixel of zero padding, then the same per-channel fixed-point requantisation as the
// pointwise layers.  NHWC, so a pixel's channels are contiguous.
//
// A thread owns 4 channels (one 32-bit word per pixel) and a strip of kStrip output pixels of
// one output row.  It loads the 3 x (columns under the strip) words once; for every output the
// nine tap words are transposed with byte permutes into one word per channel holding four taps,
// and each channel's sum is three dp4a instructions against the channel's nine weights kept as
// three packed words: no byte is ever unpacked or converted, and the int32 sums are exact.
// Threads of a warp take consecutive channel words, so loads and stores of a pixel are contiguous.
#pragma once

#include "common.cuh"

namespace prom { namespace dw {

constexpr int kThreads = 256;
constexpr int kStrip = 4;

// 4 x 4 byte transpose: words a, b, c, d hold one tap each (byte k = channel k); o[k] gets the
// four taps of channel k.
__device__ __forceinline__ void transpose4(uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t (&o)[4])
{
    const uint32_t t0 = __byte_perm(a, b, 0x5140), t1 = __byte_perm(a, b, 0x7362);
    const uint32_t t2 = __byte_perm(c, d, 0x5140), t3 = __byte_perm(c, d, 0x7362);
    o[0] = __byte_perm(t0, t2, 0x5410); o[1] = __byte_perm(t0, t2, 0x7632);
    o[2] = __byte_perm(t1, t3, 0x5410); o[3] = __byte_perm(t1, t3, 0x7632);
}

// The launch has a multiple of c / 4 threads, so a thread keeps its four channels for all the
// strips it works on: filters and constants are fetched once.
template <int STRIDE>
__global__ void __launch_bounds__(kThreads, 3)      // 80 registers: three blocks per SM beat no spills
dw3x3_kernel(const int8_t *__restrict__ x, int batch, int h, int w, int c, int ho, int wo,
             const int8_t *__restrict__ wt, const int32_t *__restrict__ bias,
             const int32_t *__restrict__ mult, const int8_t *__restrict__ shift, int lo, int hi,
             int8_t *__restrict__ y)
{
    const int cw = c >> 2;                                // channel words per pixel
    const int strips = (wo + kStrip - 1) / kStrip;
    const long long units = (long long)batch * ho * strips;
    const long long tid = (long long)blockIdx.x * kThreads + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * kThreads;
    const int ch = (int)(tid % cw) * 4;

    // this thread's filters, wk[group][channel]: taps 0-3, taps 4-7, tap 8 (low byte), and its
    // requantisation constants
    uint32_t wk[3][4];
    int cb[4], cm[4], cs[4];
    bool bad = false;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint8_t *wp = reinterpret_cast<const uint8_t *>(wt) + (size_t)(ch + k) * 9;
        wk[0][k] = (uint32_t)wp[0] | ((uint32_t)wp[1] << 8) | ((uint32_t)wp[2] << 16) | ((uint32_t)wp[3] << 24);
        wk[1][k] = (uint32_t)wp[4] | ((uint32_t)wp[5] << 8) | ((uint32_t)wp[6] << 16) | ((uint32_t)wp[7] << 24);
        wk[2][k] = (uint32_t)wp[8];
        cb[k] = __ldg(bias + ch + k); cm[k] = __ldg(mult + ch + k); cs[k] = __ldg(shift + ch + k);
        if (!requant_ok(cb[k], cm[k], cs[k])) { bad = true; cb[k] = 0; cm[k] = 0; cs[k] = 0; }
    }
    if (bad) raise_status(PROM_ERR_BAD_REQUANT);
    const bool relu127 = lo == 0 && hi == 127;
    int cb4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) cb4[k] = cb[k] * 4;

    constexpr int kCols = STRIDE * (kStrip - 1) + 3;      // input columns under a strip
    const size_t pix = (size_t)c;                         // bytes from a pixel to the next
    // 32-bit unit indices (the host keeps batch * ho * strips below 2^31)
    const unsigned ustep = (unsigned)(nthreads / cw);
    for (unsigned u = (unsigned)(tid / cw); u < (unsigned)units; u += ustep) {
        const unsigned r = u / (unsigned)strips;
        const int sp = (int)(u - r * (unsigned)strips);
        const int b = (int)(r / (unsigned)ho), i = (int)(r - (unsigned)b * (unsigned)ho);
        const int j0 = sp * kStrip;
        const int jin0 = j0 * STRIDE - 1;

        // the three input rows under this output row (null outside the image)
        const int8_t *rowp[3];
#pragma unroll
        for (int di = 0; di < 3; ++di) {
            const int ii = i * STRIDE + di - 1;
            rowp[di] = (ii >= 0 && ii < h) ? x + (((size_t)b * h + ii) * w) * pix + ch : nullptr;
        }

        // the words under the strip: xin[row][column], zeros outside the image
        uint32_t xin[3][kCols];
#pragma unroll
        for (int cidx = 0; cidx < kCols; ++cidx) {
            const int jj = jin0 + cidx;
            const bool col_ok = jj >= 0 && jj < w;
            const unsigned off = (unsigned)(jj < 0 ? 0 : jj) * (unsigned)c;
#pragma unroll
            for (int di = 0; di < 3; ++di)
                xin[di][cidx] = (col_ok && rowp[di]) ? __ldg(reinterpret_cast<const uint32_t *>(rowp[di] + off)) : 0u;
        }

        int acc[kStrip][4];
#pragma unroll
        for (int o = 0; o < kStrip; ++o) {
            const int c0 = o * STRIDE;                    // first column of this output's window
            uint32_t g0[4], g1[4];
            // taps (0,0) (0,1) (0,2) (1,0) and (1,1) (1,2) (2,0) (2,1); tap (2,2) on its own
            transpose4(xin[0][c0], xin[0][c0 + 1], xin[0][c0 + 2], xin[1][c0], g0);
            transpose4(xin[1][c0 + 1], xin[1][c0 + 2], xin[2][c0], xin[2][c0 + 1], g1);
            const uint32_t last = xin[2][c0 + 2];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                int a = __dp4a((int)g0[k], (int)wk[0][k], 0);
                a = __dp4a((int)g1[k], (int)wk[1][k], a);
                a = __dp4a((int)__byte_perm(last, 0u, 0x4440 + k), (int)wk[2][k], a);
                acc[o][k] = a;
            }
        }

        int8_t *yrow = y + (((size_t)b * ho + i) * wo + j0) * pix + ch;
#pragma unroll
        for (int o = 0; o < kStrip; ++o) {
            if (j0 + o < wo) {
                uint32_t out;
                if (relu127) {
                    // clamp [0, 127]: negative values clamp to 0 under either rounding, so the
                    // nested floors ((hi32((4 t) * mult) >> shift) + 1) >> 1 apply; the value is
                    // kept at twice its scale through a saturating pack to [0, 255] and halved
                    // with a mask, which is the clamp at 127
                    int q2[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        q2[k] = (__mulhi(acc[o][k] * 4 + cb4[k], cm[k]) >> cs[k]) + 1;
                    uint32_t wv;
                    asm("{\n\t.reg .b32 t;\n\t"
                        "cvt.pack.sat.u8.s32.b32 t, %4, %3, 0;\n\t"
                        "cvt.pack.sat.u8.s32.b32 %0, %2, %1, t;\n\t}"
                        : "=r"(wv)
                        : "r"(q2[0]), "r"(q2[1]), "r"(q2[2]), "r"(q2[3]));
                    out = (wv >> 1) & 0x7F7F7F7Fu;
                } else {
                    int q[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int t = acc[o][k] + cb[k];
                        q[k] = lo >= 0 ? requant_floor(t, cm[k], cs[k], lo, hi)
                                       : requant_exact(t, cm[k], cs[k], lo, hi);
                    }
                    // already within [-128, 127]: the saturating packs only gather the low bytes
                    asm("{\n\t.reg .b32 t;\n\t"
                        "cvt.pack.sat.s8.s32.b32 t, %4, %3, 0;\n\t"
                        "cvt.pack.sat.s8.s32.b32 %0, %2, %1, t;\n\t}"
                        : "=r"(out)
                        : "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3]));
                }
                *reinterpret_cast<uint32_t *>(yrow + (size_t)o * pix) = out;
            }
        }
    }
}

}}  // namespace prom::dw
