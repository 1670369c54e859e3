// The int8 depthwise 3x3 convolution between a block's expand and project convolutions
// (paper, Section 2; its weights are 8-bit, Section 3.1, Eq. 4-5): per channel
//     acc[b][i][j][c] = sum_{di,dj} x[b][i*s + di - 1][j*s + dj - 1][c] * w[c][di][dj]
// with one pixel of zero padding, then the same per-channel fixed-point requantisation as the
// pointwise layers.  NHWC, so a pixel's channels are contiguous.
//
// A thread owns 4 channels (one 32-bit word per pixel) and a strip of kStrip output pixels of
// kRows output rows (two rows at stride 1, one at stride 2).  It loads the words of the input rows
// and columns under the strip once.  Every input column is transposed with byte permutes into
// one word per channel that holds the column's values of all the input rows, and an output's sum
// is three dp4a instructions, one per tap column, against words that hold that column's three
// weights at the byte positions of the output's rows (zero elsewhere): a transposed column serves
// every output above it, no byte is ever unpacked or converted, and the int32 sums are exact.
// Threads of a warp take consecutive channel words, so loads and stores of a pixel are contiguous.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace prom { namespace dw {

constexpr int kThreads = 256;
constexpr int kStrip = 4;

// 4 x 4 byte transpose: words a, b, c, d hold one input row each (byte k = channel k); o[k] gets
// the four rows of channel k.
__device__ __forceinline__ void transpose4(uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t (&o)[4])
{
    const uint32_t t0 = __byte_perm(a, b, 0x5140), t1 = __byte_perm(a, b, 0x7362);
    const uint32_t t2 = __byte_perm(c, d, 0x5140), t3 = __byte_perm(c, d, 0x7362);
    o[0] = __byte_perm(t0, t2, 0x5410); o[1] = __byte_perm(t0, t2, 0x7632);
    o[2] = __byte_perm(t1, t3, 0x5410); o[3] = __byte_perm(t1, t3, 0x7632);
}

// The same for three rows; byte 3 of every result repeats byte 2 and meets a zero weight.
__device__ __forceinline__ void transpose3(uint32_t a, uint32_t b, uint32_t c, uint32_t (&o)[4])
{
    const uint32_t t0 = __byte_perm(a, b, 0x5140), t1 = __byte_perm(a, b, 0x7362);
    o[0] = __byte_perm(t0, c, 0x4410); o[1] = __byte_perm(t0, c, 0x5532);
    o[2] = __byte_perm(t1, c, 0x6610); o[3] = __byte_perm(t1, c, 0x7732);
}

__host__ __device__ constexpr int rows_per_unit(int stride) { return stride == 1 ? 2 : 1; }

// The launch has a multiple of c / 4 threads, so a thread keeps its four channels for all the
// units it works on: filters and constants are fetched once.
template <int STRIDE>
__global__ void __launch_bounds__(kThreads, 3)
dw3x3_kernel(const int8_t *__restrict__ x, int batch, int h, int w, int c, int ho, int wo,
             const int8_t *__restrict__ wt, const int32_t *__restrict__ bias,
             const int32_t *__restrict__ mult, const int8_t *__restrict__ shift, int lo, int hi,
             int8_t *__restrict__ y, int pdl, int pdl_next)
{
    // pdl: launched with programmatic dependent launch behind the kernel that writes x;
    // pdl_next: the next kernel of the stream is launched that way and may start its prologue now
    if (pdl_next) ptx::grid_dep_launch();
    constexpr int kRows = rows_per_unit(STRIDE);          // output rows of a unit
    constexpr int kRowsIn = STRIDE * (kRows - 1) + 3;     // input rows under them (3 or 4)
    constexpr int kCols = STRIDE * (kStrip - 1) + 3;      // input columns under a strip
    const int cw = c >> 2;                                // channel words per pixel
    const int strips = (wo + kStrip - 1) / kStrip;
    const int rgroups = (ho + kRows - 1) / kRows;
    const long long units = (long long)batch * rgroups * strips;
    const long long tid = (long long)blockIdx.x * kThreads + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * kThreads;
    const int ch = (int)(tid % cw) * 4;

    // this thread's filters, wk[output row][tap column][channel]: the column's three weights at
    // the bytes of the input rows that output row reads; and its requantisation constants
    uint32_t wk[kRows][3][4];
    int cb[4], cm[4], cs[4];
    bool bad = false;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint8_t *wp = reinterpret_cast<const uint8_t *>(wt) + (size_t)(ch + k) * 9;
#pragma unroll
        for (int dj = 0; dj < 3; ++dj) {
            const uint32_t col = (uint32_t)wp[dj] | ((uint32_t)wp[3 + dj] << 8) | ((uint32_t)wp[6 + dj] << 16);
#pragma unroll
            for (int rr = 0; rr < kRows; ++rr) wk[rr][dj][k] = col << (8 * rr * STRIDE);
        }
        cb[k] = __ldg(bias + ch + k); cm[k] = __ldg(mult + ch + k); cs[k] = __ldg(shift + ch + k);
        if (!requant_ok(cb[k], cm[k], cs[k])) { bad = true; cb[k] = 0; cm[k] = 0; cs[k] = 0; }
    }
    if (bad) raise_status(PROM_ERR_BAD_REQUANT);
    const bool relu127 = lo == 0 && hi == 127;
    int cb4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) cb4[k] = cb[k] * 4;

    // filters and constants are nobody's output; x is the previous kernel's (every thread waits, so
    // that a grid without work still ends after its predecessor)
    if (pdl) ptx::grid_dep_wait();
    const size_t pix = (size_t)c;                         // bytes from a pixel to the next
    // 32-bit unit indices (the host keeps the number of units below 2^31)
    const unsigned ustep = (unsigned)(nthreads / cw);
    for (unsigned u = (unsigned)(tid / cw); u < (unsigned)units; u += ustep) {
        const unsigned r = u / (unsigned)strips;
        const int sp = (int)(u - r * (unsigned)strips);
        const int b = (int)(r / (unsigned)rgroups), i0 = (int)(r - (unsigned)b * (unsigned)rgroups) * kRows;
        const int j0 = sp * kStrip;
        const int jin0 = j0 * STRIDE - 1;

        // the input rows under this unit (null outside the image)
        const int8_t *rowp[kRowsIn];
#pragma unroll
        for (int di = 0; di < kRowsIn; ++di) {
            const int ii = i0 * STRIDE + di - 1;
            rowp[di] = (ii >= 0 && ii < h) ? x + (((size_t)b * h + ii) * w) * pix + ch : nullptr;
        }

        int acc[kRows][kStrip][4];
#pragma unroll
        for (int rr = 0; rr < kRows; ++rr)
#pragma unroll
            for (int o = 0; o < kStrip; ++o)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[rr][o][k] = 0;

        // column by column: load, transpose, and add to every output whose window holds the column
#pragma unroll
        for (int cidx = 0; cidx < kCols; ++cidx) {
            const int jj = jin0 + cidx;
            const bool col_ok = jj >= 0 && jj < w;
            const unsigned off = (unsigned)(jj < 0 ? 0 : jj) * (unsigned)c;
            uint32_t xin[kRowsIn];
#pragma unroll
            for (int di = 0; di < kRowsIn; ++di)
                xin[di] = (col_ok && rowp[di]) ? __ldg(reinterpret_cast<const uint32_t *>(rowp[di] + off)) : 0u;
            uint32_t t[4];
            if constexpr (kRowsIn == 4) transpose4(xin[0], xin[1], xin[2], xin[3], t);
            else transpose3(xin[0], xin[1], xin[2], t);
#pragma unroll
            for (int o = 0; o < kStrip; ++o) {
                const int dj = cidx - o * STRIDE;         // tap column of this input column for output o
                if (dj >= 0 && dj < 3) {
#pragma unroll
                    for (int rr = 0; rr < kRows; ++rr)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            acc[rr][o][k] = __dp4a((int)t[k], (int)wk[rr][dj][k], acc[rr][o][k]);
                }
            }
        }

#pragma unroll
        for (int rr = 0; rr < kRows; ++rr) {
            if (i0 + rr >= ho) break;
            int8_t *yrow = y + (((size_t)b * ho + i0 + rr) * wo + j0) * pix + ch;
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
                            q2[k] = (__mulhi(acc[rr][o][k] * 4 + cb4[k], cm[k]) >> cs[k]) + 1;
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
                            const int t = acc[rr][o][k] + cb[k];
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
}

}}  // namespace prom::dw
