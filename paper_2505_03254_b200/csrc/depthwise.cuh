// The int8 depthwise 3x3 convolution between a block's expand and project convolutions
// (paper, Section 2; its weights are 8-bit, Section 3.1, Eq. 4-5): per channel
//     acc[b][i][j][c] = sum_{di,dj} x[b][i*s + di - 1][j*s + dj - 1][c] * w[c][di][dj]
// with one pixel of zero padding, then the same per-channel fixed-point requantisation as the
// pointwise layers.  NHWC, so a pixel's channels are contiguous.
//
// A thread owns 4 channels (one 32-bit word per pixel) and a strip of kStrip output pixels of
// one output row.  It walks over the input columns of the strip once: the 3 x 4 bytes of a
// column become floats (exactly: byte inserted into the mantissa of 2^23, one subtraction) and
// feed the up to three outputs whose window contains the column with fused multiply-adds in
// binary32, exact because |acc| <= 9 * 128 * 128 < 2^24.  The 36 weights of the thread's
// channels stay in registers as floats.  Threads of a warp take consecutive channel words, so
// loads and stores of a pixel are contiguous.
#pragma once

#include "common.cuh"

namespace prom { namespace dw {

constexpr int kThreads = 256;
constexpr int kStrip = 4;

// four signed bytes of a word -> four floats
__device__ __forceinline__ void bytes_to_floats(uint32_t wd, float (&f)[4])
{
    const uint32_t u = wd ^ 0x80808080u;                  // signed -> offset binary
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t bits = __byte_perm(u, 0x4B000000u, 0x7650 + k);   // 2^23 + byte k
        f[k] = __uint_as_float(bits) - 8388736.0f;                       // - (2^23 + 128)
    }
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

    // this thread's filters wf[tap][channel] and requantisation constants
    float wf[9][4];
    int cb[4], cm[4], cs[4];
    bool bad = false;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
        for (int t = 0; t < 9; ++t) wf[t][k] = (float)wt[(size_t)(ch + k) * 9 + t];
        cb[k] = __ldg(bias + ch + k); cm[k] = __ldg(mult + ch + k); cs[k] = __ldg(shift + ch + k);
        if (!requant_ok(cb[k], cm[k], cs[k])) { bad = true; cb[k] = 0; cm[k] = 0; cs[k] = 0; }
    }
    if (bad) raise_status(PROM_ERR_BAD_REQUANT);

    constexpr int kCols = STRIDE * (kStrip - 1) + 3;      // input columns under a strip
    const size_t pix = (size_t)c;                         // bytes from a pixel to the next
    for (long long u = tid / cw; u < units; u += nthreads / cw) {
        const int sp = (int)(u % strips);
        const long long r = u / strips;
        const int i = (int)(r % ho), b = (int)(r / ho);
        const int j0 = sp * kStrip;
        const int jin0 = j0 * STRIDE - 1;

        // the three input rows under this output row (null outside the image)
        const int8_t *rowp[3];
#pragma unroll
        for (int di = 0; di < 3; ++di) {
            const int ii = i * STRIDE + di - 1;
            rowp[di] = (ii >= 0 && ii < h) ? x + (((size_t)b * h + ii) * w) * pix + ch : nullptr;
        }

        float acc[kStrip][4];
#pragma unroll
        for (int o = 0; o < kStrip; ++o)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[o][k] = 0.0f;

#pragma unroll
        for (int cidx = 0; cidx < kCols; ++cidx) {
            const int jj = jin0 + cidx;
            const bool col_ok = jj >= 0 && jj < w;
#pragma unroll
            for (int di = 0; di < 3; ++di) {
                // a pixel outside the image reads as zeros (and converts to 0.0)
                uint32_t wd = 0;
                if (col_ok && rowp[di]) wd = __ldg(reinterpret_cast<const uint32_t *>(rowp[di] + (size_t)jj * pix));
                float f[4];
                bytes_to_floats(wd, f);
                // output o of the strip sees this column as tap dj = cidx - o * STRIDE
#pragma unroll
                for (int o = 0; o < kStrip; ++o) {
                    constexpr int kS = STRIDE;
                    const int dj = cidx - o * kS;
                    if (dj >= 0 && dj <= 2) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) acc[o][k] = fmaf(f[k], wf[di * 3 + dj][k], acc[o][k]);
                    }
                }
            }
        }

        int8_t *yrow = y + (((size_t)b * ho + i) * wo + j0) * pix + ch;
#pragma unroll
        for (int o = 0; o < kStrip; ++o) {
            if (j0 + o < wo) {
                uint32_t out = 0;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int t = (int)acc[o][k] + cb[k];
                    const int q = lo >= 0 ? requant_floor(t, cm[k], cs[k], lo, hi)
                                          : requant_exact(t, cm[k], cs[k], lo, hi);
                    out |= ((uint32_t)q & 0xFFu) << (8 * k);
                }
                *reinterpret_cast<uint32_t *>(yrow + (size_t)o * pix) = out;
            }
        }
    }
}

}}  // namespace prom::dw
