// The step before the path: float weights -> per-channel scale alpha and ternary
// 2-bit codes (paper, Section 3.1, Eq. 1-3; Figure 10, pointwise branch).
//     alpha_i = mean_j |W[i][j]|,   W-hat[i][j] = clip(round(W[i][j] / max(alpha_i, eps)), -1, 1)
// with round = ties to even (the framework's), eps = 1e-5 guarding the division
// as in the figure.  Mean and ratio are taken in binary64, so that the order of
// the sum cannot move a decision at the precision of the float32 inputs.
// One warp per output channel (rows are a few hundred weights: a block per row spent its time in
// barriers and in the latency of two dependent reads, with too few rows in flight); the row is
// read twice, the second time from cache.
#pragma once

#include "common.cuh"

namespace prom { namespace quant {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;

// One output channel (row) by one warp.  Every lane ends up with the same sum (butterfly), so the
// scale needs no exchange.
__device__ __forceinline__ void quantize_row(const float *__restrict__ row, int cin, double eps,
                                             uint8_t *__restrict__ packed_row, float *alpha_o)
{
    const int lane = threadIdx.x & 31;
    const int rowb = (cin + 3) >> 2;
    // one code of a weight at the row's scale: 0, 1 or 3 (-1), or 4 for a NaN
    auto code = [](float w, double scale) -> unsigned {
        const double v = (double)w * scale;
        if (!(v == v)) return 4u;
        double r = rint(v);                                        // ties to even
        r = r > 1.0 ? 1.0 : (r < -1.0 ? -1.0 : r);
        return (unsigned)(int)r & 3u;
    };
    bool bad = false;
    if ((cin & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15u) == 0) {
        // four weights = one 16-byte load = one byte of codes; several loads in flight per lane
        const float4 *row4 = reinterpret_cast<const float4 *>(row);
        double sum = 0.0;
#pragma unroll 4
        for (int kb = lane; kb < rowb; kb += 32) {
            const float4 v = __ldg(row4 + kb);
            sum += (fabs((double)v.x) + fabs((double)v.y)) + (fabs((double)v.z) + fabs((double)v.w));
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
        const double mean = sum / (double)cin;
        if (alpha_o && lane == 0) *alpha_o = (float)mean;
        const double scale = 1.0 / (mean < eps ? eps : mean);
#pragma unroll 4
        for (int kb = lane; kb < rowb; kb += 32) {
            const float4 v = __ldg(row4 + kb);
            const unsigned c0 = code(v.x, scale), c1 = code(v.y, scale), c2 = code(v.z, scale), c3 = code(v.w, scale);
            bad |= ((c0 | c1 | c2 | c3) & 4u) != 0;
            packed_row[kb] = (uint8_t)((c0 & 3u) | ((c1 & 3u) << 2) | ((c2 & 3u) << 4) | ((c3 & 3u) << 6));
        }
    } else {
        double sum = 0.0;
        for (int j = lane; j < cin; j += 32) sum += fabs((double)row[j]);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
        const double mean = sum / (double)cin;
        if (alpha_o && lane == 0) *alpha_o = (float)mean;
        const double scale = 1.0 / (mean < eps ? eps : mean);
        for (int kb = lane; kb < rowb; kb += 32) {
            unsigned byte = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int k = kb * 4 + e;
                if (k < cin) {
                    const unsigned c = code(row[k], scale);
                    bad |= (c & 4u) != 0;
                    byte |= (c & 3u) << (2 * e);
                }
            }
            packed_row[kb] = (uint8_t)byte;
        }
    }
    if (bad) raise_status(PROM_ERR_BAD_WEIGHT);
}

__global__ void __launch_bounds__(kThreads)
quantize_ternary_kernel(const float *__restrict__ w, int cout, int cin, double eps,
                        uint8_t *__restrict__ packed, float *__restrict__ alpha)
{
    const int rowb = (cin + 3) >> 2;
    const int warp = blockIdx.x * kWarps + (threadIdx.x >> 5), nwarps = gridDim.x * kWarps;
    for (int o = warp; o < cout; o += nwarps)
        quantize_row(w + (size_t)o * cin, cin, eps, packed + (size_t)o * rowb, alpha ? alpha + o : nullptr);
}

// Several weight matrices in one launch (all the layers of a network): the rows of all
// matrices are numbered through, and a block takes every gridDim.x-th of them.
constexpr int kMaxJobs = 64;
struct Jobs {
    int n;
    int first_row[kMaxJobs + 1];       // first global row of each matrix; first_row[n] = all rows
    int cin[kMaxJobs];
    const float *w[kMaxJobs];
    uint8_t *packed[kMaxJobs];
    float *alpha[kMaxJobs];
};

__global__ void __launch_bounds__(kThreads)
quantize_ternary_batch_kernel(const __grid_constant__ Jobs jobs, double eps)
{
    const int warp = blockIdx.x * kWarps + (threadIdx.x >> 5), nwarps = gridDim.x * kWarps;
    int j = 0;
    for (int r = warp; r < jobs.first_row[jobs.n]; r += nwarps) {
        while (r >= jobs.first_row[j + 1]) ++j;
        const int o = r - jobs.first_row[j], cin = jobs.cin[j];
        quantize_row(jobs.w[j] + (size_t)o * cin, cin, eps, jobs.packed[j] + (size_t)o * ((cin + 3) >> 2),
                     jobs.alpha[j] ? jobs.alpha[j] + o : nullptr);
    }
}

}}  // namespace prom::quant
