// The step before the path: float weights -> per-channel scale alpha and ternary
// 2-bit codes (paper, Section 3.1, Eq. 1-3; Figure 10, pointwise branch).
//     alpha_i = mean_j |W[i][j]|,   W-hat[i][j] = clip(round(W[i][j] / max(alpha_i, eps)), -1, 1)
// with round = ties to even (the framework's), eps = 1e-5 guarding the division
// as in the figure.  Mean and ratio are taken in binary64, so that the order of
// the sum cannot move a decision at the precision of the float32 inputs.
// One block per output channel; the row is read twice (the second time from cache).
#pragma once

#include "common.cuh"

namespace prom { namespace quant {

constexpr int kThreads = 128;

// One output channel (row) by the whole block.
__device__ __forceinline__ void quantize_row(const float *__restrict__ row, int cin, double eps,
                                             uint8_t *__restrict__ packed_row, float *alpha_o, double *part,
                                             double *scale_s)
{
    const int rowb = (cin + 3) >> 2;
    double sum = 0.0;
    for (int j = threadIdx.x; j < cin; j += kThreads) sum += fabs((double)row[j]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        double total = 0.0;
        for (int i = 0; i < kThreads / 32; ++i) total += part[i];
        const double mean = total / (double)cin;
        if (alpha_o) *alpha_o = (float)mean;
        *scale_s = 1.0 / (mean < eps ? eps : mean);
    }
    __syncthreads();
    const double scale = *scale_s;
    bool bad = false;
    for (int kb = threadIdx.x; kb < rowb; kb += kThreads) {
        unsigned byte = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int k = kb * 4 + e;
            if (k < cin) {
                const double v = (double)row[k] * scale;
                if (!(v == v)) { bad = true; continue; }          // NaN weight
                double r = rint(v);                                // ties to even
                r = r > 1.0 ? 1.0 : (r < -1.0 ? -1.0 : r);
                byte |= ((unsigned)(int)r & 3u) << (2 * e);
            }
        }
        packed_row[kb] = (uint8_t)byte;
    }
    if (bad) raise_status(PROM_ERR_BAD_WEIGHT);
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads)
quantize_ternary_kernel(const float *__restrict__ w, int cout, int cin, double eps,
                        uint8_t *__restrict__ packed, float *__restrict__ alpha)
{
    __shared__ double part[kThreads / 32];
    __shared__ double scale_s;
    const int rowb = (cin + 3) >> 2;
    for (int o = blockIdx.x; o < cout; o += gridDim.x)
        quantize_row(w + (size_t)o * cin, cin, eps, packed + (size_t)o * rowb, alpha ? alpha + o : nullptr, part,
                     &scale_s);
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
    __shared__ double part[kThreads / 32];
    __shared__ double scale_s;
    int j = 0;
    for (int r = blockIdx.x; r < jobs.first_row[jobs.n]; r += gridDim.x) {
        while (r >= jobs.first_row[j + 1]) ++j;
        const int o = r - jobs.first_row[j], cin = jobs.cin[j];
        quantize_row(jobs.w[j] + (size_t)o * cin, cin, eps, jobs.packed[j] + (size_t)o * ((cin + 3) >> 2),
                     jobs.alpha[j] ? jobs.alpha[j] + o : nullptr, part, &scale_s);
    }
}

}}  // namespace prom::quant
