// Shared device/host helpers of the PROM pointwise-convolution library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "prom.h"

namespace prom {

// Device status word: the largest prom_status a kernel has recorded since the
// last prom_last_device_status() call.
__device__ unsigned int g_status;
// Count of invalid weights met by the packer (one pack call at a time).
__device__ unsigned int g_pack_bad;

__device__ __forceinline__ void raise_status(unsigned int s) { atomicMax(&g_status, s); }

// Decode one 2-bit weight code: 00 -> 0, 01 -> +1, 11 -> -1 (10 is invalid and
// decodes to -2, which callers flag).
__device__ __forceinline__ int decode2(unsigned code) { return (int)(code & 1u) - (int)(code & 2u); }

__device__ __forceinline__ int weight_at(const uint8_t *w_packed, int rowb, int o, int k)
{
    unsigned byte = w_packed[(size_t)o * rowb + (k >> 2)];
    return decode2((byte >> (2 * (k & 3))) & 3u);
}

// The requantiser as defined in prom.h, in 64-bit arithmetic: one rounding of
// the exact product t*mult at 2^-(31+shift), ties away from zero, then clamp.
__device__ __forceinline__ int requant_exact(int t, int mult, int shift, int lo, int hi)
{
    long long p = (long long)t * (long long)mult;
    int s = 31 + shift;
    unsigned long long a = p < 0 ? (unsigned long long)(-p) : (unsigned long long)p;
    long long q = (long long)((a + (1ull << (s - 1))) >> s);
    if (p < 0) q = -q;
    q = q < lo ? lo : q;
    q = q > hi ? hi : q;
    return (int)q;
}

// For a clamp with act_min >= 0 the rounding of negative values is irrelevant
// (they clamp to act_min either way), so floor((p + 2^(s-1)) / 2^s) can be used:
//   q = ((hi32((t << 2) * mult) >> shift) + 1) >> 1        (nested floors, exact)
// valid for |t| < 2^29.
__device__ __forceinline__ int requant_floor(int t, int mult, int shift, int lo, int hi)
{
    int h = __mulhi(t << 2, mult);
    int q = ((h >> shift) + 1) >> 1;
    q = q < lo ? lo : q;
    q = q > hi ? hi : q;
    return q;
}

// Range check of one channel's constants (documented in prom.h).
__device__ __forceinline__ bool requant_ok(int bias, int mult, int shift)
{
    return mult >= 0 && shift >= 0 && shift <= 31 && bias >= -(1 << 28) && bias <= (1 << 28);
}

// Geometry of a layer's input: output row r (pixel (b, i, j) of a
// [batch, ho, wo] grid) reads input row ((b*hin + i*stride)*win + j*stride).
// A plain matrix is stride == 1.
struct RowMap {
    int stride, ho, wo, hin, win;
    __host__ __device__ __forceinline__ int64_t in_row(int64_t r) const
    {
        if (stride == 1) return r;
        int64_t hw = (int64_t)ho * wo;
        int64_t b = r / hw, ij = r - b * hw;
        int64_t i = ij / wo, j = ij - i * wo;
        return (b * hin + i * stride) * win + j * stride;
    }
};

}  // namespace prom
