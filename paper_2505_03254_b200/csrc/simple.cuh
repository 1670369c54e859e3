// Weight packer and the plain one-thread-per-output kernels.
#pragma once

#include "common.cuh"

namespace prom {

// Packs four ternary weights per byte along Cin.  One thread per output byte.
// *bad counts the values outside {-1,0,+1}.
__global__ void pack_ternary_kernel(const int8_t *__restrict__ w, int cout, int cin,
                                    uint8_t *__restrict__ packed, unsigned int *bad)
{
    int rowb = (cin + 3) >> 2;
    long long total = (long long)cout * rowb;
    unsigned int nbad = 0;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int o = (int)(i / rowb), kb = (int)(i - (long long)o * rowb);
        unsigned byte = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int k = kb * 4 + j;
            if (k < cin) {
                int v = w[(size_t)o * cin + k];
                if (v < -1 || v > 1) { ++nbad; v = 0; }
                byte |= ((unsigned)v & 3u) << (2 * j);   // two's-complement 2-bit code
            }
        }
        packed[i] = (uint8_t)byte;
    }
    if (nbad) atomicAdd(bad, nbad);
}

// One thread per output element; the definition written out.  Either y
// (requantised int8, plus res[i] with int8 saturation when res is set; res may be y)
// or acc_out (raw int32) is produced.
__global__ void naive_conv_kernel(const int8_t *__restrict__ x, long long m, int cin, RowMap map,
                                  const uint8_t *__restrict__ w_packed, int cout,
                                  const int32_t *__restrict__ bias,
                                  const int32_t *__restrict__ mult,
                                  const int8_t *__restrict__ shift, int act_min, int act_max,
                                  int8_t *y, int32_t *__restrict__ acc_out, const int8_t *res)
{
    int rowb = (cin + 3) >> 2;
    long long total = m * cout;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long r = i / cout;
        int o = (int)(i - r * cout);
        const int8_t *xr = x + map.in_row(r) * cin;
        int acc = 0;
        bool badw = false;
        for (int k = 0; k < cin; ++k) {
            int wv = weight_at(w_packed, rowb, o, k);
            badw |= (wv == -2);
            acc += (int)xr[k] * wv;
        }
        if (badw) raise_status(PROM_ERR_BAD_WEIGHT);
        if (acc_out) acc_out[i] = acc;
        if (y) {
            int b = bias[o], mu = mult[o], sh = shift[o];
            if (!requant_ok(b, mu, sh)) { raise_status(PROM_ERR_BAD_REQUANT); continue; }
            int q = requant_exact(acc + b, mu, sh, act_min, act_max);
            if (res) {
                q += res[i];
                q = q < -128 ? -128 : (q > 127 ? 127 : q);
            }
            y[i] = (int8_t)q;
        }
    }
}

}  // namespace prom
