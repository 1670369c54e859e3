// The small-Cin variant on CUDA cores: one thread per output row keeps the
// whole int8 row in registers (Cin <= 64), the ternary weights sit expanded to
// int8 in shared memory, and every output channel is cin/4 dp4a instructions.
// Rows are read with 16-byte vector loads; four requantised outputs are packed
// into one 32-bit store.  The reduction over Cin is short enough to stay
// inside a thread, so no cross-lane reduction is needed.
#pragma once

#include <atomic>

#include "common.cuh"

namespace prom { namespace smallk {

constexpr int kThreads = 128;
constexpr int kMaxWords = 16;   // cin <= 64

static inline bool supported(int cin, int cout)
{
    return cin >= 4 && cin <= 64 && (cin & 3) == 0 && cout >= 1 && (size_t)cout * cin <= 160 * 1024;
}

template <int KW>
__global__ void __launch_bounds__(kThreads)
smallk_kernel(const int8_t *__restrict__ x, long long m, RowMap map,
              const uint8_t *__restrict__ w_packed, int cout,
              const int32_t *__restrict__ bias, const int32_t *__restrict__ mult,
              const int8_t *__restrict__ shift, int act_min, int act_max, int8_t *__restrict__ y)
{
    constexpr int CIN = KW * 4;
    extern __shared__ uint8_t sm[];
    int *ws = reinterpret_cast<int *>(sm);                       // [cout][KW] int8x4 words
    int4 *cs = reinterpret_cast<int4 *>(sm + (((size_t)cout * CIN + 15) & ~(size_t)15)); // {bias, mult, shift, ok}
    // expand the weights (one byte of codes -> one word of four int8)
    bool bad_w = false;
    for (int i = threadIdx.x; i < cout * KW; i += kThreads) {
        unsigned byte = w_packed[i];
        unsigned word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int v = decode2((byte >> (2 * j)) & 3u);
            if (v == -2) { bad_w = true; v = 0; }
            word |= ((unsigned)v & 0xFFu) << (8 * j);
        }
        ws[i] = (int)word;
    }
    if (bad_w) raise_status(PROM_ERR_BAD_WEIGHT);
    for (int o = threadIdx.x; o < cout; o += kThreads) {
        int b = bias[o], mu = mult[o], sh = shift[o];
        int ok = requant_ok(b, mu, sh) ? 1 : 0;
        if (!ok) raise_status(PROM_ERR_BAD_REQUANT);
        cs[o] = make_int4(b, mu, sh, ok);
    }
    __syncthreads();

    const bool nonneg = act_min >= 0;
    const bool word_out = (cout & 3) == 0;
    for (long long r = blockIdx.x * (long long)kThreads + threadIdx.x; r < m;
         r += (long long)gridDim.x * kThreads) {
        int xr[KW];
        const int8_t *xp = x + map.in_row(r) * CIN;
        if constexpr ((KW & 3) == 0) {
#pragma unroll
            for (int i = 0; i < KW / 4; ++i) {
                int4 v = __ldg(reinterpret_cast<const int4 *>(xp) + i);
                xr[4 * i] = v.x; xr[4 * i + 1] = v.y; xr[4 * i + 2] = v.z; xr[4 * i + 3] = v.w;
            }
        } else if constexpr ((KW & 1) == 0) {
#pragma unroll
            for (int i = 0; i < KW / 2; ++i) {
                int2 v = __ldg(reinterpret_cast<const int2 *>(xp) + i);
                xr[2 * i] = v.x; xr[2 * i + 1] = v.y;
            }
        } else {
#pragma unroll
            for (int i = 0; i < KW; ++i) xr[i] = __ldg(reinterpret_cast<const int *>(xp) + i);
        }
        int8_t *yr = y + r * cout;
        unsigned packed = 0;
        for (int o = 0; o < cout; ++o) {
            int acc = 0;
#pragma unroll
            for (int i = 0; i < KW; ++i) acc = __dp4a(xr[i], ws[o * KW + i], acc);
            int4 c = cs[o];
            int q = 0;
            if (c.w)
                q = nonneg ? requant_floor(acc + c.x, c.y, c.z, act_min, act_max)
                           : requant_exact(acc + c.x, c.y, c.z, act_min, act_max);
            if (word_out) {
                packed |= ((unsigned)q & 0xFFu) << (8 * (o & 3));
                if ((o & 3) == 3) {
                    *reinterpret_cast<unsigned *>(yr + o - 3) = packed;
                    packed = 0;
                }
            } else if (c.w) {
                yr[o] = (int8_t)q;
            }
        }
    }
}

static inline prom_status launch(const int8_t *x, long long m, int cin, const RowMap &map,
                                 const uint8_t *w, int cout, const prom_requant &rq, int8_t *y,
                                 cudaStream_t st, std::atomic<uint64_t> &launches)
{
    if (!supported(cin, cout)) return PROM_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return PROM_ERR_CUDA;
    size_t smem = (((size_t)cout * cin + 15) & ~(size_t)15) + (size_t)cout * 16;
    long long blocks = (m + kThreads - 1) / kThreads;
    long long cap = (long long)sms * 8;
    int grid = (int)(blocks < cap ? blocks : cap);
    if (grid < 1) grid = 1;
    cudaError_t e = cudaSuccess;
#define PROM_SMALLK_CASE(KW)                                                                        \
    case KW:                                                                                        \
        if (smem > 48 * 1024)                                                                       \
            e = cudaFuncSetAttribute(smallk_kernel<KW>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                     (int)smem);                                                    \
        if (e == cudaSuccess)                                                                       \
            smallk_kernel<KW><<<grid, kThreads, smem, st>>>(x, m, map, w, cout, rq.bias, rq.mult,  \
                                                            rq.shift, rq.act_min, rq.act_max, y);  \
        break;
    switch (cin / 4) {
        PROM_SMALLK_CASE(1) PROM_SMALLK_CASE(2) PROM_SMALLK_CASE(3) PROM_SMALLK_CASE(4)
        PROM_SMALLK_CASE(5) PROM_SMALLK_CASE(6) PROM_SMALLK_CASE(7) PROM_SMALLK_CASE(8)
        PROM_SMALLK_CASE(9) PROM_SMALLK_CASE(10) PROM_SMALLK_CASE(11) PROM_SMALLK_CASE(12)
        PROM_SMALLK_CASE(13) PROM_SMALLK_CASE(14) PROM_SMALLK_CASE(15) PROM_SMALLK_CASE(16)
    default: return PROM_ERR_UNSUPPORTED;
    }
#undef PROM_SMALLK_CASE
    if (e != cudaSuccess) return PROM_ERR_CUDA;
    ++launches;
    return cudaGetLastError() == cudaSuccess ? PROM_OK : PROM_ERR_CUDA;
}

}}  // namespace prom::smallk
