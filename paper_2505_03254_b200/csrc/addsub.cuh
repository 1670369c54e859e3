// The add/subtract-only variant: the paper's own formulation (Section 2) that a
// product with a ternary weight is a signed copy of the input, so that
//     acc[m][o] = sum_{k: W[o][k]=+1} X[m][k]  -  sum_{k: W[o][k]=-1} X[m][k]
// and a zero weight costs nothing.  No multiply, multiply-add, dot-product or
// MMA instruction ever takes an activation value as an operand here; the only
// multiply per output is the shared requantisation.
//
// Step 1 (index kernel): per output channel, the positions of its +1 weights
// and of its -1 weights as two uint16 lists, each padded to a multiple of 8
// with the index of an all-zero row, plus the per-channel correction
// bias - 128*(n_plus - n_minus).  These lists are scratch memory.
// Step 2 (convolution kernel): a block stages 128 rows of X transposed in
// shared memory as unsigned bytes u = x + 128 (one 32-bit word = the same
// channel of 4 consecutive rows).  A lane owns 4 rows; it adds the even and odd
// bytes of each listed word into two packed 16-bit accumulators and spills them
// to 32-bit sums every 256 terms, before a 16-bit lane can overflow.
#pragma once

#include <atomic>
#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "hostutil.cuh"

namespace prom { namespace addsub {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRows = 128;
constexpr int kMaxCin = 1536;

struct ChannelHead {
    int n_plus8, n_minus8;   // padded list lengths (multiples of 8)
    int corr;                // bias - 128 * (n_plus - n_minus)
    int flags;               // bit 0: constants in range
};

static inline size_t list_stride(int cin) { return (size_t)((cin + 7) / 8 * 8 + 8); }

// Scratch bytes for a [cout][cin] layer: heads, then per channel a plus list and
// a minus list of list_stride(cin) uint16 each.
static inline size_t scratch_bytes(int cout, int cin)
{
    size_t heads = ((size_t)cout * sizeof(ChannelHead) + 255) & ~(size_t)255;
    return heads + (size_t)cout * 2 * list_stride(cin) * sizeof(uint16_t);
}

__global__ void build_lists_kernel(const uint8_t *__restrict__ w_packed, int cout, int cin,
                                   const int32_t *__restrict__ bias, const int32_t *__restrict__ mult,
                                   const int8_t *__restrict__ shift, uint8_t *__restrict__ scratch)
{
    int o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= cout) return;
    const int rowb = (cin + 3) >> 2;
    const size_t ls = (size_t)((cin + 7) / 8 * 8 + 8);
    size_t heads = ((size_t)cout * sizeof(ChannelHead) + 255) & ~(size_t)255;
    ChannelHead *head = reinterpret_cast<ChannelHead *>(scratch) + o;
    uint16_t *plus = reinterpret_cast<uint16_t *>(scratch + heads) + (size_t)o * 2 * ls;
    uint16_t *minus = plus + ls;
    int np = 0, nm = 0;
    bool bad = false;
    for (int k = 0; k < cin; ++k) {
        int v = weight_at(w_packed, rowb, o, k);
        if (v == 1) plus[np++] = (uint16_t)k;
        else if (v == -1) minus[nm++] = (uint16_t)k;
        else if (v == -2) bad = true;
    }
    if (bad) raise_status(PROM_ERR_BAD_WEIGHT);
    int np8 = (np + 7) & ~7, nm8 = (nm + 7) & ~7;
    for (int i = np; i < np8; ++i) plus[i] = (uint16_t)cin;     // the all-zero row
    for (int i = nm; i < nm8; ++i) minus[i] = (uint16_t)cin;
    int b = bias[o], mu = mult[o], sh = shift[o];
    int ok = requant_ok(b, mu, sh) ? 1 : 0;
    if (!ok) raise_status(PROM_ERR_BAD_REQUANT);
    head->n_plus8 = np8;
    head->n_minus8 = nm8;
    head->corr = b - 128 * (np - nm);
    head->flags = ok;
}

// Sum, over a padded index list, of the unsigned bytes of 4 rows (one word per
// listed channel).  Returns the four 32-bit sums.
__device__ __forceinline__ void list_sum(const uint32_t *__restrict__ xs_lane, int pitch_words,
                                         const uint16_t *__restrict__ list, int n8, uint32_t (&s)[4])
{
    s[0] = s[1] = s[2] = s[3] = 0;
    uint32_t ev = 0, od = 0;
    int since = 0;
    for (int i = 0; i < n8; i += 8) {
        uint4 idx = __ldg(reinterpret_cast<const uint4 *>(list + i));
        uint32_t id[4] = {idx.x, idx.y, idx.z, idx.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t w0 = xs_lane[(id[j] & 0xFFFFu) * pitch_words];
            uint32_t w1 = xs_lane[(id[j] >> 16) * pitch_words];
            ev += w0 & 0x00FF00FFu;
            od += (w0 >> 8) & 0x00FF00FFu;
            ev += w1 & 0x00FF00FFu;
            od += (w1 >> 8) & 0x00FF00FFu;
        }
        since += 8;
        if (since == 256) {      // 256 * 255 < 65536: no 16-bit lane has wrapped yet
            s[0] += ev & 0xFFFFu; s[2] += ev >> 16;
            s[1] += od & 0xFFFFu; s[3] += od >> 16;
            ev = od = 0;
            since = 0;
        }
    }
    s[0] += ev & 0xFFFFu; s[2] += ev >> 16;
    s[1] += od & 0xFFFFu; s[3] += od >> 16;
}

__global__ void __launch_bounds__(kThreads)
addsub_conv_kernel(const int8_t *__restrict__ x, long long m, int cin, RowMap map, int cout,
                   const int32_t *__restrict__ mult, const int8_t *__restrict__ shift,
                   const uint8_t *__restrict__ scratch, int act_min, int act_max,
                   int8_t *__restrict__ y)
{
    extern __shared__ uint32_t xs[];          // [cin + 1][kRows / 4 (+1 pad)] words
    constexpr int PW = kRows / 4 + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t ls = (size_t)((cin + 7) / 8 * 8 + 8);
    const size_t heads = ((size_t)cout * sizeof(ChannelHead) + 255) & ~(size_t)255;
    const ChannelHead *head = reinterpret_cast<const ChannelHead *>(scratch);
    const uint16_t *lists = reinterpret_cast<const uint16_t *>(scratch + heads);
    const bool nonneg = act_min >= 0;
    uint8_t *xs8 = reinterpret_cast<uint8_t *>(xs);

    const long long n_tiles = (m + kRows - 1) / kRows;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const long long row0 = tile * kRows;
        __syncthreads();
        // stage X^T as unsigned bytes; rows past the end and the extra row are zero
        for (int i = threadIdx.x; i < PW; i += kThreads) xs[(size_t)cin * PW + i] = 0;
        for (int i = threadIdx.x; i < kRows * cin; i += kThreads) {
            int r = i / cin, k = i - r * cin;
            long long row = row0 + r;
            uint8_t u = 0;
            if (row < m) u = (uint8_t)(x[map.in_row(row) * cin + k] ^ 0x80);
            xs8[(size_t)k * PW * 4 + r] = u;
        }
        __syncthreads();
        const uint32_t *xs_lane = xs + lane;
        const bool four = (cout & 3) == 0;
        // a warp takes 4 consecutive channels at a time so that it can store words
        for (int o4 = warp * 4; o4 < cout; o4 += kWarps * 4) {
            int q[4][4];     // [channel][row]
            bool okc[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int o = o4 + c;
                okc[c] = false;
                if (o < cout) {
                    ChannelHead h = head[o];
                    const uint16_t *pl = lists + (size_t)o * 2 * ls;
                    uint32_t sp[4], sn[4];
                    list_sum(xs_lane, PW, pl, h.n_plus8, sp);
                    list_sum(xs_lane, PW, pl + ls, h.n_minus8, sn);
                    okc[c] = (h.flags & 1) != 0;
                    int mu = mult[o], sh = shift[o];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        int t = (int)sp[j] - (int)sn[j] + h.corr;
                        q[c][j] = !okc[c] ? 0
                                  : nonneg ? requant_floor(t, mu, sh, act_min, act_max)
                                           : requant_exact(t, mu, sh, act_min, act_max);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) q[c][j] = 0;
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                long long row = row0 + lane * 4 + j;
                if (row >= m) continue;
                int8_t *yp = y + row * cout + o4;
                if (four && okc[0] && okc[1] && okc[2] && okc[3]) {
                    uint32_t wv = ((uint32_t)q[0][j] & 0xFFu) | (((uint32_t)q[1][j] & 0xFFu) << 8) |
                                  (((uint32_t)q[2][j] & 0xFFu) << 16) |
                                  (((uint32_t)q[3][j] & 0xFFu) << 24);
                    *reinterpret_cast<uint32_t *>(yp) = wv;
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (o4 + c < cout && okc[c]) yp[c] = (int8_t)q[c][j];
                }
            }
        }
    }
}

// ---- scratch owned by the library: one grow-only buffer per (device, stream) ----
struct Key {
    int dev;
    cudaStream_t st;
    bool operator==(const Key &o) const { return dev == o.dev && st == o.st; }
};
struct KeyHash {
    size_t operator()(const Key &k) const
    {
        return std::hash<void *>()((void *)k.st) ^ ((size_t)k.dev * 0x9E3779B97F4A7C15ull);
    }
};
struct Buf { uint8_t *p = nullptr; size_t bytes = 0; };

static std::mutex g_mu;
static std::unordered_map<Key, Buf, KeyHash> g_cache;

static inline uint8_t *scratch_for(cudaStream_t st, size_t bytes)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lk(g_mu);
    Buf &b = g_cache[Key{dev, st}];
    if (b.bytes < bytes) {
        if (b.p) {
            cudaStreamSynchronize(st);     // the old lists may still be in use
            cudaFree(b.p);
            b.p = nullptr; b.bytes = 0;
        }
        if (cudaMalloc(reinterpret_cast<void **>(&b.p), bytes) != cudaSuccess) return nullptr;
        b.bytes = bytes;
    }
    return b.p;
}

static inline void release_cache()
{
    std::lock_guard<std::mutex> lk(g_mu);
    for (auto &kv : g_cache)
        if (kv.second.p) cudaFree(kv.second.p);
    g_cache.clear();
}

static inline size_t conv_smem(int cin) { return (size_t)(cin + 1) * (kRows / 4 + 1) * 4; }

// Both kernels on caller-provided scratch (scratch_bytes(cout, cin), 256-aligned).
static inline prom_status launch_on(const int8_t *x, long long m, int cin, const RowMap &map,
                                    const uint8_t *w, int cout, const prom_requant &rq, int8_t *y,
                                    uint8_t *scratch, cudaStream_t st,
                                    std::atomic<uint64_t> &launches)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return PROM_ERR_CUDA;
    build_lists_kernel<<<(cout + 127) / 128, 128, 0, st>>>(w, cout, cin, rq.bias, rq.mult, rq.shift,
                                                           scratch);
    ++launches;
    if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
    size_t smem = conv_smem(cin);
    if (raise_smem_limit(addsub_conv_kernel, (int)conv_smem(kMaxCin)) != cudaSuccess) return PROM_ERR_CUDA;
    long long tiles = (m + kRows - 1) / kRows;
    int occ = smem > 100 * 1024 ? 1 : 2;
    long long cap = (long long)sms * occ;
    int grid = (int)(tiles < cap ? tiles : cap);
    addsub_conv_kernel<<<grid, kThreads, smem, st>>>(x, m, cin, map, cout, rq.mult, rq.shift,
                                                     scratch, rq.act_min, rq.act_max, y);
    ++launches;
    return cudaGetLastError() == cudaSuccess ? PROM_OK : PROM_ERR_CUDA;
}

static inline prom_status launch(const int8_t *x, long long m, int cin, const RowMap &map,
                                 const uint8_t *w, int cout, const prom_requant &rq, int8_t *y,
                                 cudaStream_t st, std::atomic<uint64_t> &launches)
{
    if (cin > kMaxCin) return PROM_ERR_UNSUPPORTED;
    uint8_t *scratch = scratch_for(st, scratch_bytes(cout, cin));
    if (!scratch) return PROM_ERR_CUDA;
    return launch_on(x, m, cin, map, w, cout, rq, y, scratch, st, launches);
}

}}  // namespace prom::addsub
