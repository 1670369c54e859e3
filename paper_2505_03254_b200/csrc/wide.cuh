// The tensor-core variant for layers whose contraction, not their bytes, is the bound
// (many input and many output channels on many rows).
//
// tc_conv_kernel keeps the weights of a channel group resident and streams the activations
// past them once per group; with Cin x Cout in the hundreds of thousands a group is only a few
// dozen channels wide, the MMAs are narrow and the activations cross the SM many times.  Here
// the roles are swapped: a CTA (one per SM) keeps a tile of 128 rows resident, all of its K
// (up to 8 chunks of 128 bytes), and streams the expanded weights of one 128-channel column
// tile after the other through a ring, so that every MMA is 128 x 128 x 32 (the tensor pipe's
// full rate) and an activation byte enters the SM once.  What an SM then has to pull from L2 is
// the weight matrix once per row tile: Cin * Cout bytes per 128 * Cin * Cout MACs, i.e. 64 bytes
// per clock at the pipe's 8192 MACs per clock, which is what one SM can take (61.5 measured).
//
// wide_prep_kernel (one CTA per column tile) expands the 2-bit weights into an int8 matrix
// [Cout padded to 128][Cin padded to 128] in global scratch, scaled for the one-multiply
// epilogue of tc.cuh where the tile's constants allow it, and writes the tile's bias digits
// and requantisation constants beside it.  The convolution kernel reads that matrix through a
// tensor map (128-byte swizzle, like the activations), the bias digits as the last "chunk" of a
// column tile, and the constants into a small ring of their own.
//
// Warp 0 issues the loads, warps 1 and 18 the MMAs, warps 2..17 are four epilogue groups, one per
// accumulator, that requantise 32 columns at a time and store through the
// output's tensor map (rows and columns outside the matrix are not written).
#pragma once

#include "tc.cuh"

namespace prom { namespace wide {

constexpr int kEpiWarps = 16;                     // four groups, one per accumulator
constexpr int kIssuer2 = 2 + kEpiWarps;           // warp of the second MMA issuer
constexpr int kThreads = 32 * (kIssuer2 + 1);     // loader, MMA issuer, sixteen epilogue warps, MMA issuer
constexpr int kNt = 128;                          // columns of a column tile = MMA N
constexpr int kChunk = 128;                       // bytes of K per chunk = swizzle span
constexpr int kMaxKc = 8;                         // resident K chunks: Cin <= 1024
constexpr int kMaxStages = 8;
constexpr int kAccs = 4;                          // accumulators of 128 columns: all 512 of tensor memory
constexpr uint32_t kStageBytes = kNt * kChunk;    // 16 KB, also one resident chunk of the row tile
constexpr uint32_t kWbiasBytes = kNt * 32;        // bias digits of a column tile (32-byte swizzled rows)
// constants of a column tile: mult[128], {bias, shift}[128], header {shmax, fast, bad, 0}
constexpr uint32_t kConstBytes = kNt * 4 + kNt * 8 + 16 + 112;
constexpr uint32_t kEpiCols = 32;                 // columns an epilogue warp stages per store
constexpr uint32_t kSlabBytes = 32 * kEpiCols;
constexpr int kBars = 2 * kMaxKc + 2 * kMaxStages + 4 * kAccs + 1;

struct Params {
    long long m;
    int cin, cout;
    int kc, ksteps_last;        // chunks of K; 32-byte MMA steps in the last one
    int n_mtiles, n_ctiles;     // row tiles, column tiles
    int nb;                     // 128-channel blocks per column tile: 1 (MMA N = 128) or 2 (N = 256)
    int groups;                 // CTAs that share a row tile's columns; n_ctiles % groups == 0
    int stages;                 // of the weight ring
    uint32_t off_w, off_const, off_out, off_aconst, off_bars;
    const uint8_t *wbias;       // [n_ctiles * nb][kWbiasBytes]
    const uint8_t *consts;      // [n_ctiles * nb][kConstBytes]
    int act_min, act_max;
};

struct PrepParams {
    int cin, cout, k_pad;
    const uint8_t *w_packed;
    const int32_t *bias, *mult;
    const int8_t *shift;
    int act_min, act_max;
    int8_t *w8;                 // [n_ctiles * 128][k_pad]
    uint8_t *wbias, *consts;
};

// The operands of column tile `tile` of one layer; all 256 threads of the CTA take part.
__device__ __forceinline__ void prep_tile(const PrepParams &p, const int tile)
{
    __shared__ int s_mult[kNt], s_bias[kNt], s_shift[kNt];
    __shared__ int s_flags[4];      // shmin, shmax, bad, slow
    const int n0 = tile * kNt;
    if (threadIdx.x == 0) { s_flags[0] = 31; s_flags[1] = 0; s_flags[2] = 0; s_flags[3] = 0; }
    __syncthreads();
    if (threadIdx.x < kNt) {
        const int n = n0 + threadIdx.x;
        int b = 0, mu = 0, sh = 0;
        if (n < p.cout) {
            b = __ldg(p.bias + n); mu = __ldg(p.mult + n); sh = __ldg(p.shift + n);
            if (!requant_ok(b, mu, sh)) { s_flags[2] = 1; b = 0; mu = 0; sh = 0; }
            atomicMin(&s_flags[0], sh);
            atomicMax(&s_flags[1], sh);
            // the one-multiply epilogue needs |acc + bias| * 2^6 below 2^31 and the scaled bias
            // within the range of its digits
            const long long ab = b < 0 ? -(long long)b : b;
            if ((((long long)128 * p.cin + ab) << 6) >= (1ll << 31) || (ab << 6) > tc::kBiasMax) s_flags[3] = 1;
        }
        s_mult[threadIdx.x] = mu; s_bias[threadIdx.x] = b; s_shift[threadIdx.x] = sh;
    }
    __syncthreads();
    const int shmax = s_flags[1];
    const bool bad = s_flags[2] != 0;
    const bool fast = !bad && s_flags[3] == 0 && p.act_min == 0 && p.act_max == 127 && shmax - s_flags[0] <= 4 &&
                      shmax <= 24 && s_flags[0] <= shmax;
    if (bad && threadIdx.x == 0) raise_status(PROM_ERR_BAD_REQUANT);

    // constants and bias digits
    uint8_t *cst = p.consts + (size_t)tile * kConstBytes;
    uint8_t *wb = p.wbias + (size_t)tile * kWbiasBytes;
    if (threadIdx.x < kNt) {
        const int c = threadIdx.x;
        reinterpret_cast<int *>(cst)[c] = s_mult[c];
        reinterpret_cast<int2 *>(cst + kNt * 4)[c] = make_int2(s_bias[c], s_shift[c]);
        uint32_t wd[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        if (fast && n0 + c < p.cout) {
            const int v = s_bias[c] << (2 + shmax - s_shift[c]);
            int h = (v >= 0 ? v + 63 : v - 63) / 127;        // nearest multiple of 127
            const int lo = v - 127 * h;                       // within [-63, 63]
            wd[0] = (uint32_t)lo & 0xFFu;
            for (int d = 0; d < tc::kBiasHiDigits; ++d) {
                const int dig = h > 127 ? 127 : (h < -127 ? -127 : h);
                h -= dig;
                const int k = d + 2;
                wd[k >> 2] |= ((uint32_t)dig & 0xFFu) << (8 * (k & 3));
            }
        }
        *reinterpret_cast<uint4 *>(wb + tc::swz_offset((uint32_t)c, 0u, 32u)) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
        *reinterpret_cast<uint4 *>(wb + tc::swz_offset((uint32_t)c, 1u, 32u)) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
    }
    if (threadIdx.x == 0) {
        int *hdr = reinterpret_cast<int *>(cst + kNt * 12);
        hdr[0] = shmax; hdr[1] = fast ? 1 : 0; hdr[2] = bad ? 1 : 0; hdr[3] = 0;
    }

    // the tile's rows of the int8 matrix, 16 bytes (16 codes = one 32-bit word) per step
    const int rowb = (p.cin + 3) >> 2, pieces = p.k_pad >> 4;
    uint32_t invalid = 0;
    for (int i = threadIdx.x; i < kNt * pieces; i += blockDim.x) {
        const int c = i / pieces, j = i - c * pieces, n = n0 + c;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (n < p.cout && j * 16 < p.cin && !bad) {
            const uint32_t w = *reinterpret_cast<const uint32_t *>(p.w_packed + (size_t)n * rowb + j * 4);
            invalid |= (w >> 1) & ~w & 0x55555555u;
            const uint32_t mag = fast ? (4u << (shmax - s_shift[c])) : 1u, neg = 256u - mag;
            uint32_t wd[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const uint32_t code = (w >> (2 * e)) & 3u;
                const uint32_t byte = code == 1u ? mag : (code == 3u ? neg : 0u);
                wd[e >> 2] |= byte << (8 * (e & 3));
            }
            val = make_uint4(wd[0], wd[1], wd[2], wd[3]);
        }
        *reinterpret_cast<uint4 *>(p.w8 + (size_t)n * p.k_pad + j * 16) = val;
    }
    if (invalid) raise_status(PROM_ERR_BAD_WEIGHT);
}

// One CTA per column tile.
__global__ void __launch_bounds__(256, 1) wide_prep_kernel(const PrepParams p) { prep_tile(p, (int)blockIdx.x); }

// The same for several layers in one launch: CTA b belongs to the layer l with first[l] <= b < first[l + 1].
constexpr int kMaxPrepLayers = 16;
struct PrepBatch {
    int n;
    int first[kMaxPrepLayers + 1];
    PrepParams layer[kMaxPrepLayers];
};

__global__ void __launch_bounds__(256, 1) wide_prep_batch_kernel(const __grid_constant__ PrepBatch t)
{
    int l = 0;
    while (l + 1 < t.n && (int)blockIdx.x >= t.first[l + 1]) ++l;
    prep_tile(t.layer[l], (int)blockIdx.x - t.first[l]);
}

// Two threads issue MMAs (warps 1 and 18), each with half of the weight ring (stages t, t + 2, ..),
// two of the four accumulators (t and t + 2) and every second column tile of a row tile: the
// k-th unit of thread t uses accumulator t + 2 (k & 1).  One thread alone cannot keep the pipe busy
// with 128-column MMAs: between the four MMAs of a chunk it spends more cycles on the barrier
// wait, the commit and its own bookkeeping than the pipe needs for them.  Epilogue group a takes
// the units of accumulator a.
__global__ void __launch_bounds__(kThreads, 1)
wide_conv_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap,
                 const __grid_constant__ CUtensorMap ymap, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + p.off_bars);
    const uint32_t bar_afull = ptx::smem_u32(bars);               // a resident chunk has landed
    const uint32_t bar_aempty = bar_afull + 8 * kMaxKc;           // ... has been read for the last time
    const uint32_t bar_wfull = bar_aempty + 8 * kMaxKc;           // weight ring
    const uint32_t bar_wempty = bar_wfull + 8 * kMaxStages;
    const uint32_t bar_tfull = bar_wempty + 8 * kMaxStages;       // accumulators
    const uint32_t bar_tempty = bar_tfull + 8 * kAccs;
    const uint32_t bar_cfull = bar_tempty + 8 * kAccs;            // constants of a unit (slot = accumulator)
    const uint32_t bar_cempty = bar_cfull + 8 * kAccs;
    const uint32_t bar_drain = bar_cempty + 8 * kAccs;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + kBars);
    volatile int *flags = reinterpret_cast<volatile int *>(bars + kBars + 1);     // [0] abort

    const int g = blockIdx.x % p.groups;
    const int worker = blockIdx.x / p.groups;
    const int nworkers = gridDim.x / p.groups;
    const int cols = p.n_ctiles / p.groups;                       // column tiles g, g + groups, ...
    const uint32_t half = (uint32_t)p.stages >> 1;                // stages per issuing thread
    // With 128-channel tiles the k-th unit of thread t uses slot t + 2 (k & 1) of four (accumulator,
    // constants); with 256-channel tiles a thread has the one slot t, twice as wide.
    const uint32_t nb = (uint32_t)p.nb, nt = nb * (uint32_t)kNt;
    const uint32_t w_stage = nb * kStageBytes;
    auto slot_of = [&](uint32_t t, uint32_t k) { return nb == 1u ? t + 2u * (k & 1u) : t; };
    auto phase_of = [&](uint32_t k) { return nb == 1u ? (k >> 1) & 1u : k & 1u; };

    // ---- prologue -----------------------------------------------------------------------------
    if (warp == 0) {
        if (lane < kMaxKc) {
            ptx::mbar_init(bar_afull + 8 * lane, 1);
            // the last unit of each issuing thread in a row tile lets go of the chunk
            ptx::mbar_init(bar_aempty + 8 * lane, cols >= 2 ? 2 : 1);
        } else if (lane < kMaxKc + kMaxStages) {
            ptx::mbar_init(bar_wfull + 8 * (lane - kMaxKc), 1);
            ptx::mbar_init(bar_wempty + 8 * (lane - kMaxKc), 1);
        } else if (lane < kMaxKc + kMaxStages + kAccs) {
            const int b = lane - kMaxKc - kMaxStages;
            ptx::mbar_init(bar_tfull + 8 * b, 1);
            ptx::mbar_init(bar_tempty + 8 * b, 4 * p.nb);      // the warps that read the slot
            ptx::mbar_init(bar_cfull + 8 * b, 1);
            ptx::mbar_init(bar_cempty + 8 * b, 4 * p.nb);
        } else if (lane == 31) {
            ptx::mbar_init(bar_drain, 2);
            flags[0] = 0;
            ptx::tma_prefetch_desc(&xmap);
            ptx::tma_prefetch_desc(&wmap);
            ptx::tma_prefetch_desc(&ymap);
        }
        ptx::mbar_init_fence();
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32((const void *)tmem_slot), 128u * kAccs);
    tc::build_aconst(smem + p.off_aconst, (int)threadIdx.x, kThreads);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---- producer -----------------------------------------------------------------------------
        // Per pair of column tiles (one for each issuing thread): their constants, then chunk by
        // chunk {the row tile's chunk for the first pair of a row tile, the chunk of either tile's
        // weights into its thread's half of the ring}, then the two tiles' bias digits.
        if (lane == 0) {
            uint32_t hs[2] = {0u, 0u}, hph[2] = {0u, 0u}, k[2] = {0u, 0u}, aph = 0;
            bool ok = true;
            // next stage of thread t's half ring, armed for tx bytes; 0 when a wait gave up
            auto w_slot = [&](int t, uint32_t tx, uint32_t &bar) -> uint32_t {
                const uint32_t st = 2u * hs[t] + (uint32_t)t;
                if (!tc::wait_bar(bar_wempty + 8 * st, hph[t] ^ 1u, flags)) { ok = false; return 0u; }
                bar = bar_wfull + 8 * st;
                ptx::mbar_expect_tx(bar, tx);
                if (++hs[t] == half) { hs[t] = 0; hph[t] ^= 1u; }
                return smem_base + p.off_w + st * w_stage;
            };
            for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers, aph ^= 1u) {
                for (int lc0 = 0; lc0 < cols && ok; lc0 += 2) {
                    const int nu = lc0 + 1 < cols ? 2 : 1;
                    int ct[2];
                    for (int t = 0; t < nu && ok; ++t) {
                        ct[t] = g + (lc0 + t) * p.groups;
                        const uint32_t slot = slot_of((uint32_t)t, k[t]);
                        if (!tc::wait_bar(bar_cempty + 8 * slot, phase_of(k[t]) ^ 1u, flags)) { ok = false; break; }
                        ptx::mbar_expect_tx(bar_cfull + 8 * slot, nb * kConstBytes);
                        ptx::bulk_load(smem_base + p.off_const + slot * nb * kConstBytes,
                                       p.consts + (size_t)ct[t] * nb * kConstBytes, nb * kConstBytes, bar_cfull + 8 * slot);
                        ++k[t];
                    }
                    for (int c = 0; c < p.kc && ok; ++c) {
                        if (lc0 == 0) {
                            if (!tc::wait_bar(bar_aempty + 8 * c, aph ^ 1u, flags)) { ok = false; break; }
                            ptx::mbar_expect_tx(bar_afull + 8 * c, kStageBytes);
                            ptx::tma_load_2d(smem_base + c * kStageBytes, &xmap, c * kChunk, mt * 128, bar_afull + 8 * c);
                        }
                        for (int t = 0; t < nu && ok; ++t) {
                            uint32_t bar = 0;
                            const uint32_t dst = w_slot(t, w_stage, bar);
                            if (ok) ptx::tma_load_2d(dst, &wmap, c * kChunk, ct[t] * (int)nt, bar);
                        }
                    }
                    for (int t = 0; t < nu && ok; ++t) {
                        uint32_t bar = 0;
                        const uint32_t dst = w_slot(t, nb * kWbiasBytes, bar);
                        if (ok) ptx::bulk_load(dst, p.wbias + (size_t)ct[t] * nb * kWbiasBytes, nb * kWbiasBytes, bar);
                    }
                }
            }
            if (!ok) {
                // let the copies in flight land before the CTA goes away
                const unsigned long long t0 = ptx::globaltimer();
                while (ptx::globaltimer() - t0 < 20000ull) {}
            }
        }
    } else if (warp == 1 || warp == kIssuer2) {
        // ---- MMA issuers ------------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t t = warp == 1 ? 0u : 1u;
            // s8 x s8 -> s32, both K-major, M = 128, N = 128 or 256
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((nt >> 3) << 17) | ((128u >> 4) << 24);
            const uint64_t d_128 = tc::smem_desc(0u, 128u), d_32 = tc::smem_desc(0u, 32u);
            const uint64_t ac_desc = d_32 | (uint64_t)((smem_base + p.off_aconst) >> 4);
            const uint32_t a_lo0 = smem_base >> 4, w_lo0 = (smem_base + p.off_w) >> 4;
            const uint32_t a_step = kStageBytes >> 4, w_step = w_stage >> 4;
            uint32_t hs = 0, hph = 0, k = 0, aph = 0;
            bool ok = true;
            for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers, aph ^= 1u) {
                for (int lc = (int)t; lc < cols && ok; lc += 2, ++k) {
                    const uint32_t acc = slot_of(t, k);
                    if (!tc::wait_bar(bar_tempty + 8 * acc, phase_of(k) ^ 1u, flags)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + acc * nt;
                    const bool first = lc == (int)t, last = lc + 2 >= cols;     // of this thread in the row tile
                    uint32_t accum = 0;
                    for (int c = 0; c < p.kc; ++c) {
                        const uint32_t st = 2u * hs + t;
                        if (first && !tc::wait_bar(bar_afull + 8 * c, aph, flags)) { ok = false; break; }
                        if (!tc::wait_bar(bar_wfull + 8 * st, hph, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t a_lo = a_lo0 + (uint32_t)c * a_step, w_lo = w_lo0 + st * w_step;
                        const int nks = c == p.kc - 1 ? p.ksteps_last : 4;
                        for (int ks = 0; ks < nks; ++ks) {
                            ptx::mma_i8(d_tmem, d_128 | (uint64_t)(a_lo + 2 * ks), d_128 | (uint64_t)(w_lo + 2 * ks), idesc, accum);
                            accum = 1;
                        }
                        ptx::mma_commit(bar_wempty + 8 * st);
                        if (last) ptx::mma_commit(bar_aempty + 8 * c);
                        if (++hs == half) { hs = 0; hph ^= 1u; }
                    }
                    if (!ok) break;
                    // the bias step: the constant block of 1s and 127s against the tile's digits
                    const uint32_t st = 2u * hs + t;
                    if (!tc::wait_bar(bar_wfull + 8 * st, hph, flags)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    ptx::mma_i8(d_tmem, ac_desc, d_32 | (uint64_t)(w_lo0 + st * w_step), idesc, 1u);
                    ptx::mma_commit(bar_wempty + 8 * st);
                    if (++hs == half) { hs = 0; hph ^= 1u; }
                    ptx::mma_commit(bar_tfull + 8 * acc);
                }
            }
            ptx::mma_commit(bar_drain);
            const unsigned long long t0 = ptx::globaltimer();
            while (!ptx::mbar_try_wait(bar_drain, 0) && ptx::globaltimer() - t0 < tc::kWaitLimitNs) {}
        }
    } else {
        // ---- epilogue ---------------------------------------------------------------------------------
        // Group grp follows issuing thread grp & 1.  With 128-channel tiles it takes that thread's
        // units with k & 1 == grp >> 1 (slot grp); with 256-channel tiles it takes every unit of the
        // thread and the half grp >> 1 of its 256 columns.
        const int q = warp & 3, grp = (warp - 2) >> 2;
        const int t = grp & 1, h = grp >> 1;
        uint8_t *slab = smem + p.off_out + (size_t)(warp - 2) * kSlabBytes;
        uint8_t *my_row = slab + lane * kEpiCols;
        const uint32_t slab_addr = ptx::smem_u32(slab);
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t acc = nb == 1u ? (uint32_t)grp : (uint32_t)t;          // slot: barriers, accumulator
        const uint32_t blk = nb == 1u ? (uint32_t)grp : 2u * (uint32_t)t + (uint32_t)h;   // 128-column block of constants
        const uint32_t tcol = blk * 128u;                                       // its accumulator columns
        const int col_in_tile = nb == 1u ? 0 : h * kNt;
        const uint8_t *cst = smem + p.off_const + blk * kConstBytes;
        const int *cm = reinterpret_cast<const int *>(cst);
        const int2 *cbs = reinterpret_cast<const int2 *>(cst + kNt * 4);
        const int *hdr = reinterpret_cast<const int *>(cst + kNt * 12);
        uint32_t k = 0;
        bool ok = true;
        for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers) {
            const int row0 = mt * 128 + q * 32;
            for (int lc = t; lc < cols && ok; lc += 2, ++k) {
                if (nb == 1u && (int)(k & 1u) != h) continue;
                const int col0 = (g + lc * p.groups) * (int)nt + col_in_tile;
                const uint32_t ph = phase_of(k);
                if (!tc::wait_bar<true>(bar_cfull + 8 * acc, ph, flags)) { ok = false; break; }
                if (!tc::wait_bar<true>(bar_tfull + 8 * acc, ph, flags)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const int shmax = hdr[0];
                const bool fast = hdr[1] != 0, bad = hdr[2] != 0;
#pragma unroll 1
                for (int pc = 0; pc < kNt / (int)kEpiCols; ++pc) {
                    const int col = col0 + pc * (int)kEpiCols;
                    const uint32_t rel = pc == kNt / (int)kEpiCols - 1 ? bar_tempty + 8 * acc : 0u;
                    if (col >= p.cout || bad) {                 // nothing of this piece exists
                        tc::release_acc(rel);
                        continue;
                    }
                    // the previous store has read the slab
                    ptx::bulk_wait_read0();
                    __syncwarp();
                    const uint32_t taddr = t_lane + tcol + pc * kEpiCols;
                    if (fast) tc::epi_fast_fixed<32>(taddr, cm + pc * kEpiCols, shmax, my_row, rel);
                    else tc::epi_exact_subtile<32>(32, p.act_min, p.act_max, taddr, cm + pc * kEpiCols,
                                                   cbs + pc * kEpiCols, my_row, rel);
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0 && row0 < p.m) {
                        ptx::tma_store_2d(&ymap, col, row0, slab_addr);
                        ptx::bulk_commit();
                    }
                }
                // the unit's constants are free for this group's next unit
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_cempty + 8 * acc);
            }
        }
        ptx::bulk_wait_read0();
    }

    // ---- teardown ---------------------------------------------------------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 128u * kAccs);
    }
}

}}  // namespace prom::wide
