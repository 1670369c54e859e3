// A run of consecutive pointwise layers on row tiles that never leave the SM.
//
// Every layer of such a run is per-pixel: output row r of layer l depends on row r of layer
// l - 1 alone.  A CTA (one per SM) therefore takes a tile of up to 128 rows through all the layers
// of the run with the activations in shared memory: the first layer's input arrives by TMA, the
// epilogue of layer l requantises its accumulators straight into the K-major, 128-byte swizzled
// operand layout that the MMAs of layer l + 1 read, and only the last layer's output goes back to
// global memory.  The intermediate tensors of the run are never written, and the grid-wide
// hand-over between two layers becomes a shared-memory barrier.
//
// The layers of a run alternate between two kinds, as the blocks of the network do:
//   P  ("project", the first layer and every second one after it): many input channels, at most
//      384 output channels.  Its input is a stream of 128-byte chunks of K that pass through a
//      small ring of shared memory; all of its (at most three) accumulators are live while the
//      chunks go by, each chunk feeding every accumulator before its ring slot is released.  Its
//      output is the resident "narrow" operand (at most three chunks).
//   E  ("expand", the layers in between): reads the narrow operand, one column tile of 128 output
//      channels ("unit") after the other; column tile c of its output is chunk c of the next P
//      layer's stream, written into the ring by the epilogue.
// The wide activations of a block therefore exist one ring slot at a time: the MMAs of the P
// layer consume chunk c while the epilogue is busy with column tile c + 1 of the E layer.  The
// first layer's chunks are put into the same ring by TMA.
//
// The weights are streamed too: wide_prep_kernel expands each layer's 2-bit codes once into an
// int8 matrix [Cout padded to 128][Cin padded to 128] in global scratch (scaled for the
// one-multiply epilogue where the constants allow it) with the bias digits and requantisation
// constants of every unit beside it; warp 0 pulls the matrix through a ring of 16 KB stages, one
// half of it for each MMA thread, and a unit's digits and constants into the slot of its accumulator.
//
// Warp 0 issues the loads, warp 1 the MMAs of the E layers, warp 18 those of the P layers, warps
// 2..17 are four epilogue groups; group g takes columns [32 g, 32 g + 32) of every unit, so that all
// sixteen warps work on the unit that the next MMAs are waiting for.  Everybody walks the same
// sequence (row tile, layer, unit) and derives barrier phases from it: accumulator and constant
// slots from a count of uses per slot, ring slots from the chunk's position in the sequence.
#pragma once

#include "tc.cuh"

namespace prom { namespace stack {

constexpr int kEpiWarps = 16;
constexpr int kIssuer2 = 2 + kEpiWarps;           // warp of the P layers' MMA issuer
constexpr int kThreads = 32 * (kIssuer2 + 1);
constexpr int kMaxLayers = 16;
constexpr int kNarrowMax = 3;                     // chunks of the narrow operand: P layers have <= 384 outputs
constexpr int kRingMax = 4;
constexpr int kMaxStages = 8;
constexpr int kAccs = 4;                          // accumulators of 128 columns: all of tensor memory
constexpr uint32_t kChunkBytes = 128u * 128u;     // 128 rows x 128 bytes of K; also a weight stage
constexpr uint32_t kWbiasBytes = 128u * 32u;      // bias digits of a unit (32-byte swizzled rows)
constexpr uint32_t kConstBytes = 128u * 4u + 128u * 8u + 16u + 112u;   // as wide_prep_kernel writes them
constexpr uint32_t kSlotBytes = 6144;             // a unit's bias digits, then its constants; 256-byte aligned
constexpr uint32_t kSlabBytes = 32u * 32u;        // staging of 32 rows x 32 columns per warp (last layer)
// barriers: ring (full, free), narrow chunks, weight ring (full, empty), accumulators (full,
// empty), constants (full, empty), drain
constexpr int kBars = 2 * kRingMax + 4 + 2 * kMaxStages + 4 * kAccs + 1;

struct Layer {
    CUtensorMap wmap;           // the int8 weight matrix, box {128, 128}
    const uint8_t *wbias;       // [n_ct][kWbiasBytes]
    const uint8_t *consts;      // [n_ct][kConstBytes]
    int cout;
    int kc, ksteps;             // chunks and 32-byte MMA steps of K
    int n_ct;                   // column tiles of 128 ("units")
    int act_min, act_max;
    int streamed;               // 1: a P layer (input through the ring); 0: an E layer (narrow operand)
    int out_mode;               // 0: the narrow operand, 1: the ring, 2: global memory (last layer)
    int slot0, nslots;          // unit ct uses accumulator slot0 + ct % nslots
    int ring_off;               // P layers: position of chunk 0 among the ring chunks of a row tile
};

struct Table {
    CUtensorMap xmap, ymap;
    long long m;
    int n_layers, n_mtiles;
    int tm;                     // rows of a tile (128, or whole image rows of a subsampled input)
    int x3d, box_r;
    int stages;                 // of the weight ring (even)
    int ring;                   // slots of the activation ring
    int chunks_per_tile;        // ring chunks a row tile sends through (all its P layers)
    uint32_t off_nar, off_ring, off_w, off_const, off_out, off_aconst, off_bars;
    int8_t *y;                  // the last layer's output [m][cout]
    int pdl, pdl_next;
    Layer layer[kMaxLayers];
};

__global__ void __launch_bounds__(kThreads, 1) stack_kernel(const __grid_constant__ Table t)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + t.off_bars);
    const uint32_t bar_rfull = ptx::smem_u32(bars);               // a ring slot holds its chunk
    const uint32_t bar_rfree = bar_rfull + 8 * kRingMax;          // ... has been read for the last time
    const uint32_t bar_nar = bar_rfree + 8 * kRingMax;            // a chunk of the narrow operand is written
    const uint32_t bar_wfull = bar_nar + 8 * 4;                   // weight ring
    const uint32_t bar_wempty = bar_wfull + 8 * kMaxStages;
    const uint32_t bar_tfull = bar_wempty + 8 * kMaxStages;       // accumulators
    const uint32_t bar_tempty = bar_tfull + 8 * kAccs;
    const uint32_t bar_cfull = bar_tempty + 8 * kAccs;            // constants of a unit (slot = accumulator)
    const uint32_t bar_cempty = bar_cfull + 8 * kAccs;
    const uint32_t bar_drain = bar_cempty + 8 * kAccs;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + kBars);
    volatile int *flags = reinterpret_cast<volatile int *>(bars + kBars + 1);     // [0] abort

    if (t.pdl_next) ptx::grid_dep_launch();

    const uint32_t half = (uint32_t)t.stages >> 1;                // stages per issuing thread
    const uint32_t R = (uint32_t)t.ring, G = (uint32_t)t.chunks_per_tile;

    // ---- prologue -----------------------------------------------------------------------------
    if (warp == 0) {
        if (lane < kRingMax) {
            ptx::mbar_init(bar_rfull + 8 * lane, kEpiWarps);
            ptx::mbar_init(bar_rfree + 8 * lane, 1);
            ptx::mbar_init(bar_nar + 8 * lane, kEpiWarps);
        } else if (lane < kRingMax + kMaxStages) {
            ptx::mbar_init(bar_wfull + 8 * (lane - kRingMax), 1);
            ptx::mbar_init(bar_wempty + 8 * (lane - kRingMax), 1);
        } else if (lane < kRingMax + kMaxStages + kAccs) {
            const int b = lane - kRingMax - kMaxStages;
            ptx::mbar_init(bar_tfull + 8 * b, 1);
            ptx::mbar_init(bar_tempty + 8 * b, kEpiWarps);
            ptx::mbar_init(bar_cfull + 8 * b, 1);
            ptx::mbar_init(bar_cempty + 8 * b, kEpiWarps);
        } else if (lane == 31) {
            ptx::mbar_init(bar_drain, 2);
            flags[0] = 0;
            ptx::tma_prefetch_desc(&t.xmap);
            ptx::tma_prefetch_desc(&t.ymap);
            ptx::tma_prefetch_desc(&t.layer[0].wmap);
        }
        ptx::mbar_init_fence();
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32((const void *)tmem_slot), 128u * kAccs);
    tc::build_aconst(smem + t.off_aconst, (int)threadIdx.x, kThreads);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---- producer -----------------------------------------------------------------------------
        // In the order the MMA threads need them: for the first layer chunk by chunk {the input
        // chunk into the activation ring, that chunk of every unit's weights}; for an E layer unit
        // by unit {its constants and bias digits, its weights, then chunk `unit` of the weights of
        // the P layer that follows}.  A P layer's constants go out right behind the first unit of
        // the E layer in front of it, long before its epilogue asks for them.
        if (lane == 0) {
            uint32_t hs[2] = {0u, 0u}, hph[2] = {0u, 0u}, par = 0, it = 0;     // par bit s: parity of slot s's uses
            bool ok = true;
            // next stage of thread w's half ring, armed for tx bytes; 0 when a wait gave up
            auto w_slot = [&](uint32_t w, uint32_t tx, uint32_t &bar) -> uint32_t {
                const uint32_t st = 2u * hs[w] + w;
                if (!tc::wait_bar(bar_wempty + 8 * st, hph[w] ^ 1u, flags)) { ok = false; return 0u; }
                bar = bar_wfull + 8 * st;
                ptx::mbar_expect_tx(bar, tx);
                if (++hs[w] == half) { hs[w] = 0; hph[w] ^= 1u; }
                return smem_base + t.off_w + st * kChunkBytes;
            };
            auto load_w = [&](uint32_t w, const Layer &L, int kchunk, int ct) {
                uint32_t bar = 0;
                const uint32_t dst = w_slot(w, kChunkBytes, bar);
                if (ok) ptx::tma_load_2d(dst, &L.wmap, kchunk * 128, ct * 128, bar);
            };
            auto load_consts = [&](const Layer &L, int ct) {
                const uint32_t slot = (uint32_t)(L.slot0 + ct % L.nslots), use = (par >> slot) & 1u;
                par ^= 1u << slot;
                if (!tc::wait_bar(bar_cempty + 8 * slot, use ^ 1u, flags)) { ok = false; return; }
                ptx::mbar_expect_tx(bar_cfull + 8 * slot, kWbiasBytes + kConstBytes);
                const uint32_t dst = smem_base + t.off_const + slot * kSlotBytes;
                ptx::bulk_load(dst, L.wbias + (size_t)ct * kWbiasBytes, kWbiasBytes, bar_cfull + 8 * slot);
                ptx::bulk_load(dst + kWbiasBytes, L.consts + (size_t)ct * kConstBytes, kConstBytes, bar_cfull + 8 * slot);
            };
            for (int mt = blockIdx.x; mt < t.n_mtiles && ok; mt += gridDim.x, ++it) {
                const Layer &L0 = t.layer[0];
                for (int j = 0; j < L0.n_ct && ok; ++j) load_consts(L0, j);
                for (int c = 0; c < L0.kc && ok; ++c) {
                    const uint32_t g = it * G + (uint32_t)c, rs = g % R;
                    if (g >= R && !tc::wait_bar(bar_rfree + 8 * rs, ((g / R) - 1u) & 1u, flags)) { ok = false; break; }
                    // the first read of what the previous kernel wrote
                    if (it == 0 && c == 0 && t.pdl) ptx::grid_dep_wait();
                    const uint32_t bar = bar_rfull + 8 * rs;
                    ptx::mbar_expect_tx(bar, 128u * (uint32_t)t.tm);
                    ptx::mbar_arrive_n(bar, kEpiWarps - 1);      // the arrivals an epilogue-written chunk would get
                    const uint32_t dst = smem_base + t.off_ring + rs * kChunkBytes;
                    if (t.x3d) ptx::tma_load_3d(dst, &t.xmap, c * 128, 0, mt * t.box_r, bar);
                    else ptx::tma_load_2d(dst, &t.xmap, c * 128, mt * t.tm, bar);
                    for (int j = 0; j < L0.n_ct && ok; ++j) load_w(1u, L0, c, j);
                }
                for (int l = 1; l < t.n_layers && ok; ++l) {
                    const Layer &L = t.layer[l];
                    if (L.streamed) continue;                   // went out with the E layer in front of it
                    const Layer *P = l + 1 < t.n_layers ? &t.layer[l + 1] : nullptr;
                    for (int ct = 0; ct < L.n_ct && ok; ++ct) {
                        load_consts(L, ct);
                        for (int s = 0; s < L.kc && ok; ++s) load_w(0u, L, s, ct);
                        if (P) {
                            if (ct == 0)
                                for (int j = 0; j < P->n_ct && ok; ++j) load_consts(*P, j);
                            for (int j = 0; j < P->n_ct && ok; ++j) load_w(1u, *P, ct, j);
                        }
                    }
                }
            }
            if (!ok) {
                // let the copies in flight land before the CTA goes away
                const unsigned long long t0 = ptx::globaltimer();
                while (ptx::globaltimer() - t0 < 20000ull) {}
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer of the E layers: narrow operand x one column tile after the other -------------
        if (lane == 0) {
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
            const uint64_t d_128 = tc::smem_desc(0u, 128u), d_32 = tc::smem_desc(0u, 32u);
            const uint64_t ac_desc = d_32 | (uint64_t)((smem_base + t.off_aconst) >> 4);
            const uint32_t w_lo0 = (smem_base + t.off_w) >> 4, a_lo0 = (smem_base + t.off_nar) >> 4;
            const uint32_t c_lo0 = (smem_base + t.off_const) >> 4;
            uint32_t hs = 0, hph = 0, par = 0;
            uint32_t nar_par = 0;           // bit c: parity of the next completion of narrow chunk c
            bool ok = true;
            for (int mt = blockIdx.x; mt < t.n_mtiles && ok; mt += gridDim.x) {
                for (int l = 0; l < t.n_layers && ok; ++l) {
                    const Layer &L = t.layer[l];
                    if (L.streamed) {
                        for (int ct = 0; ct < L.n_ct; ++ct) par ^= 1u << (L.slot0 + ct % L.nslots);
                        continue;
                    }
                    for (int ct = 0; ct < L.n_ct && ok; ++ct) {
                        const uint32_t acc = (uint32_t)(L.slot0 + ct % L.nslots), use = (par >> acc) & 1u;
                        par ^= 1u << acc;
                        if (!tc::wait_bar(bar_tempty + 8 * acc, use ^ 1u, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t d_tmem = tmem_base + acc * 128u;
                        uint32_t accum = 0;
                        for (int s = 0; s < L.kc; ++s) {
                            // the first unit of the layer waits for the narrow chunks
                            if (ct == 0 && !tc::wait_bar(bar_nar + 8 * s, (nar_par >> s) & 1u, flags)) { ok = false; break; }
                            const uint32_t st = 2u * hs;
                            if (!tc::wait_bar(bar_wfull + 8 * st, hph, flags)) { ok = false; break; }
                            ptx::tc_fence_after_sync();
                            const uint32_t a_lo = a_lo0 + (uint32_t)s * (kChunkBytes >> 4);
                            const uint32_t w_lo = w_lo0 + st * (kChunkBytes >> 4);
                            const int left = L.ksteps - 4 * s, nks = left < 4 ? left : 4;
                            for (int ks = 0; ks < nks; ++ks) {
                                ptx::mma_i8(d_tmem, d_128 | (uint64_t)(a_lo + 2 * ks), d_128 | (uint64_t)(w_lo + 2 * ks), idesc, accum);
                                accum = 1;
                            }
                            ptx::mma_commit(bar_wempty + 8 * st);
                            if (++hs == half) { hs = 0; hph ^= 1u; }
                        }
                        if (!ok) break;
                        // the bias step: the constant block of 1s and 127s against the unit's digits
                        if (!tc::wait_bar(bar_cfull + 8 * acc, use, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        ptx::mma_i8(d_tmem, ac_desc, d_32 | (uint64_t)(c_lo0 + acc * (kSlotBytes >> 4)), idesc, 1u);
                        ptx::mma_commit(bar_tfull + 8 * acc);
                    }
                    // the chunks this layer read complete once more before they are read again
                    for (int c = 0; c < L.kc; ++c) nar_par ^= 1u << c;
                }
            }
            ptx::mma_commit(bar_drain);
            const unsigned long long t0 = ptx::globaltimer();
            while (!ptx::mbar_try_wait(bar_drain, 0) && ptx::globaltimer() - t0 < tc::kWaitLimitNs) {}
        }
    } else if (warp == kIssuer2) {
        // ---- MMA issuer of the P layers: every chunk of the stream against every unit's weights -------
        if (lane == 0) {
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
            const uint64_t d_128 = tc::smem_desc(0u, 128u), d_32 = tc::smem_desc(0u, 32u);
            const uint64_t ac_desc = d_32 | (uint64_t)((smem_base + t.off_aconst) >> 4);
            const uint32_t w_lo0 = (smem_base + t.off_w) >> 4, r_lo0 = (smem_base + t.off_ring) >> 4;
            const uint32_t c_lo0 = (smem_base + t.off_const) >> 4;
            uint32_t hs = 0, hph = 0, par = 0, it = 0;
            bool ok = true;
            for (int mt = blockIdx.x; mt < t.n_mtiles && ok; mt += gridDim.x, ++it) {
                for (int l = 0; l < t.n_layers && ok; ++l) {
                    const Layer &L = t.layer[l];
                    if (!L.streamed) {
                        for (int ct = 0; ct < L.n_ct; ++ct) par ^= 1u << (L.slot0 + ct % L.nslots);
                        continue;
                    }
                    const uint32_t use = par;                   // bit of slot s: this use's parity (n_ct <= nslots here)
                    for (int j = 0; j < L.n_ct; ++j) par ^= 1u << (L.slot0 + j);
                    for (int c = 0; c < L.kc && ok; ++c) {
                        const uint32_t g = it * G + (uint32_t)(L.ring_off + c), rs = g % R;
                        if (!tc::wait_bar(bar_rfull + 8 * rs, (g / R) & 1u, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t a_lo = r_lo0 + rs * (kChunkBytes >> 4);
                        const int left = L.ksteps - 4 * c, nks = left < 4 ? left : 4;
                        for (int j = 0; j < L.n_ct; ++j) {
                            const uint32_t acc = (uint32_t)(L.slot0 + j);
                            if (c == 0) {
                                if (!tc::wait_bar(bar_tempty + 8 * acc, ((use >> acc) & 1u) ^ 1u, flags)) { ok = false; break; }
                                ptx::tc_fence_after_sync();
                            }
                            const uint32_t st = 2u * hs + 1u;
                            if (!tc::wait_bar(bar_wfull + 8 * st, hph, flags)) { ok = false; break; }
                            ptx::tc_fence_after_sync();
                            const uint32_t w_lo = w_lo0 + st * (kChunkBytes >> 4);
                            const uint32_t d_tmem = tmem_base + acc * 128u;
                            for (int ks = 0; ks < nks; ++ks)
                                ptx::mma_i8(d_tmem, d_128 | (uint64_t)(a_lo + 2 * ks), d_128 | (uint64_t)(w_lo + 2 * ks), idesc,
                                            (c | ks) ? 1u : 0u);
                            ptx::mma_commit(bar_wempty + 8 * st);
                            if (++hs == half) { hs = 0; hph ^= 1u; }
                        }
                        if (!ok) break;
                        ptx::mma_commit(bar_rfree + 8 * rs);     // every unit has read the chunk
                    }
                    for (int j = 0; j < L.n_ct && ok; ++j) {
                        const uint32_t acc = (uint32_t)(L.slot0 + j);
                        if (!tc::wait_bar(bar_cfull + 8 * acc, (use >> acc) & 1u, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        ptx::mma_i8(tmem_base + acc * 128u, ac_desc, d_32 | (uint64_t)(c_lo0 + acc * (kSlotBytes >> 4)), idesc, 1u);
                        ptx::mma_commit(bar_tfull + 8 * acc);
                    }
                }
            }
            ptx::mma_commit(bar_drain);
            const unsigned long long t0 = ptx::globaltimer();
            while (!ptx::mbar_try_wait(bar_drain, 0) && ptx::globaltimer() - t0 < tc::kWaitLimitNs) {}
        }
    } else {
        // ---- epilogue ---------------------------------------------------------------------------------
        // Warp (grp, q) requantises rows [32 q, 32 q + 32) x columns [32 grp, 32 grp + 32) of every unit:
        // into the narrow operand, into the ring, or (last layer) through a staging slab to Y.
        const int q = warp & 3, grp = (warp - 2) >> 2;
        const uint32_t r = (uint32_t)(q * 32 + lane);
        uint8_t *slab = smem + t.off_out + (size_t)(warp - 2) * kSlabBytes;
        uint8_t *my_row = slab + lane * 32;
        const uint32_t slab_addr = ptx::smem_u32(slab);
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)grp * 32u;
        // the two 16-byte pieces of this thread's 32 columns inside a 128-byte swizzled row
        const uint32_t piece0 = r * 128u + ((((uint32_t)grp * 2u) ^ (r & 7u)) << 4);
        const uint32_t piece1 = r * 128u + ((((uint32_t)grp * 2u + 1u) ^ (r & 7u)) << 4);
        uint32_t par = 0, it = 0;
        bool ok = true;
        for (int mt = blockIdx.x; mt < t.n_mtiles && ok; mt += gridDim.x, ++it) {
            const long long row0 = (long long)mt * t.tm + q * 32;
            long long rows_valid = t.tm - q * 32;
            if (t.m - row0 < rows_valid) rows_valid = t.m - row0;
            if (rows_valid > 32) rows_valid = 32;
            for (int l = 0; l < t.n_layers && ok; ++l) {
                const Layer &L = t.layer[l];
                const uint32_t g0 = L.out_mode == 1 ? it * G + (uint32_t)t.layer[l + 1].ring_off : 0u;
                for (int ct = 0; ct < L.n_ct && ok; ++ct) {
                    const uint32_t acc = (uint32_t)(L.slot0 + ct % L.nslots), ph = (par >> acc) & 1u;
                    par ^= 1u << acc;
                    if (!tc::wait_bar<true>(bar_cfull + 8 * acc, ph, flags)) { ok = false; break; }
                    if (!tc::wait_bar<true>(bar_tfull + 8 * acc, ph, flags)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint8_t *cst = smem + t.off_const + acc * kSlotBytes + kWbiasBytes;
                    const int *cm = reinterpret_cast<const int *>(cst) + grp * 32;
                    const int2 *cbs = reinterpret_cast<const int2 *>(cst + 128 * 4) + grp * 32;
                    const int *hdr = reinterpret_cast<const int *>(cst + 128 * 12);
                    const int shmax = hdr[0];
                    const bool fast = hdr[1] != 0;
                    const int col = ct * 128 + grp * 32;
                    const uint32_t rel = bar_tempty + 8 * acc;
                    const uint32_t taddr = t_lane + acc * 128u;
                    if (L.out_mode != 2) {
                        uint8_t *chunk;
                        uint32_t done;
                        if (L.out_mode == 0) {
                            chunk = smem + t.off_nar + (size_t)ct * kChunkBytes;
                            done = bar_nar + 8 * (uint32_t)ct;
                        } else {
                            // chunk ct of the next layer's stream: its ring slot must have been read
                            const uint32_t g = g0 + (uint32_t)ct, rs = g % R;
                            if (g >= R && !tc::wait_bar<true>(bar_rfree + 8 * rs, ((g / R) - 1u) & 1u, flags)) { ok = false; break; }
                            chunk = smem + t.off_ring + (size_t)rs * kChunkBytes;
                            done = bar_rfull + 8 * rs;
                        }
                        if (col >= L.cout) {
                            tc::release_acc(rel);                   // nothing of this piece exists
                        } else if (fast) {
                            uint32_t v[32];
                            ptx::tmem_ld_x32(taddr, v);
                            ptx::tmem_wait_ld();
                            tc::release_acc(rel);
                            const long long r64 = 1ll << (32 + shmax);
                            tc::fast_piece<16>(*reinterpret_cast<const uint32_t (*)[16]>(&v[0]), cm, r64, shmax,
                                               chunk + piece0, true);
                            tc::fast_piece<16>(*reinterpret_cast<const uint32_t (*)[16]>(&v[16]), cm + 16, r64, shmax,
                                               chunk + piece1, true);
                        } else {
                            tc::epi_exact<16>(taddr, cm, cbs, L.act_min, L.act_max, chunk + piece0, true, 0u);
                            tc::epi_exact<16>(taddr + 16, cm + 16, cbs + 16, L.act_min, L.act_max, chunk + piece1,
                                              true, rel);
                        }
                        ptx::fence_proxy_async_smem();          // the next layer's MMAs read these bytes
                        __syncwarp();
                        if (lane == 0) {
                            ptx::mbar_arrive(bar_cempty + 8 * acc);     // the unit's constants are free
                            ptx::mbar_arrive(done);                     // this warp's part of the chunk is written
                        }
                        continue;
                    }
                    if (col >= L.cout) {
                        tc::release_acc(rel);
                    } else {
                        ptx::bulk_wait_read0();                 // the previous store has read the slab
                        __syncwarp();
                        if (fast) tc::epi_fast_fixed<32>(taddr, cm, shmax, my_row, rel);
                        else tc::epi_exact_subtile<32>(32, L.act_min, L.act_max, taddr, cm, cbs, my_row, rel);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (rows_valid == 32) {
                            if (lane == 0) {
                                ptx::tma_store_2d(&t.ymap, col, (int)row0, slab_addr);
                                ptx::bulk_commit();
                            }
                        } else if (rows_valid > 0) {
                            // a short tile or the end of the matrix: row by row, whole 16-byte columns only
                            const uint32_t ncol = L.cout - col < 32 ? (uint32_t)(L.cout - col) : 32u;
                            if (lane < rows_valid) {
                                ptx::bulk_store(t.y + (row0 + lane) * L.cout + col, slab_addr + (uint32_t)lane * 32u, ncol);
                                ptx::bulk_commit();
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar_cempty + 8 * acc);
                }
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

}}  // namespace prom::stack
