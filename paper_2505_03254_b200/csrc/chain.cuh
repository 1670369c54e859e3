// Depth-first execution of a run of consecutive pointwise layers in one launch.
//
// Every layer of such a run is per-pixel: output row r of layer l depends on input row r
// alone (a 1x1 kernel), so a CTA that owns a tile of rows can take it through all the layers
// of the run without ever waiting for another CTA.  Each layer's output is still written to
// global memory, and the next layer reads it back from there (through L2) with TMA: the
// intermediate tensors exist exactly as in the one-launch-per-layer form; what disappears is
// the grid-wide hand-over between layers, which costs several microseconds per layer when a
// layer is a single wave of tiles.
//
// A CTA interleaves up to kMaxTasks tiles ("tasks"): the unit order is
//     for layer: for task: for subtile (nt output channels): for K chunk
// so that the store -> load round trip of one task at a layer boundary hides behind the
// other tasks' units.  Nothing is resident.  One ring of shared-memory stages feeds the
// MMAs; a stage holds one K chunk of the task's activation tile (TMA) next to the same K
// chunk of the subtile's prepared weights (a bulk copy straight from the image
// tc_prep_kernel wrote for that subtile) and, with the last chunk, the subtile's bias digits;
// the per-subtile constants of the epilogue go through a second, smaller ring.
//
// Warp roles as in tc_conv_kernel: warp 0 issues all loads (one thread), warp 1 issues the
// MMAs, warps 2..9 are two epilogue groups that take units alternately.  Completion of a
// layer for a task is a counter in shared memory: an epilogue warp adds one after the bulk
// stores of its last unit of that (layer, task) have completed, and the loading thread
// compares the counter with the number of warps that will have reported by then before it
// reads the task's rows of that layer back.
#pragma once

#include "tc.cuh"

namespace prom { namespace chain {

constexpr int kThreads = tc::kThreads;
constexpr int kMaxLayers = 16;
constexpr int kMaxTasks = 4;
constexpr int kStages = 4, kConstSlots = 8;
constexpr int kCwMax = 64;                 // K chunk: 32 or 64 bytes of a row
constexpr int kNtMax = 96;                 // subtile width
constexpr int kAccCols = 128;              // tensor-memory columns per accumulator (two of them)
constexpr uint32_t kAPart = 128u * kCwMax;                          // activation chunk of a stage
constexpr uint32_t kWPart = (uint32_t)kNtMax * kCwMax;              // weights chunk
constexpr uint32_t kStage = kAPart + kWPart + (uint32_t)kNtMax * 32u;   // ... and the bias digits
constexpr uint32_t kConstSlot = 1280;      // mult, {bias, shift}, header of one subtile (<= 96*12+16)
constexpr uint32_t kSlab = 32u * kNtMax;
constexpr uint32_t kOffOut = kStages * kStage;
constexpr uint32_t kOffConst = kOffOut + tc::kEpiWarps * kSlab;
constexpr uint32_t kOffAconst = kOffConst + kConstSlots * kConstSlot;
constexpr uint32_t kOffBars = kOffAconst + tc::kAConstBytes;
constexpr int kBarSlots = 2 * kStages + 4 + 2 * kConstSlots + 1;
constexpr uint32_t kSmemBytes = kOffBars + 8 * kBarSlots + 64 + 1024 /* alignment slack */;
static_assert(kStage % 1024 == 0 && kAPart % 1024 == 0 && (kAPart + kWPart) % 1024 == 0, "swizzle atoms");

struct Layer {
    CUtensorMap xmap, ymap;
    const uint8_t *image;       // one prepared image per subtile, image_stride bytes apart
    int8_t *y;
    uint32_t image_stride;
    uint32_t wbias_off, const_off, const_bytes;   // inside an image
    uint32_t a_tx;              // bytes one activation load brings
    int n;                      // cout
    int cw, kc, ksteps_last;
    int nt, nt_pad, n_sub;
    int store_2d;
    int x3d, box_r;
    int act_min, act_max;
};

struct Table {
    long long m_rows;
    int n_layers, n_tasks, tm;
    int pdl, pdl_next;
    Layer layer[kMaxLayers];
};

// Any width (a multiple of 8): the same in chunks of 32, 16 and 8 columns.
__device__ __noinline__ void epi_fast_any(int nt, uint32_t taddr, const int *cm, int shmax, uint8_t *dst_row,
                                          uint32_t bar_release)
{
    const bool wide = (nt & 15) == 0;
    const long long r64 = 1ll << (32 + shmax);
    int c = 0;
    for (; c + 32 <= nt; c += 32) {
        uint32_t v[32];
        ptx::tmem_ld_x32(taddr + c, v);
        ptx::tmem_wait_ld();
        if (c + 32 == nt) tc::release_acc(bar_release);
        tc::fast_piece<32>(v, cm + c, r64, shmax, dst_row + c, wide);
    }
    if (c + 16 <= nt) {
        uint32_t v[16];
        ptx::tmem_ld_x16(taddr + c, v);
        ptx::tmem_wait_ld();
        if (c + 16 == nt) tc::release_acc(bar_release);
        tc::fast_piece<16>(v, cm + c, r64, shmax, dst_row + c, wide);
        c += 16;
    }
    if (c + 8 <= nt) {
        uint32_t v[8];
        ptx::tmem_ld_x8(taddr + c, v);
        ptx::tmem_wait_ld();
        tc::release_acc(bar_release);
        tc::fast_piece<8>(v, cm + c, r64, shmax, dst_row + c, wide);
    }
}

// Position in the unit order of one round: layer, task, subtile, K chunk.
struct Pos {
    int l, g, s, c;
    bool end;
};

__device__ __forceinline__ void next_chunk(const Table &t, int ntask, Pos &p)
{
    const Layer &L = t.layer[p.l];
    if (++p.c < L.kc) return;
    p.c = 0;
    if (++p.s < L.n_sub) return;
    p.s = 0;
    if (++p.g < ntask) return;
    p.g = 0;
    if (++p.l >= t.n_layers) p.end = true;
}

// Epilogue warps that will have reported a (layer, task) as complete: four per group that
// owns at least one of its units (units alternate between the two groups).
__device__ __forceinline__ int reports_of(const Layer &L) { return L.n_sub >= 2 ? 8 : 4; }

__global__ void __launch_bounds__(kThreads, 2) tc_chain_kernel(const __grid_constant__ Table t)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kOffBars);
    const uint32_t bar_full = ptx::smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * kStages;
    const uint32_t bar_tfull = bar_empty + 8 * kStages;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_cfull = bar_tempty + 16;
    const uint32_t bar_cfree = bar_cfull + 8 * kConstSlots;
    const uint32_t bar_drain = bar_cfree + 8 * kConstSlots;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + kBarSlots);
    volatile int *flags = reinterpret_cast<volatile int *>(bars + kBarSlots) + 2;   // [0] abort
    volatile int *done = flags + 2;                                                  // [kMaxTasks]

    if (t.pdl_next) ptx::grid_dep_launch();

    // ---- prologue ---------------------------------------------------------------------------
    if (warp == 0) {
        if (lane < kStages) {
            ptx::mbar_init(bar_full + 8 * lane, 1);
            ptx::mbar_init(bar_empty + 8 * lane, 1);
        } else if (lane < kStages + 2) {
            const int b = lane - kStages;
            ptx::mbar_init(bar_tfull + 8 * b, 1);
            ptx::mbar_init(bar_tempty + 8 * b, tc::kEpiWarps / tc::kEpiGroups);
        } else if (lane >= 16 && lane < 16 + kConstSlots) {
            ptx::mbar_init(bar_cfull + 8 * (lane - 16), 1);
            ptx::mbar_init(bar_cfree + 8 * (lane - 16), tc::kEpiWarps / tc::kEpiGroups);
        } else if (lane == 31) {
            ptx::mbar_init(bar_drain, 1);
            flags[0] = 0;
            for (int g = 0; g < kMaxTasks; ++g) done[g] = 0;
        }
        ptx::mbar_init_fence();
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32((const void *)tmem_slot), 2 * kAccCols);
    tc::build_aconst(smem + kOffAconst, (int)threadIdx.x, kThreads);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // this CTA's tasks: blockIdx.x, blockIdx.x + gridDim.x, ...; kMaxTasks of them per round
    const int my_tasks = (t.n_tasks - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 0) {
        // ---- loads ------------------------------------------------------------------------------
        if (lane == 0) {
            uint32_t slot = 0, ph = 0, issued = 0;
            uint32_t wu = 0;                                      // units whose constants were loaded
            int expect[kMaxTasks];                                // reports due before a task's next layer
#pragma unroll
            for (int g = 0; g < kMaxTasks; ++g) expect[g] = 0;
            bool ok = true;
            if (t.pdl) ptx::grid_dep_wait();
            for (int base = 0; base < my_tasks && ok; base += kMaxTasks) {
                const int ntask = my_tasks - base < kMaxTasks ? my_tasks - base : kMaxTasks;
                for (int l = 0; l < t.n_layers && ok; ++l) {
                    const Layer &L = t.layer[l];
                    const int kc = L.kc, n_sub = L.n_sub, cw = L.cw, x3d = L.x3d, box_r = L.box_r;
                    const uint32_t wbytes = (uint32_t)(L.nt_pad * cw), bb = (uint32_t)L.nt_pad * 32u;
                    const uint32_t a_tx = L.a_tx, const_bytes = L.const_bytes;
                    const uint32_t wbias_off = L.wbias_off, const_off = L.const_off, istride = L.image_stride;
                    const uint8_t *image = L.image;
                    const CUtensorMap *xmap = &L.xmap;
                    const int reports = reports_of(L);
                    for (int g = 0; g < ntask && ok; ++g) {
                        const int task = (int)blockIdx.x + (base + g) * (int)gridDim.x;
                        const int c_row = x3d ? task * box_r : task * t.tm;
                        if (l > 0) {
                            // the task's rows of the previous layer must be complete in global memory
                            unsigned long long t0 = 0;
                            for (uint32_t i = 1; done[g] < expect[g]; ++i) {
                                if ((i & 255u) == 0) {
                                    t0 = tc::wait_check(t0, flags, tc::kWaitLimitNs);
                                    if (t0 == tc::kWaitGiveUp) { ok = false; break; }
                                }
                            }
                            if (!ok) break;
                            __threadfence_block();
                            asm volatile("fence.proxy.async;" ::: "memory");
                        }
                        for (int s = 0; s < n_sub && ok; ++s) {
                            const uint8_t *img = image + (size_t)s * istride;
                            for (int c = 0; c < kc; ++c) {
                                if (!tc::wait_bar(bar_empty + 8 * slot, ph ^ 1u, flags)) { ok = false; break; }
                                const uint32_t dst = smem_base + slot * kStage;
                                const uint32_t bfull = bar_full + 8 * slot;
                                const bool last = c == kc - 1;
                                if (last) {
                                    const uint32_t cs = wu & (kConstSlots - 1);
                                    if (!tc::wait_bar(bar_cfree + 8 * cs, ((wu / kConstSlots) & 1u) ^ 1u, flags)) {
                                        ok = false; break;
                                    }
                                    const uint32_t bc = bar_cfull + 8 * cs;
                                    ptx::mbar_expect_tx(bc, const_bytes);
                                    ptx::bulk_load(smem_base + kOffConst + cs * kConstSlot, img + const_off, const_bytes, bc);
                                    ++wu;
                                }
                                ptx::mbar_expect_tx(bfull, a_tx + wbytes + (last ? bb : 0u));
                                if (x3d) ptx::tma_load_3d(dst, xmap, c * cw, 0, c_row, bfull);
                                else ptx::tma_load_2d(dst, xmap, c * cw, c_row, bfull);
                                ptx::bulk_load(dst + kAPart, img + (size_t)c * wbytes, wbytes, bfull);
                                if (last) ptx::bulk_load(dst + kAPart + kWPart, img + wbias_off, bb, bfull);
                                ++issued;
                                if (++slot == kStages) { slot = 0; ph ^= 1u; }
                            }
                        }
                        expect[g] += reports;
                    }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA goes away
                for (uint32_t j = issued > (uint32_t)kStages ? issued - kStages : 0; j < issued; ++j) {
                    const unsigned long long g0 = ptx::globaltimer();
                    while (!ptx::mbar_try_wait(bar_full + 8 * (j % kStages), (j / kStages) & 1u) &&
                           ptx::globaltimer() - g0 < tc::kWaitLimitNs) {}
                }
                for (uint32_t j = wu > (uint32_t)kConstSlots ? wu - kConstSlots : 0; j < wu; ++j) {
                    const unsigned long long g0 = ptx::globaltimer();
                    while (!ptx::mbar_try_wait(bar_cfull + 8 * (j % kConstSlots), (j / kConstSlots) & 1u) &&
                           ptx::globaltimer() - g0 < tc::kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -------------------------------------------------------------------------
        if (lane == 0) {
            bool ok = true;
            const uint64_t d32 = tc::smem_desc(0u, 32u);
            const uint64_t ac_desc = d32 | (uint64_t)((smem_base + kOffAconst) >> 4);
            uint32_t slot = 0, ph = 0, u = 0;
            uint32_t a_lo = smem_base >> 4, bfull = bar_full, bempty = bar_empty;
            for (int base = 0; base < my_tasks && ok; base += kMaxTasks) {
                const int ntask = my_tasks - base < kMaxTasks ? my_tasks - base : kMaxTasks;
                for (int l = 0; l < t.n_layers && ok; ++l) {
                    const Layer &L = t.layer[l];
                    const uint64_t dcw = tc::smem_desc(0u, (uint32_t)L.cw);
                    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(L.nt_pad >> 3) << 17) |
                                           ((128u >> 4) << 24);
                    const int ks_full = L.cw >> 5, ks_last = L.ksteps_last, kc = L.kc;
                    const int units = ntask * L.n_sub;
                    for (int i = 0; i < units && ok; ++i, ++u) {
                        const uint32_t b = u & 1u;
                        if (!tc::wait_bar(bar_tempty + 8 * b, ((u >> 1) & 1u) ^ 1u, flags)) { ok = false; break; }
                        const uint32_t d_tmem = tmem_base + b * kAccCols;
                        uint32_t acc = 0;
                        for (int c = 0; c < kc; ++c) {
                            if (!tc::wait_bar(bfull, ph, flags)) { ok = false; break; }
                            ptx::tc_fence_after_sync();
                            const uint32_t b_lo = a_lo + (kAPart >> 4);
                            const bool last = c == kc - 1;
                            const int nks = last ? ks_last : ks_full;
                            for (int ks = 0; ks < nks; ++ks) {
                                ptx::mma_i8(d_tmem, dcw | (uint64_t)(a_lo + 2 * ks), dcw | (uint64_t)(b_lo + 2 * ks), idesc, acc);
                                acc = 1;
                            }
                            if (last)       // bias digits (zeros when the subtile takes the exact epilogue)
                                ptx::mma_i8(d_tmem, ac_desc, d32 | (uint64_t)(a_lo + ((kAPart + kWPart) >> 4)), idesc, 1u);
                            ptx::mma_commit(bempty);
                            a_lo += kStage >> 4; bfull += 8; bempty += 8;
                            if (++slot == kStages) { slot = 0; ph ^= 1u; a_lo = smem_base >> 4; bfull = bar_full; bempty = bar_empty; }
                        }
                        if (!ok) break;
                        ptx::mma_commit(bar_tfull + 8 * b);
                    }
                }
            }
            ptx::mma_commit(bar_drain);
            const unsigned long long g0 = ptx::globaltimer();
            while (!ptx::mbar_try_wait(bar_drain, 0) && ptx::globaltimer() - g0 < tc::kWaitLimitNs) {}
        }
    } else {
        // ---- epilogue -----------------------------------------------------------------------------
        const int q = warp & 3;
        const int grp = (warp - 2) >> 2;
        uint8_t *slab = smem + kOffOut + (size_t)(warp - 2) * kSlab;
        const uint32_t slab_addr = ptx::smem_u32(slab);
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)grp * kAccCols;
        const int m_rows = (int)t.m_rows;
        bool ok = true;
        uint32_t u = 0;
        for (int base = 0; base < my_tasks && ok; base += kMaxTasks) {
            const int ntask = my_tasks - base < kMaxTasks ? my_tasks - base : kMaxTasks;
            for (int l = 0; l < t.n_layers && ok; ++l) {
                const Layer &L = t.layer[l];
                const int nt = L.nt, nf = L.n;
                uint8_t *my_row = slab + lane * nt;
                for (int g = 0; g < ntask && ok; ++g) {
                    const int task = (int)blockIdx.x + (base + g) * (int)gridDim.x;
                    const int row0 = task * t.tm + q * 32;
                    int rows_valid = t.tm - q * 32;
                    if (m_rows - row0 < rows_valid) rows_valid = m_rows - row0;
                    if (rows_valid > 32) rows_valid = 32;
                    bool mine = false;
                    for (int s = 0; s < L.n_sub; ++s, ++u) {
                        if ((int)(u & 1u) != grp) continue;
                        mine = true;
                        const uint32_t cs = u & (kConstSlots - 1);
                        if (!tc::wait_bar<true>(bar_tfull + 8 * grp, (u >> 1) & 1u, flags) ||
                            !tc::wait_bar<true>(bar_cfull + 8 * cs, (u / kConstSlots) & 1u, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        ptx::bulk_wait_read0();        // the previous store has read the slab
                        __syncwarp();
                        const uint8_t *cslot = smem + kOffConst + cs * kConstSlot;
                        const int *cms = reinterpret_cast<const int *>(cslot);
                        const int2 *cbs = reinterpret_cast<const int2 *>(cslot + L.nt_pad * 4);
                        const int *hdr = reinterpret_cast<const int *>(cslot + L.nt_pad * 12);
                        const int shmax = hdr[0];
                        const bool fast = hdr[1] != 0, bad = hdr[2] != 0;
                        const uint32_t bar_rel = bar_tempty + 8 * grp;
                        if (fast && L.act_min == 0) {
                            switch (nt) {
                            case 32: tc::epi_fast_fixed<32>(t_lane, cms, shmax, my_row, bar_rel); break;
                            case 64: tc::epi_fast_fixed<64>(t_lane, cms, shmax, my_row, bar_rel); break;
                            case 80: tc::epi_fast_fixed<80>(t_lane, cms, shmax, my_row, bar_rel); break;
                            case 96: tc::epi_fast_fixed<96>(t_lane, cms, shmax, my_row, bar_rel); break;
                            default: epi_fast_any(nt, t_lane, cms, shmax, my_row, bar_rel); break;
                            }
                        } else {
                            tc::epi_exact_subtile<32>(nt, L.act_min, L.act_max, t_lane, cms, cbs, my_row, bar_rel);
                        }
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(bar_cfree + 8 * cs);      // constants read
                        if (!bad && rows_valid > 0) {
                            const int col = s * nt;
                            if (rows_valid == 32) {
                                if (lane == 0) {
                                    if (L.store_2d) ptx::tma_store_2d(&L.ymap, col, row0, slab_addr);
                                    else ptx::bulk_store(L.y + (long long)row0 * nf, slab_addr, 32u * (uint32_t)nf);
                                    ptx::bulk_commit();
                                }
                            } else {
                                tc::store_partial_slab(L.y + (long long)row0 * nf, slab, rows_valid, nf, nt, col,
                                                       L.store_2d != 0, lane);
                            }
                        }
                    }
                    if (!ok) break;
                    if (mine) {
                        // this warp's part of (layer, task) is complete once its stores are
                        ptx::bulk_wait_all();
                        asm volatile("fence.proxy.async;" ::: "memory");
                        __threadfence_block();
                        __syncwarp();
                        if (lane == 0) atomicAdd((int *)&done[g], 1);
                    }
                }
            }
        }
        ptx::bulk_wait_all();
    }

    // ---- teardown -------------------------------------------------------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 2 * kAccCols);
    }
}

}}  // namespace prom::chain
