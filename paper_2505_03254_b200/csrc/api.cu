// Host side of the C ABI (include/prom.h): argument checks, variant choice,
// launch planning, tensor-map creation, and the layer-sequence driver.
#include <cuda.h>
#include <cuda_runtime.h>

#include <array>
#include <atomic>
#include <map>
#include <cstdio>
#include <cmath>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "prom.h"
#include "prom_debug.h"

#include "common.cuh"
#include "hostutil.cuh"
#include "simple.cuh"
#include "tc.cuh"
#include "chain.cuh"
#include "smallk.cuh"
#include "addsub.cuh"
#include "actquant.cuh"
#include "depthwise.cuh"
#include "dwtc.cuh"
#include "wide.cuh"
#include "stack.cuh"
#include "quantize.cuh"
#include "peak.cuh"

namespace prom {

static std::atomic<uint64_t> g_launches{0};

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
    int smem_total = 0;   // shared memory per SM
    bool ok = false;
};

static DeviceInfo device_info()
{
    static std::mutex mu;
    static std::unordered_map<int, DeviceInfo> cache;
    int dev = 0;
    DeviceInfo d;
    if (cudaGetDevice(&dev) != cudaSuccess) return d;
    std::lock_guard<std::mutex> lk(mu);
    auto it = cache.find(dev);
    if (it != cache.end()) return it->second;
    if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) ==
            cudaSuccess &&
        cudaDeviceGetAttribute(&d.smem_total, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) ==
            cudaSuccess)
        d.ok = true;
    cache[dev] = d;
    return d;
}

// ---- the layer as the host sees it -----------------------------------------------
struct Conv {
    const int8_t *x;
    long long m;        // output rows
    int cin, cout;
    RowMap map;         // how output rows find their input rows
    long long in_rows;  // rows of the input matrix
    const uint8_t *w;
    prom_requant rq;
    int8_t *y;
    cudaStream_t st;
    bool pdl;           // chain to the previous kernel with programmatic dependent launch
    bool pdl_next;      // the next kernel of the sequence chains to this one
    const int8_t *res = nullptr;   // added to the output with int8 saturation (may be y)
};

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static prom_status check_requant(const prom_requant *rq)
{
    if (!rq || !rq->bias || !rq->mult || !rq->shift) return PROM_ERR_NULL;
    if (rq->act_min < -128 || rq->act_max > 127 || rq->act_min > rq->act_max)
        return PROM_ERR_BAD_REQUANT;
    return PROM_OK;
}

static prom_status check_conv(const int8_t *x, long long m, int cin, const uint8_t *w, int cout,
                              const prom_requant *rq, const int8_t *y)
{
    if (!x || !w || !y) return PROM_ERR_NULL;
    prom_status s = check_requant(rq);
    if (s != PROM_OK) return s;
    if (m < 0 || cin < 1 || cin > 4096 || cout < 1 || cout > 4096) return PROM_ERR_SHAPE;
    if (m > (1ll << 40)) return PROM_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return PROM_ERR_ALIGN;
    return PROM_OK;
}

static int grid_for(long long work_items, int threads, int sms)
{
    long long blocks = (work_items + threads - 1) / threads;
    long long cap = (long long)sms * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// With PROM_VERBOSE set in the environment the CUDA error behind a PROM_ERR_CUDA goes to stderr.
static prom_status cuda_status(cudaError_t e)
{
    if (e == cudaSuccess) return PROM_OK;
    static const bool verbose = getenv("PROM_VERBOSE") != nullptr;
    if (verbose) fprintf(stderr, "prom: CUDA error %d: %s\n", (int)e, cudaGetErrorString(e));
    return PROM_ERR_CUDA;
}

// ---- naive -------------------------------------------------------------------------------
static prom_status launch_naive(const Conv &c, int32_t *acc_out)
{
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    const int threads = 256;
    int grid = grid_for(c.m * c.cout, threads, d.sms);
    naive_conv_kernel<<<grid, threads, 0, c.st>>>(c.x, c.m, c.cin, c.map, c.w, c.cout, c.rq.bias,
                                                  c.rq.mult, c.rq.shift, c.rq.act_min,
                                                  c.rq.act_max, acc_out ? nullptr : c.y, acc_out,
                                                  acc_out ? nullptr : c.res);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

// ---- tensor-core variant: planning --------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) ==
                cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

struct TcPlan {
    tc::Params p;
    CUtensorMap xmap, ymap;
    int grid = 0;
    int per_sm = 2;        // CTAs of the launch that share an SM (picks the kernel build)
    size_t smem = 0;
    double est_us = 0;
};

// Tuning override (0 = automatic), set by prom_debug_tc_plan.
struct TcTune { int fold, nt, groups, occ, stages; };
static TcTune g_tune = {0, 0, 0, 0, 0};
// Overrides for single shapes (m, cin, cout, input stride), set by prom_debug_tc_plan_shape;
// they take precedence over g_tune for that shape.
static std::mutex g_shape_tune_mu;
static std::map<std::array<long long, 4>, TcTune> g_shape_tune;

static TcTune tune_for(long long m, int cin, int cout, int stride)
{
    std::lock_guard<std::mutex> lk(g_shape_tune_mu);
    auto it = g_shape_tune.find({m, cin, cout, stride});
    return it == g_shape_tune.end() ? g_tune : it->second;
}

// Depth-first execution of parts of a sequence, set by prom_debug_seq_chain.  Off unless asked
// for: on the network the library is timed on it is slower than one launch per layer.
static std::atomic<int> g_seq_chain{0};
// Every second layer of a sequence walks its row tiles from the last to the first, so that it
// reads first what the layer before wrote last (still in L2 when the tensor is larger than L2:
// 0.3220 -> 0.3196 ms per step on the timed network).  On unless prom_debug_seq_order(0).
static std::atomic<int> g_seq_snake{1};

static int round_up(int v, int a) { return (v + a - 1) / a * a; }

// Everything of a plan that follows from (fold, nt, groups, occ); false when it does not fit.
static bool tc_fill_plan(long long m, int cin, int cout, const RowMap &map, const DeviceInfo &d,
                         int fold, int nt, int groups, int occ, int want_stages, TcPlan &pl,
                         int cw_max = 128)
{
    tc::Params &p = pl.p;
    memset(&p, 0, sizeof(p));
    const int kf = cin * fold, nf = cout * fold;
    if (kf > 4096 || nf % nt) return false;
    const int n_sub = nf / nt;
    if (n_sub % groups) return false;
    if (n_sub > 1 && ((nt & 15) || (nf & 15))) return false;     // tensor-map stores
    if (n_sub == 1 && (nt & 7)) return false;
    const int subs = n_sub / groups;
    const int nt_pad = round_up(nt, 16);
    if (nt_pad > 256) return false;
    const int cw = kf <= 32 ? 32 : (kf <= 64 || cw_max <= 64 ? 64 : 128);
    const int kc = (kf + cw - 1) / cw;

    // tile rows
    int tm = 128, x3d = 0, box_r = 0;
    if (map.stride != 1) {
        if (fold != 1 || map.wo > 128) return false;
        box_r = 128 / map.wo;
        long long lines = m / map.wo;          // batch * ho
        if (box_r > lines) box_r = (int)lines;
        if (box_r > 256) box_r = 256;
        tm = box_r * map.wo;
        x3d = 1;
    }
    const long long rows = m / fold;
    if ((nf & 15) && (tm & 1)) return false;     // slabs of the 1-D store start on 16-byte granules
    const long long n_mtiles = (rows + tm - 1) / tm;
    if (rows + 256 >= (1ll << 31)) return false;   // row coordinates are 32-bit in the kernel

    // tensor memory: the CTAs of an SM share its 512 columns
    // occ 1: one CTA with all of the SM; occ 2: two CTAs; occ 3: one CTA on half an SM, leaving
    // the other half to the next kernel's prologue; occ 4: three CTAs
    const int share = occ == 1 ? 1 : (occ == 4 ? 3 : 2);
    const int tmem_cols = share == 1 ? 512 : (share == 2 ? 256 : 128);
    if (2 * nt_pad > tmem_cols) return false;
    // accumulator ring: an even length, so that each of the two epilogue groups keeps to its own
    // accumulators
    if (tmem_cols / nt_pad < 2) return false;
    const int nbuf = tmem_cols / nt_pad >= 4 ? 4 : 2;

    const int ncols = subs * nt_pad;
    const size_t stage_bytes = (size_t)128 * cw;
    const size_t w_bytes = (size_t)subs * kc * nt_pad * cw;
    const size_t wbias_bytes = (size_t)subs * nt_pad * 32;
    const size_t out_bytes = (size_t)tc::kEpiWarps * 32 * nt;
    const size_t fixed = w_bytes + wbias_bytes + tc::kAConstBytes + round_up((int)out_bytes, 128) +
                         (size_t)ncols * 12 + 16 + 256 + tc::kLuts * 1024 + 256 + 1024 /* alignment slack */;
    const size_t budget = share == 1 ? (size_t)d.smem_optin
                                     : (size_t)((d.smem_total - share * 1024) / share);
    if (budget > (size_t)d.smem_optin || fixed + 2 * stage_bytes > budget) return false;
    int stages = (int)((budget - fixed) / stage_bytes);
    const int share_x = (kc == 1 && subs > 1) ? 1 : 0;
    int cap = share_x ? 4 : (kc >= 4 ? tc::kMaxStages : 6);
    if (want_stages > 0) cap = want_stages;
    if (stages > cap) stages = cap;
    if (stages > tc::kMaxStages) stages = tc::kMaxStages;
    if (stages < 2) return false;
    // the packed weights of the CTA are copied into the activation stages before these are used
    {
        const size_t rowb = (size_t)(cin + 3) / 4;
        const size_t packed = fold > 1 ? (size_t)cout * rowb : (size_t)subs * nt * rowb;
        if (packed > (size_t)stages * stage_bytes) return false;
    }

    p.m_rows = rows; p.k0 = cin; p.n0 = cout; p.fold = fold; p.kf = kf; p.nf = nf;
    p.tm = tm; p.n_mtiles = (int)n_mtiles; p.nt = nt; p.nt_pad = nt_pad;
    p.n_sub = n_sub; p.groups = groups; p.subs_per_cta = subs;
    p.cw = cw; p.kc = kc;
    p.ksteps_last = (kf - (kc - 1) * cw + 31) / 32;
    p.stages = stages; p.nbuf = nbuf; p.tmem_cols = tmem_cols;
    p.share_x = share_x;
    p.store_2d = n_sub > 1 ? 1 : 0;
    p.x3d = x3d; p.box_r = box_r;
    p.tx_bytes = x3d ? (uint32_t)(cw * map.wo * box_r) : (uint32_t)stage_bytes;

    // shared-memory layout; [off_w, off_hdr + 16) is the CTA's prepared image
    uint32_t off = (uint32_t)(stages * stage_bytes);
    p.off_w = off; off += (uint32_t)w_bytes;
    p.off_wbias = off; off += (uint32_t)wbias_bytes;
    p.off_mult = off; off += (uint32_t)ncols * 4;
    p.off_bs = off; off += (uint32_t)ncols * 8;
    p.off_hdr = off; off += 16;
    p.image_bytes = off - p.off_w;
    p.image_stride = (p.image_bytes + 255u) & ~255u;
    off = (off + 255u) & ~255u;
    p.off_aconst = off; off += tc::kAConstBytes;
    p.off_out = off; off += (uint32_t)round_up((int)out_bytes, 128);
    p.off_lut = off; off += tc::kLuts * 1024;
    p.off_bars = off; off += 256;
    pl.smem = (size_t)off + 1024;
    if (occ == 1 && pl.smem * 2 + 2048 <= (size_t)d.smem_total)
        pl.smem = (size_t)d.smem_total / 2;       // keep a second CTA (and its TMEM request) off the SM
    if (pl.smem > (size_t)d.smem_optin) return false;

    const int per_sm = occ == 2 ? 2 : (occ == 4 ? 3 : 1);
    pl.per_sm = per_sm;
    const long long slots = (long long)d.sms * per_sm;
    long long workers = slots / groups;
    if (workers < 1) workers = 1;
    if (workers > n_mtiles) workers = n_mtiles;
    pl.grid = (int)(workers * groups);

    // Rough time model (microseconds), used only to rank candidate plans; the constants come
    // from timing the kernel on a B200.  A CTA pays a start-up that grows with the operands it
    // brings in, then streams its units at the rate the epilogue warps sustain, and ends with
    // the latency of its last unit (one warp draining nt columns, then the store).
    const double rounds = (double)((n_mtiles + workers - 1) / workers);
    const double ctas_per_sm = (double)pl.grid / d.sms < 1.0 ? 1.0
                               : ((double)pl.grid / d.sms > per_sm ? per_sm : (double)pl.grid / d.sms);
    const double epi_rate = 36e3 / ctas_per_sm;              // outputs per microsecond per CTA
    // an SM takes 58 bytes per clock from L2 (the copy-rate probe): 110 KB per microsecond
    const double load_rate = 110e3 / ctas_per_sm;            // bytes per microsecond per CTA
    // subtile widths with a straight-line epilogue (tc.cuh: epi_fast_fixed); any other width that
    // splits a row runs the looped epilogue, measured ~1 us per layer slower at 128 columns
    const bool straight = nt == 96 || nt == 64 || nt == 48 || nt == 32 || nt == 80;
    const double t_epi = (double)tm * nt / epi_rate * (straight || n_sub == 1 ? 1.0 : 1.5);
    const double t_load = (double)kc * tm * (kf < cw ? kf : cw) / load_rate;
    // 0.8 us per unit for the hand-overs around it (barrier waits, fences, store issue): fitted to
    // plans timed inside the chained step (32 -> 192 and 64 -> 384 prefer 96-column subtiles in
    // fewer channel groups to 64-column ones)
    const double t_first = (t_epi > t_load ? t_epi : t_load) + 0.8;
    const double t_next = share_x ? t_epi + 0.8 : t_first;
    const double startup = 1.2 + (double)p.image_bytes / 80e3 * ctas_per_sm;
    const double fill = 1.0 + 0.1 * kc;                      // first load, first MMA
    const double last = 0.45 * ((nt + 31) / 32) + 0.8;       // draining the last accumulator, store
    const double t_cta = startup + fill + rounds * (t_first + (subs - 1) * t_next) + last +
                         (occ == 1 ? 2.5 : 0.0);   // a CTA that fills its SM keeps the next kernel out
    const double t_mem = ((double)m * cin * (groups == 1 ? 1.0 : 1.0 + 0.15 * (groups - 1)) +
                          (double)m * cout) / 5.5e6;
    pl.est_us = t_cta > t_mem ? t_cta : t_mem;
    return true;
}

// Picks fold, subtile width, channel groups and occupancy.  Returns false when
// the tensor-core variant cannot run this shape.
// use: kPlanSingle (one call: the kernel builds its operands itself), kPlanDynamic (the dynamic
// layer: no row folding, a folded row could straddle two samples) or
// kPlanPrepared (a layer of a sequence, whose operands tc_prep_kernel builds once)
enum { kPlanSingle = 0, kPlanDynamic = 1, kPlanPrepared = 2 };
static bool tc_search_plan(long long m, int cin, int cout, const RowMap &map, const DeviceInfo &d,
                           int use, TcPlan &best)
{
    const bool dyn = use == kPlanDynamic;
    if (m <= 0 || (cin & 7) || (cout & 7)) return false;
    const TcTune tn = tune_for(m, cin, cout, map.stride);
    int fold = 1;
    if (map.stride == 1) {
        // Rows that are not 16-byte multiples cannot be described to TMA: two rows are folded into
        // one.  On the output side that is only needed when the row does not fit one subtile
        // (a slab of 32 whole rows is then one contiguous, 16-byte aligned range of Y anyway).
        if ((cin & 15) || ((cout & 15) && cout > 256 && m % 2 == 0)) fold = 2;
        if (m % fold) return false;
        while (fold * 2 <= 8 && fold * 2 * cin <= 128 && fold * 2 * cout <= 128 &&
               m % (fold * 2) == 0)
            fold *= 2;
        // rows of fewer than 32 bytes make poor TMA boxes (measured on the 16 -> 96 layer: 3 us
        // of 58): fold once more whatever the width, where the larger block-diagonal weights
        // are expanded once per sequence and not by every CTA
        if (use == kPlanPrepared && cin * fold < 32 && fold * 2 <= 8 && m % (fold * 2) == 0) fold *= 2;
    }
    if (dyn) {
        if ((cin & 15) || ((cout & 15) && cout > 256)) return false;
        fold = 1;
    }
    if (tn.fold > 0) fold = tn.fold;
    if (fold < 1 || fold > 8 || m % fold) return false;
    const int nf = cout * fold;
    bool found = false;
    for (int nt = 8; nt <= 256 && nt <= nf; nt += 8) {
        if (nf % nt) continue;
        if (tn.nt > 0 && nt != tn.nt) continue;
        const int n_sub = nf / nt;
        for (int groups = 1; groups <= n_sub; ++groups) {
            if (n_sub % groups) continue;
            if (tn.groups > 0 && groups != tn.groups) continue;
            for (int occ = 4; occ >= 1; --occ) {
                if (tn.occ > 0 && occ != tn.occ) continue;
                if (dyn && occ > 2) continue;
                if (tn.occ == 0 && occ >= 3) continue;      // only on request for now
                TcPlan pl;
                if (!tc_fill_plan(m, cin, cout, map, d, fold, nt, groups, occ, tn.stages, pl))
                    continue;
                if (!found || pl.est_us < best.est_us) { best = pl; found = true; }
            }
        }
    }
    return found;
}


// The search above costs tens of microseconds; its result depends only on the shape, the
// device and the tuning override, so it is remembered.
static bool tc_shape_plan(long long m, int cin, int cout, const RowMap &map, const DeviceInfo &d,
                          TcPlan &best, int use = kPlanSingle)
{
    struct Entry { bool ok; TcPlan pl; };
    static std::mutex mu;
    static std::map<std::array<long long, 15>, Entry> cache;
    int dev = 0;
    cudaGetDevice(&dev);
    const TcTune tn = tune_for(m, cin, cout, map.stride);
    const std::array<long long, 15> key = {m, cin, cout, map.stride, map.ho, map.wo, map.hin, map.win,
                                           tn.fold, tn.nt, tn.groups, tn.occ, tn.stages, dev, use};
    std::lock_guard<std::mutex> lk(mu);
    auto it = cache.find(key);
    if (it == cache.end()) {
        Entry e;
        e.ok = tc_search_plan(m, cin, cout, map, d, use, e.pl);
        if (cache.size() > 4096) cache.clear();
        it = cache.emplace(key, e).first;
    }
    if (it->second.ok) best = it->second.pl;
    return it->second.ok;
}

static bool tc_make_maps(const Conv &c, TcPlan &pl)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const tc::Params &p = pl.p;
    const CUtensorMapSwizzle sw = p.cw == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : (p.cw == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    CUresult r;
    if (!p.x3d) {
        cuuint64_t dims[2] = {(cuuint64_t)p.kf, (cuuint64_t)p.m_rows};
        cuuint64_t strides[1] = {(cuuint64_t)p.kf};
        cuuint32_t box[2] = {(cuuint32_t)p.cw, 128};
        cuuint32_t es[2] = {1, 1};
        r = enc(&pl.xmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(c.x), dims, strides,
                box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        // [channel][wo, step stride*cin][batch*ho, step stride*win*cin]
        const RowMap &mp = c.map;
        cuuint64_t dims[3] = {(cuuint64_t)c.cin, (cuuint64_t)mp.wo, (cuuint64_t)(c.m / mp.wo)};
        cuuint64_t strides[2] = {(cuuint64_t)mp.stride * c.cin,
                                 (cuuint64_t)mp.stride * mp.win * c.cin};
        cuuint32_t box[3] = {(cuuint32_t)p.cw, (cuuint32_t)mp.wo, (cuuint32_t)p.box_r};
        cuuint32_t es[3] = {1, 1, 1};
        r = enc(&pl.xmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t *>(c.x), dims, strides,
                box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return false;
    if (p.store_2d) {
        cuuint64_t dims[2] = {(cuuint64_t)p.nf, (cuuint64_t)p.m_rows};
        cuuint64_t strides[1] = {(cuuint64_t)p.nf};
        cuuint32_t box[2] = {(cuuint32_t)p.nt, 32};
        cuuint32_t es[2] = {1, 1};
        r = enc(&pl.ymap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, c.y, dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return false;
    } else {
        pl.ymap = pl.xmap;      // unused by the kernel
    }
    return true;
}

static prom_status tc_set_attr(const DeviceInfo &d)
{
    // once per device: the limit is an attribute of the (function, device) pair
    cudaError_t e = raise_smem_limit(tc::tc_conv_kernel<2>, d.smem_optin);
    if (e == cudaSuccess) e = raise_smem_limit(tc::tc_conv_kernel<3>, d.smem_optin);
    if (e == cudaSuccess) e = raise_smem_limit(tc::tc_conv_kernel<2, 1>, d.smem_optin);
    if (e == cudaSuccess) e = raise_smem_limit(tc::tc_conv_kernel<2, 2>, d.smem_optin);
    if (e == cudaSuccess) e = raise_smem_limit(tc::tc_conv_kernel<2, 4>, d.smem_optin);
    if (e == cudaSuccess) e = raise_smem_limit(tc::tc_conv_kernel<2, 3>, d.smem_optin);
    if (e == cudaSuccess) e = raise_smem_limit(tc::tc_prep_kernel, d.smem_optin);
    return e == cudaSuccess ? PROM_OK : PROM_ERR_CUDA;
}

// Fills in the pointers of a planned layer (image: prepared operands, or null).
static void tc_bind(const Conv &c, TcPlan &pl, uint8_t *image)
{
    tc::Params &p = pl.p;
    p.w_packed = c.w; p.bias = c.rq.bias; p.mult = c.rq.mult; p.shift = c.rq.shift;
    p.act_min = c.rq.act_min; p.act_max = c.rq.act_max; p.y = c.y; p.pdl = c.pdl ? 1 : 0;
    p.pdl_next = c.pdl_next ? 1 : 0;
    p.image = image;
    p.res = c.res;
}

static prom_status tc_launch_planned(const Conv &c, TcPlan &pl, int mode = 0)
{
    if (!tc_make_maps(c, pl)) return PROM_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)pl.grid);
    cfg.blockDim = dim3(tc::kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = c.st;
    cudaLaunchAttribute attr[1];
    if (c.pdl) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    cudaError_t e;
    if (mode == 1) e = cudaLaunchKernelEx(&cfg, tc::tc_conv_kernel<2, 1>, pl.xmap, pl.ymap, pl.p);
    else if (mode == 2) e = cudaLaunchKernelEx(&cfg, tc::tc_conv_kernel<2, 2>, pl.xmap, pl.ymap, pl.p);
    else if (c.res) e = cudaLaunchKernelEx(&cfg, tc::tc_conv_kernel<2, 3>, pl.xmap, pl.ymap, pl.p);
    else if (pl.p.act_min == -128 && pl.p.act_max == 127)
        e = cudaLaunchKernelEx(&cfg, tc::tc_conv_kernel<2, 4>, pl.xmap, pl.ymap, pl.p);
    else if (pl.per_sm == 3) e = cudaLaunchKernelEx(&cfg, tc::tc_conv_kernel<3>, pl.xmap, pl.ymap, pl.p);
    else e = cudaLaunchKernelEx(&cfg, tc::tc_conv_kernel<2>, pl.xmap, pl.ymap, pl.p);
    ++g_launches;
    return cuda_status(e);
}

static size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

// ---- the row-resident variant for contraction-bound layers (wide.cuh) ----------------------------
// 0: the library's choice, 1: never, 2: whenever the shape allows it
static std::atomic<int> g_wide_mode{0};
static std::atomic<int> g_wide_nb{0};        // 0: the planner's choice; 1 or 2: forced (tests)

// Global scratch of the variant (the expanded weight matrix, bias digits, constants), one buffer
// per (device, stream), grown on demand and kept until prom_shutdown().
struct WideKey {
    int dev;
    cudaStream_t st;
    bool operator<(const WideKey &o) const { return dev != o.dev ? dev < o.dev : st < o.st; }
};
struct WideBuf { uint8_t *p = nullptr; size_t bytes = 0; };
static std::mutex g_wide_mu;
static std::map<WideKey, WideBuf> g_wide_cache;

static uint8_t *wide_scratch_for(cudaStream_t st, size_t bytes)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lk(g_wide_mu);
    WideBuf &b = g_wide_cache[WideKey{dev, st}];
    if (b.bytes < bytes) {
        if (b.p) {
            cudaStreamSynchronize(st);      // an earlier call may still be reading it
            cudaFree(b.p);
            b.p = nullptr; b.bytes = 0;
        }
        if (cudaMalloc(reinterpret_cast<void **>(&b.p), bytes) != cudaSuccess) return nullptr;
        b.bytes = bytes;
    }
    return b.p;
}

static void wide_release_cache()
{
    std::lock_guard<std::mutex> lk(g_wide_mu);
    for (auto &kv : g_wide_cache)
        if (kv.second.p) cudaFree(kv.second.p);
    g_wide_cache.clear();
}

struct WidePlan {
    wide::Params p;
    int grid;
    size_t smem;
    int k_pad;
};

// Shapes the variant takes: a plain matrix, whole 16-channel slices on both sides, K within the
// resident chunks.  `worth` says whether the library picks it by itself.
static bool wide_plan(const Conv &c, const DeviceInfo &d, WidePlan &pl, bool &worth)
{
    if (c.map.stride != 1 || c.res || c.pdl || c.pdl_next) return false;
    if ((c.cin & 15) || (c.cout & 15) || c.cin < wide::kChunk || c.cin > wide::kChunk * wide::kMaxKc) return false;
    if (c.cout < 64) return false;
    if (c.m >= (1ll << 31) - 256) return false;
    wide::Params &p = pl.p;
    memset(&p, 0, sizeof(p));
    p.m = c.m; p.cin = c.cin; p.cout = c.cout;
    p.kc = (c.cin + wide::kChunk - 1) / wide::kChunk;
    p.ksteps_last = (c.cin - (p.kc - 1) * wide::kChunk + 31) / 32;
    p.n_mtiles = (int)((c.m + 127) / 128);
    pl.k_pad = p.kc * wide::kChunk;
    // shared memory: resident chunks, weight ring, constants, staging slabs, the bias step's A block, barriers
    const uint32_t a_bytes = (uint32_t)p.kc * wide::kStageBytes;
    const uint32_t const_bytes = (wide::kAccs * wide::kConstBytes + 1023u) & ~1023u;
    const uint32_t fixed = const_bytes + wide::kEpiWarps * wide::kSlabBytes + tc::kAConstBytes + 1024;
    const long long room = (long long)d.smem_optin - 1024 - a_bytes - fixed;
    // 128-channel column tiles.  256-channel tiles (half as many tcgen05 instructions per output;
    // on request, where four stages of 32 KB fit beside the resident rows) measured slower: tensor
    // memory then holds one accumulator per issuing thread, so a thread's MMAs cannot overlap the
    // read-out of its previous tile (1.6 M x 384 -> 1280: 1416 against 1090 us, x 512 -> 256: 490
    // against 300 us).
    int nb = g_wide_nb.load();
    if (nb == 0) nb = 1;
    p.nb = nb;
    int stages = (int)(room / (nb * wide::kStageBytes));
    if (stages > wide::kMaxStages) stages = wide::kMaxStages;
    stages &= ~1;                       // one half of the ring per issuing thread
    if (stages < 4) return false;
    p.stages = stages;
    p.n_ctiles = (c.cout + nb * wide::kNt - 1) / (nb * wide::kNt);
    p.off_w = a_bytes;
    p.off_aconst = p.off_w + (uint32_t)stages * nb * wide::kStageBytes;
    p.off_const = p.off_aconst + tc::kAConstBytes;
    p.off_out = p.off_const + const_bytes;
    p.off_bars = p.off_out + wide::kEpiWarps * wide::kSlabBytes;
    pl.smem = p.off_bars + 1024 + 1024;
    // few row tiles: CTAs share a row tile's columns
    int groups = 1;
    for (int g = 1; g <= p.n_ctiles; ++g)
        if (p.n_ctiles % g == 0 && (long long)p.n_mtiles * g <= d.sms) groups = g;
    p.groups = groups;
    long long workers = d.sms / groups;
    if (workers > p.n_mtiles) workers = p.n_mtiles;
    if (workers < 1) workers = 1;
    pl.grid = (int)(workers * groups);
    p.act_min = c.rq.act_min; p.act_max = c.rq.act_max;
    // measured on B200: it beats the weight-resident kernel from Cin = 512 on when there are
    // several row tiles per SM (1.4 to 1.7 times at Cin = 960); below that both are bound by the
    // cost of issuing tcgen05 instructions and the weight-resident kernel issues fewer per output
    // (a last column tile that is mostly padding costs it that margin unless Cin is large)
    const bool full_cols = 10 * c.cout > 9 * p.n_ctiles * nb * wide::kNt;
    worth = c.cin >= 512 && c.cout >= 256 && p.n_mtiles >= 4 * d.sms && (full_cols || c.cin >= 768);
    return true;
}

static prom_status launch_wide(const Conv &c, const DeviceInfo &d, WidePlan &pl)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return PROM_ERR_UNSUPPORTED;
    wide::Params &p = pl.p;
    const int blocks = p.n_ctiles * p.nb;           // of 128 channels
    const size_t w8_bytes = (size_t)blocks * wide::kNt * pl.k_pad;
    const size_t wb_bytes = (size_t)blocks * wide::kWbiasBytes;
    const size_t cs_bytes = round256((size_t)blocks * wide::kConstBytes);
    uint8_t *scratch = wide_scratch_for(c.st, w8_bytes + wb_bytes + cs_bytes);
    if (!scratch) return PROM_ERR_CUDA;
    wide::PrepParams pp;
    memset(&pp, 0, sizeof(pp));
    pp.cin = c.cin; pp.cout = c.cout; pp.k_pad = pl.k_pad; pp.w_packed = c.w;
    pp.bias = c.rq.bias; pp.mult = c.rq.mult; pp.shift = c.rq.shift;
    pp.act_min = c.rq.act_min; pp.act_max = c.rq.act_max;
    pp.w8 = reinterpret_cast<int8_t *>(scratch); pp.wbias = scratch + w8_bytes; pp.consts = scratch + w8_bytes + wb_bytes;
    p.wbias = pp.wbias; p.consts = pp.consts;
    CUtensorMap xmap, wmap, ymap;
    cuuint32_t es[2] = {1, 1};
    {
        cuuint64_t dims[2] = {(cuuint64_t)c.cin, (cuuint64_t)c.m};
        cuuint64_t strides[1] = {(cuuint64_t)c.cin};
        cuuint32_t box[2] = {(cuuint32_t)wide::kChunk, 128};
        if (enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(c.x), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PROM_ERR_UNSUPPORTED;
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)pl.k_pad, (cuuint64_t)blocks * wide::kNt};
        cuuint64_t strides[1] = {(cuuint64_t)pl.k_pad};
        cuuint32_t box[2] = {(cuuint32_t)wide::kChunk, (cuuint32_t)(p.nb * wide::kNt)};
        if (enc(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, pp.w8, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
            CUDA_SUCCESS)
            return PROM_ERR_UNSUPPORTED;
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)c.cout, (cuuint64_t)c.m};
        cuuint64_t strides[1] = {(cuuint64_t)c.cout};
        cuuint32_t box[2] = {wide::kEpiCols, 32};
        if (enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, c.y, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
            CUDA_SUCCESS)
            return PROM_ERR_UNSUPPORTED;
    }
    if (raise_smem_limit(wide::wide_conv_kernel, d.smem_optin) != cudaSuccess) return PROM_ERR_CUDA;
    wide::wide_prep_kernel<<<blocks, 256, 0, c.st>>>(pp);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
    wide::wide_conv_kernel<<<pl.grid, wide::kThreads, pl.smem, c.st>>>(xmap, wmap, ymap, p);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

static prom_status launch_tc(const Conv &c)
{
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    const int wide_mode = g_wide_mode.load();
    if (wide_mode != 1) {
        WidePlan wp;
        bool worth = false;
        if (wide_plan(c, d, wp, worth) && (worth || wide_mode == 2)) {
            const prom_status e = launch_wide(c, d, wp);
            if (e != PROM_ERR_UNSUPPORTED) return e;
        } else if (wide_mode == 2) {
            return PROM_ERR_UNSUPPORTED;
        }
    }
    TcPlan pl;
    if (!tc_shape_plan(c.m, c.cin, c.cout, c.map, d, pl)) return PROM_ERR_UNSUPPORTED;
    if (tc_set_attr(d) != PROM_OK) return PROM_ERR_CUDA;
    tc_bind(c, pl, nullptr);
    return tc_launch_planned(c, pl);
}

static bool tc_supported(const Conv &c)
{
    DeviceInfo d = device_info();
    if (!d.ok) return false;
    TcPlan pl;
    return tc_shape_plan(c.m, c.cin, c.cout, c.map, d, pl);
}

// ---- variant choice --------------------------------------------------------------------------
static prom_status run_conv(const Conv &c, prom_variant v)
{
    if (c.m == 0) return PROM_OK;
    // the residual is fused into the tensor-core and the naive kernels only
    if (c.res && (v == PROM_VARIANT_SMALLK || v == PROM_VARIANT_ADDSUB)) return PROM_ERR_UNSUPPORTED;
    switch (v) {
    case PROM_VARIANT_NAIVE: return launch_naive(c, nullptr);
    case PROM_VARIANT_TC: return launch_tc(c);
    case PROM_VARIANT_SMALLK: return smallk::launch(c.x, c.m, c.cin, c.map, c.w, c.cout, c.rq, c.y,
                                                    c.st, g_launches);
    case PROM_VARIANT_ADDSUB: return addsub::launch(c.x, c.m, c.cin, c.map, c.w, c.cout, c.rq, c.y,
                                                    c.st, g_launches);
    case PROM_VARIANT_AUTO:
        if (tc_supported(c)) return launch_tc(c);
        if (!c.res && smallk::supported(c.cin, c.cout))
            return smallk::launch(c.x, c.m, c.cin, c.map, c.w, c.cout, c.rq, c.y, c.st, g_launches);
        return launch_naive(c, nullptr);
    default: return PROM_ERR_UNSUPPORTED;
    }
}


// Shapes of a sequence; false when it does not chain.
struct SeqShape {
    std::vector<long long> m;      // output rows per layer
    std::vector<RowMap> map;
    std::vector<int> h, w;
};

static bool seq_shapes(const prom_layer *layers, int n, int batch, int h0, int w0, SeqShape &s)
{
    if (!layers || n < 1 || batch < 1 || h0 < 1 || w0 < 1) return false;
    int h = h0, w = w0;
    for (int i = 0; i < n; ++i) {
        const prom_layer &l = layers[i];
        if (l.cin < 1 || l.cin > 4096 || l.cout < 1 || l.cout > 4096) return false;
        if (i > 0 && l.cin != layers[i - 1].cout) return false;
        if (l.in_stride != 1 && l.in_stride != 2) return false;
        if (h % l.in_stride || w % l.in_stride) return false;
        // the block's input (the previous layer's input) has this layer's output shape
        if (l.add_block_input &&
            (i < 1 || l.in_stride != 1 || layers[i - 1].in_stride != 1 || l.cout != layers[i - 1].cin))
            return false;
        RowMap mp;
        mp.stride = l.in_stride; mp.hin = h; mp.win = w;
        h /= l.in_stride; w /= l.in_stride;
        mp.ho = h; mp.wo = w;
        if (l.dw_w) {                 // the depthwise convolution applies the stride itself
            if (l.cin & 3) return false;
            mp.stride = 1; mp.hin = h; mp.win = w;
        }
        s.map.push_back(mp);
        s.m.push_back((long long)batch * h * w);
        s.h.push_back(h); s.w.push_back(w);
    }
    return true;
}

// Workspace regions: a and b take the outputs of even and odd layers in turn; b also ends with
// room for the largest depthwise output (the input of the pointwise convolution behind it).
static void seq_regions(const prom_layer *layers, int n, const SeqShape &s, size_t &a, size_t &b,
                        size_t *dw_off = nullptr)
{
    a = b = 0;
    size_t c = 0;
    for (int i = 0; i < n; ++i) {
        if (i + 1 < n) {
            size_t bytes = round256((size_t)s.m[i] * layers[i].cout);
            if (i & 1) { if (bytes > b) b = bytes; }
            else { if (bytes > a) a = bytes; }
        }
        if (layers[i].dw_w) {
            size_t bytes = round256((size_t)s.m[i] * layers[i].cin);
            if (bytes > c) c = bytes;
        }
    }
    if (dw_off) *dw_off = a + b;
    b += c;
}

// ---- depth-first chains (chain.cuh) ---------------------------------------------------------
// A chain is a run of consecutive layers of a sequence that one launch of tc_chain_kernel takes
// tile by tile through all of them: same number of rows in every layer (only the first may
// subsample its input), channel counts that are multiples of 16, the clamp [0, 127], no
// depthwise convolution and no skip connection, and few enough tiles that a CTA interleaves
// at most chain::kMaxTasks of them.  Each layer of a chain writes to a buffer of its own in the
// workspace (a ping-pong pair would be overwritten by tiles that are layers ahead).
struct ChainPlan {
    int first = 0, last = 0;             // layers [first, last]
    int tm = 128, n_tasks = 0, grid = 0, box_r = 0;
    std::vector<TcPlan> prep;            // per layer: the plan whose image layout the kernel reads
    // kind 1: the run stays in shared memory (stack.cuh); `prep` is then empty
    int kind = 0;
    stack::Table st;                     // everything but pointers and tensor maps
    size_t smem = 0;
};

// Global scratch of one layer of a resident run: the int8 matrix, bias digits and constants that
// wide_prep_kernel writes, column tile after column tile.
struct StackScratch { size_t w8, wbias, consts, total; int n_ct, k_pad; };
static StackScratch stack_scratch(int cin, int cout)
{
    StackScratch z;
    z.n_ct = (cout + 127) / 128;
    z.k_pad = (cin + 127) / 128 * 128;
    z.w8 = (size_t)z.n_ct * 128 * z.k_pad;
    z.wbias = (size_t)z.n_ct * stack::kWbiasBytes;
    z.consts = round256((size_t)z.n_ct * stack::kConstBytes);
    z.total = z.w8 + z.wbias + z.consts;
    return z;
}

// The layers of a resident run alternate: P layers (the first and every second one after it; at
// most 384 output channels) and E layers (at most 384 input channels).
static bool stack_layer_ok(const prom_layer &l, bool is_p)
{
    if (l.dw_w || l.add_block_input || l.cin % 16 || l.cout % 16 || l.cin > 4096 || l.cout > 4096) return false;
    return is_p ? l.cout <= 128 * stack::kNarrowMax : l.cin <= 128 * stack::kNarrowMax;
}

// Roles, accumulator slots, shared-memory layout and rings of a resident run over the layers
// [c.first, c.last]; false when it does not fit.
static bool stack_fill(const prom_layer *layers, const DeviceInfo &d, ChainPlan &c)
{
    stack::Table &t = c.st;
    memset(&t, 0, sizeof(t));
    const int n = c.last - c.first + 1;
    if (n < 2 || n > stack::kMaxLayers) return false;
    int narrow = 1, ring_chunks = 0;
    for (int l = 0; l < n; ++l) {
        const prom_layer &pl = layers[c.first + l];
        stack::Layer &L = t.layer[l];
        L.cout = pl.cout;
        L.kc = (pl.cin + 127) / 128;
        L.ksteps = (pl.cin + 31) / 32;
        L.n_ct = (pl.cout + 127) / 128;
        L.act_min = pl.rq.act_min; L.act_max = pl.rq.act_max;
        L.streamed = (l & 1) ? 0 : 1;
        L.out_mode = l == n - 1 ? 2 : (L.streamed ? 0 : 1);
        if (L.streamed) {
            if (L.n_ct > stack::kNarrowMax) return false;
            L.ring_off = ring_chunks;
            ring_chunks += L.kc;
            if (L.out_mode == 0 && L.n_ct > narrow) narrow = L.n_ct;
        } else if (L.kc > stack::kNarrowMax) {
            return false;
        }
    }
    // accumulators: a P layer keeps all of its units' live, two of the four slots unless it has three
    // units; the E layer in front of it takes what is left
    for (int l = 0; l < n; ++l) {
        stack::Layer &L = t.layer[l];
        if (L.streamed) {
            L.nslots = L.n_ct == 3 ? 3 : 2;
            L.slot0 = stack::kAccs - L.nslots;
        } else {
            const bool tight = l + 1 < n && t.layer[l + 1].n_ct == 3;
            L.slot0 = 0;
            L.nslots = tight ? 1 : 2;
        }
    }
    t.n_layers = n;
    t.tm = c.tm; t.box_r = c.box_r; t.x3d = c.box_r > 0 ? 1 : 0;
    t.n_mtiles = c.n_tasks;
    t.chunks_per_tile = ring_chunks;
    t.ring = 3;
    const uint32_t const_bytes = stack::kAccs * stack::kSlotBytes;
    const uint32_t fixed = const_bytes + stack::kEpiWarps * stack::kSlabBytes + tc::kAConstBytes + 1024;
    const uint32_t act_bytes = (uint32_t)(narrow + t.ring) * stack::kChunkBytes;
    const long long room = (long long)d.smem_optin - 1024 - act_bytes - fixed;
    int stages = (int)(room / stack::kChunkBytes);
    if (stages > stack::kMaxStages) stages = stack::kMaxStages;
    stages &= ~1;                   // one half of the ring per issuing thread
    if (stages < 4) return false;
    t.stages = stages;
    t.off_nar = 0;
    t.off_ring = (uint32_t)narrow * stack::kChunkBytes;
    t.off_w = t.off_ring + (uint32_t)t.ring * stack::kChunkBytes;
    t.off_aconst = t.off_w + (uint32_t)stages * stack::kChunkBytes;
    t.off_const = t.off_aconst + tc::kAConstBytes;
    t.off_out = t.off_const + const_bytes;
    t.off_bars = t.off_out + stack::kEpiWarps * stack::kSlabBytes;
    c.smem = t.off_bars + 1024 + 1024;
    // one CTA per SM whatever the size: each allocates all of tensor memory
    if (c.smem < (size_t)d.smem_optin / 2 + 2048) c.smem = (size_t)d.smem_optin / 2 + 2048;
    return true;
}

static int chain_nt(int cout)
{
    if (cout % 16) return 0;
    if (cout <= chain::kNtMax) return cout;
    for (int nt = chain::kNtMax; nt >= 16; nt -= 16)
        if (cout % nt == 0) return nt;
    return 0;
}

static bool chain_layer_ok(const prom_layer &l)
{
    return !l.dw_w && !l.add_block_input && l.cin % 16 == 0 && l.cin >= 32 && l.cout % 16 == 0 &&
           l.rq.act_min == 0 && l.rq.act_max == 127 && chain_nt(l.cout) > 0;
}

static bool chain_prep_plan(long long m, int cin, int cout, const DeviceInfo &d, TcPlan &pl)
{
    const int nt = chain_nt(cout);
    const RowMap plain{1, 1, 1, 1, 1};
    return nt > 0 && tc_fill_plan(m, cin, cout, plain, d, 1, nt, cout / nt, 1, 0, pl, chain::kCwMax) &&
           pl.p.cw <= chain::kCwMax && pl.p.nt_pad <= chain::kNtMax &&
           (uint32_t)pl.p.nt_pad * 12u + 16u <= chain::kConstSlot;
}

static void find_chains(const prom_layer *layers, int n, const SeqShape &s, const DeviceInfo &d,
                        std::vector<ChainPlan> &out)
{
    out.clear();
    const int mode = g_seq_chain.load();
    if (!mode) return;
    int i = 0;
    while (mode == 2 && i < n) {
        // runs that stay in shared memory: P, E, P, E, ...
        if (!stack_layer_ok(layers[i], true) || s.m[i] <= 0 || s.m[i] + 256 >= (1ll << 31)) { ++i; continue; }
        ChainPlan c;
        c.kind = 1;
        c.first = i;
        const RowMap &mp = s.map[i];
        if (mp.stride != 1) {
            if (mp.wo > 128) { ++i; continue; }
            c.box_r = 128 / mp.wo;
            const long long lines = s.m[i] / mp.wo;
            if (c.box_r > lines) c.box_r = (int)lines;
            c.tm = c.box_r * mp.wo;
        }
        c.n_tasks = (int)((s.m[i] + c.tm - 1) / c.tm);
        int j = i + 1;
        while (j < n && j - i < stack::kMaxLayers && s.m[j] == s.m[i] && s.map[j].stride == 1 &&
               stack_layer_ok(layers[j], ((j - i) & 1) == 0))
            ++j;
        // the longest run that fits
        bool found = false;
        for (; j - i >= 2 && !found; --j) {
            // a skip connection into layer j reads the output of layer j - 2, which must exist
            if (j < n && layers[j].add_block_input) continue;
            c.last = j - 1;
            found = stack_fill(layers, d, c);
        }
        if (!found) { ++i; continue; }
        c.grid = c.n_tasks < d.sms ? c.n_tasks : d.sms;
        out.push_back(c);
        i = c.last + 1;
    }
    if (mode == 2) return;
    while (i < n) {
        if (!chain_layer_ok(layers[i]) || s.m[i] <= 0) { ++i; continue; }
        ChainPlan c;
        c.first = i;
        const RowMap &mp = s.map[i];
        if (mp.stride != 1) {
            if (mp.wo > 128) { ++i; continue; }
            c.box_r = 128 / mp.wo;
            const long long lines = s.m[i] / mp.wo;
            if (c.box_r > lines) c.box_r = (int)lines;
            c.tm = c.box_r * mp.wo;
        }
        const long long tasks = (s.m[i] + c.tm - 1) / c.tm;
        if (tasks > (long long)chain::kMaxTasks * 2 * d.sms || s.m[i] + 256 >= (1ll << 31)) { ++i; continue; }
        c.n_tasks = (int)tasks;
        int j = i;
        for (; j < n && j - i < chain::kMaxLayers; ++j) {
            if (!chain_layer_ok(layers[j]) || s.m[j] != s.m[i] || (j > i && s.map[j].stride != 1)) break;
            TcPlan pl;
            if (!chain_prep_plan(s.m[j], layers[j].cin, layers[j].cout, d, pl)) break;
            c.prep.push_back(pl);
        }
        if (j - i < 2) { ++i; continue; }
        c.last = j - 1;
        c.grid = c.n_tasks < 2 * d.sms ? c.n_tasks : 2 * d.sms;
        out.push_back(c);
        i = j;
    }
}

static bool make_x_map(CUtensorMap *map, const int8_t *x, int cin, long long rows, int cw, const RowMap *strided,
                       int box_r)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const CUtensorMapSwizzle sw = cw == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : (cw == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    cuuint32_t es[3] = {1, 1, 1};
    if (!strided) {
        cuuint64_t dims[2] = {(cuuint64_t)cin, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)cin};
        cuuint32_t box[2] = {(cuuint32_t)cw, 128};
        return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(x), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    // [channel][wo, step stride*cin][batch*ho, step stride*win*cin]
    const RowMap &mp = *strided;
    cuuint64_t dims[3] = {(cuuint64_t)cin, (cuuint64_t)mp.wo, (cuuint64_t)(rows / mp.wo)};
    cuuint64_t strides[2] = {(cuuint64_t)mp.stride * cin, (cuuint64_t)mp.stride * mp.win * cin};
    cuuint32_t box[3] = {(cuuint32_t)cw, (cuuint32_t)mp.wo, (cuuint32_t)box_r};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t *>(x), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool make_y_map(CUtensorMap *map, int8_t *y, int nf, long long rows, int nt)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)nf, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)nf};
    cuuint32_t box[2] = {(cuuint32_t)nt, 32};
    cuuint32_t es[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, y, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Where everything of a sequence sits in the caller's workspace.
struct SeqLayout {
    size_t ra = 0, rb = 0, dw_off = 0;     // the two ping-pong regions (b ends with the depthwise buffer)
    std::vector<size_t> img_off;           // per layer: prepared image of a one-launch layer, or -1
    size_t img_total = 0;
    std::vector<ChainPlan> chains;
    std::vector<int> chain_of;             // per layer: its chain, or -1
    std::vector<size_t> cimg_off, cbuf_off;   // per chain layer: images, output buffer
    size_t cimg_total = 0, cbuf_total = 0;
    size_t base() const { return ra + rb; }
    size_t with_images() const { return round256(base()) + img_total; }
    size_t with_chains() const { return round256(with_images()) + cimg_total + cbuf_total; }
};

static void seq_layout(const prom_layer *layers, int n, const SeqShape &s, const DeviceInfo &d, bool want_tc,
                       SeqLayout &L, bool allow_chains = true)
{
    seq_regions(layers, n, s, L.ra, L.rb, &L.dw_off);
    L.chain_of.assign(n, -1);
    L.img_off.assign(n, (size_t)-1);
    L.cimg_off.assign(n, 0);
    L.cbuf_off.assign(n, 0);
    if (!want_tc || !d.ok) return;
    if (allow_chains) find_chains(layers, n, s, d, L.chains);
    for (size_t c = 0; c < L.chains.size(); ++c)
        for (int i = L.chains[c].first; i <= L.chains[c].last; ++i) L.chain_of[i] = (int)c;
    for (int i = 0; i < n; ++i) {
        if (L.chain_of[i] >= 0) {
            const ChainPlan &c = L.chains[L.chain_of[i]];
            L.cimg_off[i] = L.cimg_total;
            if (c.kind == 1) {
                L.cimg_total += round256(stack_scratch(layers[i].cin, layers[i].cout).total);
                continue;
            }
            const tc::Params &p = c.prep[i - c.first].p;
            L.cimg_total += round256((size_t)p.groups * p.image_stride);
            continue;
        }
        TcPlan pl;
        if (tc_shape_plan(s.m[i], layers[i].cin, layers[i].cout, s.map[i], d, pl, kPlanPrepared)) {
            L.img_off[i] = L.img_total;
            L.img_total += round256((size_t)pl.p.groups * pl.p.image_stride);
        }
    }
    for (int i = 0; i < n; ++i)
        if (L.chain_of[i] >= 0 && i + 1 < n) {
            // (the inner layers of a resident run have no output tensor)
            const ChainPlan &c = L.chains[L.chain_of[i]];
            if (c.kind == 1 && i != c.last) continue;
            L.cbuf_off[i] = L.cimg_total + L.cbuf_total;
            L.cbuf_total += round256((size_t)s.m[i] * layers[i].cout);
        }
}


// ---- depthwise 3x3 on the tensor cores (dwtc.cuh) ---------------------------------------------
// 0: the library's choice, 1: CUDA cores only, 2: tensor cores or PROM_ERR_UNSUPPORTED
static std::atomic<int> g_dw_variant{0};

// Launch configuration of a kernel that may be chained to its predecessor in the stream with
// programmatic dependent launch (attr must outlive the launch call).
static void fill_launch_cfg(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int grid, int threads, size_t smem,
                            cudaStream_t st, bool pdl)
{
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    if (pdl) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
}

static prom_status launch_dw_tc(const int8_t *x, int batch, int h, int w, int c, const int8_t *wt,
                                const prom_requant *rq, int8_t *y, const DeviceInfo &d, cudaStream_t st,
                                bool pdl, bool pdl_next)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return PROM_ERR_UNSUPPORTED;
    const int slices = c / 16;
    int ns = dwtc::kMaxSlices;
    while (slices % ns) --ns;
    dwtc::Params p;
    memset(&p, 0, sizeof(p));
    p.batch = batch; p.h = h; p.w = w; p.c = c; p.ns = ns; p.groups = slices / ns;
    p.tiles_y = (h + dwtc::kTileH - 1) / dwtc::kTileH;
    p.tiles_x = (w + dwtc::kTileW - 1) / dwtc::kTileW;
    p.tiles = (long long)batch * p.tiles_y * p.tiles_x;
    p.wt = wt; p.bias = rq->bias; p.mult = rq->mult; p.shift = rq->shift; p.lo = rq->act_min; p.hi = rq->act_max;
    p.y = y;
    if (p.groups > 2 * d.sms || p.tiles >= (1ll << 31)) return PROM_ERR_UNSUPPORTED;
    // {channel in slice, x, y, slice, image}: the slice is a dimension of its own (16 bytes apart),
    // so that the patches of a group's slices land one after the other in shared memory
    CUtensorMap map;
    cuuint64_t dims[5] = {16, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)slices, (cuuint64_t)batch};
    cuuint64_t strides[4] = {(cuuint64_t)c, (cuuint64_t)w * c, 16, (cuuint64_t)h * w * c};
    cuuint32_t box[5] = {16, (cuuint32_t)dwtc::kPatchW, (cuuint32_t)dwtc::kPatchH, (cuuint32_t)ns, 1};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 5, const_cast<int8_t *>(x), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return PROM_ERR_UNSUPPORTED;
    if (raise_smem_limit(dwtc::dw3x3_tc_kernel, (int)dwtc::kSmemBytes) != cudaSuccess) return PROM_ERR_CUDA;
    long long workers = (2ll * d.sms) / p.groups;
    if (workers < 1) workers = 1;
    if (workers > p.tiles) workers = p.tiles;
    const int grid = (int)(workers * p.groups);
    p.pdl = pdl ? 1 : 0;
    p.pdl_next = pdl_next ? 1 : 0;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_launch_cfg(cfg, attr, grid, dwtc::kThreads, dwtc::kSmemBytes, st, pdl);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, dwtc::dw3x3_tc_kernel, map, p);
    ++g_launches;
    return cuda_status(e);
}

// pdl / pdl_next: the call is a link of a layer sequence (programmatic dependent launch behind the
// kernel that writes x; the next kernel of the stream is launched that way)
static prom_status dw_conv3x3(const int8_t *x_dev, int batch, int h, int w, int c, int stride,
                              const int8_t *w_dev, const prom_requant *rq, int8_t *y_dev, void *cuda_stream,
                              bool pdl, bool pdl_next)
{
    if (batch < 0 || h < 1 || w < 1 || c < 1 || c > 4096 || (stride != 1 && stride != 2)) return PROM_ERR_SHAPE;
    if (c & 3) return PROM_ERR_UNSUPPORTED;
    if (!rq) return PROM_ERR_NULL;
    prom_status e = check_requant(rq);
    if (e != PROM_OK) return e;
    if (batch == 0) return PROM_OK;
    if (!x_dev || !w_dev || !y_dev) return PROM_ERR_NULL;
    if (!aligned16(x_dev) || !aligned16(y_dev)) return PROM_ERR_ALIGN;
    if (reinterpret_cast<const void *>(x_dev) == reinterpret_cast<const void *>(y_dev)) return PROM_ERR_ALIGN;
    const int ho = (h - 1) / stride + 1, wo = (w - 1) / stride + 1;
    if ((long long)batch * h * w * c >= (1ll << 40)) return PROM_ERR_SHAPE;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    // stride 1 and whole slices of 16 channels: TMA patches and tensor-core taps
    const int dw_variant = g_dw_variant.load();
    // (left to itself the library keeps images of fewer than 100 pixels on the CUDA cores: a 7 x 7
    // image fills 49 of a tile's 128 rows, and [128,7,7,960] takes 18.6 us there against 14.8 us)
    if (dw_variant != 1 && stride == 1 && (c & 15) == 0 &&
        !(dw_variant == 0 && ((long long)batch * h * w < 128 || h * w < 100))) {
        const prom_status e = launch_dw_tc(x_dev, batch, h, w, c, w_dev, rq, y_dev, d,
                                           static_cast<cudaStream_t>(cuda_stream), pdl, pdl_next);
        if (e != PROM_ERR_UNSUPPORTED) return e;
    }
    if (dw_variant == 2) return PROM_ERR_UNSUPPORTED;
    const int rows = dw::rows_per_unit(stride);
    const long long units = (long long)batch * ((ho + rows - 1) / rows) * ((wo + dw::kStrip - 1) / dw::kStrip);
    if (units >= (1ll << 31)) return PROM_ERR_SHAPE;
    const long long total = units * (c >> 2);
    // a multiple of c / 4 threads, so that a thread keeps its channels: blocks in multiples of
    // (c / 4) / gcd(c / 4, threads per block)
    int step = c >> 2;
    for (int a = step, b = dw::kThreads; b;) { const int r = a % b; a = b; b = r; if (!b) step = (c >> 2) / a; }
    long long blocks = (total + dw::kThreads - 1) / dw::kThreads;
    const long long cap = (long long)d.sms * 16;
    if (blocks > cap) blocks = cap;
    blocks = (blocks + step - 1) / step * step;
    const int grid = (int)blocks;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_launch_cfg(cfg, attr, grid, dw::kThreads, 0, st, pdl);
    const int f_pdl = pdl ? 1 : 0, f_next = pdl_next ? 1 : 0;
    cudaError_t le;
    if (stride == 1)
        le = cudaLaunchKernelEx(&cfg, dw::dw3x3_kernel<1>, x_dev, batch, h, w, c, ho, wo, w_dev, rq->bias, rq->mult,
                                rq->shift, rq->act_min, rq->act_max, y_dev, f_pdl, f_next);
    else
        le = cudaLaunchKernelEx(&cfg, dw::dw3x3_kernel<2>, x_dev, batch, h, w, c, ho, wo, w_dev, rq->bias, rq->mult,
                                rq->shift, rq->act_min, rq->act_max, y_dev, f_pdl, f_next);
    ++g_launches;
    return cuda_status(le);
}

// One launch of tc_chain_kernel for layers [c.first, c.last]; conv[] holds every layer's pointers.
static prom_status launch_chain(const prom_layer *layers, const SeqShape &s, const ChainPlan &c,
                                const std::vector<Conv> &conv, uint8_t *const *images, bool pdl, bool pdl_next,
                                cudaStream_t st)
{
    chain::Table t;
    memset(&t, 0, sizeof(t));
    t.m_rows = s.m[c.first];
    t.n_layers = c.last - c.first + 1;
    t.n_tasks = c.n_tasks;
    t.tm = c.tm;
    t.pdl = pdl ? 1 : 0;
    t.pdl_next = pdl_next ? 1 : 0;
    for (int i = c.first; i <= c.last; ++i) {
        chain::Layer &L = t.layer[i - c.first];
        const tc::Params &p = c.prep[i - c.first].p;
        const bool strided = i == c.first && s.map[i].stride != 1;
        if (!make_x_map(&L.xmap, conv[i].x, layers[i].cin, s.m[i], p.cw, strided ? &s.map[i] : nullptr, c.box_r))
            return PROM_ERR_CUDA;
        L.store_2d = p.n_sub > 1 ? 1 : 0;
        if (L.store_2d) {
            if (!make_y_map(&L.ymap, conv[i].y, layers[i].cout, s.m[i], p.nt)) return PROM_ERR_CUDA;
        } else {
            L.ymap = L.xmap;       // unused
        }
        L.image = images[i];
        L.y = conv[i].y;
        L.image_stride = p.image_stride;
        L.wbias_off = p.off_wbias - p.off_w;
        L.const_off = p.off_mult - p.off_w;
        L.const_bytes = (uint32_t)p.nt_pad * 12u + 16u;
        L.a_tx = strided ? (uint32_t)(p.cw * s.map[i].wo * c.box_r) : 128u * (uint32_t)p.cw;
        L.n = layers[i].cout;
        L.cw = p.cw; L.kc = p.kc; L.ksteps_last = p.ksteps_last;
        L.nt = p.nt; L.nt_pad = p.nt_pad; L.n_sub = p.n_sub;
        L.x3d = strided ? 1 : 0;
        L.box_r = c.box_r;
        L.act_min = layers[i].rq.act_min; L.act_max = layers[i].rq.act_max;
    }
    if (raise_smem_limit(chain::tc_chain_kernel, (int)chain::kSmemBytes) != cudaSuccess) return PROM_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)c.grid);
    cfg.blockDim = dim3(chain::kThreads);
    cfg.dynamicSmemBytes = chain::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (pdl) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    const cudaError_t e = cudaLaunchKernelEx(&cfg, chain::tc_chain_kernel, t);
    ++g_launches;
    return cuda_status(e);
}

// One launch of stack_kernel for the layers [c.first, c.last] of a resident run.
static prom_status launch_stack(const prom_layer *layers, const SeqShape &s, const ChainPlan &c,
                                const std::vector<Conv> &conv, uint8_t *const *scratch, const DeviceInfo &d,
                                bool pdl, bool pdl_next, cudaStream_t st)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return PROM_ERR_CUDA;
    stack::Table t = c.st;
    t.m = s.m[c.first];
    t.pdl = pdl ? 1 : 0;
    t.pdl_next = pdl_next ? 1 : 0;
    t.y = conv[c.last].y;
    const bool strided = s.map[c.first].stride != 1;
    if (!make_x_map(&t.xmap, conv[c.first].x, layers[c.first].cin, s.m[c.first], 128,
                    strided ? &s.map[c.first] : nullptr, c.box_r))
        return PROM_ERR_CUDA;
    if (!make_y_map(&t.ymap, conv[c.last].y, layers[c.last].cout, s.m[c.last], 32)) return PROM_ERR_CUDA;
    cuuint32_t es[2] = {1, 1};
    for (int i = c.first; i <= c.last; ++i) {
        stack::Layer &L = t.layer[i - c.first];
        const StackScratch z = stack_scratch(layers[i].cin, layers[i].cout);
        cuuint64_t dims[2] = {(cuuint64_t)z.k_pad, (cuuint64_t)z.n_ct * 128};
        cuuint64_t strides[1] = {(cuuint64_t)z.k_pad};
        cuuint32_t box[2] = {128, 128};
        if (enc(&L.wmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, scratch[i], dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PROM_ERR_CUDA;
        L.wbias = scratch[i] + z.w8;
        L.consts = scratch[i] + z.w8 + z.wbias;
    }
    if (raise_smem_limit(stack::stack_kernel, d.smem_optin) != cudaSuccess) return PROM_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_launch_cfg(cfg, attr, c.grid, stack::kThreads, c.smem, st, pdl);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, stack::stack_kernel, t);
    ++g_launches;
    return cuda_status(e);
}

static prom_status run_seq(const prom_layer *layers, int n, const int8_t *x0, int batch, int h0,
                           int w0, void *ws, size_t ws_bytes, int8_t *y_out, prom_variant variant,
                           cudaStream_t st)
{
    SeqShape s;
    if (!seq_shapes(layers, n, batch, h0, w0, s)) return PROM_ERR_SHAPE;
    // validate everything before the first launch
    for (int i = 0; i < n; ++i) {
        if (!layers[i].w_packed) return PROM_ERR_NULL;
        if (layers[i].dw_w) {
            prom_status de = check_requant(&layers[i].dw_rq);
            if (de != PROM_OK) return de;
        }
        prom_status e = check_requant(&layers[i].rq);
        if (e != PROM_OK) return e;
        if (!aligned16(layers[i].w_packed)) return PROM_ERR_ALIGN;
        if (layers[i].add_block_input &&
            (variant == PROM_VARIANT_SMALLK || variant == PROM_VARIANT_ADDSUB))
            return PROM_ERR_UNSUPPORTED;
    }
    DeviceInfo d = device_info();
    const bool want_tc = variant == PROM_VARIANT_TC || variant == PROM_VARIANT_AUTO;
    SeqLayout lay;
    seq_layout(layers, n, s, d, want_tc, lay);
    const size_t ra = lay.ra, rb = lay.rb;
    if (ra + rb > 0) {
        if (!ws) return PROM_ERR_NULL;
        if (!aligned16(ws)) return PROM_ERR_ALIGN;
        if (ws_bytes < ra + rb) return PROM_ERR_WORKSPACE;
    }
    if (!d.ok) return PROM_ERR_CUDA;
    int8_t *reg[2] = {static_cast<int8_t *>(ws), static_cast<int8_t *>(ws) + ra};
    int8_t *dw_buf = static_cast<int8_t *>(ws) + lay.dw_off;      // depthwise outputs

    // The images and the chains are optimisations: a workspace without room for them still works.
    uint8_t *img_base = nullptr, *chain_base = nullptr;
    if (ws && lay.img_total + lay.cimg_total > 0 && ws_bytes >= lay.with_images())
        img_base = static_cast<uint8_t *>(ws) + round256(lay.base());
    if (ws && !lay.chains.empty() && ws_bytes >= lay.with_chains())
        chain_base = static_cast<uint8_t *>(ws) + round256(lay.with_images());
    if (!chain_base && !lay.chains.empty()) {
        // no room: plan again without chains (their layers then want one-launch images)
        lay = SeqLayout();
        seq_layout(layers, n, s, d, want_tc, lay, false);
        img_base = nullptr;
        if (ws && lay.img_total > 0 && ws_bytes >= lay.with_images())
            img_base = static_cast<uint8_t *>(ws) + round256(lay.base());
    }

    // plan: which layers run on the tensor cores, and where their prepared operands go
    std::vector<Conv> conv(n);
    std::vector<TcPlan> plan(n);
    std::vector<char> is_tc(n, 0);
    std::vector<uint8_t *> chain_img(n, nullptr);
    const int8_t *cur = x0;
    long long in_rows = (long long)batch * h0 * w0;
    for (int i = 0; i < n; ++i) {
        Conv &c = conv[i];
        const bool chained = lay.chain_of[i] >= 0;
        // behind a depthwise convolution the pointwise layer reads that convolution's output
        c.x = layers[i].dw_w ? dw_buf : cur; c.m = s.m[i]; c.cin = layers[i].cin; c.cout = layers[i].cout;
        c.map = s.map[i]; c.in_rows = layers[i].dw_w ? s.m[i] : in_rows;
        c.w = layers[i].w_packed; c.rq = layers[i].rq;
        c.y = (i == n - 1) ? y_out
              : (chained ? reinterpret_cast<int8_t *>(chain_base + lay.cbuf_off[i]) : reg[i & 1]);
        c.st = st;
        c.pdl = i > 0;
        c.pdl_next = i + 1 < n;
        // The block's input is the output of layer i-2, which sits where this layer's output
        // goes (unless a chain wrote it to a buffer of its own: then the sum reads from there).
        if (layers[i].add_block_input) c.res = i == 1 ? x0 : conv[i - 2].y;
        if (chained) {
            chain_img[i] = chain_base + lay.cimg_off[i];
        } else if (want_tc && c.m > 0 && tc_shape_plan(c.m, c.cin, c.cout, c.map, d, plan[i], kPlanPrepared)) {
            is_tc[i] = 1;
            tc_bind(c, plan[i], img_base && lay.img_off[i] != (size_t)-1 ? img_base + lay.img_off[i] : nullptr);
        } else if (variant == PROM_VARIANT_TC && c.m > 0) {
            return PROM_ERR_UNSUPPORTED;
        }
        cur = c.y;
        in_rows = c.m;
    }
    if (want_tc && tc_set_attr(d) != PROM_OK) return PROM_ERR_CUDA;
    // tile order: opposite to that of the kernel that wrote the layer's input (a depthwise
    // convolution and the kernels off the tensor cores walk forwards)
    if (g_seq_snake.load()) {
        bool writer_rev = true;             // the first layer walks forwards
        for (int i = 0; i < n; ++i) {
            if (layers[i].dw_w) writer_rev = false;
            const bool rev = is_tc[i] && lay.chain_of[i] < 0 && !writer_rev;
            if (is_tc[i]) plan[i].p.reverse = rev ? 1 : 0;
            writer_rev = rev;
        }
    }

    // one launch prepares the operands of every tensor-core layer (of a chain: one image per subtile)
    if (img_base || chain_base) {
        int i = 0;
        while (i < n) {
            tc::PrepTable t;
            memset(&t, 0, sizeof(t));
            size_t smem = 0;
            int ctas = 0;
            for (; i < n && t.n < tc::kMaxPrepLayers; ++i) {
                const TcPlan *pl = nullptr;
                if (lay.chain_of[i] >= 0) {
                    const ChainPlan &c = lay.chains[lay.chain_of[i]];
                    if (c.kind == 1) continue;          // prepared by the batch below
                    TcPlan tmp = c.prep[i - c.first];
                    tc_bind(conv[i], tmp, chain_img[i]);
                    t.layer[t.n] = tmp.p;
                    pl = &c.prep[i - c.first];
                } else if (is_tc[i] && plan[i].p.image) {
                    t.layer[t.n] = plan[i].p;
                    pl = &plan[i];
                } else {
                    continue;
                }
                t.first[t.n] = ctas;
                ctas += pl->p.groups;
                if (pl->smem > smem) smem = pl->smem;
                ++t.n;
            }
            if (t.n == 0) break;
            t.first[t.n] = ctas;
            tc::tc_prep_kernel<<<ctas, tc::kThreads, smem, st>>>(t);
            ++g_launches;
            if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
        }
    }

    // ... and one launch the operands of the runs that stay in shared memory
    if (chain_base) {
        int i = 0;
        while (i < n) {
            wide::PrepBatch b;
            memset(&b, 0, sizeof(b));
            int ctas = 0;
            for (; i < n && b.n < wide::kMaxPrepLayers; ++i) {
                if (lay.chain_of[i] < 0 || lay.chains[lay.chain_of[i]].kind != 1) continue;
                const StackScratch z = stack_scratch(layers[i].cin, layers[i].cout);
                wide::PrepParams &pp = b.layer[b.n];
                pp.cin = layers[i].cin; pp.cout = layers[i].cout; pp.k_pad = z.k_pad; pp.w_packed = layers[i].w_packed;
                pp.bias = layers[i].rq.bias; pp.mult = layers[i].rq.mult; pp.shift = layers[i].rq.shift;
                pp.act_min = layers[i].rq.act_min; pp.act_max = layers[i].rq.act_max;
                pp.w8 = reinterpret_cast<int8_t *>(chain_img[i]);
                pp.wbias = chain_img[i] + z.w8;
                pp.consts = chain_img[i] + z.w8 + z.wbias;
                b.first[b.n] = ctas;
                ctas += z.n_ct;
                ++b.n;
            }
            if (b.n == 0) break;
            b.first[b.n] = ctas;
            wide::wide_prep_batch_kernel<<<ctas, 256, 0, st>>>(b);
            ++g_launches;
            if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
        }
    }

    for (int i = 0; i < n; ++i) {
        if (lay.chain_of[i] >= 0) {
            const ChainPlan &c = lay.chains[lay.chain_of[i]];
            prom_status e = c.kind == 1
                ? launch_stack(layers, s, c, conv, chain_img.data(), d, c.first > 0, c.last + 1 < n, st)
                : launch_chain(layers, s, c, conv, chain_img.data(), c.first > 0, c.last + 1 < n, st);
            if (e != PROM_OK) return e;
            i = c.last;
            continue;
        }
        if (layers[i].dw_w && s.m[i] > 0) {
            const int stride = layers[i].in_stride;
            const int8_t *src = i == 0 ? x0 : conv[i - 1].y;
            // chained like the pointwise kernels: behind layer i-1's kernel (which releases its
            // dependents at entry) and in front of layer i's, which waits for it before its loads
            prom_status de = dw_conv3x3(src, batch, s.h[i] * stride, s.w[i] * stride, layers[i].cin, stride,
                                        layers[i].dw_w, &layers[i].dw_rq, dw_buf, st, i > 0, true);
            if (de != PROM_OK) return de;
        }
        prom_status e = is_tc[i] ? tc_launch_planned(conv[i], plan[i]) : run_conv(conv[i], variant);
        if (e != PROM_OK) return e;
    }
    return PROM_OK;
}

// ---- the add/sub variant on built-in scratch (no allocation anywhere) --------------------
// The index lists of the add/sub variant normally live in a buffer the library
// grows with cudaMalloc.  This copy of the scratch is part of the loaded module
// instead: PROM_STATIC_SCRATCH_BYTES of device memory on every GPU that loads
// the library, held until the process exits.  In host code the array's name is
// only a handle for the runtime, not a device address; the address a kernel can
// use comes from cudaGetSymbolAddress, asked once per device.
static __device__ __align__(256) uint8_t g_static_scratch[PROM_STATIC_SCRATCH_BYTES];

static uint8_t *static_scratch_address()
{
    static std::mutex mu;
    static std::unordered_map<int, uint8_t *> by_device;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lk(mu);
    auto it = by_device.find(dev);
    if (it != by_device.end()) return it->second;
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return nullptr;
    by_device[dev] = static_cast<uint8_t *>(p);
    return static_cast<uint8_t *>(p);
}

// scale_y[b] = 127 / max(gamma_y[b], eps): between the two passes of the dynamic layer
__global__ void dyn_scale_kernel(const float *__restrict__ gamma_y, int batch, float eps,
                                        float *__restrict__ scale_y)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) {
        const float g = gamma_y[b];
        scale_y[b] = __fdiv_rn(127.0f, g < eps ? eps : g);
    }
}

}  // namespace prom

using namespace prom;

extern "C" {

size_t prom_packed_bytes(int cout, int cin)
{
    if (cout < 0 || cin < 0) return 0;
    return (size_t)cout * (size_t)((cin + 3) / 4);
}

prom_status prom_pack_ternary(const int8_t *w_dev, int cout, int cin, uint8_t *packed_dev,
                              size_t packed_bytes, void *cuda_stream)
{
    if (!w_dev || !packed_dev) return PROM_ERR_NULL;
    if (cout < 1 || cin < 1 || cout > 4096 || cin > 4096) return PROM_ERR_SHAPE;
    if (packed_bytes < prom_packed_bytes(cout, cin)) return PROM_ERR_WORKSPACE;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned int *bad = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void **>(&bad), g_pack_bad) != cudaSuccess)
        return PROM_ERR_CUDA;
    if (cudaMemsetAsync(bad, 0, sizeof(unsigned int), st) != cudaSuccess) return PROM_ERR_CUDA;
    long long total = (long long)cout * ((cin + 3) / 4);
    pack_ternary_kernel<<<grid_for(total, 256, d.sms), 256, 0, st>>>(w_dev, cout, cin, packed_dev,
                                                                     bad);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
    unsigned int host_bad = 0;
    if (cudaMemcpyAsync(&host_bad, bad, sizeof(host_bad), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return PROM_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PROM_ERR_CUDA;
    return host_bad ? PROM_ERR_BAD_WEIGHT : PROM_OK;
}

prom_status prom_quantize_ternary(const float *w_dev, int cout, int cin, uint8_t *packed_dev,
                                  size_t packed_bytes, float *alpha_dev, void *cuda_stream)
{
    if (!w_dev || !packed_dev) return PROM_ERR_NULL;
    if (cout < 1 || cin < 1 || cout > 4096 || cin > 4096) return PROM_ERR_SHAPE;
    if (packed_bytes < prom_packed_bytes(cout, cin)) return PROM_ERR_WORKSPACE;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    const int want = (cout + quant::kWarps - 1) / quant::kWarps;        // a warp per row
    const int grid = want < d.sms * 16 ? want : d.sms * 16;
    quant::quantize_ternary_kernel<<<grid, quant::kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        w_dev, cout, cin, 1e-5, packed_dev, alpha_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_quantize_ternary_batch(const prom_quantize_job *jobs, int n, void *cuda_stream)
{
    if (!jobs) return PROM_ERR_NULL;
    if (n < 0) return PROM_ERR_SHAPE;
    for (int i = 0; i < n; ++i) {
        const prom_quantize_job &j = jobs[i];
        if (!j.w_dev || !j.packed_dev) return PROM_ERR_NULL;
        if (j.cout < 1 || j.cin < 1 || j.cout > 4096 || j.cin > 4096) return PROM_ERR_SHAPE;
        if (j.packed_bytes < prom_packed_bytes(j.cout, j.cin)) return PROM_ERR_WORKSPACE;
    }
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    for (int base = 0; base < n; base += quant::kMaxJobs) {
        quant::Jobs t;
        memset(&t, 0, sizeof(t));
        t.n = n - base < quant::kMaxJobs ? n - base : quant::kMaxJobs;
        int rows = 0;
        for (int i = 0; i < t.n; ++i) {
            const prom_quantize_job &j = jobs[base + i];
            t.first_row[i] = rows;
            rows += j.cout;
            t.cin[i] = j.cin; t.w[i] = j.w_dev; t.packed[i] = j.packed_dev; t.alpha[i] = j.alpha_dev;
        }
        t.first_row[t.n] = rows;
        const int want = (rows + quant::kWarps - 1) / quant::kWarps;      // a warp per row
        const int grid = want < d.sms * 16 ? want : d.sms * 16;
        quant::quantize_ternary_batch_kernel<<<grid, quant::kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
            t, 1e-5);
        ++g_launches;
        if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
    }
    return PROM_OK;
}

prom_status prom_dw_conv3x3_i8(const int8_t *x_dev, int batch, int h, int w, int c, int stride,
                               const int8_t *w_dev, const prom_requant *rq, int8_t *y_dev,
                               void *cuda_stream)
{
    return dw_conv3x3(x_dev, batch, h, w, c, stride, w_dev, rq, y_dev, cuda_stream, false, false);
}

prom_status prom_pw_conv_i8_dyn(const int8_t *x_dev, int batch, int64_t rows_per_sample, int cin,
                                const uint8_t *w_packed_dev, int cout, const float *alpha_dev,
                                const float *gamma_x_dev, int8_t *q_dev, float *gamma_y_dev,
                                float *scale_y_dev, void *cuda_stream)
{
    if (batch < 0 || rows_per_sample < 1 || cin < 1 || cout < 1 || cin > 4096 || cout > 4096)
        return PROM_ERR_SHAPE;
    const long long m = (long long)batch * rows_per_sample;
    if (rows_per_sample >= (1ll << 31) || m >= (1ll << 31)) return PROM_ERR_SHAPE;
    if (batch == 0) return PROM_OK;
    if (!x_dev || !w_packed_dev || !alpha_dev || !gamma_x_dev || !q_dev || !gamma_y_dev || !scale_y_dev)
        return PROM_ERR_NULL;
    if (!aligned16(x_dev) || !aligned16(w_packed_dev) || !aligned16(q_dev)) return PROM_ERR_ALIGN;
    if (reinterpret_cast<const void *>(x_dev) == reinterpret_cast<const void *>(q_dev)) return PROM_ERR_ALIGN;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    TcPlan pl;
    const RowMap plain{1, 1, 1, 1, 1};
    if (!tc_shape_plan(m, cin, cout, plain, d, pl, kPlanDynamic)) return PROM_ERR_UNSUPPORTED;
    if (tc_set_attr(d) != PROM_OK) return PROM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Conv c;
    memset(&c, 0, sizeof(c));
    c.x = x_dev; c.m = m; c.cin = cin; c.cout = cout; c.map = plain; c.in_rows = m;
    c.w = w_packed_dev; c.y = q_dev; c.st = st; c.pdl = false; c.pdl_next = false;
    c.rq.bias = nullptr; c.rq.shift = nullptr;
    c.rq.mult = reinterpret_cast<const int32_t *>(alpha_dev);     // bit patterns of alpha
    c.rq.act_min = -128; c.rq.act_max = 127;                      // keeps the weights at +-1
    tc_bind(c, pl, nullptr);
    pl.p.dyn = 1;
    pl.p.rows_per_sample = (int)rows_per_sample;
    pl.p.batch = batch;
    pl.p.gamma_x = gamma_x_dev;
    pl.p.gamma_y = gamma_y_dev;
    pl.p.scale_y = scale_y_dev;
    if (cudaMemsetAsync(gamma_y_dev, 0, sizeof(float) * (size_t)batch, st) != cudaSuccess)
        return PROM_ERR_CUDA;
    prom_status e = tc_launch_planned(c, pl, 1);
    if (e != PROM_OK) return e;
    dyn_scale_kernel<<<(batch + 127) / 128, 128, 0, st>>>(gamma_y_dev, batch, 1e-5f, scale_y_dev);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return PROM_ERR_CUDA;
    return tc_launch_planned(c, pl, 2);
}

prom_status prom_quantize_act_absmax(const float *x_dev, int batch, int64_t per_sample,
                                     int8_t *q_dev, float *gamma_dev, float *scale_dev,
                                     void *cuda_stream)
{
    if (batch < 0 || per_sample < 1 || per_sample > (1ll << 40)) return PROM_ERR_SHAPE;
    if (batch == 0) return PROM_OK;
    if (!x_dev || !q_dev || !gamma_dev || !scale_dev) return PROM_ERR_NULL;
    if (!aligned16(x_dev) || !aligned16(q_dev)) return PROM_ERR_ALIGN;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const float eps = 1e-5f;

    // fused route: the smallest cluster whose slices fit shared memory
    const size_t room = (size_t)d.smem_optin - 4096;
    int cluster = 0, slice = 0;
    if (per_sample % 16 == 0) {
        for (int c = 1; c <= actq::kMaxCluster; c *= 2) {
            const long long s = ((per_sample + c - 1) / c + 15) / 16 * 16;
            if ((size_t)s * 4 <= room) { cluster = c; slice = (int)s; break; }
        }
    }
    if (cluster) {
        const cudaError_t attr_err = raise_smem_limit(actq::act_quant_cluster_kernel, d.smem_optin - 4096);
        if (attr_err != cudaSuccess) return cuda_status(attr_err);
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)cluster);       // one cluster, for the occupancy query
        cfg.blockDim = dim3(actq::kThreads);
        cfg.dynamicSmemBytes = (size_t)slice * 4;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cluster;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        // as many clusters as are resident at once, each walking over its share of the samples
        // (asked once per shape: the query costs tens of microseconds on the host)
        static std::mutex mu;
        static std::map<std::array<long long, 3>, int> known;
        int dev = 0;
        cudaGetDevice(&dev);
        int resident = 0;
        {
            std::lock_guard<std::mutex> lk(mu);
            const std::array<long long, 3> key = {dev, cluster, slice};
            auto it = known.find(key);
            if (it == known.end()) {
                if (cudaOccupancyMaxActiveClusters(&resident, actq::act_quant_cluster_kernel, &cfg) !=
                    cudaSuccess)
                    resident = 0;
                cudaGetLastError();
                known[key] = resident;
            } else {
                resident = it->second;
            }
        }
        if (resident > 0) {
            const int nclusters = resident < batch ? resident : batch;
            cfg.gridDim = dim3((unsigned)(nclusters * cluster));
            cudaError_t e = cudaLaunchKernelEx(&cfg, actq::act_quant_cluster_kernel, x_dev, batch,
                                               (long long)per_sample, slice, eps, q_dev, gamma_dev,
                                               scale_dev);
            ++g_launches;
            return cuda_status(e);
        }
    }

    // the same clusters reading their slices twice (the second time from L2): samples whose
    // slices do not fit shared memory (as fast as the staged route at the bench's size, but the
    // second read is from HBM again whenever L2 has lost the slice)
    if (per_sample % 16 == 0) {
        const int c = actq::kMaxCluster;
        const long long s = ((per_sample + c - 1) / c + 15) / 16 * 16;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)c);
        cfg.blockDim = dim3(actq::kThreads);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)c;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        static std::mutex mu;
        static std::map<int, int> known;
        int dev = 0;
        cudaGetDevice(&dev);
        int resident = 0;
        {
            std::lock_guard<std::mutex> lk(mu);
            auto it = known.find(dev);
            if (it == known.end()) {
                if (cudaOccupancyMaxActiveClusters(&resident, actq::act_quant_reread_kernel, &cfg) !=
                    cudaSuccess)
                    resident = 0;
                cudaGetLastError();
                known[dev] = resident;
            } else {
                resident = it->second;
            }
        }
        if (resident > 0 && s * 4 <= (8ll << 20)) {
            const int nclusters = resident < batch ? resident : batch;
            cfg.gridDim = dim3((unsigned)(nclusters * c));
            cudaError_t e = cudaLaunchKernelEx(&cfg, actq::act_quant_reread_kernel, x_dev, batch,
                                               (long long)per_sample, s, eps, q_dev, gamma_dev, scale_dev);
            ++g_launches;
            return cuda_status(e);
        }
    }

    // two passes
    if (cudaMemsetAsync(gamma_dev, 0, sizeof(float) * (size_t)batch, st) != cudaSuccess) return PROM_ERR_CUDA;
    long long bx = (per_sample + actq::kThreads * 8 - 1) / (actq::kThreads * 8);
    const long long cap = (long long)d.sms * 8 / batch + 1;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    const dim3 grid((unsigned)bx, (unsigned)batch);
    if (batch > 65535) return PROM_ERR_SHAPE;
    actq::act_absmax_kernel<<<grid, actq::kThreads, 0, st>>>(x_dev, (long long)per_sample, gamma_dev);
    ++g_launches;
    actq::act_quant_kernel<<<grid, actq::kThreads, 0, st>>>(x_dev, (long long)per_sample, eps, gamma_dev, q_dev,
                                                            scale_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_requant_from_scale(double scale, int32_t *mult, int8_t *shift)
{
    if (!mult || !shift) return PROM_ERR_NULL;
    if (!(scale > 0.0) || scale >= 1.0) return PROM_ERR_BAD_REQUANT;
    // scale = f * 2^(e+1) with f in [0.5, 1): mult = round(f * 2^31), shift = -(e+1)
    int e = ilogb(scale);                        // floor(log2(scale)), <= -1
    int sh = -(e + 1);
    double m = nearbyint(scalbn(scale, 31 + sh));
    if (m >= 2147483648.0) { m = 1073741824.0; --sh; }
    if (sh < 0 || sh > 31) return PROM_ERR_BAD_REQUANT;
    *mult = (int32_t)m;
    *shift = (int8_t)sh;
    return PROM_OK;
}

prom_status prom_pw_conv_i8(const int8_t *x_dev, int64_t m, int cin, const uint8_t *w_packed_dev,
                            int cout, const prom_requant *rq, int8_t *y_dev, prom_variant variant,
                            void *cuda_stream)
{
    // an empty matrix has no rows to read or write: its pointers may be anything
    if (m == 0 && cin >= 1 && cin <= 4096 && cout >= 1 && cout <= 4096 && w_packed_dev && rq)
        return check_requant(rq);
    prom_status s = check_conv(x_dev, m, cin, w_packed_dev, cout, rq, y_dev);
    if (s != PROM_OK) return s;
    Conv c;
    c.x = x_dev; c.m = m; c.cin = cin; c.cout = cout;
    c.map = RowMap{1, 1, 1, 1, 1};
    c.in_rows = m;
    c.w = w_packed_dev; c.rq = *rq; c.y = y_dev;
    c.st = static_cast<cudaStream_t>(cuda_stream);
    c.pdl = false;
    c.pdl_next = false;
    return run_conv(c, variant);
}

// ---- one layer with operands prepared ahead of the call --------------------------------------
static bool prepared_plan(long long m, int cin, int cout, const DeviceInfo &d, TcPlan &pl)
{
    return m > 0 && tc_shape_plan(m, cin, cout, RowMap{1, 1, 1, 1, 1}, d, pl, kPlanPrepared);
}

size_t prom_pw_prepared_bytes(int64_t m, int cin, int cout)
{
    if (m < 1 || cin < 1 || cin > 4096 || cout < 1 || cout > 4096) return 0;
    DeviceInfo d = device_info();
    if (!d.ok) { d.sms = 148; d.smem_optin = 232448; d.smem_total = 233472; d.ok = true; }
    TcPlan pl;
    if (!prepared_plan(m, cin, cout, d, pl)) return 0;
    return round256((size_t)pl.p.groups * pl.p.image_stride);
}

prom_status prom_pw_prepare(int64_t m, int cin, const uint8_t *w_packed_dev, int cout, const prom_requant *rq,
                            void *prepared_dev, size_t prepared_bytes, void *cuda_stream)
{
    if (!w_packed_dev || !prepared_dev) return PROM_ERR_NULL;
    prom_status e = check_requant(rq);
    if (e != PROM_OK) return e;
    if (m < 1 || cin < 1 || cin > 4096 || cout < 1 || cout > 4096) return PROM_ERR_SHAPE;
    if (!aligned16(w_packed_dev) || !aligned16(prepared_dev)) return PROM_ERR_ALIGN;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    TcPlan pl;
    if (!prepared_plan(m, cin, cout, d, pl)) return PROM_ERR_UNSUPPORTED;
    if (prepared_bytes < round256((size_t)pl.p.groups * pl.p.image_stride)) return PROM_ERR_WORKSPACE;
    if (tc_set_attr(d) != PROM_OK) return PROM_ERR_CUDA;
    Conv c;
    c.x = nullptr; c.m = m; c.cin = cin; c.cout = cout; c.map = RowMap{1, 1, 1, 1, 1}; c.in_rows = m;
    c.w = w_packed_dev; c.rq = *rq; c.y = nullptr; c.st = static_cast<cudaStream_t>(cuda_stream);
    c.pdl = false; c.pdl_next = false;
    tc_bind(c, pl, static_cast<uint8_t *>(prepared_dev));
    tc::PrepTable t;
    memset(&t, 0, sizeof(t));
    t.n = 1;
    t.first[0] = 0;
    t.first[1] = pl.p.groups;
    t.layer[0] = pl.p;
    tc::tc_prep_kernel<<<pl.p.groups, tc::kThreads, pl.smem, c.st>>>(t);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_pw_conv_i8_prepared(const int8_t *x_dev, int64_t m, int cin, int cout, const void *prepared_dev,
                                     int act_min, int act_max, int8_t *y_dev, void *cuda_stream)
{
    if (act_min < -128 || act_max > 127 || act_min > act_max) return PROM_ERR_BAD_REQUANT;
    if (cin < 1 || cin > 4096 || cout < 1 || cout > 4096 || m < 0 || m > (1ll << 40)) return PROM_ERR_SHAPE;
    if (m == 0) return PROM_OK;
    if (!x_dev || !prepared_dev || !y_dev) return PROM_ERR_NULL;
    if (!aligned16(x_dev) || !aligned16(prepared_dev) || !aligned16(y_dev)) return PROM_ERR_ALIGN;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    TcPlan pl;
    if (!prepared_plan(m, cin, cout, d, pl)) return PROM_ERR_UNSUPPORTED;
    if (tc_set_attr(d) != PROM_OK) return PROM_ERR_CUDA;
    Conv c;
    c.x = x_dev; c.m = m; c.cin = cin; c.cout = cout; c.map = RowMap{1, 1, 1, 1, 1}; c.in_rows = m;
    c.w = nullptr; c.rq = prom_requant{nullptr, nullptr, nullptr, act_min, act_max}; c.y = y_dev;
    c.st = static_cast<cudaStream_t>(cuda_stream);
    c.pdl = false; c.pdl_next = false;
    tc_bind(c, pl, const_cast<uint8_t *>(static_cast<const uint8_t *>(prepared_dev)));
    return tc_launch_planned(c, pl);
}

prom_status prom_pw_conv_i8_res(const int8_t *x_dev, int64_t m, int cin, const uint8_t *w_packed_dev,
                                int cout, const prom_requant *rq, const int8_t *res_dev,
                                int8_t *y_dev, prom_variant variant, void *cuda_stream)
{
    if (m == 0 && cin >= 1 && cin <= 4096 && cout >= 1 && cout <= 4096 && w_packed_dev && rq)
        return check_requant(rq);
    prom_status s = check_conv(x_dev, m, cin, w_packed_dev, cout, rq, y_dev);
    if (s != PROM_OK) return s;
    if (!res_dev) return PROM_ERR_NULL;
    if (!aligned16(res_dev)) return PROM_ERR_ALIGN;
    Conv c;
    c.x = x_dev; c.m = m; c.cin = cin; c.cout = cout;
    c.map = RowMap{1, 1, 1, 1, 1};
    c.in_rows = m;
    c.w = w_packed_dev; c.rq = *rq; c.y = y_dev;
    c.st = static_cast<cudaStream_t>(cuda_stream);
    c.pdl = false;
    c.pdl_next = false;
    c.res = res_dev;
    return run_conv(c, variant);
}

prom_status prom_pw_conv_i8_acc32(const int8_t *x_dev, int64_t m, int cin,
                                  const uint8_t *w_packed_dev, int cout, int32_t *acc_dev,
                                  void *cuda_stream)
{
    if (!x_dev || !w_packed_dev || !acc_dev) return PROM_ERR_NULL;
    if (m < 0 || cin < 1 || cin > 4096 || cout < 1 || cout > 4096) return PROM_ERR_SHAPE;
    if (m == 0) return PROM_OK;
    Conv c;
    c.x = x_dev; c.m = m; c.cin = cin; c.cout = cout;
    c.map = RowMap{1, 1, 1, 1, 1};
    c.in_rows = m;
    c.w = w_packed_dev;
    c.rq = prom_requant{nullptr, nullptr, nullptr, 0, 127};
    c.y = nullptr;
    c.st = static_cast<cudaStream_t>(cuda_stream);
    c.pdl = false;
    c.pdl_next = false;
    return launch_naive(c, acc_dev);
}

prom_status prom_pw_conv_i8_host(const int8_t *x_host, int64_t m, int cin,
                                 const uint8_t *w_packed_dev, int cout, const prom_requant *rq,
                                 int8_t *y_host, void *workspace_dev, size_t workspace_bytes,
                                 prom_variant variant, void *cuda_stream)
{
    if (!x_host || !y_host || !workspace_dev) return PROM_ERR_NULL;
    if (m < 0 || cin < 1 || cout < 1) return PROM_ERR_SHAPE;
    size_t xb = round256((size_t)m * cin), yb = round256((size_t)m * cout);
    if (workspace_bytes < xb + yb) return PROM_ERR_WORKSPACE;
    if (!aligned16(workspace_dev)) return PROM_ERR_ALIGN;
    int8_t *xd = static_cast<int8_t *>(workspace_dev);
    int8_t *yd = xd + xb;
    prom_status s = check_conv(xd, m, cin, w_packed_dev, cout, rq, yd);
    if (s != PROM_OK) return s;
    if (m == 0) return PROM_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(xd, x_host, (size_t)m * cin, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return PROM_ERR_CUDA;
    s = prom_pw_conv_i8(xd, m, cin, w_packed_dev, cout, rq, yd, variant, cuda_stream);
    if (s != PROM_OK) return s;
    return cuda_status(cudaMemcpyAsync(y_host, yd, (size_t)m * cout, cudaMemcpyDeviceToHost, st));
}

size_t prom_layer_seq_workspace_bytes(const prom_layer *layers, int n, int batch, int h0, int w0)
{
    SeqShape s;
    if (!seq_shapes(layers, n, batch, h0, w0, s)) return 0;
    DeviceInfo d = device_info();
    SeqLayout lay;
    seq_layout(layers, n, s, d, true, lay);
    if (!lay.chains.empty()) return lay.with_chains();
    return lay.img_total ? lay.with_images() : lay.base();
}

prom_status prom_pw_layer_seq(const prom_layer *layers, int n, const int8_t *x0_dev, int batch,
                              int h0, int w0, void *workspace_dev, size_t workspace_bytes,
                              int8_t *y_out_dev, prom_variant variant, void *cuda_stream)
{
    if (!layers || !x0_dev || !y_out_dev) return PROM_ERR_NULL;
    if (!aligned16(x0_dev) || !aligned16(y_out_dev)) return PROM_ERR_ALIGN;
    return run_seq(layers, n, x0_dev, batch, h0, w0, workspace_dev, workspace_bytes, y_out_dev,
                   variant, static_cast<cudaStream_t>(cuda_stream));
}

size_t prom_layer_seq_host_workspace_bytes(const prom_layer *layers, int n, int batch, int h0,
                                           int w0)
{
    SeqShape s;
    if (!seq_shapes(layers, n, batch, h0, w0, s)) return 0;
    const size_t core = round256(prom_layer_seq_workspace_bytes(layers, n, batch, h0, w0));
    size_t xin = round256((size_t)batch * h0 * w0 * layers[0].cin);
    size_t yout = round256((size_t)s.m[n - 1] * layers[n - 1].cout);
    return core + xin + yout;
}

prom_status prom_pw_layer_seq_host(const prom_layer *layers, int n, const int8_t *x0_host,
                                   int batch, int h0, int w0, void *workspace_dev,
                                   size_t workspace_bytes, int8_t *y_out_host, prom_variant variant,
                                   void *cuda_stream)
{
    if (!layers || !x0_host || !y_out_host || !workspace_dev) return PROM_ERR_NULL;
    if (!aligned16(workspace_dev)) return PROM_ERR_ALIGN;
    SeqShape s;
    if (!seq_shapes(layers, n, batch, h0, w0, s)) return PROM_ERR_SHAPE;
    const size_t core = round256(prom_layer_seq_workspace_bytes(layers, n, batch, h0, w0));
    size_t xin_raw = (size_t)batch * h0 * w0 * layers[0].cin;
    size_t yout_raw = (size_t)s.m[n - 1] * layers[n - 1].cout;
    size_t xin = round256(xin_raw), yout = round256(yout_raw);
    if (workspace_bytes < core + xin + yout) return PROM_ERR_WORKSPACE;
    int8_t *base = static_cast<int8_t *>(workspace_dev);
    int8_t *xd = base + core, *yd = xd + xin;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(xd, x0_host, xin_raw, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return PROM_ERR_CUDA;
    prom_status e = run_seq(layers, n, xd, batch, h0, w0, base, core, yd, variant, st);
    if (e != PROM_OK) return e;
    return cuda_status(cudaMemcpyAsync(y_out_host, yd, yout_raw, cudaMemcpyDeviceToHost, st));
}

prom_status prom_pw_conv_i8_addsub_static(const int8_t *x_dev, int64_t m, int cin,
                                          const uint8_t *w_packed_dev, int cout,
                                          const prom_requant *rq, int8_t *y_dev,
                                          void *cuda_stream)
{
    // an empty matrix has no rows to read or write: its pointers may be anything
    if (m == 0 && cin >= 1 && cin <= 4096 && cout >= 1 && cout <= 4096 && w_packed_dev && rq)
        return check_requant(rq);
    prom_status s = check_conv(x_dev, m, cin, w_packed_dev, cout, rq, y_dev);
    if (s != PROM_OK) return s;
    if (cin > addsub::kMaxCin) return PROM_ERR_UNSUPPORTED;
    if (addsub::scratch_bytes(cout, cin) > (size_t)PROM_STATIC_SCRATCH_BYTES)
        return PROM_ERR_WORKSPACE;
    if (m == 0) return PROM_OK;
    uint8_t *scratch = static_scratch_address();
    if (!scratch) return PROM_ERR_CUDA;
    return addsub::launch_on(x_dev, m, cin, RowMap{1, 1, 1, 1, 1}, w_packed_dev, cout, *rq, y_dev,
                             scratch, static_cast<cudaStream_t>(cuda_stream), g_launches);
}

prom_status prom_last_device_status(void *cuda_stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned int v = 0;
    if (cudaMemcpyFromSymbolAsync(&v, g_status, sizeof(v), 0, cudaMemcpyDeviceToHost, st) !=
        cudaSuccess)
        return PROM_ERR_CUDA;
    unsigned int zero = 0;
    if (cudaMemcpyToSymbolAsync(g_status, &zero, sizeof(zero), 0, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return PROM_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PROM_ERR_CUDA;
    return static_cast<prom_status>(v);
}

uint64_t prom_launch_count(void) { return g_launches.load(); }

void prom_debug_tc_plan_shape(int64_t m, int cin, int cout, int stride, int fold, int nt, int groups,
                              int occ, int stages)
{
    std::lock_guard<std::mutex> lk(g_shape_tune_mu);
    const std::array<long long, 4> key = {m, cin, cout, stride};
    if (!fold && !nt && !groups && !occ && !stages) g_shape_tune.erase(key);
    else g_shape_tune[key] = TcTune{fold, nt, groups, occ, stages};
}

void prom_debug_tc_plan(int fold, int nt, int groups, int occ, int stages)
{
    std::lock_guard<std::mutex> lk(g_shape_tune_mu);
    g_tune = TcTune{fold, nt, groups, occ, stages};
}

prom_status prom_debug_wait_timeout(uint64_t limit_ns, int *gave_up_dev, void *cuda_stream)
{
    if (limit_ns < 1000 || limit_ns > 100000000ull) return PROM_ERR_SHAPE;
    tc::wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        (unsigned long long)limit_ns, gave_up_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_debug_i8_mma_rate(int iters, long long *cycles_dev, int cycles_len, int *grid_out,
                                   void *cuda_stream)
{
    if (!cycles_dev || !grid_out) return PROM_ERR_NULL;
    if (iters < 1 || iters > (1 << 20)) return PROM_ERR_SHAPE;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    if (cycles_len < d.sms) return PROM_ERR_WORKSPACE;
    if (raise_smem_limit(peak::i8_mma_rate_kernel, peak::kMmaSmem) != cudaSuccess) return PROM_ERR_CUDA;
    *grid_out = d.sms;
    peak::i8_mma_rate_kernel<<<d.sms, peak::kMmaThreads, peak::kMmaSmem,
                               static_cast<cudaStream_t>(cuda_stream)>>>(iters, cycles_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_debug_alu_rate(int op, int iters, int *sink_dev, long long *cycles_dev,
                                int cycles_len, int *grid_out, void *cuda_stream)
{
    if (!sink_dev || !cycles_dev || !grid_out) return PROM_ERR_NULL;
    if (op < 0 || op > 6 || iters < 1 || iters > (1 << 24)) return PROM_ERR_SHAPE;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    const int grid = 2 * d.sms;
    if (cycles_len < grid) return PROM_ERR_WORKSPACE;
    *grid_out = grid;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (op == 0) peak::alu_rate_kernel<0><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    else if (op == 1) peak::alu_rate_kernel<1><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    else if (op == 2) peak::alu_rate_kernel<2><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    else if (op == 3) peak::alu_rate_kernel<3><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    else if (op == 4) peak::alu_rate_kernel<4><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    else if (op == 5) peak::alu_rate_kernel<5><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    else peak::alu_rate_kernel<6><<<grid, peak::kAluThreads, 0, st>>>(iters, 1, sink_dev, cycles_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_debug_mma_issue_rate(int n, int warps, int iters, long long *cycles_dev, int cycles_len,
                                      int *grid_out, void *cuda_stream)
{
    if (!cycles_dev || !grid_out) return PROM_ERR_NULL;
    if (n < 16 || n > 256 || (n & 15) || warps < 1 || warps > 4 || iters < 1 || iters > (1 << 20))
        return PROM_ERR_SHAPE;
    if (warps * 2 * (n > 64 ? n : 64) > 512) return PROM_ERR_SHAPE;     // tensor-memory columns
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    if (cycles_len < 4 * d.sms) return PROM_ERR_WORKSPACE;
    *grid_out = d.sms;
    if (raise_smem_limit(peak::mma_issue_rate_kernel, peak::kMmaSmem) != cudaSuccess) return PROM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(cycles_dev, 0, sizeof(long long) * 4 * (size_t)d.sms, st) != cudaSuccess) return PROM_ERR_CUDA;
    peak::mma_issue_rate_kernel<<<d.sms, peak::kMmaThreads, peak::kMmaSmem, st>>>(iters, n, warps, cycles_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_debug_l2_copy_rate(const void *region_dev, uint64_t region_bytes, int iters, int stages,
                                    long long *cycles_dev, int cycles_len, int *grid_out, void *cuda_stream)
{
    if (!region_dev || !cycles_dev || !grid_out) return PROM_ERR_NULL;
    if (!aligned16(region_dev)) return PROM_ERR_ALIGN;
    if (region_bytes < peak::kCopyBytes || region_bytes % peak::kCopyBytes || iters < 1 || iters > (1 << 20) ||
        stages < 1 || stages > peak::kCopyMaxStages)
        return PROM_ERR_SHAPE;
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    if (cycles_len < d.sms) return PROM_ERR_WORKSPACE;
    *grid_out = d.sms;
    const int smem = peak::kCopyMaxStages * (int)peak::kCopyBytes + 256;
    if (raise_smem_limit(peak::l2_copy_rate_kernel, smem) != cudaSuccess) return PROM_ERR_CUDA;
    peak::l2_copy_rate_kernel<<<d.sms, 32, smem, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint8_t *>(region_dev), (unsigned long long)region_bytes, iters, stages, cycles_dev);
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

prom_status prom_debug_mma_beside(int mode, int iters, int nwarps, int stages, const void *region_dev,
                                  uint64_t region_bytes, long long *out_dev, int out_len, int *grid_out,
                                  void *cuda_stream)
{
    if (!out_dev || !grid_out) return PROM_ERR_NULL;
    if ((mode != 0 && mode != 1) || iters < 1 || iters > (1 << 20)) return PROM_ERR_SHAPE;
    if (mode == 0) {
        if (stages < 0 || stages > 3) return PROM_ERR_SHAPE;
        if (stages > 0) {
            if (!region_dev) return PROM_ERR_NULL;
            if (!aligned16(region_dev)) return PROM_ERR_ALIGN;
            if (region_bytes < peak::kCopyBytes || region_bytes % peak::kCopyBytes) return PROM_ERR_SHAPE;
        }
    } else if ((nwarps != 4 && nwarps != 8 && nwarps != 16) || (stages != 0 && stages != 1)) {
        return PROM_ERR_SHAPE;
    }
    DeviceInfo d = device_info();
    if (!d.ok) return PROM_ERR_CUDA;
    if (out_len < 8 * d.sms) return PROM_ERR_WORKSPACE;
    *grid_out = d.sms;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(out_dev, 0, sizeof(long long) * 8 * (size_t)d.sms, st) != cudaSuccess) return PROM_ERR_CUDA;
    const uint8_t *src = static_cast<const uint8_t *>(region_dev);
    if (mode == 0) {
        if (raise_smem_limit(peak::beside_mma_kernel<0>, peak::kBesideSmem) != cudaSuccess) return PROM_ERR_CUDA;
        peak::beside_mma_kernel<0><<<d.sms, peak::kBesideThreads, peak::kBesideSmem, st>>>(
            iters, 0, stages, src, (unsigned long long)region_bytes, out_dev);
    } else {
        if (raise_smem_limit(peak::beside_mma_kernel<1>, peak::kBesideSmem) != cudaSuccess) return PROM_ERR_CUDA;
        peak::beside_mma_kernel<1><<<d.sms, peak::kBesideThreads, peak::kBesideSmem, st>>>(
            iters, nwarps, stages, src, (unsigned long long)region_bytes, out_dev);
    }
    ++g_launches;
    return cuda_status(cudaGetLastError());
}

void prom_debug_seq_order(int alternate) { g_seq_snake.store(alternate ? 1 : 0); }
void prom_debug_seq_chain(int mode) { g_seq_chain.store(mode == 2 ? 2 : (mode ? 1 : 0)); }

void prom_debug_dw_variant(int variant) { g_dw_variant.store(variant < 0 || variant > 2 ? 0 : variant); }

void prom_debug_tc_wide(int mode, int blocks)
{
    g_wide_mode.store(mode < 0 || mode > 2 ? 0 : mode);
    g_wide_nb.store(blocks == 1 || blocks == 2 ? blocks : 0);
}

int64_t prom_debug_layer_seq_output_offset(const prom_layer *layers, int n, int batch, int h0, int w0,
                                           int layer, int *chained)
{
    SeqShape s;
    if (!seq_shapes(layers, n, batch, h0, w0, s) || layer < 0 || layer >= n - 1) return -1;
    DeviceInfo d = device_info();
    SeqLayout lay;
    seq_layout(layers, n, s, d, true, lay);
    const bool in_chain = lay.chain_of[layer] >= 0;
    if (chained) *chained = in_chain ? 1 : 0;
    if (in_chain) {
        const ChainPlan &c = lay.chains[lay.chain_of[layer]];
        if (c.kind == 1 && layer != c.last) return -2;      // never written: it stays in shared memory
        return (int64_t)(round256(lay.with_images()) + lay.cbuf_off[layer]);
    }
    return (layer & 1) ? (int64_t)lay.ra : 0;
}

int prom_debug_once_per_device(int device, int key)
{
    static OncePerDevice table;
    return table.first(device, reinterpret_cast<const void *>((intptr_t)key)) ? 1 : 0;
}

int prom_debug_tc_plan_query(int64_t m, int cin, int cout, int *out9)
{
    if (!out9) return 0;
    DeviceInfo d = device_info();
    if (!d.ok) {
        // no device to ask: the plan for a B200 as shipped (148 SMs, 227 KB of shared memory a
        // CTA can opt into, 228 KB per SM), so that the planner can be exercised anywhere
        d.sms = 148; d.smem_optin = 232448; d.smem_total = 233472; d.ok = true;
    }
    TcPlan pl;
    if (!tc_shape_plan(m, cin, cout, RowMap{1, 1, 1, 1, 1}, d, pl)) return 0;
    const tc::Params &p = pl.p;
    out9[0] = p.fold; out9[1] = p.nt; out9[2] = p.groups; out9[3] = pl.grid; out9[4] = p.stages;
    out9[5] = p.nbuf; out9[6] = (int)pl.smem; out9[7] = p.cw; out9[8] = (int)(pl.est_us * 100);
    return 1;
}

void prom_shutdown(void)
{
    addsub::release_cache();
    wide_release_cache();
}

const char *prom_status_string(prom_status s)
{
    switch (s) {
    case PROM_OK: return "ok";
    case PROM_ERR_NULL: return "null pointer";
    case PROM_ERR_SHAPE: return "bad shape";
    case PROM_ERR_ALIGN: return "misaligned pointer";
    case PROM_ERR_BAD_WEIGHT: return "weight outside {-1,0,+1}";
    case PROM_ERR_BAD_REQUANT: return "requantisation constants out of range";
    case PROM_ERR_WORKSPACE: return "workspace too small";
    case PROM_ERR_UNSUPPORTED: return "variant does not support this shape";
    case PROM_ERR_CUDA: return "CUDA call failed";
    case PROM_ERR_TIMEOUT: return "device-side wait ran out";
    default: return "unknown status";
    }
}

}  // extern "C"
