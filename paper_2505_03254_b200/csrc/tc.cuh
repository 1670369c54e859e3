// The tensor-core variant: TMA-staged int8 activation tiles, ternary weights
// expanded from their 2-bit form into shared memory once per CTA, tcgen05
// int8 MMAs accumulating in tensor memory, and a fused requantising epilogue
// whose int8 rows leave through bulk (TMA) stores.
//
// Work decomposition
//   tile      = `tm` consecutive output rows (<= 128; one MMA M block)
//   subtile   = `nt` consecutive output channels (one accumulator, <= 256)
//   K chunk   = `cw` bytes of a row (32, 64 or 128: one TMA box, one swizzle span)
//   unit      = (tile, subtile)
// A CTA keeps the expanded weights of its subtiles resident for its whole
// life and walks over tiles.  Warp 0 issues TMA loads, warp 1 issues MMAs,
// warps 2..9 are two epilogue groups of four warps (one TMEM lane quarter
// each) that take units alternately.
//
// Row folding: with fold f the matrices are viewed as X'[M/f][f*cin],
// Y'[M/f][f*cout] and the weights as the block diagonal diag(W, .., W); X' and
// Y' are byte for byte the same memory as X and Y.  It makes channel counts
// that are not multiples of 16 legal for TMA and gives tiny layers wider tiles.
//
// Fast epilogue (clamp [0,127], shifts of the CTA's channels within 4 of one
// another, no overflow): channel c's weights are expanded as
// +-2^(2+shmax-shift[c]) and its bias, scaled the same way, enters the
// accumulator through one extra MMA k-step (a constant A block of 1s and 127s
// against a block of base-127 bias digits), so that TMEM holds
// t' = (acc + bias) * 2^(2+shmax-shift[c]) and
//     v1 = (hi32(t' * mult) + 2^shmax) >> shmax
// equals floor(t*mult / 2^(30+shift)) + 1 exactly; the result is
// sat_u8(v1) >> 1.  Everything else takes the 64-bit definition.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace prom { namespace tc {

constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr int kEpiGroups = 2;
constexpr unsigned long long kWaitLimitNs = 100000000ull;   // 0.1 s: far beyond any legitimate wait
constexpr int kMaxStages = 8;
constexpr int kMaxBufs = 4;
constexpr int kLuts = 6;                 // magnitude 1, then 4, 8, 16, 32, 64
constexpr int kAConstBytes = 128 * 32;
constexpr int kBiasHiDigits = 30;        // A-const row: 1, 1, then 30 x 127
constexpr int kBiasMax = 127 * 127 * kBiasHiDigits;
constexpr int kNoColumn = -1000;        // marks a padding column (no int8 shift has this value)

struct Params {
    long long m_rows;   // rows of the folded problem
    int k0, n0;         // layer cin, cout
    int fold;
    int kf, nf;         // folded cin, cout
    int tm;             // rows per tile
    int n_mtiles;
    int nt, nt_pad;     // subtile width, MMA N
    int n_sub, groups, subs_per_cta;
    int cw;             // chunk row bytes (32, 64, 128) = swizzle span
    int kc;             // K chunks per tile
    int ksteps_last;    // 32-wide MMA steps in the last chunk
    int stages, nbuf, tmem_cols;
    int share_x;        // kc == 1: one activation load serves all subtiles of the tile
    int store_2d;       // 0: rows of a slab are contiguous in Y (one subtile), 1: tensor-map store
    int x3d, box_r;     // 3-D activation map (strided input); rows of dim 2 per tile
    uint32_t tx_bytes;
    uint32_t off_w, off_wbias, off_mult, off_bs, off_hdr, off_aconst, off_out, off_lut, off_bars;
    // A CTA's prepared operands (expanded weights, bias digits, multipliers, {bias, shift},
    // header) are one contiguous range of shared memory, [off_w, off_hdr + 16).  When `image`
    // is set it holds that range for every channel group, image_stride bytes apart, written
    // by tc_prep_kernel; the convolution kernel then copies it in instead of building it.
    uint8_t *image;
    uint32_t image_bytes, image_stride;
    const uint8_t *w_packed;
    const int32_t *bias, *mult;
    const int8_t *shift;
    int act_min, act_max;
    int8_t *y;
    int pdl;            // launched with programmatic dependent launch
    int pdl_next;       // the next kernel in the stream is launched that way
    int reverse;        // row tiles are taken from the last to the first
    // The dynamic layer (kernel modes 1 and 2): `mult` then holds the bit patterns of the
    // float per-channel factors alpha, bias and shift are not read, and rows belong to
    // samples of rows_per_sample rows each.
    int dyn;                    // 0: static requantisation
    int rows_per_sample;
    int batch;
    const float *gamma_x;       // [batch] per-sample maximum behind the int8 input
    float *gamma_y;             // [batch] mode 1: maxima of the dequantised output (as bit patterns)
    const float *scale_y;       // [batch] mode 2: 127 / max(gamma_y, eps)
    // Kernel mode 3: an int8 tensor of Y's shape added to the requantised output with
    // saturation.  It may be Y itself: a warp reads the bytes of a slab before it stores there.
    const int8_t *res;
};

// Bounded wait on an mbarrier phase.  The clock is read only every 1024 polls (a
// poll that finds the phase incomplete already suspends the thread for a while), so
// that a wait which ends within microseconds never pays for a timer read.
constexpr unsigned long long kWaitGiveUp = ~0ull;

// The rare part of a wait, out of line: returns the time the wait began (set on the first call),
// or kWaitGiveUp when another thread has given up or this wait has run past its limit.
__device__ __noinline__ unsigned long long wait_check(unsigned long long t0, volatile int *abort_flag,
                                                      unsigned long long limit_ns)
{
    if (*abort_flag) return kWaitGiveUp;
    const unsigned long long now = ptx::globaltimer();
    if (t0 == 0) return now;
    if (now - t0 > limit_ns) {
        *abort_flag = 1;
        raise_status(PROM_ERR_TIMEOUT);
        return kWaitGiveUp;
    }
    return t0;
}

template <bool BACKOFF = false>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                         unsigned long long limit_ns = kWaitLimitNs)
{
    unsigned long long t0 = 0;
    for (uint32_t i = 1;; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if constexpr (BACKOFF) __nanosleep(20);      // whole warps wait here: poll gently
        if ((i & 1023u) == 0) {
            t0 = wait_check(t0, abort_flag, limit_ns);
            if (t0 == kWaitGiveUp) return false;
        }
    }
}

// K-major operand with rows of `cw` bytes swizzled over a span of `cw` bytes:
// 8-row atoms of 8*cw bytes, one after the other.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t cw)
{
    const uint64_t mode = cw == 128 ? 2ull : (cw == 64 ? 4ull : 6ull);
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)((8u * cw) >> 4) << 32) |
           (1ull << 46) | (mode << 61);
}

// 16-byte piece j of row n inside a swizzled block with rows of cw bytes.
__device__ __forceinline__ uint32_t swz_offset(uint32_t n, uint32_t j, uint32_t cw)
{
    const uint32_t x = cw == 128 ? (n & 7u) : (cw == 64 ? ((n >> 1) & 3u) : ((n >> 2) & 1u));
    return n * cw + ((j ^ x) << 4);
}

template <int NC>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&v)[NC])
{
    if constexpr (NC == 32) ptx::tmem_ld_x32(taddr, v);
    else if constexpr (NC == 16) ptx::tmem_ld_x16(taddr, v);
    else ptx::tmem_ld_x8(taddr, v);
}

// Once a warp has read the last columns of an accumulator into registers it hands the
// accumulator back (one arrival per warp), so that the next MMA overlaps the arithmetic
// on those registers.  bar == 0: not the last columns.
__device__ __forceinline__ void release_acc(uint32_t bar)
{
    if (bar) {
        ptx::tc_fence_before_sync();
        __syncwarp();
        if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(bar);
    }
}

// Rows of the staging slab are nt bytes apart: 16-byte aligned only when nt is a
// multiple of 16 (`wide`), 8-byte aligned otherwise.
template <int NC>
__device__ __forceinline__ void put_row(uint8_t *dst, const uint32_t (&out)[NC / 4], bool wide)
{
    if (NC >= 16 && wide) {
#pragma unroll
        for (int i = 0; i < NC / 16; ++i)
            *reinterpret_cast<uint4 *>(dst + 16 * i) =
                make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < NC / 8; ++i)
            *reinterpret_cast<uint2 *>(dst + 8 * i) = make_uint2(out[2 * i], out[2 * i + 1]);
    }
}

// The 64-bit definition (any clamp, any shifts).
template <int NC>
__device__ __forceinline__ void epi_exact(uint32_t taddr, const int *__restrict__ cm,
                                          const int2 *__restrict__ cbs, int lo, int hi, uint8_t *dst,
                                          bool wide, uint32_t release_bar)
{
    uint32_t v[NC];
    tmem_ld<NC>(taddr, v);
    ptx::tmem_wait_ld();
    release_acc(release_bar);
    uint32_t out[NC / 4];
#pragma unroll
    for (int c = 0; c < NC; c += 4) {
        uint32_t w = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int2 bs = cbs[c + e];
            const int q = requant_exact((int)v[c + e] + bs.x, cm[c + e], bs.y, lo, hi);
            w |= ((uint32_t)q & 0xFFu) << (8 * e);
        }
        out[c / 4] = w;
    }
    put_row<NC>(dst, out, wide);
}

// One output of the fast epilogue for the full int8 range: the rounding term loses one unit
// when the product is negative (ties go away from zero), and the shift drops the extra bit.
__device__ __forceinline__ int fast_signed(int v, int mu, long long r64, int shmax)
{
    return (int)(((long long)v * mu + (r64 + (long long)(v >> 31))) >> 32) >> (shmax + 1);
}

// NC accumulator columns of this thread's row, already in registers: the high word of a
// 64-bit multiply-add (rounding term in the addend), one shift, saturating pack, halve.
// SIGNED: the clamp is [-128, 127] instead of [0, 127].
template <int NC, bool SIGNED = false>
__device__ __forceinline__ void fast_piece(const uint32_t (&v)[NC], const int *__restrict__ cm,
                                           long long r64, int shmax, uint8_t *dst, bool wide)
{
    uint32_t out[NC / 4];
#pragma unroll
    for (int c = 0; c < NC; c += 4) {
        const int4 mu = *reinterpret_cast<const int4 *>(cm + c);
        if constexpr (SIGNED) {
            const int q0 = fast_signed((int)v[c], mu.x, r64, shmax);
            const int q1 = fast_signed((int)v[c + 1], mu.y, r64, shmax);
            const int q2 = fast_signed((int)v[c + 2], mu.z, r64, shmax);
            const int q3 = fast_signed((int)v[c + 3], mu.w, r64, shmax);
            out[c / 4] = ptx::pack_sat_s8(q1, q0, ptx::pack_sat_s8(q3, q2, 0u));
            continue;
        }
        const int q0 = (int)(((long long)(int)v[c] * mu.x + r64) >> 32) >> shmax;
        const int q1 = (int)(((long long)(int)v[c + 1] * mu.y + r64) >> 32) >> shmax;
        const int q2 = (int)(((long long)(int)v[c + 2] * mu.z + r64) >> 32) >> shmax;
        const int q3 = (int)(((long long)(int)v[c + 3] * mu.w + r64) >> 32) >> shmax;
        uint32_t w = ptx::pack_sat_u8(q3, q2, 0u);
        w = ptx::pack_sat_u8(q1, q0, w);
        out[c / 4] = (w >> 1) & 0x7F7F7F7Fu;
    }
    put_row<NC>(dst, out, wide);
}

// The fast epilogue over one subtile, in chunks of CH (32 or 16), then 16 and 8 columns.  The
// accumulator goes back to the MMA thread as soon as its last columns are in registers.
template <int CH, bool SIGNED = false>
__device__ __forceinline__ void epi_fast_subtile(const Params &p, uint32_t taddr, const int *cm,
                                                 int shmax, uint8_t *dst_row, uint32_t bar_release)
{
    const bool wide = (p.nt & 15) == 0;
    const long long r64 = 1ll << (32 + shmax);   // rounding term, in the addend of the 64-bit product
    const int tail = p.nt & (CH - 1);            // columns after the last full chunk
    int c = 0;
    for (; c + CH <= p.nt; c += CH) {
        uint32_t v[CH];
        tmem_ld<CH>(taddr + c, v);
        ptx::tmem_wait_ld();
        if (tail == 0 && c + CH == p.nt) release_acc(bar_release);
        fast_piece<CH, SIGNED>(v, cm + c, r64, shmax, dst_row + c, wide);
    }
    if (CH > 16 && c + 16 <= p.nt) {
        uint32_t v[16];
        ptx::tmem_ld_x16(taddr + c, v);
        ptx::tmem_wait_ld();
        if (c + 16 == p.nt) release_acc(bar_release);
        fast_piece<16, SIGNED>(v, cm + c, r64, shmax, dst_row + c, wide);
        c += 16;
    }
    if (c + 8 <= p.nt) {
        uint32_t v[8];
        ptx::tmem_ld_x8(taddr + c, v);
        ptx::tmem_wait_ld();
        release_acc(bar_release);
        fast_piece<8, SIGNED>(v, cm + c, r64, shmax, dst_row + c, wide);
    }
}

// The fast epilogue over one subtile of a width known at compile time: straight-line code.
template <int NT, bool SIGNED = false>
__device__ __forceinline__ void epi_fast_fixed(uint32_t taddr, const int *cm, int shmax, uint8_t *dst_row,
                                               uint32_t bar_release)
{
    constexpr bool wide = (NT & 15) == 0;
    const long long r64 = 1ll << (32 + shmax);
    constexpr int full = NT & ~31;
#pragma unroll
    for (int c = 0; c < full; c += 32) {
        uint32_t v[32];
        ptx::tmem_ld_x32(taddr + c, v);
        ptx::tmem_wait_ld();
        if (c + 32 == NT) release_acc(bar_release);
        fast_piece<32, SIGNED>(v, cm + c, r64, shmax, dst_row + c, wide);
    }
    if constexpr ((NT & 16) != 0) {
        uint32_t v[16];
        ptx::tmem_ld_x16(taddr + full, v);
        ptx::tmem_wait_ld();
        if (full + 16 == NT) release_acc(bar_release);
        fast_piece<16, SIGNED>(v, cm + full, r64, shmax, dst_row + full, wide);
    }
    if constexpr ((NT & 8) != 0) {
        constexpr int c8 = NT & ~15;
        uint32_t v[8];
        ptx::tmem_ld_x8(taddr + c8, v);
        ptx::tmem_wait_ld();
        release_acc(bar_release);
        fast_piece<8, SIGNED>(v, cm + c8, r64, shmax, dst_row + c8, wide);
    }
}

// The exact epilogue over one subtile, in chunks of CH (32 or 16), then 16 and 8 columns.
template <int CH>
__device__ __noinline__ void epi_exact_subtile(int nt, int act_min, int act_max, uint32_t taddr,
                                               const int *cm, const int2 *cbs, uint8_t *dst_row,
                                               uint32_t bar_release)
{
    const bool wide = (nt & 15) == 0;
    const int tail = nt & (CH - 1);    // columns after the last full chunk
    int c = 0;
    for (; c + CH <= nt; c += CH) {
        const uint32_t rel = (tail == 0 && c + CH == nt) ? bar_release : 0u;
        epi_exact<CH>(taddr + c, cm + c, cbs + c, act_min, act_max, dst_row + c, wide, rel);
    }
    if (CH > 16 && c + 16 <= nt) {
        const uint32_t rel = (c + 16 == nt) ? bar_release : 0u;
        epi_exact<16>(taddr + c, cm + c, cbs + c, act_min, act_max, dst_row + c, wide, rel);
        c += 16;
    }
    if (c + 8 <= nt)
        epi_exact<8>(taddr + c, cm + c, cbs + c, act_min, act_max, dst_row + c, wide, bar_release);
}

// Stores the first rows_valid rows of a warp's 32 x nt staging slab (a short tile or the end of
// the matrix); yp points at the slab's first row in Y.  Out of line: it runs at most once per CTA.
__device__ __noinline__ void store_partial_slab(int8_t *yp, const uint8_t *slab, int rows_valid, int nf,
                                                int nt, int col, bool store_2d, int lane)
{
    const uint32_t slab_addr = ptx::smem_u32(slab);
    if (!store_2d) {
        // one subtile spans the row: the slab is one contiguous range of Y
        if (lane == 0 && rows_valid > 0) {
            const uint32_t bytes = (uint32_t)(rows_valid * nf);
            const uint32_t whole = bytes & ~15u;      // bulk copies move 16-byte granules
            if (whole) {
                ptx::bulk_store(yp, slab_addr, whole);
                ptx::bulk_commit();
            }
            if (bytes & 15u)                          // odd last row of an 8-multiple width
                *reinterpret_cast<uint2 *>(yp + whole) = *reinterpret_cast<const uint2 *>(slab + whole);
        }
    } else if (lane < rows_valid) {
        // the slab leaves row by row
        ptx::bulk_store(yp + (long long)lane * nf + col, slab_addr + (uint32_t)(lane * nt), (uint32_t)nt);
        ptx::bulk_commit();
    }
}

// ---- the dynamic layer's epilogues ---------------------------------------------------------
// y = acc * alpha[column] * dq[sample]: the int32 accumulator becomes a float exactly (the
// magic-number form holds below 2^22; |acc| <= 4096 * 127), then two correctly rounded products
// in this order.
__device__ __forceinline__ float dyn_value(uint32_t acc, int alpha_bits, float dq)
{
    const float f = __fadd_rn(__int_as_float((int)acc + 0x4B400000), -12582912.0f);
    return __fmul_rn(__fmul_rn(f, __int_as_float(alpha_bits)), dq);
}

// NC accumulator columns of this thread's row, already in registers.
// Mode 1: the largest |y| among them joins m.
template <int NC>
__device__ __forceinline__ float dyn_piece_max(const uint32_t (&v)[NC], const int *__restrict__ cm, float dq,
                                               float m)
{
#pragma unroll
    for (int e = 0; e < NC; e += 4) {
        const int4 mu = *reinterpret_cast<const int4 *>(cm + e);
        m = fmaxf(m, fabsf(dyn_value(v[e], mu.x, dq)));
        m = fmaxf(m, fabsf(dyn_value(v[e + 1], mu.y, dq)));
        m = fmaxf(m, fabsf(dyn_value(v[e + 2], mu.z, dq)));
        m = fmaxf(m, fabsf(dyn_value(v[e + 3], mu.w, dq)));
    }
    return m;
}

// Mode 2: y quantised with the sample's scale (ties to even through the magic-number add,
// saturating packs clip to [-128, 127]) and staged like the static epilogue's bytes.
template <int NC>
__device__ __forceinline__ void dyn_piece_quant(const uint32_t (&v)[NC], const int *__restrict__ cm, float dq,
                                                float sc, uint8_t *dst, bool wide)
{
    uint32_t out[NC / 4];
#pragma unroll
    for (int e = 0; e < NC; e += 4) {
        const int4 mu = *reinterpret_cast<const int4 *>(cm + e);
        const int a4[4] = {mu.x, mu.y, mu.z, mu.w};
        int r[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float y = dyn_value(v[e + j], a4[j], dq);
            r[j] = __float_as_int(__fadd_rn(__fmul_rn(y, sc), 12582912.0f)) - 0x4B400000;
        }
        uint32_t w;
        asm("{\n\t.reg .b32 t;\n\t"
            "cvt.pack.sat.s8.s32.b32 t, %4, %3, 0;\n\t"
            "cvt.pack.sat.s8.s32.b32 %0, %2, %1, t;\n\t}"
            : "=r"(w)
            : "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]));
        out[e / 4] = w;
    }
    put_row<NC>(dst, out, wide);
}

// One subtile in chunks of CH, then 16 and 8 columns (nt is a multiple of 8).  QUANT false:
// returns the largest |y| of the row; true: stages the codes and returns 0.
template <int CH, bool QUANT>
__device__ __forceinline__ float epi_dyn_subtile(const Params &p, uint32_t taddr, const int *cm, float dq,
                                                 float sc, uint8_t *dst_row, uint32_t bar_release)
{
    const bool wide = (p.nt & 15) == 0;
    const int tail = p.nt & (CH - 1);
    float m = 0.0f;
    int c = 0;
    for (; c + CH <= p.nt; c += CH) {
        uint32_t v[CH];
        tmem_ld<CH>(taddr + c, v);
        ptx::tmem_wait_ld();
        if (tail == 0 && c + CH == p.nt) release_acc(bar_release);
        if constexpr (QUANT) dyn_piece_quant<CH>(v, cm + c, dq, sc, dst_row + c, wide);
        else m = dyn_piece_max<CH>(v, cm + c, dq, m);
    }
    if (CH > 16 && c + 16 <= p.nt) {
        uint32_t v[16];
        ptx::tmem_ld_x16(taddr + c, v);
        ptx::tmem_wait_ld();
        if (c + 16 == p.nt) release_acc(bar_release);
        if constexpr (QUANT) dyn_piece_quant<16>(v, cm + c, dq, sc, dst_row + c, wide);
        else m = dyn_piece_max<16>(v, cm + c, dq, m);
        c += 16;
    }
    if (c + 8 <= p.nt) {
        uint32_t v[8];
        ptx::tmem_ld_x8(taddr + c, v);
        ptx::tmem_wait_ld();
        release_acc(bar_release);
        if constexpr (QUANT) dyn_piece_quant<8>(v, cm + c, dq, sc, dst_row + c, wide);
        else m = dyn_piece_max<8>(v, cm + c, dq, m);
    }
    return m;
}

// Where the parts of a CTA's shared memory are.
struct View {
    uint8_t *smem;
    uint32_t smem_base;
    uint8_t *w_smem, *wbias_smem, *aconst_smem;
    int *cmult;          // mult per resident column
    int2 *cbs;           // {bias, shift} per resident column
    int *hdr;            // {shmax, fast epilogue, bad constants, 0}
    uint32_t *lut;       // [kLuts][256]
    volatile int *flags; // [0] abort, [1] shmin, [2] shmax, [3] bad constants, [4] slow path
    uint32_t bar_wload;
};

__device__ __forceinline__ View make_view(const Params &p, uint8_t *smem, uint64_t *bars)
{
    View v;
    v.smem = smem;
    v.smem_base = ptx::smem_u32(smem);
    v.w_smem = smem + p.off_w;
    v.wbias_smem = smem + p.off_wbias;
    v.aconst_smem = smem + p.off_aconst;
    v.cmult = reinterpret_cast<int *>(smem + p.off_mult);
    v.cbs = reinterpret_cast<int2 *>(smem + p.off_bs);
    v.hdr = reinterpret_cast<int *>(smem + p.off_hdr);
    v.lut = reinterpret_cast<uint32_t *>(smem + p.off_lut);
    constexpr int kBarSlots = 2 * kMaxStages + 2 * kMaxBufs + 2;
    v.flags = reinterpret_cast<volatile int *>(bars + kBarSlots + 1);
    v.bar_wload = ptx::smem_u32(bars) + 8 * (kBarSlots - 1);
    return v;
}

// The constant A block of the bias step: bytes 0,1 = 1, bytes 2..31 = 127.
__device__ __forceinline__ void build_aconst(uint8_t *aconst_smem, int tid, int nthreads)
{
    for (int i = tid; i < 128 * 2; i += nthreads) {
        const uint32_t r = (uint32_t)i >> 1, j = (uint32_t)i & 1u;
        const uint4 val = j == 0 ? make_uint4(0x7F7F0101u, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu)
                                 : make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);
        *reinterpret_cast<uint4 *>(aconst_smem + swz_offset(r, j, 32u)) = val;
    }
}

// Builds the prepared operands of channel group g in shared memory: requantisation
// constants checked and stored, the fast/exact decision, bias digits, and the 2-bit weights
// expanded into the K-major swizzled int8 operand layout.  All kThreads threads take part
// (three block-wide syncs inside); on return the header is written but not yet synchronised.
// Thread 0 starts the bulk copy of the group's packed weights into the not yet used
// activation stages; meanwhile every thread requests the constants of its channels and
// builds the code tables.
__device__ __forceinline__ void build_image(const Params &p, const int g, const View &vw)
{
    uint8_t *const smem = vw.smem;
    const uint32_t smem_base = vw.smem_base;
    uint8_t *const w_smem = vw.w_smem, *const wbias_smem = vw.wbias_smem;
    int *const cmult = vw.cmult;
    int2 *const cbs = vw.cbs;
    int *const hdr = vw.hdr;
    uint32_t *const lut = vw.lut;
    volatile int *const flags = vw.flags;
    const uint32_t bar_wload = vw.bar_wload;
    const int ncols_res = p.subs_per_cta * p.nt_pad;
    const uint32_t cw = (uint32_t)p.cw;
    // Thread 0 sets up the barriers and starts the bulk copy of this CTA's packed (2-bit)
    // weights into the not yet used activation stages; meanwhile every thread requests the
    // constants of its channels and builds the code tables.  Three block-wide syncs in all.
    const int rowb = (p.k0 + 3) >> 2;
    const uint8_t *wq = smem;                    // packed weights: rows of rowb bytes
    if (threadIdx.x == 0) {
        ptx::mbar_init(bar_wload, 1);
        ptx::mbar_init_fence();
        flags[0] = 0; flags[1] = 31; flags[2] = 0; flags[3] = 0; flags[4] = 0;
        if (p.fold > 1) {
            // small layer: the whole packed matrix, indexed by channel
            const uint32_t bytes = (uint32_t)(p.n0 * rowb);
            ptx::mbar_expect_tx(bar_wload, bytes);
            ptx::bulk_load(smem_base, p.w_packed, bytes, bar_wload);
        } else {
            // the rows of each resident subtile, subtile after subtile
            const uint32_t bytes = (uint32_t)(p.nt * rowb);
            ptx::mbar_expect_tx(bar_wload, bytes * (uint32_t)p.subs_per_cta);
            for (int ls = 0; ls < p.subs_per_cta; ++ls)
                ptx::bulk_load(smem_base + (uint32_t)ls * bytes,
                               p.w_packed + (size_t)(g + ls * p.groups) * bytes, bytes, bar_wload);
        }
    }

    // constants of up to kConstPerThread resident channels per thread, requested early
    constexpr int kConstPerThread = 4;
    int cb_[kConstPerThread], cm_[kConstPerThread], cs_[kConstPerThread];
#pragma unroll
    for (int u = 0; u < kConstPerThread; ++u) {
        const int i = u * kThreads + (int)threadIdx.x;
        cb_[u] = 0; cm_[u] = 0; cs_[u] = kNoColumn;         // padding column, or none
        if (i < ncols_res) {
            const int ls = i / p.nt_pad, c = i - ls * p.nt_pad;
            const int nfold = (g + ls * p.groups) * p.nt + c;
            if (c < p.nt && nfold < p.nf) {
                const int n = nfold % p.n0;
                cm_[u] = __ldg(p.mult + n);
                cb_[u] = p.dyn ? 0 : __ldg(p.bias + n);
                cs_[u] = p.dyn ? 0 : (int)__ldg(p.shift + n);
            }
        }
    }
    // code tables: byte of four 2-bit codes -> four int8 of magnitude 1, 4, 8, .., 64
    for (int i = threadIdx.x; i < kLuts * 256; i += kThreads) {
        const uint32_t t = (uint32_t)i >> 8, byte = (uint32_t)i & 255u;
        const uint32_t mag = t == 0 ? 1u : (2u << t), neg = 256u - mag;
        uint32_t w4 = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t code = (byte >> (2 * e)) & 3u;
            const uint32_t val = code == 1u ? mag : (code == 3u ? neg : 0u);
            w4 |= val << (8 * e);
        }
        lut[i] = w4;
    }
    __syncthreads();                                        // barriers and flags are set up

    // range check, shift span, and whether every channel can take the fast epilogue: with
    // the largest weight magnitude (2^6) |acc + bias| * 2^6 must stay below 2^31 and the
    // scaled bias within the digit range
    {
        int mn = 31, mx = 0, bad = 0, slow = 0;
        auto take = [&](int i, int b, int mu, int sh) {
            if (sh != kNoColumn) {
                if (!requant_ok(b, mu, sh)) { bad = 1; b = 0; mu = 0; sh = 0; }
                mn = min(mn, sh); mx = max(mx, sh);
                const long long ab = b < 0 ? -(long long)b : b;
                if ((((long long)128 * p.k0 + ab) << 6) >= (1ll << 31) || (ab << 6) > kBiasMax) slow = 1;
            } else {
                sh = 0;
            }
            cmult[i] = mu;
            cbs[i] = make_int2(b, sh);
        };
#pragma unroll
        for (int u = 0; u < kConstPerThread; ++u) {
            const int i = u * kThreads + (int)threadIdx.x;
            if (i < ncols_res) take(i, cb_[u], cm_[u], cs_[u]);
        }
        for (int i = kConstPerThread * kThreads + (int)threadIdx.x; i < ncols_res; i += kThreads) {
            const int ls = i / p.nt_pad, c = i - ls * p.nt_pad;
            const int nfold = (g + ls * p.groups) * p.nt + c;
            int b = 0, mu = 0, sh = kNoColumn;
            if (c < p.nt && nfold < p.nf) {
                const int n = nfold % p.n0;
                b = __ldg(p.bias + n); mu = __ldg(p.mult + n); sh = __ldg(p.shift + n);
            }
            take(i, b, mu, sh);
        }
        if (bad) flags[3] = 1;
        if (slow) flags[4] = 1;
        if (mn <= mx) {
            atomicMin((int *)&flags[1], mn);
            atomicMax((int *)&flags[2], mx);
        }
    }
    __syncthreads();
    const int shmax = flags[2];
    const bool bad_consts = flags[3] != 0;
    const bool fast = !p.dyn && flags[4] == 0 && (p.act_min == 0 || p.act_min == -128) && p.act_max == 127 &&
                      shmax - flags[1] <= 4 && shmax <= 24;

    // bias digits of the resident channels (fast path): row n of a 32-byte-swizzled block
    if (fast)
        for (int i = threadIdx.x; i < ncols_res; i += kThreads) {
            const int ls = i / p.nt_pad, c = i - ls * p.nt_pad;
            const int2 bs = cbs[i];
            const int v = bs.x << (2 + shmax - bs.y);
            int h = (v >= 0 ? v + 63 : v - 63) / 127;        // nearest multiple of 127
            const int lo = v - 127 * h;                       // within [-63, 63]
            uint32_t wd[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) wd[e] = 0;
            wd[0] = (uint32_t)lo & 0xFFu;
#pragma unroll
            for (int d = 0; d < kBiasHiDigits; ++d) {
                const int dig = h > 127 ? 127 : (h < -127 ? -127 : h);
                h -= dig;
                const int k = d + 2;
                wd[k >> 2] |= ((uint32_t)dig & 0xFFu) << (8 * (k & 3));
            }
            uint8_t *blk = wbias_smem + (size_t)ls * p.nt_pad * 32;
            *reinterpret_cast<uint4 *>(blk + swz_offset((uint32_t)c, 0u, 32u)) =
                make_uint4(wd[0], wd[1], wd[2], wd[3]);
            *reinterpret_cast<uint4 *>(blk + swz_offset((uint32_t)c, 1u, 32u)) =
                make_uint4(wd[4], wd[5], wd[6], wd[7]);
        }
    else   // no bias step: the block is all zeros, so that a kernel which always issues the step adds nothing
        for (int i = threadIdx.x; i < ncols_res * 2; i += kThreads)
            *reinterpret_cast<uint4 *>(wbias_smem + (size_t)i * 16) = make_uint4(0u, 0u, 0u, 0u);

    // expand the resident weights from the packed copy into the K-major swizzled operand
    // layout: one table look-up per byte of four codes
    {
        const bool quick = (p.k0 & 15) == 0;
        const int cpr = p.cw >> 4;                        // 16-byte pieces per row
        const int cpr_log2 = cpr == 8 ? 3 : (cpr == 4 ? 2 : 1);
        const int per_blk = p.nt_pad * cpr;
        const int nblk = p.subs_per_cta * p.kc;
        uint32_t invalid = 0;
        const bool have_w = wait_bar<true>(bar_wload, 0u, flags);
        for (int blk = 0; have_w && blk < nblk; ++blk) {
            const int ls = blk / p.kc, chunk = blk - ls * p.kc;
            const int sub = g + ls * p.groups;
            uint8_t *dst_blk = w_smem + (size_t)blk * p.nt_pad * cw;
            const int jmax = (chunk == p.kc - 1) ? p.ksteps_last * 2 : cpr;   // pieces ever read
            for (int idx = threadIdx.x; idx < per_blk; idx += kThreads) {
                const int n = idx >> cpr_log2, j = idx & (cpr - 1);
                if (j >= jmax) continue;
                const int nfold = sub * p.nt + n, kbase = chunk * p.cw + j * 16;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (n < p.nt && nfold < p.nf && kbase < p.kf) {
                    const int t = fast ? 1 + shmax - cbs[ls * p.nt_pad + n].y : 0;
                    int pn = 0, pk = 0;                    // diagonal block of the folded weights
                    if (p.fold > 1) {
                        while ((pn + 1) * p.n0 <= nfold) ++pn;
                        while ((pk + 1) * p.k0 <= kbase) ++pk;
                    }
                    // row of this channel in the packed copy
                    const int row = p.fold > 1 ? nfold - pn * p.n0 : ls * p.nt + n;
                    if (quick) {
                        if (pn == pk) {
                            const uint32_t w = *reinterpret_cast<const uint32_t *>(
                                wq + (size_t)row * rowb + ((kbase - pk * p.k0) >> 2));
                            invalid |= (w >> 1) & ~w & 0x55555555u;
                            const uint32_t *tb = lut + t * 256;
                            val.x = tb[w & 0xFFu];
                            val.y = tb[(w >> 8) & 0xFFu];
                            val.z = tb[(w >> 16) & 0xFFu];
                            val.w = tb[w >> 24];
                        }
                    } else {
                        // cin is 8 modulo 16: a piece may straddle two diagonal blocks; the part of
                        // it that lies in this channel's block pn is the K range [pn k0, (pn + 1) k0)
                        const uint32_t mag = t == 0 ? 1u : (2u << t), neg = 256u - mag;
                        uint32_t wd[4] = {0, 0, 0, 0};
                        const int k_lo = pn * p.k0, k_hi = min(k_lo + p.k0, p.kf);
                        const int e_lo = max(0, k_lo - kbase), e_hi = min(16, k_hi - kbase);
                        for (int e = e_lo; e < e_hi; ++e) {
                            int wv = weight_at(wq, rowb, row, kbase + e - k_lo);
                            if (wv == -2) { invalid = 1; wv = 0; }
                            const uint32_t byte = wv == 0 ? 0u : (wv > 0 ? mag : neg);
                            wd[e >> 2] |= byte << (8 * (e & 3));
                        }
                        val = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                    }
                }
                *reinterpret_cast<uint4 *>(dst_blk + swz_offset((uint32_t)n, (uint32_t)j, cw)) = val;
            }
        }
        if (invalid) raise_status(PROM_ERR_BAD_WEIGHT);
        if (bad_consts && threadIdx.x == 0) raise_status(PROM_ERR_BAD_REQUANT);
    }
    if (threadIdx.x == 0) {
        hdr[0] = shmax; hdr[1] = fast ? 1 : 0; hdr[2] = bad_consts ? 1 : 0;
        hdr[3] = ((p.act_min & 0xFF) << 8) | (p.act_max & 0xFF);     // the clamp these operands were built for
    }
}

// MINB: CTAs of this kernel that share an SM (2 with 96 registers a thread, 3 with 64).
// MODE 0: static fixed-point requantisation.  MODE 1 and 2: the two passes of the dynamic layer
// (per-sample maxima of the dequantised output; output quantised with the per-sample scale).
// MODE 3: mode 0 plus a residual tensor added to the output with int8 saturation.
// MODE 4: mode 0 for the clamp [-128, 127] (the host launches it for exactly that clamp; the
// kernel the benchmark step runs stays free of the second fast epilogue).
template <int MINB, int MODE = 0>
__global__ void __launch_bounds__(kThreads, MINB)
tc_conv_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap ymap,
               const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte aligned base, by pointer arithmetic (a cast through an integer would make every
    // access below a generic one)
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int CH = MINB >= 3 ? 16 : 32;     // columns per tensor-memory load in the epilogue

    uint8_t *w_smem = smem + p.off_w;
    uint8_t *wbias_smem = smem + p.off_wbias;
    uint8_t *aconst_smem = smem + p.off_aconst;
    int *cmult = reinterpret_cast<int *>(smem + p.off_mult);        // mult per resident column
    int2 *cbs = reinterpret_cast<int2 *>(smem + p.off_bs);          // {bias, shift} per column
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + p.off_bars);
    // barrier slots: full[kMaxStages], empty[kMaxStages], tfull[kMaxBufs], tempty[kMaxBufs], drain
    const uint32_t bar_full = ptx::smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * kMaxStages;
    const uint32_t bar_tfull = bar_empty + 8 * kMaxStages;
    const uint32_t bar_tempty = bar_tfull + 8 * kMaxBufs;
    const uint32_t bar_drain = bar_tempty + 8 * kMaxBufs;
    const uint32_t bar_wload = bar_drain + 8;
    constexpr int kBarSlots = 2 * kMaxStages + 2 * kMaxBufs + 2;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + kBarSlots);
    volatile int *flags = reinterpret_cast<volatile int *>(bars + kBarSlots + 1);
    // flags[0] abort, flags[1] shmin, flags[2] shmax, flags[3] bad constants, flags[4] slow path

    const int g = blockIdx.x % p.groups;
    const int worker = blockIdx.x / p.groups;
    const int nworkers = gridDim.x / p.groups;
    const uint32_t cw = (uint32_t)p.cw;
    const uint32_t stage_bytes = 128u * cw;

    // Let the next kernel of the stream start its own prologue as soon as there is room for
    // it; it waits for this grid to finish before it touches activations.
    if (p.pdl_next) ptx::grid_dep_launch();

    // ---- prologue: nothing here depends on the previous kernel's output -------------
    if (threadIdx.x == 0 && p.image) {
        // prepared by tc_prep_kernel: one bulk copy, started before anything else
        ptx::mbar_init(bar_wload, 1);
        ptx::mbar_init_fence();
        ptx::mbar_expect_tx(bar_wload, p.image_bytes);
        ptx::bulk_load(smem_base + p.off_w, p.image + (size_t)g * p.image_stride, p.image_bytes,
                       bar_wload);
        flags[0] = 0;
    }
    if (warp == 0) {
        // the pipeline's barriers, one lane each
        if (lane < p.stages) {
            ptx::mbar_init(bar_full + 8 * lane, 1);
            ptx::mbar_init(bar_empty + 8 * lane, 1);
        } else if (lane >= 16 && lane < 16 + p.nbuf) {
            ptx::mbar_init(bar_tfull + 8 * (lane - 16), 1);
            ptx::mbar_init(bar_tempty + 8 * (lane - 16), kEpiWarps / kEpiGroups);
        } else if (lane == 31) {
            ptx::mbar_init(bar_drain, 1);
            ptx::tma_prefetch_desc(&xmap);
            if (p.store_2d) ptx::tma_prefetch_desc(&ymap);
        }
        ptx::mbar_init_fence();
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32((const void *)tmem_slot), (uint32_t)p.tmem_cols);
    const View vw = make_view(p, smem, bars);
    // With a prepared image, warp 0 (the producer) does not take part in the rest of the
    // prologue: it announces the barriers and goes straight to its loads, which need neither
    // weights nor constants, while the other nine warps wait for the image.
    const bool split = p.image != nullptr;
    if (split) {
        if (warp == 0) {
            __syncwarp();
            ptx::named_arrive(1, kThreads);
        } else {
            build_aconst(aconst_smem, (int)threadIdx.x - 32, kThreads - 32);
            ptx::named_sync(1, kThreads);
            // an image that never lands stops the whole CTA (the header is then never read)
            if (!wait_bar<true>(bar_wload, 0u, flags)) flags[0] = 1;
            ptx::fence_proxy_async_smem();
            ptx::tc_fence_before_sync();
            ptx::named_sync(2, kThreads - 32);
            ptx::tc_fence_after_sync();
        }
    } else {
        build_aconst(aconst_smem, (int)threadIdx.x, kThreads);
        build_image(p, g, vw);
        ptx::fence_proxy_async_smem();
        ptx::tc_fence_before_sync();
        __syncthreads();
        ptx::tc_fence_after_sync();
    }
    const bool solo = split && warp == 0;        // has not seen the image or tensor memory
    const bool no_image = !solo && split && flags[0] != 0;
    const uint32_t tmem_base = solo ? 0u : *tmem_slot;
    const int shmax = solo || no_image ? 0 : vw.hdr[0];
    const bool fast = solo || no_image ? false : vw.hdr[1] != 0;
    // operands prepared for another clamp than this launch's are refused like bad constants
    const bool wrong_clamp = !solo && split && !no_image &&
                             vw.hdr[3] != (((p.act_min & 0xFF) << 8) | (p.act_max & 0xFF));
    if (wrong_clamp && threadIdx.x == 32) raise_status(PROM_ERR_BAD_REQUANT);
    const bool bad_consts = solo ? false : (no_image || wrong_clamp || vw.hdr[2] != 0);
    if (bad_consts && threadIdx.x == 32) flags[0] = 1;      // stops the producer too

    // instruction descriptor: s8 x s8 -> s32, both K-major, M = 128, N = nt_pad
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.nt_pad >> 3) << 17) |
                           ((128u >> 4) << 24);
    const int loads_per_tile = p.share_x ? 1 : p.subs_per_cta * p.kc;
    // One load per unit (one K chunk, one subtile): the k-th unit uses stage k % stages, and the
    // epilogue, which learns of the MMA's completion anyway, frees that stage for the producer;
    // this spares the MMA thread one of its four tcgen05 instructions per unit.
    const bool epi_frees = p.kc == 1 && p.subs_per_cta == 1;

    if (!bad_consts) {
        // The two single-thread roles below run beside many busy epilogue warps, so every
        // instruction on their per-unit path costs tens of cycles: ring positions, phases and
        // descriptors are advanced by additions, never recomputed with divisions.
        if (warp == 0) {
            // ---- TMA producer ----------------------------------------------------
            if (lane == 0) {
                uint32_t s = 0, ph = 0, issued = 0;
                uint32_t dst = smem_base, bfull = bar_full, bempty = bar_empty;
                const int cx_end = p.share_x ? p.cw : p.kc * p.cw;
                bool ok = true;
                // Only this thread reads what the previous kernel wrote; everything else in the
                // CTA follows from its loads, so it alone waits for that kernel to finish.
                if (p.pdl) ptx::grid_dep_wait();
                for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers) {
                    const int mtx = p.reverse ? p.n_mtiles - 1 - mt : mt;
                    const int c_row = p.x3d ? mtx * p.box_r : mtx * p.tm;
                    int cx = 0;
                    for (int l = 0; l < loads_per_tile; ++l) {
                        if (!wait_bar(bempty, ph ^ 1u, flags)) { ok = false; break; }
                        ptx::mbar_expect_tx(bfull, p.tx_bytes);
                        if (p.x3d) ptx::tma_load_3d(dst, &xmap, cx, 0, c_row, bfull);
                        else ptx::tma_load_2d(dst, &xmap, cx, c_row, bfull);
                        ++issued;
                        cx += p.cw;
                        if (cx == cx_end) cx = 0;
                        ++s; dst += stage_bytes; bfull += 8; bempty += 8;
                        if (s == (uint32_t)p.stages) {
                            s = 0; ph ^= 1u; dst = smem_base; bfull = bar_full; bempty = bar_empty;
                        }
                    }
                }
                if (!ok) {
                    // let the copies already issued land before the CTA goes away
                    const uint32_t first = issued > (uint32_t)p.stages ? issued - p.stages : 0;
                    for (uint32_t j = first; j < issued; ++j) {
                        const unsigned long long t0 = ptx::globaltimer();
                        while (!ptx::mbar_try_wait(bar_full + 8 * (j % p.stages),
                                                   (j / p.stages) & 1u) &&
                               ptx::globaltimer() - t0 < kWaitLimitNs) {}
                    }
                }
            }
        } else if (warp == 1) {
            // ---- MMA issuer ---------------------------------------------------------
            if (lane == 0) {
                bool ok = true;
                // descriptors: constant high word, low word = (address >> 4) | LBO field
                const uint64_t d_cw = smem_desc(0u, cw), d_32 = smem_desc(0u, 32u);
                const uint32_t a_lo0 = smem_base >> 4, a_step = stage_bytes >> 4;
                const uint32_t b_lo0 = ptx::smem_u32(w_smem) >> 4, b_step = ((uint32_t)p.nt_pad * cw) >> 4;
                const uint32_t wb_lo0 = ptx::smem_u32(wbias_smem) >> 4, wb_step = ((uint32_t)p.nt_pad * 32u) >> 4;
                const uint64_t ac_desc = d_32 | (uint64_t)(ptx::smem_u32(aconst_smem) >> 4);
                const int ks_full = p.cw >> 5;
                uint32_t s = 0, ph = 0, a_lo = a_lo0, bfull = bar_full, bempty = bar_empty;
                uint32_t b = 0, tph = 0, d_tmem = tmem_base, btfull = bar_tfull, btempty = bar_tempty;
                if (epi_frees) {
                    // One load, one accumulator per tile: the shortest path this thread can take.
                    // It competes for issue slots with the epilogue warps, so what it executes
                    // per tile is what bounds the tile rate of streaming layers.
                    const uint64_t b_desc = d_cw | (uint64_t)b_lo0, wb_desc = d_32 | (uint64_t)wb_lo0;
                    const uint32_t a_end = a_lo0 + (uint32_t)p.stages * a_step;
                    const uint32_t bfull_end = bar_full + 8u * (uint32_t)p.stages;
                    const uint32_t btfull_end = bar_tfull + 8u * (uint32_t)p.nbuf;
                    const uint32_t tempty_off = bar_tempty - bar_tfull;
                    const int nks = p.ksteps_last;
                    int left = (p.n_mtiles - worker + nworkers - 1) / nworkers;
                    for (; left > 0 && ok; --left) {
                        if (!ptx::mbar_try_wait(btfull + tempty_off, tph ^ 1u) &&
                            !wait_bar(btfull + tempty_off, tph ^ 1u, flags)) { ok = false; break; }
                        if (!ptx::mbar_try_wait(bfull, ph) && !wait_bar(bfull, ph, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        ptx::mma_i8(d_tmem, d_cw | (uint64_t)a_lo, b_desc, idesc, 0u);
                        for (int ks = 1; ks < nks; ++ks)
                            ptx::mma_i8(d_tmem, d_cw | (uint64_t)(a_lo + 2 * ks), b_desc + 2 * ks, idesc, 1u);
                        if (fast) ptx::mma_i8(d_tmem, ac_desc, wb_desc, idesc, 1u);
                        ptx::mma_commit(btfull);
                        a_lo += a_step; bfull += 8;
                        if (bfull == bfull_end) { ph ^= 1u; a_lo = a_lo0; bfull = bar_full; }
                        d_tmem += p.nt_pad; btfull += 8;
                        if (btfull == btfull_end) { tph ^= 1u; d_tmem = tmem_base; btfull = bar_tfull; }
                    }
                    (void)a_end;
                } else
                for (int mt = worker; mt < p.n_mtiles && ok; mt += nworkers) {
                    uint32_t b_lo = b_lo0, wb_lo = wb_lo0;
                    for (int ls = 0; ls < p.subs_per_cta && ok; ++ls) {
                        if (!wait_bar(btempty, tph ^ 1u, flags)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        uint32_t acc = 0;
                        for (int chunk = 0; chunk < p.kc; ++chunk) {
                            if (!p.share_x || ls == 0) {
                                if (!wait_bar(bfull, ph, flags)) { ok = false; break; }
                                ptx::tc_fence_after_sync();
                            }
                            const int nks = (chunk == p.kc - 1) ? p.ksteps_last : ks_full;
                            for (int ks = 0; ks < nks; ++ks) {
                                ptx::mma_i8(d_tmem, d_cw | (uint64_t)(a_lo + 2 * ks),
                                            d_cw | (uint64_t)(b_lo + 2 * ks), idesc, acc);
                                acc = 1;
                            }
                            b_lo += b_step;
                            if (!p.share_x || ls == p.subs_per_cta - 1) {
                                if (!epi_frees) ptx::mma_commit(bempty);
                                ++s; a_lo += a_step; bfull += 8; bempty += 8;
                                if (s == (uint32_t)p.stages) {
                                    s = 0; ph ^= 1u; a_lo = a_lo0; bfull = bar_full; bempty = bar_empty;
                                }
                            }
                        }
                        if (!ok) break;
                        if (fast) ptx::mma_i8(d_tmem, ac_desc, d_32 | (uint64_t)wb_lo, idesc, 1u);
                        wb_lo += wb_step;
                        ptx::mma_commit(btfull);
                        ++b; d_tmem += p.nt_pad; btfull += 8; btempty += 8;
                        if (b == (uint32_t)p.nbuf) {
                            b = 0; tph ^= 1u; d_tmem = tmem_base; btfull = bar_tfull; btempty = bar_tempty;
                        }
                    }
                }
                // every MMA has finished before tensor memory is released
                ptx::mma_commit(bar_drain);
                const unsigned long long t0 = ptx::globaltimer();
                while (!ptx::mbar_try_wait(bar_drain, 0) && ptx::globaltimer() - t0 < kWaitLimitNs) {}
            }
        } else {
            // ---- epilogue ---------------------------------------------------------------
            // Everything a warp does per unit besides the arithmetic is a chain of dependent
            // scalar instructions issued among many busy warps, tens of cycles each: positions,
            // addresses and phases advance by additions, and a full slab takes the short path.
            const int q = warp & 3;                     // TMEM lane quarter of this warp
            if constexpr (MODE == 3) {
                // the residual was written two kernels back: complete once the previous one is
                if (p.pdl) ptx::grid_dep_wait();
            }
            // Unit u goes to group u % 2 and accumulator u % nbuf; nbuf is even, so a group meets
            // each of its accumulators in cyclic order and never waits on a barrier that is more
            // than one phase away.
            const int grp = (warp - 2) >> 2;
            uint8_t *slab = smem + p.off_out + (size_t)(warp - 2) * 32 * p.nt;
            uint8_t *my_row = slab + lane * p.nt;
            const uint32_t slab_addr = ptx::smem_u32(slab);
            const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
            const int subs = p.subs_per_cta;
            const int m_rows = (int)p.m_rows;           // the planner keeps rows below 2^31
            bool ok = true;
            int mt0 = worker, ls = grp;                 // this group's first unit
            while (ls >= subs) { ls -= subs; mt0 += nworkers; }
            // the next unit of the group is two further on: with one subtile per CTA that is two
            // tiles on, otherwise two subtiles on and at most one step to the next tile
            const int dls = subs == 1 ? 0 : kEpiGroups;
            // (in a sequence every second layer walks its tiles backwards: what the layer before
            // wrote last, and is still in L2, is read first)
            const int dir = p.reverse ? -1 : 1;
            const int drow = subs == 1 ? dir * kEpiGroups * nworkers * p.tm : 0, drow_wrap = dir * nworkers * p.tm;
            const bool whole_tile = p.tm - q * 32 >= 32;     // a tile gives this warp 32 rows
            int row0 = (p.reverse ? p.n_mtiles - 1 - mt0 : mt0) * p.tm + q * 32;   // first row of this warp's slab
            const unsigned row_span = (unsigned)(p.n_mtiles * p.tm);
            const uint32_t slab_bytes = 32u * (uint32_t)p.nf;
            int col = (g + ls * p.groups) * p.nt;       // first column of the subtile
            const int dcol = dls * p.groups * p.nt;
            const bool store_2d = p.store_2d != 0;
            // accumulators of this group: grp alone (two in the ring) or grp and grp + 2 (four)
            const uint32_t btoggle = p.nbuf == 4 ? 2u : 0u;
            uint32_t b = (uint32_t)grp, tph = 0;
            uint32_t st = (uint32_t)grp % (uint32_t)p.stages;    // stage of this group's unit (epi_frees)
            while ((unsigned)(row0 - q * 32) < row_span && ok) {
                // The residual (mode 3): the bytes that sit where this slab goes in Y, in 8-byte
                // granules across the warp.  The first kResHeld granules of a lane are requested
                // before the wait for the accumulator, so that their latency hides behind it.
                constexpr int kResHeld = 6;
                uint2 res_held[kResHeld];
                int res_total = 0, res_g8 = 1;
                const int8_t *res_p = nullptr;
                if constexpr (MODE == 3) {
                    int rows_valid = p.tm - q * 32;
                    if (m_rows - row0 < rows_valid) rows_valid = m_rows - row0;
                    if (rows_valid > 32) rows_valid = 32;
                    res_g8 = p.nt >> 3;
                    res_total = rows_valid * res_g8;
                    res_p = p.res + (long long)row0 * p.nf + col;
#pragma unroll
                    for (int j = 0; j < kResHeld; ++j) {
                        const int i = lane + 32 * j;
                        res_held[j] = make_uint2(0u, 0u);
                        if (i < res_total) {
                            const int r = i / res_g8, c = (i - r * res_g8) * 8;
                            res_held[j] = __ldcg(reinterpret_cast<const uint2 *>(res_p + (long long)r * p.nf + c));
                        }
                    }
                    // the rest is asked into L2
                    for (int i = lane + 32 * kResHeld; i < res_total; i += 32) {
                        const int r = i / res_g8, c = (i - r * res_g8) * 8;
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(res_p + (long long)r * p.nf + c));
                    }
                }
                if (!wait_bar<true>(bar_tfull + 8 * b, tph, flags)) { ok = false; break; }
                if (epi_frees) {
                    if (q == 0 && lane == 0) ptx::mbar_arrive(bar_empty + 8 * st);
                    st += kEpiGroups;
                    if (st >= (uint32_t)p.stages) st -= p.stages;
                }
                ptx::tc_fence_after_sync();
                // the previous bulk store must have read the slab before it is rewritten
                ptx::bulk_wait_read0();
                __syncwarp();
                const uint32_t taddr = t_lane + b * p.nt_pad;
                const int *cms = cmult + ls * p.nt_pad;
                const uint32_t bar_rel = bar_tempty + 8 * b;
                if constexpr (MODE == 0 || MODE == 3 || MODE == 4) {
                    // the fast epilogue's clamp: [0, 127] in mode 0, [-128, 127] in mode 4, either in mode 3
                    const bool full_range = MODE == 4 || (MODE == 3 && p.act_min < 0);
                    if (fast && !full_range) {
                        // the widths of the network's large layers get straight-line code
                        if (CH == 32 && p.nt == 96) epi_fast_fixed<96>(taddr, cms, shmax, my_row, bar_rel);
                        else if (CH == 32 && p.nt == 64) epi_fast_fixed<64>(taddr, cms, shmax, my_row, bar_rel);
                        else if (CH == 32 && p.nt == 48) epi_fast_fixed<48>(taddr, cms, shmax, my_row, bar_rel);
                        else if (CH == 32 && p.nt == 32) epi_fast_fixed<32>(taddr, cms, shmax, my_row, bar_rel);
                        else if (CH == 32 && p.nt == 80) epi_fast_fixed<80>(taddr, cms, shmax, my_row, bar_rel);
                        else epi_fast_subtile<CH>(p, taddr, cms, shmax, my_row, bar_rel);
                    }
                    else if (fast) epi_fast_subtile<CH, true>(p, taddr, cms, shmax, my_row, bar_rel);
                    else epi_exact_subtile<CH>(p.nt, p.act_min, p.act_max, taddr, cms, cbs + ls * p.nt_pad, my_row, bar_rel);
                    if constexpr (MODE == 3) {
                        __syncwarp();
                        auto add_to_slab = [&](int i, uint2 rv) {
                            const int r = i / res_g8, c = (i - r * res_g8) * 8;
                            uint2 *sp = reinterpret_cast<uint2 *>(slab + r * p.nt + c);
                            uint2 sv = *sp;
                            sv.x = __vaddss4(sv.x, rv.x);
                            sv.y = __vaddss4(sv.y, rv.y);
                            *sp = sv;
                        };
#pragma unroll
                        for (int j = 0; j < kResHeld; ++j)
                            if (lane + 32 * j < res_total) add_to_slab(lane + 32 * j, res_held[j]);
                        for (int i = lane + 32 * kResHeld; i < res_total; i += 32) {
                            const int r = i / res_g8, c = (i - r * res_g8) * 8;
                            add_to_slab(i, __ldcg(reinterpret_cast<const uint2 *>(res_p + (long long)r * p.nf + c)));
                        }
                    }
                } else {
                    // this thread's row and its sample (rows past the end borrow the last sample's
                    // factors; they are neither counted nor stored)
                    const int row = row0 + lane;
                    int smp = row / p.rows_per_sample;
                    smp = smp < p.batch ? smp : p.batch - 1;
                    const float gx = __ldg(p.gamma_x + smp);
                    const float dq = __fdiv_rn(gx < 1e-5f ? 1e-5f : gx, 127.0f);
                    if constexpr (MODE == 1) {
                        float mx = epi_dyn_subtile<CH, false>(p, taddr, cms, dq, 0.0f, nullptr, bar_rel);
                        if (row >= m_rows || p.tm - q * 32 <= lane) mx = 0.0f;
                        // one atomic per warp when its 32 rows share a sample, else one per row
                        const int smp0 = __shfl_sync(0xFFFFFFFFu, smp, 0);
                        if (__all_sync(0xFFFFFFFFu, smp == smp0)) {
#pragma unroll
                            for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, d));
                            if (lane == 0 && mx > 0.0f)
                                atomicMax(reinterpret_cast<unsigned int *>(p.gamma_y + smp0), __float_as_uint(mx));
                        } else if (mx > 0.0f) {
                            atomicMax(reinterpret_cast<unsigned int *>(p.gamma_y + smp), __float_as_uint(mx));
                        }
                        // nothing is stored in this pass
                        ls += dls; row0 += drow; col += dcol;
                        if (ls >= subs) { ls -= subs; row0 += drow_wrap; col -= p.nf; }
                        b ^= btoggle;
                        if (b < (uint32_t)kEpiGroups) tph ^= 1u;
                        continue;
                    } else {
                        epi_dyn_subtile<CH, true>(p, taddr, cms, dq, __ldg(p.scale_y + smp), my_row, bar_rel);
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (whole_tile && row0 + 32 <= m_rows) {
                    // a whole slab: one copy
                    if (lane == 0) {
                        if (store_2d) ptx::tma_store_2d(&ymap, col, row0, slab_addr);
                        else ptx::bulk_store(p.y + (long long)row0 * p.nf, slab_addr, slab_bytes);
                        ptx::bulk_commit();
                    }
                } else {
                    // a short tile or the end of the matrix
                    int rows_valid = p.tm - q * 32;
                    if (m_rows - row0 < rows_valid) rows_valid = m_rows - row0;
                    if (rows_valid > 32) rows_valid = 32;
                    store_partial_slab(p.y + (long long)row0 * p.nf, slab, rows_valid, p.nf, p.nt, col,
                                       store_2d, lane);
                }
                // this group's next unit and accumulator
                ls += dls; row0 += drow; col += dcol;
                if (ls >= subs) { ls -= subs; row0 += drow_wrap; col -= p.nf; }
                b ^= btoggle;
                if (b < (uint32_t)kEpiGroups) tph ^= 1u;
            }
            // the stores complete with the grid; only their reads of the slab must be over
            ptx::bulk_wait_read0();
        }
    }

    // ---- teardown -------------------------------------------------------------------------
    // A CTA whose roles were skipped has not waited for the previous kernel yet; it must, or
    // this grid could end (and release the next one) while that kernel is still running.
    if (p.pdl && bad_consts && threadIdx.x == 0) ptx::grid_dep_wait();
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}


// Test aid: one warp waits, with the library's bounded wait and a limit of `limit_ns`, on an
// mbarrier phase that nothing will ever complete.  The wait gives up by itself, records
// PROM_ERR_TIMEOUT in the device status word and the kernel returns normally.
__global__ void __launch_bounds__(32, 1) wait_timeout_probe_kernel(unsigned long long limit_ns, int *gave_up)
{
    __shared__ uint64_t bar;
    __shared__ int flag;
    if (threadIdx.x == 0) {
        flag = 0;
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        ptx::mbar_init_fence();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool done = wait_bar(ptx::smem_u32(&bar), 0u, &flag, limit_ns);
        if (gave_up) *gave_up = done ? 0 : 1;
    }
}

// Prepared operands for a whole layer sequence in one launch: CTA b builds the image of
// (layer, channel group) = the b-th entry of the table and writes it to that layer's
// `image` buffer.  Shared-memory offsets are those of the layer's convolution launch.
constexpr int kMaxPrepLayers = 48;
struct PrepTable {
    int n;
    int first[kMaxPrepLayers + 1];     // first CTA of each layer; first[n] = grid size
    Params layer[kMaxPrepLayers];
};

__global__ void __launch_bounds__(kThreads, 1)
tc_prep_kernel(const __grid_constant__ PrepTable t)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    int l = 0;
    while (l + 1 < t.n && (int)blockIdx.x >= t.first[l + 1]) ++l;
    const Params &p = t.layer[l];
    const int g = (int)blockIdx.x - t.first[l];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + p.off_bars);
    const View vw = make_view(p, smem, bars);
    build_image(p, g, vw);
    ptx::fence_proxy_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
        ptx::bulk_store(p.image + (size_t)g * p.image_stride, vw.smem_base + p.off_w, p.image_bytes);
        ptx::bulk_commit();
        ptx::bulk_wait_all();
    }
}

}}  // namespace prom::tc
