/*
 * CPU oracle for the ternary pointwise-convolution path of PROM.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain-loop statement of
 * what the path computes.  It shares no code with the CUDA library and must
 * never be called by it; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may use it.  Nothing here is blocked, fused, vectorised by
 * hand or reordered: every function is the definition written out so that it
 * can be checked against the paper by eye.  Rows are split over OpenMP
 * threads and that is the only parallelism.
 *
 * Notation (paper, Section 3.1): X is the int8 activation matrix [M, Cin]
 * (NHWC pixels flattened to rows), W-hat is the ternary weight matrix
 * [Cout, Cin] with entries in {-1, 0, +1}, and the layer output before
 * scaling is  acc[m][o] = sum_k X[m][k] * W-hat[o][k]   (Section 3.1,
 * inference form: the input is convolved directly with the ternary weights
 * and scaled afterwards; Figure 12, inference branch).
 *
 * The paper scales the integer result by the per-output-channel factor alpha
 * and the activation scale in floating point (Figure 12).  The build's
 * contract replaces that by a static fixed-point requantisation per output
 * channel; the reading taken is
 *     t = acc + bias[o]
 *     p = t * mult[o]                    (exact, 64-bit)
 *     q = sign(p) * floor((|p| + 2^(s-1)) / 2^s),   s = 31 + shift[o]
 *     y = min(act_max, max(act_min, q))
 * i.e. one rounding of the exact product, ties away from zero.
 *
 * Pins (tests/test_oracle_*.py): brute force over all ternary matrices on
 * tiny shapes against Python big integers, the add/sub identity of Section 2,
 * all-zero and one-hot weights, an int64 library matmul, exact rational
 * arithmetic for the requantiser, hand-built ties, and byte tables for the
 * 2-bit codes.  No function in this file is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- threads ----------------------------------------------------------- */

int prom_ref_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void prom_ref_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---- 2-bit storage of ternary weights ---------------------------------- */
/*
 * The paper stores a ternary weight in 2 bits (Section 4, "Memory"; the
 * storage column of Table 1 is consistent with it) but prints no format.
 * Reading taken: the 2-bit two's-complement code of the value
 *     0 -> 00,  +1 -> 01,  -1 -> 11,  (10 is never produced and is invalid)
 * four codes per byte along Cin, weight k of output channel o in byte
 * o*ceil(Cin/4) + k/4 at bits 2*(k%4) and 2*(k%4)+1; a row is padded to a
 * whole byte with code 00.
 */

size_t prom_ref_packed_bytes(int cout, int cin)
{
    return (size_t)cout * (size_t)((cin + 3) / 4);
}

/* Returns the number of entries of w that are not in {-1,0,+1}; packed is
 * written only when that number is 0. */
long prom_ref_pack(const int8_t *w, int cout, int cin, uint8_t *packed)
{
    long bad = 0;
    for (long i = 0; i < (long)cout * cin; ++i)
        if (w[i] < -1 || w[i] > 1) ++bad;
    if (bad) return bad;
    int rowb = (cin + 3) / 4;
    memset(packed, 0, (size_t)cout * rowb);
    for (int o = 0; o < cout; ++o)
        for (int k = 0; k < cin; ++k) {
            int v = w[(long)o * cin + k];
            unsigned code = (v == 0) ? 0u : (v == 1 ? 1u : 3u);
            packed[(long)o * rowb + k / 4] |= (uint8_t)(code << (2 * (k % 4)));
        }
    return 0;
}

/* Returns the number of invalid codes (10) met, padding codes that are not 00
 * included; w is written in any case (an invalid code decodes to 0). */
long prom_ref_unpack(const uint8_t *packed, int cout, int cin, int8_t *w)
{
    long bad = 0;
    int rowb = (cin + 3) / 4;
    for (int o = 0; o < cout; ++o)
        for (int k = 0; k < rowb * 4; ++k) {
            unsigned code = (packed[(long)o * rowb + k / 4] >> (2 * (k % 4))) & 3u;
            int v = 0;
            if (code == 1u) v = 1;
            else if (code == 3u) v = -1;
            else if (code == 2u) ++bad;
            if (k < cin) w[(long)o * cin + k] = (int8_t)v;
            else if (code != 0u && code != 2u) ++bad;
        }
    return bad;
}

/* ---- requantisation ----------------------------------------------------- */

int32_t prom_ref_requant_scalar(int32_t t, int32_t mult, int shift,
                                int act_min, int act_max)
{
    int64_t p = (int64_t)t * (int64_t)mult;
    int s = 31 + shift;
    int64_t half = (int64_t)1 << (s - 1);
    int64_t a = p < 0 ? -p : p;
    int64_t q = (a + half) >> s;          /* a + half >= 0: the shift is a floor */
    if (p < 0) q = -q;
    if (q < act_min) q = act_min;
    if (q > act_max) q = act_max;
    return (int32_t)q;
}

void prom_ref_requant(const int32_t *t, long n, int32_t mult, int shift,
                      int act_min, int act_max, int32_t *q)
{
    for (long i = 0; i < n; ++i)
        q[i] = prom_ref_requant_scalar(t[i], mult, shift, act_min, act_max);
}

/* ---- the convolution, multiply form ------------------------------------- */
/*
 * x: [m, cin] int8, rows `x_row_stride` bytes apart (cin when dense);
 * w: [cout, cin] int8 with ternary values; acc (optional): [m, cout] int32;
 * y (optional): [m, cout] int8.  bias/mult/shift: [cout].
 */
void prom_ref_conv_mul(const int8_t *x, long m, int cin, long x_row_stride,
                       const int8_t *w, int cout,
                       const int32_t *bias, const int32_t *mult, const int8_t *shift,
                       int act_min, int act_max,
                       int32_t *acc_out, int8_t *y)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < m; ++r) {
        const int8_t *xr = x + r * x_row_stride;
        for (int o = 0; o < cout; ++o) {
            const int8_t *wo = w + (long)o * cin;
            int32_t acc = 0;
            for (int k = 0; k < cin; ++k)
                acc += (int32_t)xr[k] * (int32_t)wo[k];
            if (acc_out) acc_out[r * cout + o] = acc;
            if (y) {
                int32_t t = acc + bias[o];
                y[r * cout + o] = (int8_t)prom_ref_requant_scalar(
                    t, mult[o], shift[o], act_min, act_max);
            }
        }
    }
}

/* ---- the convolution, add/subtract form (Section 2: a product with a
 * ternary weight reduces to a sum of input channels) ---------------------- */
void prom_ref_conv_addsub(const int8_t *x, long m, int cin, long x_row_stride,
                          const int8_t *w, int cout,
                          const int32_t *bias, const int32_t *mult, const int8_t *shift,
                          int act_min, int act_max,
                          int32_t *acc_out, int8_t *y)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < m; ++r) {
        const int8_t *xr = x + r * x_row_stride;
        for (int o = 0; o < cout; ++o) {
            const int8_t *wo = w + (long)o * cin;
            int32_t plus = 0, minus = 0;
            for (int k = 0; k < cin; ++k) {
                if (wo[k] == 1) plus += xr[k];
                else if (wo[k] == -1) minus += xr[k];
                /* a zero weight needs no work */
            }
            int32_t acc = plus - minus;
            if (acc_out) acc_out[r * cout + o] = acc;
            if (y) {
                int32_t t = acc + bias[o];
                y[r * cout + o] = (int8_t)prom_ref_requant_scalar(
                    t, mult[o], shift[o], act_min, act_max);
            }
        }
    }
}

/* ---- spatial subsampling: the depthwise stand-in ------------------------ */
/*
 * The depthwise 3x3 convolution between expand and project (Section 2) is
 * modelled as the identity on values plus its spatial stride: output pixel
 * (i, j) of a stride-2 site is input pixel (2i, 2j).  in: [batch, h, w, c],
 * out: [batch, h/stride, w/stride, c].
 */
void prom_ref_subsample(const int8_t *in, int batch, int h, int w, int c,
                        int stride, int8_t *out)
{
    int ho = h / stride, wo = w / stride;
    for (int b = 0; b < batch; ++b)
        for (int i = 0; i < ho; ++i)
            for (int j = 0; j < wo; ++j)
                memcpy(out + (((long)b * ho + i) * wo + j) * c,
                       in + (((long)b * h + i * stride) * w + j * stride) * c,
                       (size_t)c);
}

/*
 * The skip connection of an inverted-residual block (Section 2): when a
 * block keeps the shape of its input, the input is added to the output of
 * the project convolution.  Both tensors are int8 on one scale here (the
 * paper adds in floating point after dequantising), so the sum is the
 * integer sum clamped to the int8 range.
 */
void prom_ref_residual_add(const int8_t *y_layer, const int8_t *block_in, long n,
                           int8_t *out)
{
    for (long i = 0; i < n; ++i) {
        int s = (int)y_layer[i] + (int)block_in[i];
        if (s < -128) s = -128;
        if (s > 127) s = 127;
        out[i] = (int8_t)s;
    }
}

/* ---- the layer sequence -------------------------------------------------- */
/*
 * Runs n pointwise layers back to back: the output of layer i is the input
 * of layer i+1; a layer with in_stride 2 reads pixel (2i, 2j) of its input
 * for its own pixel (i, j), in place of materialising the subsampled tensor.
 * cin/cout/in_stride: [n]; w: n pointers to ternary [cout, cin];
 * bias/mult/shift: n pointers to [cout] arrays.  Returns 0, or -1 when the
 * shapes do not chain or a buffer cannot be had.
 */
int prom_ref_layer_seq(int n, const int *cin, const int *cout, const int *in_stride,
                       const int8_t *const *w,
                       const int32_t *const *bias, const int32_t *const *mult,
                       const int8_t *const *shift,
                       int act_min, int act_max,
                       const int8_t *x0, int batch, int h0, int w0,
                       int8_t *y_out)
{
    int h = h0, wd = w0;
    const int8_t *cur = x0;
    int8_t *own = NULL;
    for (int l = 0; l < n; ++l) {
        if (l > 0 && cin[l] != cout[l - 1]) { free(own); return -1; }
        int st = in_stride[l];
        if (st != 1 && st != 2) { free(own); return -1; }
        if (h % st || wd % st) { free(own); return -1; }
        int ho = h / st, wo = wd / st;
        long m = (long)batch * ho * wo;
        int8_t *dst = (l == n - 1) ? y_out : (int8_t *)malloc((size_t)m * cout[l]);
        if (!dst) { free(own); return -1; }
#pragma omp parallel for schedule(static)
        for (long r = 0; r < m; ++r) {
            long b = r / ((long)ho * wo);
            long ij = r % ((long)ho * wo);
            long i = ij / wo, j = ij % wo;
            const int8_t *xr = cur + (((long)b * h + i * st) * wd + j * st) * cin[l];
            for (int o = 0; o < cout[l]; ++o) {
                const int8_t *wl = w[l] + (long)o * cin[l];
                int32_t acc = 0;
                for (int k = 0; k < cin[l]; ++k)
                    acc += (int32_t)xr[k] * (int32_t)wl[k];
                dst[r * cout[l] + o] = (int8_t)prom_ref_requant_scalar(
                    acc + bias[l][o], mult[l][o], shift[l][o], act_min, act_max);
            }
        }
        free(own);
        own = (l == n - 1) ? NULL : dst;
        cur = dst;
        h = ho; wd = wo;
    }
    return 0;
}

/* ---- ternary absmean quantiser (the step before the path) ---------------- */
/*
 * Paper, Section 3.1, Eq. 1-3, and the pointwise branch of the quantiser in
 * Figure 10: per output channel i
 *     alpha_i = mean_j |W[i][j]|
 *     W-hat[i][j] = max(-1, min(1, round(W[i][j] / alpha_i)))
 * Readings taken where the paper is at odds with itself: the division guard
 * is the figure's (the mean is clamped from below by eps = 1e-5) rather than
 * Eq. 3's (eps added to the mean); `round` is the framework's, i.e. ties go
 * to the even integer, so a ratio of exactly 0.5 gives 0 and 1.5 gives 2 -> 1.
 * The paper fixes no summation order; mean and ratio are taken in binary64 so
 * that the order cannot matter at the precision of the float32 inputs.
 * w: [cout][cin] float32; q: [cout][cin] in {-1,0,+1}; alpha: [cout].
 */
void prom_ref_quantize_ternary(const float *w, int cout, int cin, double eps,
                               int8_t *q, double *alpha)
{
    for (int i = 0; i < cout; ++i) {
        double sum = 0.0;
        for (int j = 0; j < cin; ++j) sum += fabs((double)w[(long)i * cin + j]);
        double mean = sum / (double)cin;
        alpha[i] = mean;
        double scale = 1.0 / (mean < eps ? eps : mean);
        for (int j = 0; j < cin; ++j) {
            double r = nearbyint((double)w[(long)i * cin + j] * scale);   /* ties to even */
            if (r > 1.0) r = 1.0;
            if (r < -1.0) r = -1.0;
            q[(long)i * cin + j] = (int8_t)r;
        }
    }
}

/*
 * The fixed-point pair that stands for a real per-channel scale (the paper
 * scales by alpha and the activation scales in floating point, Figure 12; the
 * build's contract wants mult in [2^30, 2^31) and a right shift): the shift is
 * the one that puts scale * 2^(31+shift) into [2^30, 2^31], and mult is that
 * number rounded to nearest (a result of 2^31 is renormalised to 2^30 with the
 * shift one smaller).  Returns 0, or -1 when scale is not positive or the
 * shift would leave [0, 31].
 */
int prom_ref_requant_from_scale(double scale, int32_t *mult, int *shift)
{
    if (!(scale > 0.0) || isinf(scale)) return -1;
    int sh = 0;
    double v = scale * 2147483648.0;            /* scale * 2^31 */
    while (v >= 2147483648.0) { v /= 2.0; --sh; }
    while (v < 1073741824.0) { v *= 2.0; ++sh; if (sh > 64) return -1; }
    double m = floor(v + 0.5);
    if (m >= 2147483648.0) { m = 1073741824.0; --sh; }
    if (sh < 0 || sh > 31) return -1;
    *mult = (int32_t)m;
    *shift = sh;
    return 0;
}

/*
 * Per-sample absmax quantisation of activations to 8 bits: paper, Section 3.1
 * ("Activations", the two equations after Eq. 5, numbered 6 and 7 here) and the
 * activation figure of the pseudocode appendix.  For sample i over all its
 * channels and pixels
 *     gamma_i = max |X[i][...]|
 *     scale_i = 127 / max(gamma_i, eps)
 *     X-hat[i][...] = max(-128, min(127, round(X[i][...] * scale_i)))
 * Readings: the text's second equation divides by (gamma_i + eps) and leaves the
 * 127 out, which would map every value into [-1, 1] before rounding; the figure
 * multiplies by 127 / clamp(gamma_i, eps), and that is what is computed here.
 * `round` is the framework's (ties to even).  The rounding decision is taken in
 * binary32, the precision the paper's framework computes in: the quotient and
 * the product are each one correctly rounded binary32 operation (volatile keeps
 * the compiler from carrying extra precision or fusing them), so a second
 * implementation that uses the same two operations must agree bit for bit.
 * x: [batch][per_sample] float32 (any layout inside a sample: the maximum does
 * not care); q: same shape, int8; gamma, scale: [batch].
 */
void prom_ref_quantize_act_absmax(const float *x, int batch, long per_sample, float eps,
                                  int8_t *q, float *gamma, float *scale)
{
    for (int i = 0; i < batch; ++i) {
        const float *xi = x + (long)i * per_sample;
        float mx = 0.0f;
        for (long j = 0; j < per_sample; ++j) {
            float a = fabsf(xi[j]);
            if (a > mx) mx = a;
        }
        gamma[i] = mx;
        volatile float den = mx < eps ? eps : mx;
        volatile float sc = 127.0f / den;
        scale[i] = sc;
        for (long j = 0; j < per_sample; ++j) {
            volatile float prod = xi[j] * sc;
            float r = nearbyintf(prod);                     /* ties to even */
            if (r > 127.0f) r = 127.0f;
            if (r < -128.0f) r = -128.0f;
            q[(long)i * per_sample + j] = (int8_t)r;
        }
    }
}

/*
 * A pointwise layer in the paper's own inference dataflow (pseudocode appendix, the
 * inference branch of the quantised convolution module, followed by the activation
 * quantiser of the next module; Section 3.1, Eq. 6-7):
 *     acc[m][o] = sum_k X-hat[m][k] * W-hat[o][k]                  (integers, exact)
 *     y[m][o]   = acc[m][o] * alpha[o] * dq[b(m)]                  (dequantise)
 *     gamma_y[b] = max_{m in sample b, o} |y[m][o]|
 *     q[m][o]   = clip(round(y[m][o] * 127 / max(gamma_y[b], eps)), -128, 127)
 * where X-hat was produced by the activation quantiser with per-sample maximum gamma_x[b],
 * dq[b] = max(gamma_x[b], eps) / 127 is the reciprocal of its scale, and sample b owns rows
 * [b * rows_per_sample, (b + 1) * rows_per_sample).
 * Readings: the module divides by the weight scale (1 / alpha) and by the activation scale;
 * here the result is multiplied by alpha and by dq, the same real numbers, so that each step
 * is one binary32 rounding of a product; BatchNorm and PReLU, separate float modules in the
 * paper, are not part of this function.  All float steps are single correctly rounded
 * binary32 operations in the order written (volatile stops the compiler from fusing or
 * widening), so that a second implementation with the same steps agrees bit for bit.
 * y (optional): [m][cout] float32; q: [m][cout] int8; gamma_y, scale_y: [batch].
 */
void prom_ref_conv_dyn(const int8_t *x, int batch, long rows_per_sample, int cin,
                       const int8_t *w, int cout, const float *alpha, const float *gamma_x,
                       float eps, float *y_out, int8_t *q, float *gamma_y, float *scale_y)
{
    long m = (long)batch * rows_per_sample;
    float *y = (float *)malloc(sizeof(float) * (size_t)m * (size_t)cout);
    for (int b = 0; b < batch; ++b) {
        volatile float gx = gamma_x[b] < eps ? eps : gamma_x[b];
        volatile float dq = gx / 127.0f;
        float mx = 0.0f;
        for (long r = b * rows_per_sample; r < (b + 1) * rows_per_sample; ++r) {
            for (int o = 0; o < cout; ++o) {
                int32_t acc = 0;
                for (int k = 0; k < cin; ++k)
                    acc += (int32_t)x[r * cin + k] * (int32_t)w[(long)o * cin + k];
                volatile float t = (float)acc;          /* exact: |acc| < 2^24 */
                volatile float u = t * alpha[o];
                volatile float v = u * dq;
                y[r * cout + o] = v;
                float a = fabsf(v);
                if (a > mx) mx = a;
            }
        }
        gamma_y[b] = mx;
        volatile float den = mx < eps ? eps : mx;
        volatile float sc = 127.0f / den;
        scale_y[b] = sc;
        for (long r = b * rows_per_sample; r < (b + 1) * rows_per_sample; ++r) {
            for (int o = 0; o < cout; ++o) {
                volatile float prod = y[r * cout + o] * sc;
                float rr = nearbyintf(prod);
                if (rr > 127.0f) rr = 127.0f;
                if (rr < -128.0f) rr = -128.0f;
                q[r * cout + o] = (int8_t)rr;
            }
        }
    }
    if (y_out) memcpy(y_out, y, sizeof(float) * (size_t)m * (size_t)cout);
    free(y);
}

/*
 * The int8 depthwise 3x3 convolution that sits between the expand and the project
 * convolution of a block (paper, Section 2: depthwise-separable block; Section 3.1: its
 * weights are 8-bit, quantised per channel by absmax, Eq. 4-5).  Each channel is filtered
 * on its own, with one pixel of zero padding and the block's stride:
 *     acc[b][i][j][c] = sum_{di,dj in 0..2} x[b][i*s + di - 1][j*s + dj - 1][c] * w[c][di][dj]
 * (pixels outside the image count as 0), output size ho = (h - 1) / s + 1, wo likewise,
 * followed by the same fixed-point requantisation per channel as the pointwise layers
 * (bias, mult, shift, clamp).  The padding and the size are the reference network's
 * (3x3, padding 1), which the paper takes over unchanged; it prints neither.
 * x: [batch][h][w][c] int8; w: [c][3][3] int8; y: [batch][ho][wo][c] int8;
 * acc_out (optional): same shape as y, int32.
 */
void prom_ref_dw3x3(const int8_t *x, int batch, int h, int w, int c, int stride,
                    const int8_t *wt, const int32_t *bias, const int32_t *mult,
                    const int8_t *shift, int act_min, int act_max, int32_t *acc_out, int8_t *y)
{
    int ho = (h - 1) / stride + 1, wo = (w - 1) / stride + 1;
#pragma omp parallel for schedule(static)
    for (long bi = 0; bi < (long)batch * ho; ++bi) {
        int b = (int)(bi / ho), i = (int)(bi % ho);
        for (int j = 0; j < wo; ++j) {
            for (int ch = 0; ch < c; ++ch) {
                int32_t acc = 0;
                for (int di = 0; di < 3; ++di) {
                    for (int dj = 0; dj < 3; ++dj) {
                        int ii = i * stride + di - 1, jj = j * stride + dj - 1;
                        if (ii < 0 || ii >= h || jj < 0 || jj >= w) continue;
                        acc += (int32_t)x[(((long)b * h + ii) * w + jj) * c + ch] *
                               (int32_t)wt[(long)ch * 9 + di * 3 + dj];
                    }
                }
                long o = (((long)b * ho + i) * wo + j) * c + ch;
                if (acc_out) acc_out[o] = acc;
                if (y)
                    y[o] = (int8_t)prom_ref_requant_scalar(acc + bias[ch], mult[ch], shift[ch],
                                                           act_min, act_max);
            }
        }
    }
}
