/*
 * prom.h -- C ABI of the B200 (sm_100a) ternary pointwise-convolution library.
 *
 * The library computes the inference form of PROM's quantised 1x1 convolution
 * (paper, Section 3.1 and Figure 12, inference branch): int8 activations are
 * convolved directly with ternary weights W-hat in {-1,0,+1}^{Cout x Cin}, so
 * that every product is a signed copy of an input value (Section 2), and the
 * integer result is scaled per output channel afterwards.
 *
 * Layout: activations are NHWC, i.e. a row-major matrix X[M][Cin] with
 * M = batch*H*W; the output is Y[M][Cout]; weights are [Cout][Cin].
 *
 * For every row m and output channel o the library returns exactly
 *
 *     acc = sum_k X[m][k] * W[o][k]                       (int32, exact)
 *     t   = acc + bias[o]
 *     p   = t * mult[o]                                   (exact)
 *     q   = sign(p) * floor((|p| + 2^(s-1)) / 2^s),  s = 31 + shift[o]
 *     Y[m][o] = min(act_max, max(act_min, q))
 *
 * The paper applies the per-channel weight scale and the activation scale in
 * floating point, after the integer convolution (Figure 12, inference branch); this library
 * takes them, with BatchNorm and the next layer's activation scale folded in,
 * as the fixed-point pair (mult, shift): one rounding of the exact product,
 * ties away from zero.  Integer sums and this rounding are exact, so there is
 * one correct byte per output.
 *
 * General conventions
 *   - Every pointer named *_dev is device memory of the current CUDA device,
 *     owned by the caller; *_host is host memory (pinned for overlap).
 *   - The library allocates nothing the caller must free.  It keeps small
 *     internal caches (tensor-map plans; per device and stream, the index
 *     lists of the add/sub variant and the expanded weight matrix of the
 *     row-resident tensor-core kernel, which single calls with Cin >= 512 and
 *     Cout >= 256 on many rows use: device memory obtained with cudaMalloc on
 *     first use, so the first such call on a stream should not be made while
 *     that stream is being captured) that prom_shutdown() releases.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Convolution calls are asynchronous on that stream.
 *   - Errors are return codes; nothing aborts or traps.  Argument errors are
 *     found on the host before any launch.  Conditions only the device can
 *     see (constants out of range, a bounded wait that ran out) are recorded
 *     in a device status word read by prom_last_device_status().
 *   - Calls are re-entrant across streams; two calls that write the same
 *     output race like any two kernels would.
 */
#ifndef PROM_H_
#define PROM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PROM_OK = 0,
    PROM_ERR_NULL,         /* a required pointer is NULL */
    PROM_ERR_SHAPE,        /* a size is non-positive, too large, or shapes do not chain */
    PROM_ERR_ALIGN,        /* a base pointer is not 16-byte aligned */
    PROM_ERR_BAD_WEIGHT,   /* a weight outside {-1,0,+1} / an invalid 2-bit code */
    PROM_ERR_BAD_REQUANT,  /* mult/shift/bias/clamp outside the documented range */
    PROM_ERR_WORKSPACE,    /* workspace too small */
    PROM_ERR_UNSUPPORTED,  /* the requested variant cannot run this shape */
    PROM_ERR_CUDA,         /* a CUDA runtime/driver call failed */
    PROM_ERR_TIMEOUT       /* a bounded device-side wait ran out */
} prom_status;

typedef enum {
    PROM_VARIANT_AUTO = 0, /* the library picks TC where it applies, else SMALLK, else NAIVE */
    PROM_VARIANT_TC,       /* TMA + tcgen05 int8 MMA into TMEM, fused epilogue */
    PROM_VARIANT_SMALLK,   /* CUDA-core dot products for small Cin */
    PROM_VARIANT_ADDSUB,   /* additions and subtractions only on activation values */
    PROM_VARIANT_NAIVE     /* one thread per output, plain loops (tests) */
} prom_variant;

/* Per-output-channel requantisation (stands in for the paper's division by the
 * weight and activation scales, Figure 12).  bias/mult/shift: device arrays of
 * `cout` entries.  Ranges: 0 <= mult < 2^31, 0 <= shift <= 31,
 * |bias| <= 2^28, -128 <= act_min <= act_max <= 127.  The clamp is checked on
 * the host; the arrays are checked on the device by the kernels that read
 * them (a violation sets PROM_ERR_BAD_REQUANT in the device status word and
 * the affected output tile is left unwritten). */
typedef struct {
    const int32_t *bias;
    const int32_t *mult;
    const int8_t  *shift;
    int act_min, act_max;
} prom_requant;

/* One layer of a sequence.  in_stride (1 or 2) is the spatial subsampling
 * applied to this layer's input.  With dw_w == NULL the depthwise convolution
 * that sits between an expand and a project convolution (Section 2) is
 * modelled as the identity on values plus its stride: output pixel (i, j)
 * reads input pixel (in_stride*i, in_stride*j).  With dw_w set, the int8
 * depthwise 3x3 convolution of prom_dw_conv3x3_i8 (weights dw_w [cin][3][3],
 * constants dw_rq, stride in_stride) runs on the layer's input first and the
 * pointwise convolution reads its output; the input's height and width must
 * then be multiples of in_stride.  With add_block_input nonzero the input of
 * the previous layer (in an inverted-residual block, Section 2: the block's
 * input, when this layer is the project convolution and the previous one the
 * expand convolution) is added to this layer's output as in
 * prom_pw_conv_i8_res; both layers must then have in_stride 1 and this
 * layer's cout must equal the previous layer's cin (PROM_ERR_SHAPE
 * otherwise), and the variants SMALLK and ADDSUB refuse the sequence
 * (PROM_ERR_UNSUPPORTED). */
typedef struct {
    int cin, cout;
    int in_stride;
    const uint8_t *w_packed;   /* device, prom_packed_bytes(cout, cin) bytes */
    prom_requant rq;
    const int8_t *dw_w;        /* device, or NULL: no depthwise convolution in front */
    prom_requant dw_rq;        /* read only when dw_w is set */
    int add_block_input;       /* nonzero: add the previous layer's input to the output */
} prom_layer;

/* Bytes of the 2-bit form of a [cout][cin] ternary matrix: cout*ceil(cin/4).
 * The paper counts a ternary weight as 2 bits of storage (Section 4, Memory;
 * Table 1) without fixing a format; this library's is: code 00 = 0, 01 = +1,
 * 11 = -1 (10 invalid); weight k of channel o in byte o*ceil(cin/4) + k/4 at
 * bits 2*(k%4), 2*(k%4)+1; rows padded to a whole byte with 00. */
size_t prom_packed_bytes(int cout, int cin);

/* Packs device int8 ternary weights w_dev[cout][cin] into packed_dev.
 * Weights are quantised once, ahead of inference (Figure 12, inference
 * branch): this runs once per layer, off the hot path.  Synchronises `cuda_stream`.  Returns
 * PROM_ERR_BAD_WEIGHT (packed_dev contents then unspecified) if any value is
 * outside {-1,0,+1}; PROM_ERR_WORKSPACE if packed_bytes is too small. */
prom_status prom_pack_ternary(const int8_t *w_dev, int cout, int cin,
                              uint8_t *packed_dev, size_t packed_bytes,
                              void *cuda_stream);

/* The step before the path: quantises float weights w_dev[cout][cin] to ternary
 * and writes them in the 2-bit form straight away (Section 3.1, Eq. 1-3;
 * Figure 10, pointwise branch): alpha_i = mean_j |W[i][j]|,
 * W-hat = clip(round(W / max(alpha_i, 1e-5)), -1, 1), ties to the even integer
 * as the framework's round does, the division guarded as in the figure (Eq. 3
 * adds the epsilon instead).  alpha_dev (cout floats, may be NULL) receives the
 * per-channel scales, by which the paper multiplies the integer result
 * afterwards.  Asynchronous on `cuda_stream`; a NaN weight sets
 * PROM_ERR_BAD_WEIGHT in the device status word. */
prom_status prom_quantize_ternary(const float *w_dev, int cout, int cin,
                                  uint8_t *packed_dev, size_t packed_bytes,
                                  float *alpha_dev, void *cuda_stream);

/* The same quantiser over several weight matrices (all the layers of a network)
 * in one launch: the per-layer call is bound by launch latency, not by the few
 * megabytes it moves.  jobs: host array of n entries, each as the arguments of
 * prom_quantize_ternary (alpha_dev may be NULL).  Everything is checked before
 * the launch.  Asynchronous on `cuda_stream`. */
typedef struct {
    const float *w_dev;
    int cout, cin;
    uint8_t *packed_dev;
    size_t packed_bytes;
    float *alpha_dev;
} prom_quantize_job;
prom_status prom_quantize_ternary_batch(const prom_quantize_job *jobs, int n, void *cuda_stream);

/* The int8 depthwise 3x3 convolution between a block's expand and project convolutions
 * (paper, Section 2: depthwise-separable blocks; Section 3.1: its weights are 8-bit, Eq. 4-5).
 * Per channel, with one pixel of zero padding and stride 1 or 2,
 *     acc[b][i][j][c] = sum_{di,dj in 0..2} x[b][i*s + di - 1][j*s + dj - 1][c] * w[c][di][dj]
 * and y = requant(acc + bias[c], mult[c], shift[c]) clamped to [act_min, act_max], the
 * requantisation of prom_pw_conv_i8.  Output size: ho = (h - 1) / stride + 1, wo likewise.
 *   x_dev  [batch][h][w][c] int8, device, 16-byte aligned (NHWC)
 *   w_dev  [c][3][3] int8, device (the paper quantises them per channel by absmax:
 *          prom_quantize_act_absmax over a [c][9] float matrix, 16-byte aligned, gives exactly that)
 *   rq     per-channel constants as for prom_pw_conv_i8 (device arrays of c entries)
 *   y_dev  [batch][ho][wo][c] int8, device, 16-byte aligned, not x_dev
 * c must be a multiple of 4 (PROM_ERR_UNSUPPORTED otherwise).  Asynchronous on the stream.
 * Constants out of range surface as PROM_ERR_BAD_REQUANT in prom_last_device_status. */
prom_status prom_dw_conv3x3_i8(const int8_t *x_dev, int batch, int h, int w, int c, int stride,
                               const int8_t *w_dev, const prom_requant *rq, int8_t *y_dev,
                               void *cuda_stream);

/* A pointwise layer in the paper's own inference dataflow: pseudocode appendix, inference
 * branch of the quantised convolution module (integer convolution first, the scales applied to
 * its result), followed by the activation quantiser of the next module (Section 3.1,
 * Eq. 6-7).  With b(m) = m / rows_per_sample the sample of row m,
 *     acc[m][o] = sum_k x[m][k] * W-hat[o][k]                        exact integers
 *     y[m][o]   = acc[m][o] * alpha[o] * (max(gamma_x[b], 1e-5) / 127)  dequantised output
 *     gamma_y[b] = max |y| over the sample,  scale_y[b] = 127 / max(gamma_y[b], 1e-5)
 *     q[m][o]   = clip(round(y[m][o] * scale_y[b]), -128, 127)        ties to even
 * Every float step is one correctly rounded binary32 operation in the order written, so the
 * outputs are reproducible bit for bit.  y itself is never written: the tensor cores run the
 * convolution twice (first pass: maxima, second pass: codes), which costs a second read of x
 * instead of writing and re-reading four bytes per output.
 *   x_dev        [batch * rows_per_sample][cin] int8, device, 16-byte aligned (the activation
 *                quantiser's output; gamma_x_dev [batch] are the maxima it reported)
 *   w_packed_dev packed ternary weights (prom_pack_ternary / prom_quantize_ternary)
 *   alpha_dev    [cout] float32 > 0, the weight scales (prom_quantize_ternary's alpha), times
 *                whatever per-channel factor the caller folds in
 *   q_dev        [batch * rows_per_sample][cout] int8, device, 16-byte aligned, not x_dev
 *   gamma_y_dev, scale_y_dev  [batch] float32 outputs
 * Tensor-core variant only: cin a multiple of 16, cout a multiple of 8 (of 16 above 256), else
 * PROM_ERR_UNSUPPORTED.  Asynchronous on the stream (one memset, three launches).  Other errors
 * as for prom_pw_conv_i8; weights outside {-1,0,+1} surface as PROM_ERR_BAD_WEIGHT in
 * prom_last_device_status. */
prom_status prom_pw_conv_i8_dyn(const int8_t *x_dev, int batch, int64_t rows_per_sample, int cin,
                                const uint8_t *w_packed_dev, int cout, const float *alpha_dev,
                                const float *gamma_x_dev, int8_t *q_dev, float *gamma_y_dev,
                                float *scale_y_dev, void *cuda_stream);

/* Per-sample absmax quantisation of float activations to int8: paper, Section 3.1
 * ("Activations", Eq. 6-7) and the activation figure of the pseudocode appendix.  For each of
 * the `batch` samples, over all `per_sample` values of the sample (any layout inside it),
 *     gamma = max |x|,  scale = 127 / max(gamma, 1e-5),  q = clip(round(x * scale), -128, 127),
 * round = ties to even.  The quotient and the product are single correctly rounded binary32
 * operations, so q, gamma and scale are reproducible bit for bit.  Non-finite inputs are not
 * supported (NaNs are ignored by the maximum and give an unspecified code).
 *   x_dev      [batch][per_sample] float32, device, 16-byte aligned
 *   q_dev      [batch][per_sample] int8, device, 16-byte aligned
 *   gamma_dev, scale_dev  [batch] float32, device (Eq. 6's gamma and the factor applied)
 * Asynchronous on the stream.  When per_sample is a multiple of 16 a thread-block cluster of
 * up to 8 CTAs works on each sample and exchanges the maxima through distributed shared
 * memory: if the sample fits the shared memory of 8 SMs (per_sample <= about 450 000) it is
 * staged there and read from HBM once, larger samples are read twice (the second time from L2
 * while it still holds them).  Other sizes take two kernels and read every value twice.
 * Errors: PROM_ERR_NULL, PROM_ERR_SHAPE (batch < 0, per_sample < 1, batch > 65535 on the
 * two-pass route), PROM_ERR_ALIGN, PROM_ERR_CUDA; a copy that does not land within 0.1 s sets
 * PROM_ERR_TIMEOUT in prom_last_device_status.  batch == 0 is a no-op. */
prom_status prom_quantize_act_absmax(const float *x_dev, int batch, int64_t per_sample,
                                     int8_t *q_dev, float *gamma_dev, float *scale_dev,
                                     void *cuda_stream);

/* Host helper: the fixed-point pair for a real per-channel scale (alpha_i times
 * the activation scales and whatever BatchNorm folds in; Figure 12 divides by
 * these in floating point): mult in [2^30, 2^31) and shift in [0, 31] with
 * mult * 2^-(31+shift) the nearest such number to `scale`.  0 < scale < 1;
 * PROM_ERR_BAD_REQUANT when the shift would leave its range. */
prom_status prom_requant_from_scale(double scale, int32_t *mult, int8_t *shift);

/* One ternary pointwise convolution with fused requantisation (Section 3.1,
 * inference form; formula at the top of this file).
 *   x_dev        [m][cin]  int8, dense rows, 16-byte aligned base
 *   w_packed_dev 2-bit weights of [cout][cin], 16-byte aligned base
 *   y_dev        [m][cout] int8, 16-byte aligned base, must not overlap x_dev
 * m >= 0 (m == 0 is a no-op for which x_dev and y_dev may be NULL), 1 <= cin <= 4096,
 * 1 <= cout <= 4096.
 * TC needs cin % 8 == 0 and cout % 8 == 0 (and even m when cin or cout is not
 * a multiple of 16); SMALLK needs cin % 4 == 0 and cin <= 64; ADDSUB and NAIVE
 * take any shape.  An explicit variant that cannot run the shape returns
 * PROM_ERR_UNSUPPORTED; AUTO always finds one. */
prom_status prom_pw_conv_i8(const int8_t *x_dev, int64_t m, int cin,
                            const uint8_t *w_packed_dev, int cout,
                            const prom_requant *rq, int8_t *y_dev,
                            prom_variant variant, void *cuda_stream);

/* The same layer with its operands prepared ahead of the call.  The paper's
 * weights are quantised once, before inference (Figure 12, inference branch);
 * the same holds for everything this library derives from them: the 2-bit
 * codes expanded to the int8 operand layout of the tensor cores, the bias
 * digits and the per-channel constants.  prom_pw_prepare writes that form of a
 * layer into a caller-owned buffer once (one small kernel, asynchronous on the
 * stream), and prom_pw_conv_i8_prepared runs the tensor-core variant from it,
 * so that a call no longer rebuilds the operands in every CTA.
 *   prom_pw_prepared_bytes  size of the buffer for a layer of m rows (the
 *       launch plan, and with it the layout, depends on m, cin, cout and the
 *       device); 0 when the tensor-core variant cannot run the shape
 *   prom_pw_prepare         rq: constants and clamp as for prom_pw_conv_i8
 *       (their ranges are checked on the device: PROM_ERR_BAD_REQUANT in
 *       prom_last_device_status); prepared_dev: device, 16-byte aligned,
 *       prepared_bytes >= prom_pw_prepared_bytes (PROM_ERR_WORKSPACE otherwise)
 *   prom_pw_conv_i8_prepared  same m, cin, cout as at preparation; the clamp
 *       [act_min, act_max] is given again and must equal the prepared one;
 *       x_dev, y_dev as in prom_pw_conv_i8
 * The buffer stays valid for any number of calls on the device it was
 * prepared on; its contents are private to this build of the library.
 * PROM_ERR_UNSUPPORTED where PROM_VARIANT_TC would be. */
size_t prom_pw_prepared_bytes(int64_t m, int cin, int cout);
prom_status prom_pw_prepare(int64_t m, int cin, const uint8_t *w_packed_dev, int cout,
                            const prom_requant *rq, void *prepared_dev, size_t prepared_bytes,
                            void *cuda_stream);
prom_status prom_pw_conv_i8_prepared(const int8_t *x_dev, int64_t m, int cin, int cout,
                                     const void *prepared_dev, int act_min, int act_max,
                                     int8_t *y_dev, void *cuda_stream);

/* The project convolution of an inverted-residual block with the block's
 * skip connection (Section 2): the layer of prom_pw_conv_i8, then
 *   y[r][o] = clamp(y[r][o] + res[r][o], -128, 127),
 * both terms on the output's scale (the requantisation constants are chosen
 * so; the paper adds in floating point after dequantising).  The kernel adds
 * in its epilogue: the sum costs one more read of m*cout bytes and no pass of
 * its own.
 *   res_dev  [m][cout] int8, 16-byte aligned base; it may be y_dev itself
 *            (the sum is then formed in place) but must not overlap y_dev
 *            in any other way, nor x_dev at all
 * Everything else as in prom_pw_conv_i8.  Variants: AUTO, TC and NAIVE; SMALLK
 * and ADDSUB return PROM_ERR_UNSUPPORTED, and AUTO falls back on NAIVE where
 * TC does not apply. */
prom_status prom_pw_conv_i8_res(const int8_t *x_dev, int64_t m, int cin,
                                const uint8_t *w_packed_dev, int cout,
                                const prom_requant *rq, const int8_t *res_dev,
                                int8_t *y_dev, prom_variant variant,
                                void *cuda_stream);

/* Test/debug: the raw accumulators acc[m][cout] (int32) of the same layer,
 * computed by the plain one-thread-per-output kernel. */
prom_status prom_pw_conv_i8_acc32(const int8_t *x_dev, int64_t m, int cin,
                                  const uint8_t *w_packed_dev, int cout,
                                  int32_t *acc_dev, void *cuda_stream);

/* Same convolution with HOST activations and output: copies x_host to the
 * device, runs, copies the result back, all asynchronous on `cuda_stream`
 * (pinned host memory is needed for the copies to be asynchronous).
 * workspace_dev must hold m*cin + m*cout bytes (each rounded up to 256). */
prom_status prom_pw_conv_i8_host(const int8_t *x_host, int64_t m, int cin,
                                 const uint8_t *w_packed_dev, int cout,
                                 const prom_requant *rq, int8_t *y_host,
                                 void *workspace_dev, size_t workspace_bytes,
                                 prom_variant variant, void *cuda_stream);

/* A sequence of pointwise layers, each reading the previous one's output
 * (the expand -> depthwise -> project block structure of Section 2 with the
 * depthwise stage reduced to its stride).  Input x0_dev is
 * [batch][h0][w0][layers[0].cin]; the result y_out_dev is
 * [batch][h][w][layers[n-1].cout] with h, w divided by every in_stride.
 * Intermediate activations live in the caller's workspace (two ping-pong
 * regions), followed by the prepared operands of the tensor-core layers
 * (expanded weights, bias digits, constants; rebuilt by one small kernel at
 * the start of every call, so the call stays stateless);
 * prom_layer_seq_workspace_bytes gives the size needed (0 on a shape error).
 * A workspace that only holds the two activation regions still works, more
 * slowly.  `variant` applies to every layer (AUTO picks per layer).  The
 * kernels of one call are chained with programmatic dependent launch and can
 * be captured into a CUDA graph. */
size_t prom_layer_seq_workspace_bytes(const prom_layer *layers, int n,
                                      int batch, int h0, int w0);
prom_status prom_pw_layer_seq(const prom_layer *layers, int n,
                              const int8_t *x0_dev, int batch, int h0, int w0,
                              void *workspace_dev, size_t workspace_bytes,
                              int8_t *y_out_dev,
                              prom_variant variant, void *cuda_stream);

/* Same sequence with HOST input and output; the workspace must additionally
 * hold the input and the output (prom_layer_seq_host_workspace_bytes). */
size_t prom_layer_seq_host_workspace_bytes(const prom_layer *layers, int n,
                                           int batch, int h0, int w0);
prom_status prom_pw_layer_seq_host(const prom_layer *layers, int n,
                                   const int8_t *x0_host, int batch, int h0, int w0,
                                   void *workspace_dev, size_t workspace_bytes,
                                   int8_t *y_out_host,
                                   prom_variant variant, void *cuda_stream);

/* The ADDSUB variant of prom_pw_conv_i8 for callers that must not allocate.
 * (The paper has no counterpart; this exists for integration reasons only.)
 *
 * Who needs it: the ordinary ADDSUB variant keeps its per-layer index lists in
 * a buffer the library obtains with cudaMalloc on first use and replaces with a
 * larger one (cudaFree + cudaMalloc) when a bigger layer comes along.  Those
 * calls synchronise the whole device and can fail outright in a process whose
 * memory pool or inference engine has already claimed all free device memory;
 * a serving loop with a fixed memory budget, or a plug-in that runs inside
 * someone else's arena, cannot afford either.  This entry point calls no
 * cudaMalloc, cudaFree or other allocating routine, ever.
 *
 * How: the index lists go into a fixed array of PROM_STATIC_SCRATCH_BYTES that
 * is part of the library's device image, so every GPU that loads the library
 * holds that much memory until the process ends.  A layer fits when
 *     256*ceil(cout*16/256) + 4*cout*(8*ceil(cin/8) + 8)  <=  PROM_STATIC_SCRATCH_BYTES
 * (and cin <= 1536, the variant's own limit); cout = 1280, cin = 960 needs
 * about 4.8 MiB.  A larger layer is refused with PROM_ERR_WORKSPACE before
 * anything is launched.
 *
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  All calls
 * on a device share the one array and each call rewrites the part it uses, so
 * nothing needs clearing between calls, but two calls that may overlap on the
 * GPU (different streams, no ordering between them) race on it: order them.
 * Arguments, result and error codes are otherwise those of prom_pw_conv_i8
 * with PROM_VARIANT_ADDSUB. */
#define PROM_STATIC_SCRATCH_BYTES (6u << 20)
prom_status prom_pw_conv_i8_addsub_static(const int8_t *x_dev, int64_t m, int cin,
                                          const uint8_t *w_packed_dev, int cout,
                                          const prom_requant *rq, int8_t *y_dev,
                                          void *cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the device status word:
 * PROM_OK, PROM_ERR_BAD_REQUANT, PROM_ERR_BAD_WEIGHT (invalid 2-bit code met
 * by a kernel) or PROM_ERR_TIMEOUT. */
prom_status prom_last_device_status(void *cuda_stream);

/* Number of kernels this library has launched since it was loaded (all
 * streams, this process); used by the benchmark to count launches. */
uint64_t prom_launch_count(void);

/* Frees the library's internal caches (all devices).  Optional. */
void prom_shutdown(void);

const char *prom_status_string(prom_status s);

#ifdef __cplusplus
}
#endif
#endif /* PROM_H_ */
