/*
 * prom_debug.h -- tuning, measurement and test aids of the ternary
 * pointwise-convolution library.  Nothing here is needed to run the path of
 * prom.h; results of that path never depend on anything set here.  The paper
 * has no counterpart for any of these.
 */
#ifndef PROM_DEBUG_H_
#define PROM_DEBUG_H_

#include "prom.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Tuning aid for the TC variant: forces the row fold (1, 2, 4, 8), the subtile
 * width, the number of output-channel groups, the way CTAs share an SM (1: one
 * CTA with all of tensor memory; 2: two CTAs of the kernel per SM; 3: one
 * half-sized CTA per SM; 4: three CTAs per SM, on a build of the kernel with 64
 * registers a thread) and the depth of the activation ring of later calls;
 * 0 leaves a choice to the library.  A forced combination that does not fit
 * makes TC report PROM_ERR_UNSUPPORTED.  The override is process-wide (one
 * lock guards it; a call that plans while another thread changes it sees the
 * old or the new override, never a mixture).  prom_debug_tc_plan_query writes
 * the plan the library would use for a plain [m][cin] x [cout] layer ({fold,
 * nt, groups, grid, stages, accumulators, shared bytes, chunk bytes, estimate
 * in 1/100 us}) and returns 1, or returns 0 if TC cannot run it.  Without a
 * CUDA device it plans for a B200's nominal limits (148 SMs, 227 KB of shared
 * memory per CTA). */
void prom_debug_tc_plan(int fold, int nt, int groups, int occ, int stages);
/* The same override for one shape only (m rows, cin, cout, input stride of the
 * layer); it takes precedence over prom_debug_tc_plan for that shape.  All five
 * values 0 removes it. */
void prom_debug_tc_plan_shape(int64_t m, int cin, int cout, int stride, int fold, int nt,
                              int groups, int occ, int stages);
int prom_debug_tc_plan_query(int64_t m, int cin, int cout, int *out9);

/* Depth-first launches inside prom_pw_layer_seq: 0 = none, one launch per layer
 * (default); 1 = every run of consecutive layers that qualifies (same number
 * of rows in all of them, only the first may subsample its input; channel
 * counts that are multiples of 16 with cin >= 32; clamp [0, 127]; no depthwise
 * convolution, no skip connection; at most 8 tiles of 128 rows per SM) is
 * executed by one launch in which a CTA takes its tiles of rows through all
 * the layers of the run.  Every layer's output is still written to the
 * workspace (each to a buffer of its own) and read back from there by the next
 * layer.  Results do not depend on the mode; the workspace size does
 * (prom_layer_seq_workspace_bytes follows the mode; a workspace that is too
 * small for the depth-first buffers falls back to one launch per layer).
 * 2 = runs that stay in shared memory: consecutive layers on the same rows
 * (only the first may subsample), channel counts multiples of 16, no depthwise
 * convolution and no skip connection, alternately at most 384 output channels
 * (the first layer and every second one after it) and at most 384 input
 * channels (the layers in between), any clamp; one launch takes a tile of rows
 * through all of them and only the run's last layer writes a tensor (to a
 * buffer of its own in the workspace, or to y_out).  The inner layers have no
 * output tensor: prom_debug_layer_seq_output_offset returns -2 for them.
 * Process-wide. */
void prom_debug_seq_chain(int mode);
/* Order of the row tiles inside the tensor-core layers of prom_pw_layer_seq:
 * 1 (default) = every second layer walks its tiles from the last to the first,
 * so that it reads first what the layer before wrote last; 0 = every layer
 * from the first to the last.  Results do not depend on it.  Process-wide. */
void prom_debug_seq_order(int alternate);

/* Which kernel prom_dw_conv3x3_i8 runs: 0 = the library's choice (default: TMA
 * patches and tensor-core taps for stride 1 with a channel count that is a
 * multiple of 16 and images of at least 100 pixels, CUDA cores otherwise), 1 = CUDA cores only, 2 = tensor cores
 * or PROM_ERR_UNSUPPORTED.  Results do not depend on it.  Process-wide. */
void prom_debug_dw_variant(int variant);

/* Which kernel the tensor-core variant of a single pointwise call runs: 0 = the
 * library's choice (the row-resident kernel, which keeps 128 rows with all their
 * input channels in shared memory and streams the weight matrix past them, for
 * layers with Cin >= 512, Cout >= 256 (nearly a multiple of 128 unless Cin >= 768)
 * and at least four tiles of 128 rows per SM;
 * the weight-resident kernel otherwise), 1 = the weight-resident kernel only, 2 = the row-resident kernel
 * or PROM_ERR_UNSUPPORTED (it takes plain matrices with Cin and Cout multiples
 * of 16, 128 <= Cin <= 1024, Cout >= 64, no residual).  blocks: 128-channel
 * blocks per column tile of that kernel, 1 (MMA N = 128) or 2 (N = 256; refused
 * where four 32 KB stages do not fit beside the resident rows), 0 = the
 * planner's choice.  Results do not depend on either.  Process-wide. */
void prom_debug_tc_wide(int mode, int blocks);

/* Where layer `layer`'s output ([rows][cout] int8) sits in the workspace of a
 * prom_pw_layer_seq call whose workspace has prom_layer_seq_workspace_bytes
 * bytes, with AUTO or TC as the variant: the byte offset from the workspace's
 * start, -1 for the last layer (its output is y_out_dev) or a bad argument,
 * -2 for a layer inside a shared-memory run (prom_debug_seq_chain(2)) that is
 * not the run's last: it writes no tensor.  *chained (may be NULL) receives 1
 * when the layer runs inside a multi-layer launch.  A layer's output stays intact until the layer two further on has
 * run (ping-pong regions) or, inside a depth-first launch, until the next
 * call. */
int64_t prom_debug_layer_seq_output_offset(const prom_layer *layers, int n, int batch, int h0,
                                           int w0, int layer, int *chained);

/* Failure-detection check: launches one warp that waits, with the library's
 * bounded mbarrier wait and a limit of limit_ns nanoseconds (1000 ..
 * 100 000 000), on a barrier phase nothing ever completes.  The wait gives up
 * by itself and the kernel returns normally; afterwards
 * prom_last_device_status reports PROM_ERR_TIMEOUT.  gave_up_dev (device int,
 * may be NULL) receives 1.  Nothing traps, faults or waits without a limit. */
prom_status prom_debug_wait_timeout(uint64_t limit_ns, int *gave_up_dev, void *cuda_stream);

/* Rate probes for the roofline figures.  Both launch one grid over all SMs and
 * write, per CTA, the SM clock cycles of its measured loop into cycles_dev
 * (device, cycles_len >= the grid size, which *grid_out receives); the host
 * times the launch itself with events.
 *   i8_mma_rate: one CTA per SM, one thread issuing iters x 4
 *     tcgen05.mma.kind::i8 instructions of shape 128 x 256 x 32 on fixed
 *     shared-memory operands into two alternating accumulators, one commit and
 *     a bounded wait at the end: 2 * 128 * 256 * 32 * 4 * iters operations per CTA.
 *     1 <= iters <= 2^20.
 *   alu_rate: op 0 = mul.hi.s32 (the requantiser's multiply), 1 = mad.lo.s32,
 *     2 = fma.rn.f32, 3 = mad.wide.s32 (high word fed back), 4 = cvt.pack.sat.u8.s32,
 *     5 = shr.s32, 6 = fma.rn.f64; two CTAs of 512 threads per SM, 8 independent chains per
 *     thread, 64 * iters instructions per thread.  sink_dev: one device int.
 * Asynchronous on the stream. */
prom_status prom_debug_i8_mma_rate(int iters, long long *cycles_dev, int cycles_len, int *grid_out,
                                   void *cuda_stream);
prom_status prom_debug_alu_rate(int op, int iters, int *sink_dev, long long *cycles_dev,
                                int cycles_len, int *grid_out, void *cuda_stream);

/* Two more probes: rates that bound kernels made of small MMAs and kernels
 * that stream an operand out of L2.
 *   mma_issue_rate: how often an SM accepts a tcgen05.mma.kind::i8 of shape
 *     128 x n x 32 (n a multiple of 16, 16..256) when `warps` threads (1..4, one
 *     per warp, each with two accumulators of its own: warps * 2 * max(n, 64)
 *     <= 512 tensor-memory columns, else PROM_ERR_SHAPE) issue iters x 4 of them
 *     each.  cycles_dev[4 * cta + w] = SM clocks of warp w; cycles_len >= 4 x the
 *     grid size.
 *   l2_copy_rate: what one SM can pull from L2.  One thread per SM keeps `stages`
 *     (1..8) bulk copies of 16 KB in flight out of region_dev (device, 16-byte
 *     aligned, region_bytes a multiple of 16 KB and at least that; keep it below
 *     the L2 size), iters copies per SM.  cycles_dev[cta] = SM clocks.
 * Both write the grid size to *grid_out and are asynchronous on the stream. */
prom_status prom_debug_mma_issue_rate(int n, int warps, int iters, long long *cycles_dev, int cycles_len,
                                      int *grid_out, void *cuda_stream);
prom_status prom_debug_l2_copy_rate(const void *region_dev, uint64_t region_bytes, int iters, int stages,
                                    long long *cycles_dev, int cycles_len, int *grid_out, void *cuda_stream);

/* What shares an SM with the MMAs, one CTA per SM.
 *   mode 0: one thread issues iters x 4 tcgen05.mma.kind::i8 of shape
 *     128 x 128 x 32 while a second thread keeps `stages` (0 = none, 1..3) bulk
 *     copies of 16 KB in flight out of region_dev (as for l2_copy_rate) into
 *     other shared memory, until the MMAs are done.
 *   mode 1: nwarps (4, 8 or 16) warps each read iters times 32 lanes x 32
 *     columns of tensor memory (tcgen05.ld 32x32b.x32, wait, fold) while, if
 *     stages == 1, another thread issues the same MMAs into other columns until
 *     the readers are done (stages == 0: no MMAs).
 * out_dev[8 * cta + i], out_len >= 8 x the grid size: i = 0 SM clocks of the
 * measured loop (mode 1: of the slowest reading warp), 1 = MMAs issued,
 * 2 = SM clocks of the MMA loop, 3 = copies issued.  Asynchronous on the
 * stream; all waits bounded. */
prom_status prom_debug_mma_beside(int mode, int iters, int nwarps, int stages, const void *region_dev,
                                  uint64_t region_bytes, long long *out_dev, int out_len, int *grid_out,
                                  void *cuda_stream);

/* Bookkeeping check, no CUDA call: returns 1 the first time (device, key) is
 * asked about on the table used for per-device kernel attributes, 0
 * afterwards (the table behind this entry is a separate instance). */
int prom_debug_once_per_device(int device, int key);

#ifdef __cplusplus
}
#endif
#endif /* PROM_DEBUG_H_ */
