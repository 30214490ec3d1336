/*
 * qbp.h -- C ABI of libqbp: the 8-bit training hot path (Quantized
 * Back-Propagation with Gradients Bifurcation, followed by Range
 * Batch-Normalization) as hand-written CUDA kernels for sm_100a.
 *
 * Paper: "Scalable Methods for 8-bit Training of Neural Networks"
 * (arXiv 1805.11046).  Each entry point cites the passage that defines the
 * operation it performs.
 *
 * Conventions (all entry points)
 *   - Every tensor pointer is a DEVICE pointer owned by the caller.  Scalars
 *     the GPU produces (scale, zero-point, range) stay on the device in a
 *     qbp_qparams.  The library allocates no device memory and keeps no
 *     results between calls; scratch comes from the caller's workspace `ws`
 *     (device memory, 256-byte aligned) of at least qbp_*_workspace_bytes().
 *     (Host-side objects it does keep: the per-device function attributes,
 *     and, for the layer calls, one stream and two events per host thread
 *     and device -- see qbp_layer_fwd.)
 *   - `stream` is a cudaStream_t passed as void*; work is enqueued on it and
 *     the call returns without synchronising the host.
 *   - Layouts: matrices row-major and dense; activations NHWC; filters KRSC.
 *     Code tensors (int8/uint8) that feed an integer product must start on a
 *     16-byte boundary and have an innermost extent that is a multiple of 16.
 *   - Return value: QBP_OK or a negative qbp_status.  Argument and shape
 *     errors are found on the host before anything is launched; the reason
 *     is kept per thread and returned by qbp_last_error().
 *   - Device status word.  Calls are asynchronous, so a failure on the device
 *     cannot be a return value of the call that enqueued the work.  The
 *     tensor-core products (qbp_gemm_s8, qbp_conv_s8_implicit, qbp_wgrad_s16)
 *     and the layer calls keep an int32 status word in the FIRST FOUR BYTES of
 *     the workspace `ws` they are given: the call clears it, and a kernel
 *     whose bounded wait (about one second) runs out sets it to
 *     QBP_ERR_TIMEOUT, frees what it holds and ends normally -- the outputs
 *     are then invalid.  Read it with qbp_device_status(ws, stream) (which
 *     synchronises the stream) before `ws` is handed to another call.
 *     qbp_layer_fwd clears the word of the layer's workspace once; every
 *     product of that forward and of the following qbp_layer_bwd can only
 *     raise it, so one read after the backward call covers the whole step.
 *   - Stored codes are signed: stored = unsigned code - 2^(M-1), and the
 *     stored zero-point is shifted the same way, so that (q - zero_point) is
 *     the value every product works on.
 */
#ifndef QBP_H_
#define QBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QBP_OK = 0,
    QBP_ERR_INVALID_ARG = -1,       /* NULL/misaligned pointer, negative size, bad enum */
    QBP_ERR_UNSUPPORTED_SHAPE = -2, /* shape outside what the kernels implement         */
    QBP_ERR_OVERFLOW_K = -3,        /* reduction too long for the int32 accumulator     */
    QBP_ERR_WORKSPACE = -4,         /* ws NULL or smaller than *_workspace_bytes()      */
    QBP_ERR_CUDA = -5,              /* a CUDA call failed; message holds its text       */
    QBP_ERR_TIMEOUT = -6            /* a bounded device-side wait gave up (status word) */
} qbp_status;

/* Quantisation parameters of one tensor (or one channel), device resident.
 * x ~= scale * (q - zero_point).  vmin/vmax are the clamping values used,
 * after widening to contain 0 (Appendix B). */
typedef struct {
    float   scale;
    int32_t zero_point;
    float   vmin;
    float   vmax;
} qbp_qparams;

/* Convolution geometry.  Input [N,H,W,C], filter [K,R,S,C], output [N,P,Q,K]
 * with P = (H + 2*pad - R)/stride + 1 (Q likewise).  The integer products
 * implement stride 1 with R = S = 2*pad + 1 ("same" convolution, R in {1,3}). */
typedef struct {
    int32_t N, H, W, C;
    int32_t K, R, S;
    int32_t stride, pad;
} qbp_conv_desc;

enum { QBP_PER_TENSOR = 0, QBP_PER_CHANNEL = 1 };
enum { QBP_ROUND_NEAREST = 0, QBP_ROUND_STOCHASTIC = 1 };
enum { QBP_CONV_FPROP = 0, QBP_CONV_DGRAD = 1 };

/* Text of the last error raised on the calling thread ("" if none). */
const char *qbp_last_error(void);

/* Diagnostics (no counterpart in the paper).  While tracing is enabled every
 * kernel the library launches is bracketed by a CUDA event pair on its stream
 * (process-wide, one host thread at a time).  After synchronising the
 * stream(s), qbp_trace_count() records can be read: kernel name and device
 * time in milliseconds.  qbp_trace_enable(1) discards earlier records; (0)
 * stops tracing and discards them. */
int qbp_trace_enable(int on);
int qbp_trace_count(void);
int qbp_trace_read(int index, char *name, int name_cap, float *ms);

/* Device status word of the calls that used workspace `ws` (see Conventions;
 * no counterpart in the paper).  Copies the word at the start of `ws` to the
 * host on `stream`, SYNCHRONISES that stream, and returns QBP_OK or
 * QBP_ERR_TIMEOUT. */
int qbp_device_status(const void *ws, void *stream);

/* Self-test of the bounded waits (diagnostics; no counterpart in the paper):
 * launches one warp that waits, through the same wait routines the product
 * kernels use but with a limit of `limit_cycles` SM clock cycles (1..1e8), on
 * a barrier that nothing ever signals.  The wait gives up, the kernel raises
 * the status word at the start of `ws` (at least 4 bytes, cleared by this
 * call) and ends normally; qbp_device_status(ws, stream) then returns
 * QBP_ERR_TIMEOUT and the device remains usable. */
int qbp_selftest_bounded_wait(void *ws, size_t ws_bytes, uint32_t limit_cycles, void *stream);

/* ------------------------------------------------------------------------
 * Range quantiser -- Section 4 "Quantization methods" and Appendix B:
 *   scale = (vmax - vmin) / (2^M - 1), zero-point = round(-vmin / scale),
 *   output = round(x / scale + zero-point), clamped to the M-bit codes;
 * clamping values = the tensor's min and max, widened to contain 0.  Nearest
 * rounding (ties to even) for weights and activations; stochastic rounding
 * for gradients (Section 4: convergence needed it) -- up with probability
 * frac, the draw being 16 bits of the Philox4x32-10 word of the element (the
 * high half-word for 8-bit codes, the low half-word for 16-bit codes): key =
 * seed, counter = (i/4 low, i/4 high, tensor_id, 0), word i%4, i = flat
 * index.  All arithmetic is IEEE fp32 in a fixed order, so codes are
 * reproducible bit for bit.
 *
 * x [rows x cols], cols innermost (the channel dimension).  granularity
 * QBP_PER_CHANNEL keeps one qbp_qparams per column (qp_out has `cols`
 * entries), else one.  range_in (nullable): take vmin/vmax from these
 * qbp_qparams (same count as qp_out) instead of scanning x -- the range the
 * preceding Range BN already knows (Section 4).  row_sums (nullable, [rows],
 * per-tensor only): sum over the columns of each row's stored codes.
 * col_sums (nullable, [cols], per-tensor only): sum over rows, int64.
 * rows*cols == 0 is valid and launches nothing but the parameter kernel.
 * ---------------------------------------------------------------------- */
size_t qbp_quantize_workspace_bytes(int64_t rows, int64_t cols, int granularity);

int qbp_quantize_s8(const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                    uint64_t seed, uint32_t tensor_id, const qbp_qparams *range_in,
                    int8_t *q, qbp_qparams *qp_out, int32_t *row_sums, int64_t *col_sums,
                    void *ws, size_t ws_bytes, void *stream);

/* Clamping values for activations as Appendix B takes them (the mean, over K
 * chunks of the tensor, of each chunk's largest and smallest value, which
 * narrows the quantisation steps of tensors with a high dynamic range): x [rows x cols] is
 * cut into `chunks` equal contiguous groups of rows (rows a multiple of
 * chunks, chunks <= 4096); range_out->vmax receives the average of the groups'
 * maxima, range_out->vmin the average of their minima (sums in double, in
 * chunk order; scale and zero_point of the record are left 0).  Pass range_out
 * as range_in to qbp_quantize_s8: values beyond the clamp saturate at the end
 * codes.  Device pointers; workspace of qbp_range_chunked_workspace_bytes(). */
size_t qbp_range_chunked_workspace_bytes(void);

int qbp_range_chunked(const float *x, int64_t rows, int64_t cols, int64_t chunks,
                      qbp_qparams *range_out, void *ws, size_t ws_bytes, void *stream);

/* qbp_quantize_s8 for callers that cannot provide a workspace (the paper has
 * no counterpart; this is a packaging variant of the same kernels).  Some
 * hosts of this library may not allocate device memory at the point where
 * they quantise: code running under a fixed memory plan or inside a region
 * where cudaMalloc is forbidden (it synchronises the device and can fail late),
 * or a plugin that is handed its tensors and nothing else.  For them the range
 * scan's scratch lives inside the library: a file-scope device array of
 * 2 * 4 * 1024 * QBP_STATIC_MAX_CHANNELS + 256 bytes (2 MiB + 256) that every
 * GPU which loads the library holds until the process exits.  The call itself
 * allocates nothing (no cudaMalloc / cudaFree, no allocating library call).
 *
 * Same arguments and results as qbp_quantize_s8 without range_in, row_sums,
 * col_sums and ws.  Limits: per-channel granularity needs cols <=
 * QBP_STATIC_MAX_CHANNELS, otherwise QBP_ERR_UNSUPPORTED_SHAPE and nothing is
 * launched; per-tensor granularity has no size limit.  Argument errors are
 * reported before anything touches the device.
 *
 * The first call on each device resolves the array's device address (once per
 * device, with that device current); make that first call outside any stream
 * capture.  All calls on a device share the one array: it keeps the previous
 * call's partial ranges, which is harmless (each call overwrites every entry
 * it later reads, nothing has to start at zero), but two calls whose kernels
 * overlap on the GPU (different streams, or different host threads) race on
 * it -- serialise them on one stream, or use qbp_quantize_s8 with separate
 * workspaces. */
#define QBP_STATIC_MAX_CHANNELS 256
int qbp_quantize_s8_static(const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                           uint64_t seed, uint32_t tensor_id, int8_t *q, qbp_qparams *qp_out,
                           void *stream);

/* 16-bit variant.  Any of q (int16 codes), hi (signed high byte) and lo
 * (unsigned low byte), q = 256*hi + lo, may be NULL, but not all three. */
int qbp_quantize_s16(const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                     uint64_t seed, uint32_t tensor_id, const qbp_qparams *range_in,
                     int16_t *q, int8_t *hi, uint8_t *lo, qbp_qparams *qp_out,
                     void *ws, size_t ws_bytes, void *stream);

/* Gradients Bifurcation (Sections 1 and 4, Section 6 "Putting it all
 * together"): from one read of the fp32 gradient g, write its 8-bit copy
 * (for the layer gradient) and its 16-bit copy as byte limbs (for the weight
 * gradient); both per-tensor, both stochastically rounded, from the streams
 * tensor_id8 and tensor_id16 (equal ids: both copies draw from one word per
 * element, the 8-bit copy from its high half, the 16-bit copy from its low
 * half -- independent draws at half the generator work).  row_sums8
 * (nullable): as in qbp_quantize_s8. */
int qbp_bifurcate(const float *g, int64_t rows, int64_t cols, uint64_t seed,
                  uint32_t tensor_id8, uint32_t tensor_id16,
                  int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8,
                  int8_t *hi, uint8_t *lo, qbp_qparams *qp16,
                  void *ws, size_t ws_bytes, void *stream);

/* qbp_bifurcate for one shard of a gradient whose minibatch is spread over
 * several GPUs (Gradients Bifurcation, Sections 1, 4 and 6; data-parallel
 * form).  g is this GPU's [rows x cols] part of the whole gradient tensor:
 * index_base (a multiple of 4) is the flat index of g[0] in the whole tensor,
 * so that every element keeps the Philox word it has in the undivided tensor,
 * and range_in carries the clamping values of the WHOLE tensor (the min and
 * max, combined over the GPUs by the caller), so that all shards share one
 * scale.  The codes are then, bit for bit, the rows of the codes that the
 * undivided call would produce.  No workspace: nothing is scanned. */
int qbp_bifurcate_shard(const float *g, int64_t rows, int64_t cols, uint64_t seed,
                        uint32_t tensor_id8, uint32_t tensor_id16, uint64_t index_base,
                        const qbp_qparams *range_in,
                        int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8,
                        int8_t *hi, uint8_t *lo, qbp_qparams *qp16, void *stream);

/* Dequantisation of integer accumulators that were combined outside the
 * product: out[i] = (float)acc[i] * (qa->scale * qb->scale), as the products
 * themselves do it.  For Eq. (grad_weight) under data parallelism: each GPU
 * takes its int64 accumulators from qbp_wgrad_s16 (acc_out), the caller adds
 * them up over the GPUs (exact, order-free), then dequantises here. */
int qbp_dequant_s64(const int64_t *acc, int64_t count, const qbp_qparams *qa, const qbp_qparams *qb,
                    float *out, void *stream);

/* ------------------------------------------------------------------------
 * 8-bit products -- Section 1 (the weighted sums y = W x are where the work
 * is), Eq. (grad_layer) g_{l-1} = g_l W^T; int32 accumulation:
 *   acc[m,n] = sum_k (A[m,k] - za)(B[k,n] - zb),  C[m,n] = (float)acc * (sa*sb).
 * A is [M x K] (transA: stored [K x M]), B is [K x N] (transB: stored
 * [N x K]).  qa/qb give the operands' scale and zero-point (device).  acc_out
 * and C are each nullable, not both.  K*255*255 must fit int32 (K <= 33025),
 * else QBP_ERR_OVERFLOW_K.  M, N, K multiples of 16.
 * ---------------------------------------------------------------------- */
size_t qbp_gemm_s8_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Optional extra work of a product's epilogue.
 *
 * (1) Statistics.  Section 3's Range BN needs the mean, minimum and maximum
 * of every output channel of the layer; they are taken here from the fp32
 * outputs as they are written, so that the normalisation that follows needs
 * no statistics pass of its own.  col_sum (double), col_min, col_max: [N]
 * each (device), all three or none; they receive the sum / minimum / maximum
 * over the M rows of each column of C (of each output channel over all
 * positions for a convolution).  qbp_gemm_s8: N <= QBP_EPILOGUE_MAX_COLUMNS,
 * else QBP_ERR_UNSUPPORTED_SHAPE; qbp_conv_s8_implicit: any number of
 * channels (at most 256 per SM of the device).
 *
 * (2) ReLU and requantisation, for a product whose output feeds the next
 * layer directly (no Range BN in between; Appendix B's quantiser with
 * clamping values the caller knows beforehand, e.g. from the previous step):
 * relu != 0 rectifies the fp32 output (C then holds the rectified values);
 * with q_out the 8-bit codes of that output under the clamping values of
 * requant_range (its vmin / vmax; nearest rounding; values beyond the clamp
 * saturate) are written to q_out [M x N], their parameters to qp_out and,
 * if row_sums_out is given, each row's sum of stored codes to row_sums_out
 * [M].  C may then be NULL.  Not together with (1); runs on the single-CTA
 * kernel.
 *
 * ep == NULL: none of it. */
#define QBP_EPILOGUE_MAX_COLUMNS 256
typedef struct qbp_epilogue {
    double *col_sum;
    float *col_min;
    float *col_max;
    int32_t relu;
    const qbp_qparams *requant_range;
    int8_t *q_out;
    qbp_qparams *qp_out;
    int32_t *row_sums_out;
} qbp_epilogue;

int qbp_gemm_s8(int transA, int transB, int64_t M, int64_t N, int64_t K,
                const int8_t *A, const qbp_qparams *qa,
                const int8_t *B, const qbp_qparams *qb,
                int32_t *acc_out, float *C, const qbp_epilogue *ep,
                void *ws, size_t ws_bytes, void *stream);

/* qbp_gemm_s8 with the code sums along the reduction supplied by the caller
 * (the zero-point correction of Appendix B's scheme needs them; qbp_gemm_s8
 * computes them in two small kernels per call).  a_sums [M] (nullable): the
 * sum over k of the stored codes of row m of op(A); b_sums [N] (nullable): the
 * sum over k of column n of op(B); int32 (K <= 33025 codes always fit).  The
 * row_sums output of qbp_quantize_s8 / qbp_requant is a_sums of a
 * non-transposed A (and b_sums of a transposed B). */
int qbp_gemm_s8_sums(int transA, int transB, int64_t M, int64_t N, int64_t K,
                     const int8_t *A, const qbp_qparams *qa, const int32_t *a_sums,
                     const int8_t *B, const qbp_qparams *qb, const int32_t *b_sums,
                     int32_t *acc_out, float *C, const qbp_epilogue *ep,
                     void *ws, size_t ws_bytes, void *stream);

/* The same products for a convolution, computed as an implicit GEMM over
 * the filter taps (no im2col buffer).  QBP_CONV_FPROP: x [N,H,W,C] ->
 * [N,P,Q,K].  QBP_CONV_DGRAD (Eq. grad_layer): g [N,P,Q,K] -> [N,H,W,C].
 * Padding is real zero, i.e. contributes nothing to (q - zero_point). */
size_t qbp_conv_s8_workspace_bytes(int mode, const qbp_conv_desc *d);

int qbp_conv_s8_implicit(int mode, const qbp_conv_desc *d,
                         const int8_t *in, const qbp_qparams *q_in,
                         const int8_t *w, const qbp_qparams *q_w,
                         int32_t *acc_out, float *out, const qbp_epilogue *ep,
                         void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------
 * Weight gradient -- Eq. (grad_weight) g_W = g_l I_{l-1}^T with the 16-bit
 * copy of g_l and the 8-bit layer input (Sections 6 and 7):
 *   d == NULL: acc[k,n]     = sum_m (x[m,k] - zx)(g16[m,n] - zg)     dW [K x N]
 *   d != NULL: acc[k,r,s,c] = sum over (n,p,q) with the tap in bounds of
 *              (g16[n,p,q,k] - zg)(x[n,p+r-pad,q+s-pad,c] - zx)      dW [K,R,S,C]
 * g16 = 256*g_hi + g_lo.  Each limb runs on the int8 tensor cores with an
 * int32 accumulator over at most 65536 reduction rows at a time (the low
 * limb's bound is 128*255*rows <= 2^31-1, rows <= 65793); partial results
 * are combined in int64, exactly.  acc_out (int64) and dW each nullable, not
 * both; dW = (float)acc * (sx*sg).
 * ---------------------------------------------------------------------- */
size_t qbp_wgrad_s16_workspace_bytes(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K);

int qbp_wgrad_s16(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K,
                  const int8_t *x, const qbp_qparams *qx,
                  const int8_t *g_hi, const uint8_t *g_lo, const qbp_qparams *qg16,
                  int64_t *acc_out, float *dW,
                  void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------
 * Range Batch-Normalization -- Section 3, Eq. (range):
 *   xhat = (x - mu) / (C(n) * range(x - mu)),  C(n) = 1/sqrt(2 ln n),
 *   range = max - min, per channel over the n rows; y = gamma*xhat + beta
 *   (gamma/beta nullable: 1, 0), optionally followed by ReLU.  A channel of
 *   zero range yields xhat = 0.  n >= 2.
 * x, y [n x C], C innermost.  save_mean/min/max [C] are written for the
 * backward pass.  out_range (nullable): the exact per-tensor min and max of
 * y, which the next layer's quantiser can take as range_in (Section 4).
 * ---------------------------------------------------------------------- */
size_t qbp_rangebn_workspace_bytes(int64_t n, int64_t C);

int qbp_rangebn_fwd(const float *x, int64_t n, int64_t C, const float *gamma, const float *beta,
                    int relu, float *y, float *save_mean, float *save_min, float *save_max,
                    qbp_qparams *out_range, void *ws, size_t ws_bytes, void *stream);

/* Requantisation for the next layer, fused into the pass that writes an
 * activation.  Section 4 ("Quantization methods"): the minimum and maximum of
 * an activation are known from the Range BN that produced it, so finding the
 * quantiser's scale costs no further pass over the tensor.  The exact range
 * of y follows from the per-channel statistics (y is a monotone function of x
 * in each channel, evaluated in a fixed fp32 order, so its extremes sit at the
 * channel's min and max); the apply pass then writes, beside y or instead of
 * it, the 8-bit codes that qbp_quantize_s8(y, per-tensor, nearest) would
 * produce, bit for bit:
 *   q        [n x C] int8 codes (required)
 *   qp       their parameters (required)
 *   row_sums  [n] sum of each row's stored codes (nullable) -- the code sums
 *             the next product's zero-point correction needs (Appendix B);
 *   chan_sums [C] sum of each channel's stored codes over all rows, int64
 *             (nullable) -- what the next layer's weight gradient needs for
 *             its zero-point terms (fewer than 2^22 rows). */
typedef struct {
    int8_t      *q;
    qbp_qparams *qp;
    int32_t     *row_sums;
    int64_t     *chan_sums;
} qbp_requant;

/* qbp_rangebn_fwd with the fused requantisation rq (nullable); y may be NULL
 * when rq is given (the fp32 activation is then never written). */
int qbp_rangebn_fwd_q8(const float *x, int64_t n, int64_t C, const float *gamma, const float *beta,
                       int relu, float *y, float *save_mean, float *save_min, float *save_max,
                       qbp_qparams *out_range, const qbp_requant *rq,
                       void *ws, size_t ws_bytes, void *stream);

/* The two passes as separate calls, for a minibatch that is spread over
 * several GPUs (Section 3: the mean and the range are those of the whole
 * minibatch).  _stats leaves the per-channel sum (fp64), minimum and maximum
 * of this GPU's n rows in col_sum / col_min / col_max [C]; the caller combines
 * them over the GPUs (sum, min, max -- all order-free up to fp64 rounding of
 * the sum); _apply normalises this GPU's n_rows rows with the combined
 * statistics of n_stat >= n_rows rows (mean = sum / n_stat, C(n_stat)) and
 * fills save_* for the backward pass.  y / out_range / rq as above. */
int qbp_rangebn_fwd_stats(const float *x, int64_t n, int64_t C,
                          double *col_sum, float *col_min, float *col_max,
                          void *ws, size_t ws_bytes, void *stream);
int qbp_rangebn_fwd_apply(const float *x, int64_t n_rows, int64_t n_stat, int64_t C,
                          const double *col_sum, const float *col_min, const float *col_max,
                          const float *gamma, const float *beta, int relu,
                          float *y, float *save_mean, float *save_min, float *save_max,
                          qbp_qparams *out_range, const qbp_requant *rq, void *stream);

/* Backward -- Section 7: the derivative of max (min) is one at every
 * coordinate attaining it and zero elsewhere; otherwise the chain rule:
 *   dbeta = sum dy, dgamma = sum dy*xhat, s = 1/(C(n)(max-min)),
 *   dx = s*(gamma*dy - gamma*dbeta/n - C(n)*gamma*dgamma*([x==max]-[x==min])).
 * With relu, dy is first zeroed where the forward output was not positive. */
int qbp_rangebn_bwd(const float *dy, const float *x, int64_t n, int64_t C,
                    const float *gamma, const float *beta, int relu,
                    const float *save_mean, const float *save_min, const float *save_max,
                    float *dx, float *dgamma, float *dbeta,
                    void *ws, size_t ws_bytes, void *stream);

/* The backward passes as separate calls for a minibatch spread over several
 * GPUs: _stats leaves this GPU's sum dy and sum dy*xhat per channel (fp64,
 * [C] each; save_* are the combined statistics of the forward); the caller
 * adds them up over the GPUs; _apply writes dx for this GPU's rows and the
 * complete dgamma / dbeta (nullable) from the combined sums, with n_stat the
 * rows of the whole minibatch. */
int qbp_rangebn_bwd_stats(const float *dy, const float *x, int64_t n_rows, int64_t n_stat, int64_t C,
                          const float *gamma, const float *beta, int relu,
                          const float *save_mean, const float *save_min, const float *save_max,
                          double *sum_dy, double *sum_dyxhat,
                          void *ws, size_t ws_bytes, void *stream);
int qbp_rangebn_bwd_apply(const float *dy, const float *x, int64_t n_rows, int64_t n_stat, int64_t C,
                          const float *gamma, const float *beta, int relu,
                          const float *save_mean, const float *save_min, const float *save_max,
                          const double *sum_dy, const double *sum_dyxhat,
                          float *dx, float *dgamma, float *dbeta,
                          void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------
 * Whole layer -- Sections 4 and 6: forward = quantise x and w to 8 bits
 * (nearest) -> 8-bit product -> Range BN (+ReLU); backward = Range BN
 * backward -> bifurcate the gradient (8-bit and 16-bit copies, stochastic)
 * -> layer gradient from the 8-bit copy and the forward's weight codes, and
 * weight gradient from the 16-bit copy and the forward's input codes.
 * Linear: conv.R == 0, x [batch x in_features], w [in_features x
 * out_features] (y = x w).  Conv: x NHWC, w KRSC.
 * ---------------------------------------------------------------------- */
typedef struct {
    qbp_conv_desc conv;          /* conv.R == 0 selects the linear layer   */
    int64_t batch, in_features, out_features;   /* linear layer only       */
    int32_t relu;
    uint64_t seed;               /* Philox key of the stochastic rounding  */
    uint32_t tensor_id8, tensor_id16;
} qbp_layer_desc;

/* Caller-owned buffers: what the forward leaves for the backward, and the
 * backward's own intermediates (kept visible so that each stage can be
 * checked on its own).  Element counts: x_codes = |x|, w_codes = |w|; z, g,
 * g8, g_hi, g_lo = rows*channels of the product's output (rows = batch or
 * N*P*Q); z is the fp32 output of the product (the input of Range BN), g the
 * fp32 gradient arriving at it.  The g* members are used by the backward only.
 * g may be NULL: the backward pass then quantises the gradient as it computes
 * it and never writes it as fp32 (the exact range of the gradient follows from
 * per-channel extremes of dy that the statistics pass of the Range BN backward
 * takes: Section 4 takes a tensor's range from the operator that makes it).
 * That needs dy and z 16-byte aligned and the channel count a multiple of 4;
 * qbp_layer_bwd says so otherwise.
 * g_lo holds the low bytes of the 16-bit codes with their top bit flipped, i.e.
 * the signed bytes lo - 128 (g16 = 256*g_hi + (lo - 128) + 128): both limbs
 * then have one operand type and the layer's weight gradient runs them as one
 * product of twice the columns. */
typedef struct {
    int8_t *x_codes;  qbp_qparams *qx;
    int8_t *w_codes;  qbp_qparams *qw;
    float  *z;
    float  *save_mean, *save_min, *save_max;
    float  *g;
    int8_t *g8;       qbp_qparams *qg8;
    int8_t *g_hi;     uint8_t *g_lo;   qbp_qparams *qg16;
    /* nullable; convolution layers: [C] per-channel sums of the input codes over all positions, written by the
     * forward (by its quantiser, or handed on as in->chan_sums by the layer before) and read by the backward, whose
     * weight gradient then builds its zero-point terms from these totals and the border positions instead of a
     * pass over the three code tensors.  Fewer than 2^22 positions. */
    int64_t *x_chan_sums;
} qbp_layer_ctx;

size_t qbp_layer_workspace_bytes(const qbp_layer_desc *L);

/* A convolution layer with a small filter runs the filter's one-block kernels
 * on a stream of the library's own, forked from `stream` once the range of the
 * activation (forward) or gradient (backward) is enqueued and joined again
 * before the product, so that they overlap the pass that writes the codes.
 * That stream and its two events are created at the first such call of a host
 * thread on a device: make that call before any stream capture.  Under stream
 * capture the fork and join become part of the captured graph. */
int qbp_layer_fwd(const qbp_layer_desc *L, const float *x, const float *w,
                  const float *gamma, const float *beta, float *y, const qbp_layer_ctx *saved,
                  void *ws, size_t ws_bytes, void *stream);

/* Chained layers (Section 4: the quantiser of an activation takes its range
 * from the Range BN that produced the activation -- no range scan and no
 * separate quantisation pass between layers).
 *   in  (nullable): the input arrives already quantised -- the `out` record of
 *       the previous layer's call.  x must then be NULL, and in->q / in->qp
 *       must be the saved->x_codes / saved->qx of this layer (the backward
 *       pass reads the input codes from there), and in->chan_sums, if
 *       saved->x_chan_sums is used, that same buffer.  in->row_sums NULL: the
 *       code sums are computed here.
 *   out (nullable): also write the 8-bit codes of this layer's output for the
 *       next layer (see qbp_requant); y may then be NULL.
 * With in == NULL and out == NULL this is qbp_layer_fwd.
 *
 * Recompute instead of store (forward only; Section 7 argues the method's
 * gain in memory and bandwidth): with saved->z == NULL, y == NULL and out
 * given, a convolution layer of at most QBP_EPILOGUE_MAX_COLUMNS output
 * channels never writes the fp32 output of its product.  The convolution is
 * run twice: the first run leaves only the per-channel statistics of the
 * Range BN, the second normalises, rectifies and requantises in its epilogue
 * and writes one byte per output.  The codes and statistics are the same, bit
 * for bit, as with z kept; qbp_layer_bwd needs z and refuses such a record. */
int qbp_layer_fwd_chained(const qbp_layer_desc *L, const float *x, const qbp_requant *in,
                          const float *w, const float *gamma, const float *beta,
                          float *y, const qbp_requant *out, const qbp_layer_ctx *saved,
                          void *ws, size_t ws_bytes, void *stream);

int qbp_layer_bwd(const qbp_layer_desc *L, const qbp_layer_ctx *saved, const float *dy,
                  const float *gamma, const float *beta,
                  float *dx, float *dw, float *dgamma, float *dbeta,
                  void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------
 * Weight update -- Section 6 "Putting it all together": the updates are the
 * one operation kept in float32 (they accumulate small changes and run once
 * per minibatch).  The paper names stochastic gradient descent and no further
 * detail; this is the usual step with optional momentum and weight decay:
 *   g = dw + weight_decay * w;  v = momentum * v + g (momentum_buf non-NULL);
 *   w = w - lr * v   (or w - lr * g without a buffer),
 * each operation rounded to fp32 on its own, in this order.  w (master
 * weights, or gamma / beta of a Range BN) and momentum_buf are updated in
 * place; `count` elements.
 * ---------------------------------------------------------------------- */
int qbp_sgd_update(float *w, const float *dw, float *momentum_buf, int64_t count,
                   float lr, float momentum, float weight_decay, void *stream);

/* ------------------------------------------------------------------------
 * Appendix C -- Ternarized Back-Propagation: 1-bit weights and activations,
 * ternary gradients, every forward MAC an XNOR + popcount.
 *
 * Binary and ternary tensors are int8 codes with zero-point 0 here: the
 * +-1 dot product that XNOR + popcount computes is run by the int8 tensor
 * cores through qbp_gemm_s8 / qbp_conv_s8_implicit / qbp_wgrad_s16, whose
 * integer accumulators are that result exactly.
 *
 * qbp_binarize_s8: q[i] = +1 for x[i] >= 0 (also -0.0), else -1; n elements;
 * x 4-byte aligned (device), q (device).  qp_out (nullable, device) receives
 * scale 1, zero-point 0, the parameters to pass with q to a product.
 * Allocates nothing.
 *
 * qbp_stc_ternarize_s8: the stochastic ternarisation the appendix and its
 * Algorithm 1 use (not spelled out there; the one of the ternary-gradient
 * work the paper cites): s = max |g| over the n elements; a sample keeps
 * element i as sign(g[i]) with probability |g[i]| / s, else 0.  The draw is
 * taken in fp32: u = (word >> 8) * 2^-24 with the element's Philox4x32-10
 * word (block i / 4, word i % 4, counter words 2 and 3 = tensor_id and the
 * sample index, key = seed), kept iff u * s < |g[i]| (s > 0).  q[i] = the
 * sum of the element's `samples` (1..127) samples, in [-samples, samples];
 * qp_out: scale = s / samples (1 when s = 0), zero-point 0, vmin / vmax =
 * -s / s, so that scale * q[i] estimates g[i] without bias.  samples = 1 is
 * a ternary tensor.  ws of qbp_stc_ternarize_workspace_bytes() bytes.
 *
 * qbp_tbp_weight_gradient: Algorithm 1 (multiple stochastic ternarisation
 * sampling): the weight gradient of a binarised layer as the mean over
 * `samples` ternarisations of g of the product (ternary g)^T (binary a).
 * The samples are added per element first (the product is linear in them)
 * and one 16-bit x 8-bit product is run.  d == NULL: a [rows x K] (+-1
 * codes, parameters qa from qbp_binarize_s8), g [rows x N] fp32, gW [K x N];
 * d != NULL: a is the layer's NHWC input, g its NHWC output gradient, gW
 * [K][R][S][C] (rows, N, K are then taken from d).  t_hi / t_lo (device,
 * rows * N bytes each, 16-byte aligned) receive the byte limbs of the summed
 * samples, qp_t their parameters; acc_out (int64, nullable) the integer
 * accumulators, gW (nullable) = accumulator * qa.scale * qp_t.scale.  Shape
 * limits and errors as qbp_wgrad_s16.
 * ---------------------------------------------------------------------- */
int qbp_binarize_s8(const float *x, int64_t n, int8_t *q, qbp_qparams *qp_out, void *stream);
size_t qbp_stc_ternarize_workspace_bytes(void);
int qbp_stc_ternarize_s8(const float *g, int64_t n, int samples, uint64_t seed, uint32_t tensor_id,
                         int8_t *q, qbp_qparams *qp_out, void *ws, size_t ws_bytes, void *stream);
size_t qbp_tbp_weight_gradient_workspace_bytes(const qbp_conv_desc *d, int64_t rows, int64_t N, int64_t K);
int qbp_tbp_weight_gradient(const qbp_conv_desc *d, int64_t rows, int64_t N, int64_t K,
                            const int8_t *a_codes, const qbp_qparams *qa, const float *g,
                            int samples, uint64_t seed, uint32_t tensor_id,
                            int8_t *t_hi, uint8_t *t_lo, qbp_qparams *qp_t,
                            int64_t *acc_out, float *gW, void *ws, size_t ws_bytes, void *stream);

/* Bit rows and the literal XNOR + popcount products (Appendix C), for operands
 * kept at one bit per element (an eighth of the bytes of the code tensors).
 *
 * qbp_pack_bits: codes [rows x cols] (int8, device) to bit rows: element c of
 * a row is bit c % 32 of word c / 32 (1 for a code > 0; with mask != 0 for a
 * code != 0: the non-zero plane of a ternary tensor, whose sign plane is the
 * mask == 0 form); ceil(cols / 32) words per row, spare bits 0.
 *
 * qbp_xnor_gemm_bits: A_bits [M rows], B_bits [N rows] of K bits each;
 * C [M x N] (int32) = K - 2 popcount(a xor b), the dot product of the +-1
 * rows.  qbp_gated_xnor_gemm_bits: the same for a ternary left operand given
 * as its non-zero and sign planes: C = popcount(nz & ~(sg xor b)) -
 * popcount(nz & (sg xor b)).  Plain CUDA-core kernels bound by the popcount
 * unit; the same integers as qbp_gemm_s8 on the byte codes, which is the
 * faster route when the operands are bytes already.  M <= 4194240.  Allocate
 * nothing. */
int qbp_pack_bits(const int8_t *codes, int64_t rows, int64_t cols, int mask, uint32_t *words, void *stream);
int qbp_xnor_gemm_bits(int64_t M, int64_t N, int64_t K, const uint32_t *A_bits, const uint32_t *B_bits,
                       int32_t *C, void *stream);
int qbp_gated_xnor_gemm_bits(int64_t M, int64_t N, int64_t K, const uint32_t *nz_bits,
                             const uint32_t *sign_bits, const uint32_t *B_bits, int32_t *C, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* QBP_H_ */
