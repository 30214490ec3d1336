// Whole quantised layer (Sections 4 and 6): the composition of the library's
// own entry points in the order the method prescribes.
//   forward : quantise x, w to 8 bits (nearest) -> 8-bit product -> Range BN (+ReLU)
//   backward: Range BN backward -> gradient bifurcation (8-bit and 16-bit copies,
//             stochastic rounding) -> layer gradient from the 8-bit copy and the
//             forward's weight codes; weight gradient from the 16-bit copy and
//             the forward's input codes.
// The straight-through estimator through the quantiser is the identity here:
// the clamping values are the tensor's own min and max, so nothing is clipped.
// Everything is enqueued on the caller's stream; temporaries live in the
// caller's workspace.
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

struct LayerShape {
    bool conv;
    int64_t rows;        // batch, or N*H*W
    int64_t cin, cout;   // reduced / produced channels of the forward product
    int64_t x_elems, w_elems;
};

static int layer_shape(const qbp_layer_desc *L, LayerShape &s)
{
    if (!L) return fail(QBP_ERR_INVALID_ARG, "layer: descriptor is NULL");
    s.conv = L->conv.R != 0;
    if (s.conv) {
        const qbp_conv_desc &d = L->conv;
        if (d.N <= 0 || d.H <= 0 || d.W <= 0 || d.C <= 0 || d.K <= 0 || d.R <= 0 || d.S <= 0)
            return fail(QBP_ERR_INVALID_ARG, "layer: bad convolution geometry");
        // what every product of the step implements, checked before anything is launched
        if (!conv_supported(&d) || !wgrad_conv_supported(&d))
            return fail(QBP_ERR_UNSUPPORTED_SHAPE,
                        "layer: needs stride 1, R = S in {1,3}, pad = (R-1)/2, C and K multiples of 32");
        if ((int64_t)d.R * d.S * std::max(d.C, d.K) > 33025)
            return fail(QBP_ERR_OVERFLOW_K, "layer: reduction length exceeds 33025");
        s.rows = (int64_t)d.N * d.H * d.W; s.cin = d.C; s.cout = d.K;
        s.x_elems = s.rows * d.C; s.w_elems = (int64_t)d.K * d.R * d.S * d.C;
    } else {
        if (L->batch <= 0 || L->in_features <= 0 || L->out_features <= 0)
            return fail(QBP_ERR_INVALID_ARG, "layer: batch, in_features, out_features must be positive");
        if (L->batch % 16 || L->in_features % 16 || L->out_features % 16)
            return fail(QBP_ERR_UNSUPPORTED_SHAPE, "layer: batch, in_features, out_features must be multiples of 16");
        if (L->in_features > 33025 || L->out_features > 33025)
            return fail(QBP_ERR_OVERFLOW_K, "layer: in_features and out_features are reduction lengths of 8-bit products (at most 33025)");
        s.rows = L->batch; s.cin = L->in_features; s.cout = L->out_features;
        s.x_elems = s.rows * s.cin; s.w_elems = s.cin * s.cout;
    }
    if (s.rows < 2) return fail(QBP_ERR_INVALID_ARG, "layer: Range BN needs at least 2 rows");
    return QBP_OK;
}

// The layer's workspace: [0, kLayerHead) the sticky status word of the whole step (cleared once by the forward
// call, raised by any product whose bounded wait runs out, never overwritten by a later step), then the scratch
// the steps share (they run one after another on the stream), then the buffers that live across steps.
constexpr size_t kLayerHead = 256;

// A small filter's kernels (one block each, some ten microseconds of latency) need the quantiser parameters of the
// activation or gradient they are paired with, but not its codes: they run on a stream of the library's own beside
// the pass that writes those codes, forked from the caller's stream after the parameters and joined before the
// product.  One stream and two events per host thread and device, made at first use (a first call should therefore
// come before any stream capture); when they cannot be made the kernels simply run in line.
struct SideStream { cudaStream_t s; cudaEvent_t fork, join; bool ok; };
static SideStream *side_stream()
{
    thread_local SideStream cache[kMaxDevices] = {};
    thread_local bool tried[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    SideStream &c = cache[dev];
    if (!tried[dev]) {
        tried[dev] = true;
        c.ok = cudaStreamCreateWithFlags(&c.s, cudaStreamNonBlocking) == cudaSuccess &&
               cudaEventCreateWithFlags(&c.fork, cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&c.join, cudaEventDisableTiming) == cudaSuccess;
        if (!c.ok) (void)cudaGetLastError();
    }
    return c.ok ? &c : nullptr;
}
// Runs what the caller enqueues on `side` between the event `fork` (already recorded on st) and the rest of st.
static int side_begin(SideStream *sd) { QBP_CUDA_OK(cudaStreamWaitEvent(sd->s, sd->fork, 0)); return QBP_OK; }
static int side_end(SideStream *sd, cudaStream_t st)
{
    QBP_CUDA_OK(cudaEventRecord(sd->join, sd->s));
    QBP_CUDA_OK(cudaStreamWaitEvent(st, sd->join, 0));
    return QBP_OK;
}

static size_t step_scratch_bytes(const qbp_layer_desc *L, const LayerShape &s)
{
    size_t b = qbp_quantize_workspace_bytes(s.rows, std::max(s.cin, s.cout), QBP_PER_TENSOR);
    b = std::max(b, qbp_rangebn_workspace_bytes(s.rows, s.cout));
    if (s.conv) {
        b = std::max(b, qbp_conv_s8_workspace_bytes(QBP_CONV_FPROP, &L->conv));
        b = std::max(b, qbp_wgrad_s16_workspace_bytes(&L->conv, 0, 0, 0));
    } else {
        b = std::max(b, qbp_gemm_s8_workspace_bytes(s.rows, std::max(s.cin, s.cout), std::max(s.cin, s.cout)));
        b = std::max(b, qbp_wgrad_s16_workspace_bytes(nullptr, s.rows, s.cout, s.cin));
    }
    return align_up(b, 256);
}

// Buffers that live across steps, behind the shared step scratch: the per-row sums of the codes feeding the
// next product (written by the quantiser that makes the codes) and the range partials of the gradient
// (written by the Range BN backward pass that makes the gradient).
// (a convolution's epilogue takes the output's per-channel statistics for any number of channels that leaves a CTA one
// column tile: 256 channels per tile, one CTA per SM)
static bool epilogue_stats(const LayerShape &s) { return s.conv && (s.cout + 255) / 256 <= sm_count(); }
static size_t colstat_cells(const LayerShape &s) { return epilogue_stats(s) ? (size_t)colstat_rows_max() * (size_t)s.cout : 0; }
static size_t chained_bytes(const LayerShape &s)
{
    // ... and the per-channel (sum, min, max) partials of the layer output that the convolution's epilogue leaves
    // for the Range BN forward, and the per-channel constants of the normalisation for the recompute fusion
    return align_up(sizeof(int32_t) * (size_t)s.rows, 256) + align_up(sizeof(float2) * rangebn_range_parts_capacity(s.cout), 256) +
           2 * align_up(sizeof(float) * colstat_cells(s), 256) + align_up(sizeof(double) * colstat_cells(s), 256) +
           align_up(sizeof(float4) * (size_t)s.cout, 256) + align_up(sizeof(int32_t) * 16 * (size_t)std::max(s.cin, s.cout), 256) +
           align_up(sizeof(int64_t) * (size_t)s.cout, 256);
}
// The forward column terms that come with the filter's codes (the piece before the last of the region above).
static int32_t *colterm_buffer(const qbp_layer_desc *L, const LayerShape &s, void *ws_after_head)
{
    return reinterpret_cast<int32_t *>(static_cast<char *>(ws_after_head) + step_scratch_bytes(L, s) + chained_bytes(s) -
                                       align_up(sizeof(int64_t) * (size_t)s.cout, 256) -
                                       align_up(sizeof(int32_t) * 16 * (size_t)std::max(s.cin, s.cout), 256));
}
// The per-channel totals of the 16-bit gradient codes (last piece of the region above).
static int64_t *tot_g_buffer(const qbp_layer_desc *L, const LayerShape &s, void *ws_after_head)
{
    return reinterpret_cast<int64_t *>(static_cast<char *>(ws_after_head) + step_scratch_bytes(L, s) + chained_bytes(s) -
                                       align_up(sizeof(int64_t) * (size_t)s.cout, 256));
}

// Recompute instead of store (motivated by Section 7's memory and bandwidth argument): convolution -> Range BN
// (+ReLU) -> 8-bit codes for the next layer without ever writing the fp32 output of the product.  The
// convolution runs twice: the first run leaves only the per-channel statistics (its epilogue stores nothing), the
// second run normalises, rectifies and requantises in its epilogue and writes one byte per output.
static int conv_rangebn_recompute(const qbp_conv_desc *d, const int8_t *x_codes, const qbp_qparams *qx, const int32_t *in_sums,
                                  const int8_t *w_codes, const qbp_qparams *qw, const float *gamma, const float *beta, int relu,
                                  float *save_mean, float *save_min, float *save_max, const qbp_requant *out,
                                  ColStatParts parts, float4 *fold, const int32_t *colterm, int *status, void *ws, size_t scratch,
                                  cudaStream_t st)
{
    const int64_t rows = (int64_t)d->N * d->H * d->W;
    const EpilogueTail first{nullptr, 0, nullptr, nullptr, nullptr, 0, colterm};
    int rc = conv_s8_impl(QBP_CONV_FPROP, d, x_codes, qx, w_codes, qw, nullptr, nullptr, in_sums, &parts, status, ws, scratch, st,
                          colterm ? &first : nullptr);
    if (rc) return rc;
    if ((rc = rangebn_fold_from_parts(rows, d->K, gamma, beta, relu, save_mean, save_min, save_max, parts, out->qp, fold, st))) return rc;
    const EpilogueTail tail{fold, relu, out->qp, out->q, out->row_sums, 1, colterm};
    rc = conv_s8_impl(QBP_CONV_FPROP, d, x_codes, qx, w_codes, qw, nullptr, nullptr, in_sums, nullptr, status, ws, scratch, st, &tail);
    if (rc || !out->chan_sums) return rc;
    return launch_colsum(out->q, true, rows, d->K, out->chan_sums, st);
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) size_t qbp_layer_workspace_bytes(const qbp_layer_desc *L)
{
    LayerShape s;
    if (layer_shape(L, s)) return 0;
    return kLayerHead + step_scratch_bytes(L, s) + chained_bytes(s);
}

extern "C" __attribute__((visibility("default"))) int qbp_layer_fwd(const qbp_layer_desc *L, const float *x,
                                                                   const float *w, const float *gamma,
                                                                   const float *beta, float *y,
                                                                   const qbp_layer_ctx *saved, void *ws,
                                                                   size_t ws_bytes, void *stream)
{
    if (!x || !y) return fail(QBP_ERR_INVALID_ARG, "layer_fwd: NULL argument");
    return qbp_layer_fwd_chained(L, x, nullptr, w, gamma, beta, y, nullptr, saved, ws, ws_bytes, stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_layer_fwd_chained(const qbp_layer_desc *L, const float *x,
                                                                           const qbp_requant *in, const float *w,
                                                                           const float *gamma, const float *beta,
                                                                           float *y, const qbp_requant *out,
                                                                           const qbp_layer_ctx *saved, void *ws,
                                                                           size_t ws_bytes, void *stream)
{
    LayerShape s;
    int rc = layer_shape(L, s);
    if (rc) return rc;
    if (!w || !saved) return fail(QBP_ERR_INVALID_ARG, "layer_fwd: NULL argument");
    if ((x != nullptr) == (in != nullptr))
        return fail(QBP_ERR_INVALID_ARG, "layer_fwd: exactly one of x (fp32 input) and in (input already quantised) is needed");
    if (!y && !out) return fail(QBP_ERR_INVALID_ARG, "layer_fwd: neither y nor 8-bit output codes wanted");
    if (out && (!out->q || !out->qp)) return fail(QBP_ERR_INVALID_ARG, "layer_fwd: the output record needs q and qp");
    if (!saved->x_codes || !saved->qx || !saved->w_codes || !saved->qw || !saved->save_mean ||
        !saved->save_min || !saved->save_max)
        return fail(QBP_ERR_INVALID_ARG, "layer_fwd: the saved-state record has a NULL buffer");
    // saved->z == NULL: the fp32 output of the product is not kept (forward only): the convolution is run twice instead
    const bool recompute = saved->z == nullptr;
    if (recompute && !(s.conv && s.cout <= QBP_EPILOGUE_MAX_COLUMNS && out && !y))
        return fail(QBP_ERR_INVALID_ARG, "layer_fwd: without saved->z the layer must be a convolution of at most %d output "
                    "channels that writes 8-bit codes only (out given, y NULL)", QBP_EPILOGUE_MAX_COLUMNS);
    if (in && (in->q != saved->x_codes || in->qp != saved->qx))
        return fail(QBP_ERR_INVALID_ARG, "layer_fwd: in->q / in->qp must be the layer's saved x_codes / qx");
    const bool want_totals = s.conv && saved->x_chan_sums != nullptr;
    if (want_totals && s.rows >= (1ll << 22)) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "layer_fwd: x_chan_sums for fewer than 2^22 positions");
    if (want_totals && in && in->chan_sums && in->chan_sums != saved->x_chan_sums)
        return fail(QBP_ERR_INVALID_ARG, "layer_fwd: in->chan_sums must be the layer's saved x_chan_sums");
    if (!ws || ws_bytes < qbp_layer_workspace_bytes(L))
        return fail(QBP_ERR_WORKSPACE, "layer_fwd: workspace of %zu bytes needed, %zu given",
                    qbp_layer_workspace_bytes(L), ws_bytes);
    const size_t scratch = step_scratch_bytes(L, s);
    cudaStream_t st = (cudaStream_t)stream;
    int *status = static_cast<int *>(ws);
    QBP_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
    ws = static_cast<char *>(ws) + kLayerHead;

    // activations: nearest rounding, clamping values = min and max (Appendix B) -- or already quantised by the
    // Range BN of the layer before (Section 4)
    // (convolution: each pixel's code sum is needed for the zero-point correction of the product)
    int32_t *row_sums = reinterpret_cast<int32_t *>(static_cast<char *>(ws) + scratch);
    const int32_t *in_sums = s.conv ? row_sums : nullptr;
    // (a small filter's launch runs beside the pass that writes the input codes)
    const bool small_filter = s.conv && filter_prep_supported(&L->conv, w, saved->w_codes);
    SideStream *sd = (x && small_filter) ? side_stream() : nullptr;
    if (x) {
        bool left = false;
        rc = quantize_s8_with_totals(x, s.rows, s.cin, saved->x_codes, saved->qx, s.conv ? row_sums : nullptr,
                                     want_totals ? saved->x_chan_sums : nullptr, &left, ws, scratch, st, sd ? sd->fork : nullptr);
        if (rc) return rc;
        // (a shape the quantiser cannot take the totals of: one pass over the codes)
        if (want_totals && !left && (rc = launch_colsum(saved->x_codes, true, s.rows, s.cin, saved->x_chan_sums, st))) return rc;
    } else if (s.conv) {
        if (in->row_sums) in_sums = in->row_sums;
        else if ((rc = launch_rowsum(in->q, true, s.rows, s.cin, row_sums, st))) return rc;
        if (want_totals && !in->chan_sums && (rc = launch_colsum(in->q, true, s.rows, s.cin, saved->x_chan_sums, st))) return rc;
    }
    // weights: nearest rounding, clamping values = min and max (a small filter: scan, codes, code sums and the forward
    // product's column terms in one launch)
    const int64_t w_rows = s.conv ? (int64_t)L->conv.K * L->conv.R * L->conv.S : s.cin;
    const int32_t *colterm = nullptr;
    if (small_filter) {
        int32_t *ct = colterm_buffer(L, s, ws);
        if (sd && (rc = side_begin(sd))) return rc;
        if ((rc = launch_filter_prep(&L->conv, w, saved->qx, saved->w_codes, saved->qw, ct, sd ? sd->s : st))) return rc;
        if (sd && (rc = side_end(sd, st))) return rc;
        colterm = ct;
    } else {
        rc = qbp_quantize_s8(w, w_rows, s.w_elems / w_rows, QBP_PER_TENSOR, QBP_ROUND_NEAREST, 0, 0, nullptr,
                             saved->w_codes, saved->qw, nullptr, nullptr, ws, scratch, stream);
        if (rc) return rc;
    }
    const EpilogueTail with_colterm{nullptr, 0, nullptr, nullptr, nullptr, 0, colterm};
    ColStatParts parts{nullptr, nullptr, nullptr, 0};
    if (epilogue_stats(s)) {
        char *base = static_cast<char *>(ws) + scratch + align_up(sizeof(int32_t) * (size_t)s.rows, 256) +
                     align_up(sizeof(float2) * rangebn_range_parts_capacity(s.cout), 256);
        parts.lo = reinterpret_cast<float *>(base);
        parts.hi = reinterpret_cast<float *>(base + align_up(sizeof(float) * colstat_cells(s), 256));
        parts.sum = reinterpret_cast<double *>(base + 2 * align_up(sizeof(float) * colstat_cells(s), 256));
    }
    if (recompute) {
        float4 *fold = reinterpret_cast<float4 *>(reinterpret_cast<char *>(parts.sum) + align_up(sizeof(double) * colstat_cells(s), 256));
        return conv_rangebn_recompute(&L->conv, saved->x_codes, saved->qx, in_sums, saved->w_codes, saved->qw, gamma, beta, L->relu,
                                      saved->save_mean, saved->save_min, saved->save_max, out, parts, fold, colterm, status, ws,
                                      scratch, st);
    }
    if (s.conv)
        rc = conv_s8_impl(QBP_CONV_FPROP, &L->conv, saved->x_codes, saved->qx, saved->w_codes, saved->qw, nullptr, saved->z,
                          in_sums, parts.sum ? &parts : nullptr, status, ws, scratch, st, colterm ? &with_colterm : nullptr);
    else
        rc = gemm_s8_impl(0, 0, s.rows, s.cout, s.cin, saved->x_codes, saved->qx, saved->w_codes, saved->qw, nullptr,
                          saved->z, nullptr, status, ws, scratch, st);
    if (rc) return rc;
    // the convolution's epilogue has left the statistics of z: no pass over z for them
    if (parts.sum)
        return rangebn_fwd_from_parts(saved->z, s.rows, s.cout, gamma, beta, L->relu, y, saved->save_mean, saved->save_min,
                                      saved->save_max, parts, nullptr, out, st);
    return qbp_rangebn_fwd_q8(saved->z, s.rows, s.cout, gamma, beta, L->relu, y, saved->save_mean, saved->save_min,
                              saved->save_max, nullptr, out, ws, scratch, stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_layer_bwd(const qbp_layer_desc *L, const qbp_layer_ctx *saved,
                                                                   const float *dy, const float *gamma,
                                                                   const float *beta, float *dx, float *dw,
                                                                   float *dgamma, float *dbeta, void *ws,
                                                                   size_t ws_bytes, void *stream)
{
    LayerShape s;
    int rc = layer_shape(L, s);
    if (rc) return rc;
    if (!saved || !dy || !dx || !dw) return fail(QBP_ERR_INVALID_ARG, "layer_bwd: NULL argument");
    if (!ws || ws_bytes < qbp_layer_workspace_bytes(L))
        return fail(QBP_ERR_WORKSPACE, "layer_bwd: workspace of %zu bytes needed, %zu given",
                    qbp_layer_workspace_bytes(L), ws_bytes);
    if (!saved->g8 || !saved->qg8 || !saved->g_hi || !saved->g_lo || !saved->qg16 || !saved->z)
        return fail(QBP_ERR_INVALID_ARG, "layer_bwd: the saved-state record has a NULL buffer (the backward pass needs z and the gradient buffers)");
    const size_t scratch = step_scratch_bytes(L, s);
    float *g = saved->g;
    int8_t *g8 = saved->g8, *ghi = saved->g_hi;
    uint8_t *glo = saved->g_lo;
    qbp_qparams *qp8 = saved->qg8, *qp16 = saved->qg16;

    cudaStream_t st = (cudaStream_t)stream;
    int *status = static_cast<int *>(ws);          // the forward call cleared it; the backward only ever raises it
    ws = static_cast<char *>(ws) + kLayerHead;
    int32_t *row_sums = reinterpret_cast<int32_t *>(static_cast<char *>(ws) + scratch);
    float2 *range_parts = reinterpret_cast<float2 *>(static_cast<char *>(ws) + scratch + align_up(sizeof(int32_t) * (size_t)s.rows, 256));
    // two copies of the gradient: 8 bits for the layer gradient, 16 bits for the weight gradient
    // (convolution with the input's per-channel code totals at hand: the bifurcation leaves the gradient's, and the
    // weight gradient reads only the border positions again for its zero-point terms)
    // ... and when the weight-gradient product has a spare chunk of MMA rows, it takes the gradient's totals itself
    const bool self_totals = s.conv && saved->x_chan_sums && wgrad_self_totals(&L->conv) && s.rows < (1ll << 22);
    const bool totals = s.conv && saved->x_chan_sums && (self_totals || quantizer_totals_supported(s.cout)) && s.rows < (1ll << 22);
    int64_t *tot_g = totals ? tot_g_buffer(L, s, ws) : nullptr;
    // (a small filter: the layer gradient's column terms in one launch, beside the bifurcation -- they need the
    // gradient's parameters only; else two kernels inside the product's call)
    const bool small = s.conv && (int64_t)L->conv.R * L->conv.S * L->conv.C <= 12288 && s.w_elems <= 49152 && L->conv.C % 4 == 0;
    SideStream *sd = small ? side_stream() : nullptr;
    // Range BN backward and the two copies of its result.  Where the shape allows, in two passes over (dy, z): the
    // statistics pass also takes the extremes of dy, from which the exact range of the gradient follows (Section 4:
    // the range without a scan), and the second pass quantises the gradient as it computes it -- the fp32 gradient is
    // written only when the caller keeps saved->g.  Else: the pass that writes the gradient leaves its range, and the
    // bifurcation reads the gradient back.
    const bool two_pass = rangebn_bwd_bifurcate_supported(dy, saved->z, g, s.rows, s.cout, s.conv);
    if (two_pass) {
        rc = rangebn_bwd_bifurcate_impl(dy, saved->z, s.rows, s.cout, gamma, beta, L->relu, saved->save_mean, saved->save_min,
                                        saved->save_max, g, dgamma, dbeta, L->seed, L->tensor_id8, L->tensor_id16, g8, qp8,
                                        s.conv ? row_sums : nullptr, ghi, glo, qp16, true, ws, scratch, st, sd ? sd->fork : nullptr,
                                        self_totals ? nullptr : tot_g);
    } else {
        if (!g) return fail(QBP_ERR_INVALID_ARG, "layer_bwd: this shape needs saved->g (the fp32 gradient is written and read back)");
        int nparts = 0;
        rc = rangebn_bwd_impl(dy, saved->z, s.rows, s.cout, gamma, beta, L->relu, saved->save_mean, saved->save_min,
                              saved->save_max, g, dgamma, dbeta, ws, scratch, range_parts, &nparts, st);
        if (rc) return rc;
        rc = bifurcate_with_range_partials(g, s.rows, s.cout, L->seed, L->tensor_id8, L->tensor_id16, g8, qp8,
                                           s.conv ? row_sums : nullptr, ghi, glo, qp16, range_parts, nparts, st,
                                           self_totals ? nullptr : tot_g, true, sd ? sd->fork : nullptr);
    }
    if (rc) return rc;
    if (s.conv) {
        int32_t *ct = small ? colterm_buffer(L, s, ws) : nullptr;
        if (small) {
            if (sd && (rc = side_begin(sd))) return rc;
            if ((rc = launch_filter_dgrad_colterm(&L->conv, saved->w_codes, qp8, ct, sd ? sd->s : st))) return rc;
            if (sd && (rc = side_end(sd, st))) return rc;
        }
        const EpilogueTail with_colterm{nullptr, 0, nullptr, nullptr, nullptr, 0, ct};
        rc = conv_s8_impl(QBP_CONV_DGRAD, &L->conv, g8, qp8, saved->w_codes, saved->qw, nullptr, dx, row_sums, nullptr, status, ws, scratch, st,
                          small ? &with_colterm : nullptr);
        if (rc) return rc;
        return wgrad_s16_impl(&L->conv, 0, 0, 0, saved->x_codes, saved->qx, ghi, glo, qp16, nullptr, dw, status, ws, scratch, st,
                              totals ? saved->x_chan_sums : nullptr, tot_g, !self_totals, true);
    }
    // dx [batch x in] = g8 [batch x out] . w^T, w stored [in x out]
    rc = gemm_s8_impl(0, 1, s.rows, s.cin, s.cout, g8, qp8, saved->w_codes, saved->qw, nullptr, dx, nullptr, status, ws, scratch, st);
    if (rc) return rc;
    return wgrad_s16_impl(nullptr, s.rows, s.cout, s.cin, saved->x_codes, saved->qx, ghi, glo, qp16, nullptr, dw, status, ws,
                          scratch, st, nullptr, nullptr, true, true);
}
