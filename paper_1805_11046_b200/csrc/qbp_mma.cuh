// Declarations shared by the tensor-core product files: TMA tensor-map
// construction on the host, the parameter block of the tcgen05 kernels, and
// the small helper launchers (row/column sums of codes).
#pragma once

#include <cuda.h>

#include "qbp_common.cuh"

namespace qbp {

// ---- sums of stored codes (qbp_quant.cu) -------------------------------------
int launch_rowsum(const void *q, bool is_signed, int64_t rows, int64_t cols, int32_t *sums, cudaStream_t st);
int launch_colsum(const void *q, bool is_signed, int64_t rows, int64_t cols, int64_t *sums, cudaStream_t st);

// ---- per-tensor range scan (qbp_quant.cu): *qp = 8-bit parameters of [min(lowest, 0), max(highest, 0)] -------------
size_t range_scan_ws_bytes();
int range_scan(const float *x, int64_t n, void *ws, size_t ws_bytes, qbp_qparams *qp, cudaStream_t st);

// ---- pieces the whole-layer composition chains without a pass of their own ------
// Range BN backward that also leaves per-block (min, max) of dx (qbp_rangebn.cu), and the gradient
// bifurcation that starts from such partials instead of scanning (qbp_quant.cu).
int rangebn_bwd_impl(const float *dy, const float *x, int64_t n, int64_t C, const float *gamma, const float *beta,
                     int relu, const float *save_mean, const float *save_min, const float *save_max, float *dx,
                     float *dgamma, float *dbeta, void *ws, size_t ws_bytes, float2 *range_parts, int *nparts,
                     cudaStream_t st);
size_t rangebn_range_parts_capacity(int64_t C);
// Range BN backward and the bifurcation of the gradient in two passes, the fp32 gradient optional (qbp_rangebn.cu).
bool rangebn_bwd_bifurcate_supported(const float *dy, const float *x, const float *g_out, int64_t n, int64_t C, bool row_sums);
int rangebn_bwd_bifurcate_impl(const float *dy, const float *x, int64_t n, int64_t C, const float *gamma, const float *beta,
                               int relu, const float *save_mean, const float *save_min, const float *save_max, float *g_out,
                               float *dgamma, float *dbeta, uint64_t seed, uint32_t id8, uint32_t id16, int8_t *q8,
                               qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi, uint8_t *lo, qbp_qparams *qp16, bool lo_signed,
                               void *ws, size_t ws_bytes, cudaStream_t st, cudaEvent_t after_range = nullptr,
                               int64_t *tot16 = nullptr);      // tot16 (nullable) [C]: per-channel totals of the stored 16-bit codes
int launch_range_finalize(const float2 *partials, int nparts, qbp_qparams *qp8, qbp_qparams *qp16, cudaStream_t st,
                          cudaEvent_t after_range = nullptr);
int bifurcate_with_range_partials(const float *g, int64_t rows, int64_t cols, uint64_t seed, uint32_t tensor_id8,
                                  uint32_t tensor_id16, int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi,
                                  uint8_t *lo, qbp_qparams *qp16, const float2 *partials, int nparts, cudaStream_t st,
                                  int64_t *tot16 = nullptr, bool lo_signed = false, cudaEvent_t after_range = nullptr);
// after_range (here and in quantize_s8_with_totals; nullable): an event recorded on the stream as soon as the quantiser's
// parameters are enqueued, before the pass that writes the codes.
// Whether the quantising kernels can leave per-channel totals for a tensor of `cols` channels.
bool quantizer_totals_supported(int64_t cols);
int quantize_s8_with_totals(const float *x, int64_t rows, int64_t cols, int8_t *q, qbp_qparams *qp_out, int32_t *row_sums,
                            int64_t *tot8, bool *left, void *ws, size_t ws_bytes, cudaStream_t st, cudaEvent_t after_range = nullptr);
// The convolution products with the per-pixel channel sums of the input codes supplied by the caller
// (nullable: computed here) (qbp_mma.cu).
// Per-column (sum, min, max) of a product's fp32 output as partial rows [rows][N], one per CTA
// of the tensor-core kernel; `rows` is filled in by the launch.  colstat_rows_max(): the most rows a launch leaves.
struct ColStatParts { float *lo, *hi; double *sum; int rows; };
int colstat_rows_max();
int rangebn_fold_from_parts(int64_t n, int64_t C, const float *gamma, const float *beta, int relu, float *save_mean,
                            float *save_min, float *save_max, const ColStatParts &parts, qbp_qparams *qp8_out,
                            float4 *fold, cudaStream_t st);
// Optional tail of a product's epilogue: per-column normalisation (fold: (mean, scale, gamma, beta) per output
// column, as rangebn_fold_from_parts leaves them), ReLU, and 8-bit codes of the result with parameters *rq
// (q [M x N], row_sums [M] nullable).  keep_terms: the zero-point term kernels ran for the same operands in the
// call just before on the same workspace and are not run again.
// colterm (nullable): the column terms [16][N] of this product, already computed (launch_filter_prep).
struct EpilogueTail { const float4 *fold; int relu; const qbp_qparams *rq; int8_t *q; int32_t *row_sums; int keep_terms; const int32_t *colterm; };
// A small filter quantised and its forward column terms computed in one launch (qbp_mma.cu).
bool filter_prep_supported(const qbp_conv_desc *d, const float *w, const int8_t *codes);
int launch_filter_prep(const qbp_conv_desc *d, const float *w, const qbp_qparams *q_in, int8_t *codes, qbp_qparams *qw,
                       int32_t *colterm, cudaStream_t st);
// ... and the layer-gradient product's column terms [16][C] from such a filter's codes, in one launch.
int launch_filter_dgrad_colterm(const qbp_conv_desc *d, const int8_t *codes, const qbp_qparams *q_g, int32_t *colterm, cudaStream_t st);

// ext_status (here and below; nullable): a status word the caller owns and has cleared -- the product raises it when
// a bounded wait runs out and never clears it; NULL: the word is the first int of `ws`, cleared by the call itself.
int conv_s8_impl(int mode, const qbp_conv_desc *d, const int8_t *in, const qbp_qparams *q_in, const int8_t *wgt,
                 const qbp_qparams *q_w, int32_t *acc_out, float *out, const int32_t *in_chan_sum, ColStatParts *stats,
                 int *ext_status, void *ws, size_t ws_bytes, cudaStream_t st, const EpilogueTail *tail = nullptr);
int gemm_s8_impl(int transA, int transB, int64_t M, int64_t N, int64_t K, const int8_t *A, const qbp_qparams *qa,
                 const int8_t *B, const qbp_qparams *qb, int32_t *acc_out, float *C, const qbp_epilogue *ep,
                 int *ext_status, void *ws, size_t ws_bytes, cudaStream_t st, const int32_t *a_sums = nullptr,
                 const int32_t *b_sums = nullptr);
// tot_x [C] / tot_g16 [K] (convolution; nullable, both or none): per-channel totals of the stored x codes and of the
// stored 16-bit gradient codes (256 * hi + lo) over all positions, left by the kernels that wrote the codes.
// lo_signed: g_lo holds the low bytes with the top bit flipped, i.e. the signed bytes lo - 128 (lo_signed in
// bifurcate_with_range_partials): g16 - zg = 256 * hi + (lo - 128) - (zg - 128), so the two limbs have one operand
// type and run as one product of twice the columns (the x tile is read from shared memory once, not once per limb),
// with zg - 128 as the zero-point.
int wgrad_s16_impl(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K, const int8_t *x, const qbp_qparams *qx,
                   const int8_t *g_hi, const uint8_t *g_lo, const qbp_qparams *qg16, int64_t *acc_out, float *dW,
                   int *ext_status, void *ws, size_t ws_bytes, cudaStream_t st, const int64_t *tot_x = nullptr,
                   const int64_t *tot_g16 = nullptr, bool tot_g_filled = true, bool lo_signed = false);
// tot_g_filled == false: tot_g16 is a buffer [K] that the product fills itself (possible when wgrad_self_totals(d)).
bool wgrad_self_totals(const qbp_conv_desc *d);
// Bifurcation with optional per-channel totals of the 16-bit codes (tot16 [cols], zeroed here) -- see above.
// Shapes the convolution products / the convolution weight gradient implement.
bool conv_supported(const qbp_conv_desc *d);
bool wgrad_conv_supported(const qbp_conv_desc *d);
// Range BN forward from such partials instead of a statistics pass over x (qbp_rangebn.cu).
// out_range / rq (each nullable): the exact range of y / its 8-bit codes for the next layer (see qbp_requant).
int rangebn_fwd_from_parts(const float *x, int64_t n, int64_t C, const float *gamma, const float *beta, int relu, float *y,
                           float *save_mean, float *save_min, float *save_max, const ColStatParts &parts,
                           qbp_qparams *out_range, const qbp_requant *rq, cudaStream_t st);

// ---- TMA tensor maps ---------------------------------------------------------
// A dense byte matrix [rows x cols] (cols innermost) read in boxes of
// box_cols x box_rows; box_cols in {32, 64, 128} selects the matching swizzle.
int make_map_2d(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols);
// A dense NHWC byte tensor read in boxes of box_c x bw x bh x bn.
int make_map_nhwc(CUtensorMap *map, const void *base, uint64_t N, uint64_t H, uint64_t W, uint64_t C, uint32_t bn,
                  uint32_t bh, uint32_t bw, uint32_t box_c);

// fp32 output matrix [rows x cols] stored by TMA in boxes of 32 rows x 32 columns (128-byte swizzled slabs).
int make_map_out_2d(CUtensorMap *map, float *base, uint64_t rows, uint64_t cols);

// ---- the dense product on CTA pairs (qbp_mma2.cu) -------------------------------
bool gemm2_eligible(int64_t M, int64_t N, int64_t K);
int launch_gemm2(int transA, int transB, int64_t M, int64_t N, int64_t K, const int8_t *A, const qbp_qparams *qa,
                 const int8_t *B, const qbp_qparams *qb, int32_t *acc_out, float *C, const int32_t *rowterm,
                 const int32_t *colterm, int *status, bool clear_status, cudaStream_t st);

// ---- the dense weight gradient on CTA pairs (qbp_wgrad2.cu) ----------------------
bool wgrad2_eligible(int64_t M, int64_t N, int64_t K);
int launch_wgrad2(int64_t M, int64_t N, int64_t K, const int8_t *x, const qbp_qparams *qx, const int8_t *g_hi,
                  const uint8_t *g_lo, const qbp_qparams *qg16, int64_t *acc_out, float *dW, const long long *rowterm,
                  const long long *colterm, int *status, cudaStream_t st, bool lo_signed = false);

// ---- shared-memory operand descriptors ---------------------------------------
// How one operand tile of a pipeline stage is laid out and walked by the MMAs.
struct OperandLayout {
    uint32_t tile_bytes;    // bytes of this operand per stage
    uint32_t desc_lo;       // descriptor bits 16..31 (leading byte offset), address added at run time
    uint32_t desc_hi;       // descriptor bits 32..63 (stride byte offset, version, swizzle)
    uint32_t kstep;         // start-address advance per MMA (K = 32), in 16-byte units
    uint32_t major;         // 0 = K-major, 1 = MN-major (instruction descriptor bit)
};

// K-major tile: `rows` rows of `row_bytes` (32/64/128, swizzled alike) reduction bytes.
OperandLayout layout_kmajor(uint32_t rows, uint32_t row_bytes);
// MN-major tile: `krows` reduction rows of `row_bytes` (32/64/128) M/N bytes each;
// `chunks` such tiles side by side (chunk_stride bytes apart) widen M/N beyond row_bytes.
OperandLayout layout_mnmajor(uint32_t krows, uint32_t row_bytes, uint32_t chunks, uint32_t chunk_stride);

// ---- division by launch-time constants ----------------------------------------
// Division of a non-negative int (< 2^31) by a positive constant known at launch: multiply-high and
// shift (Granlund & Montgomery, "Division by invariant integers using multiplication").  The producer
// and MMA-issue threads run one dependent instruction at a time, so 32-bit divisions (some 25 dependent
// instructions each) per tile and per stage would dominate short tiles.
struct FastDiv {
    uint32_t mul, shr, d;
#ifdef __CUDACC__
    __device__ __forceinline__ int div(int n) const { return d == 1 ? n : (int)(__umulhi((uint32_t)n, mul) >> shr); }
    __device__ __forceinline__ void divmod(int n, int &q, int &r) const { q = div(n); r = n - q * (int)d; }
#endif
};
inline FastDiv make_fastdiv(int d)
{
    FastDiv f; f.d = (uint32_t)d; f.mul = 0; f.shr = 0;
    if (d > 1) {
        int lg = 0; while ((1ll << lg) < d) ++lg;
        const int p = 31 + lg;
        f.mul = (uint32_t)(((1ull << p) + (uint64_t)d - 1) / (uint64_t)d);
        f.shr = (uint32_t)(p - 32);
    }
    return f;
}

uint32_t make_idesc(bool a_signed, bool b_signed, uint32_t a_major, uint32_t b_major, uint32_t m, uint32_t n);

}  // namespace qbp
