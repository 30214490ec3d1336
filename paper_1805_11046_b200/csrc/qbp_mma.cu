// 8-bit integer products on the 5th-generation tensor cores:
//   y = W x and g_{l-1} = g_l W^T (Section 1; Eq. (grad_layer)) for linear
//   layers (GEMM) and for convolutions (implicit GEMM over the filter taps).
//
// This file: the persistent single-CTA kernel (convolutions, narrow GEMMs) and the entry points; the dense GEMM of
// at least one 256 x 256 tile runs on CTA pairs (qbp_mma2.cu).  One CTA per SM walks output tiles of 128 (or 2 x 128)
// rows x BN columns.  Warp 0 drives TMA (cp.async.bulk.tensor into 128B/64B/32B-swizzled shared-memory stages),
// warp 1 issues tcgen05.mma kind::i8 with int32 accumulators in tensor memory (the whole warp runs the loop, an
// elected lane issues: see issue_stage), up to twelve epilogue warps read accumulators back (tcgen05.ld), apply the
// zero-point correction, dequantise and store through swizzled slabs and TMA.  A 3 x 3 convolution loads the
// pixel box of a tile once with its border and takes the nine taps as shifted windows of that tile.  Stages are
// handed over with mbarriers; tcgen05.commit releases a stage when the MMAs that read it are done.  Every wait is
// bounded; on expiry the CTA raises the status word at the start of the workspace and leaves through the normal exit.
//
// The raw MMA sums stored codes; padding taps are zero-filled by TMA and so
// contribute nothing to the raw sum.  The sum over (q_a - z_a)(q_b - z_b) is
// recovered in the epilogue from code sums prepared by small helper kernels:
//   acc = raw + rowterm[m] + colterm[class(m)][n]
// where, for a convolution, class(m) says which taps of output pixel m fall
// inside the image (real-zero padding contributes nothing).
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

// =============================================================== tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return (EncodeTiledFn)p;
    }();
    return fn;
}

static CUtensorMapSwizzle swizzle_for(uint32_t inner_bytes)
{
    return inner_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
         : inner_bytes == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                              : CU_TENSOR_MAP_SWIZZLE_32B;
}

int make_map_2d(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    if (box_cols != 32 && box_cols != 64 && box_cols != 128) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "box of %u bytes", box_cols);
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_cols), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled(2d %llu x %llu, box %u x %u) failed: %d",
                                       (unsigned long long)rows, (unsigned long long)cols, box_rows, box_cols, (int)r);
    return QBP_OK;
}

int make_map_nhwc(CUtensorMap *map, const void *base, uint64_t N, uint64_t H, uint64_t W, uint64_t C, uint32_t bn,
                  uint32_t bh, uint32_t bw, uint32_t box_c)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    if (box_c != 32 && box_c != 64 && box_c != 128) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "box of %u bytes", box_c);
    cuuint64_t dims[4] = {C, W, H, N};
    cuuint64_t strides[3] = {C, W * C, H * W * C};
    cuuint32_t box[4] = {box_c, bw, bh, bn};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_c), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled(nhwc) failed: %d", (int)r);
    return QBP_OK;
}

// fp32 output matrix [rows x cols] stored in boxes of 32 rows x 32 columns (128-byte swizzled slabs).
int make_map_out_2d(CUtensorMap *map, float *base, uint64_t rows, uint64_t cols)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(float)};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled(fp32 output %llu x %llu) failed: %d",
                                       (unsigned long long)rows, (unsigned long long)cols, (int)r);
    return QBP_OK;
}

// fp32 NHWC output stored in boxes of 32 channels x (sw x sh x sn = 32 pixels).
int make_map_out_nhwc(CUtensorMap *map, float *base, uint64_t N, uint64_t H, uint64_t W, uint64_t C, uint32_t sn,
                      uint32_t sh, uint32_t sw)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t dims[4] = {C, W, H, N};
    cuuint64_t strides[3] = {C * sizeof(float), W * C * sizeof(float), H * W * C * sizeof(float)};
    cuuint32_t box[4] = {32, sw, sh, sn};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(QBP_ERR_CUDA, "cuTensorMapEncodeTiled(fp32 nhwc output) failed: %d", (int)r);
    return QBP_OK;
}

// ========================================================= operand descriptors
// Shared-memory matrix descriptor (64 bit): start address >> 4 in bits 0..13,
// leading byte offset >> 4 in 16..29, stride byte offset >> 4 in 32..45, the
// constant 1 in 46..47, swizzle mode in 61..63 (2 = 128B, 4 = 64B, 6 = 32B).
static uint32_t swizzle_code(uint32_t row_bytes) { return row_bytes == 128 ? 2u : row_bytes == 64 ? 4u : 6u; }

OperandLayout layout_kmajor(uint32_t rows, uint32_t row_bytes)
{
    OperandLayout L;
    L.tile_bytes = rows * row_bytes;
    L.desc_lo = 1u << 16;                                    // leading offset: unused for swizzled K-major
    L.desc_hi = ((8u * row_bytes) >> 4) | (1u << 14) | (swizzle_code(row_bytes) << 29);   // 8-row groups
    L.kstep = 32u >> 4;                                      // next 32 reduction bytes inside the swizzled row
    L.major = 0;
    return L;
}

OperandLayout layout_mnmajor(uint32_t krows, uint32_t row_bytes, uint32_t chunks, uint32_t chunk_stride)
{
    OperandLayout L;
    L.tile_bytes = chunks > 1 ? chunks * chunk_stride : krows * row_bytes;
    L.desc_lo = ((chunks > 1 ? chunk_stride : krows * row_bytes) >> 4) << 16;   // between M/N chunks
    L.desc_hi = ((8u * row_bytes) >> 4) | (1u << 14) | (swizzle_code(row_bytes) << 29);   // between 8-row K groups
    L.kstep = (32u * row_bytes) >> 4;                        // next 32 reduction rows
    L.major = 1;
    return L;
}

// Instruction descriptor of tcgen05.mma kind::i8: accumulator type in bits 4..5
// (2 = s32), A/B type in 7..9 / 10..12 (0 = u8, 1 = s8), A/B major in 15 / 16,
// N >> 3 in 17..22, M >> 4 in 24..28.
uint32_t make_idesc(bool a_signed, bool b_signed, uint32_t a_major, uint32_t b_major, uint32_t m, uint32_t n)
{
    return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | ((b_signed ? 1u : 0u) << 10) | (a_major << 15) | (b_major << 16) |
           ((n >> 3) << 17) | ((m >> 4) << 24);
}

// ================================================================== the kernel
enum { MODE_GEMM = 0, MODE_FPROP = 1, MODE_DGRAD = 2 };
constexpr int kMaxStages = 16;
constexpr int kMaxStageMmas = 256;                    // bound on the MMAs of one pipeline stage (several halo tiles per stage)
constexpr int kMaxAccBufs = 8;                        // accumulator buffers in tensor memory (512 columns in all)
constexpr int kEpiWarps = 12;                         // three per tensor-memory lane quadrant
constexpr int kMmaThreads = 64 + 32 * kEpiWarps;      // TMA warp, MMA warp, epilogue warps
constexpr int kGroupM = 8;           // GEMM raster: tiles walk down kGroupM tile rows before moving one column right
constexpr uint32_t kStageSlab = 32 * 128;             // epilogue staging per warp: 32 rows x 32 fp32
constexpr uint32_t kSmemBudget = 226u * 1024u;        // dynamic shared memory of the kernel

struct MmaParams {
    CUtensorMap mapA, mapB, mapC;
    OperandLayout a, b;
    uint32_t idesc;
    int mode;
    int stages, k_iters, mma_per_iter, bn, tmem_cols;
    int msub;                     // 128-row accumulator sub-tiles per CTA tile (1 or 2)
    int nbuf;                     // accumulator buffers in tensor memory: as many as fit (even when msub == 1)
    int a_loads, b_loads;         // TMA loads per operand tile (M/N-major operands wider than one swizzled row)
    uint32_t a_load_bytes, b_load_bytes;
    int ips;                      // k iterations (operand tiles) per pipeline stage (at most 32: one lane each)
    int halo;                     // conv: a stage holds whole halo tiles of the pixel box (one per channel chunk); the
                                  // taps are shifted windows of a tile instead of loads of their own
    int halo_w;                   // pixels per row of a halo tile (box width + 2)
    int halo_rb;                  // halo tiles: 0 forward (K-major filter tiles), else the row bytes of the M/N-major filter tiles
    int groups;                   // pipeline stages per output tile
    int stage_mmas;               // MMAs per stage
    int b_stage_tiles;            // filter tiles consumed per stage (resident filter)
    uint32_t stage_tx;            // bytes the TMA loads of one stage deliver
    int egroups;                  // msub == 1: groups of four epilogue warps that take tiles in turn (at most 3, at most nbuf)
    int ewarps;                   // epilogue warps at work (the rest of the kEpiWarps idle): 8 when msub == 2, else 4 * egroups
    int nslab;                    // epilogue staging slabs per warp (2: a store is still reading one while the next is filled)
    // Per-column statistics of the fp32 output (for the Range BN that follows, Section 3): every working epilogue
    // warp keeps (sum, min, max) of the columns in shared memory; when the kernel ends the CTA's warps add them up
    // into row blockIdx.x of these partial arrays [rows][N].  NULL: not wanted.  Up to 256 columns every CTA keeps all of
    // them (stat_cols = N); beyond (convolutions only) the grid is a multiple of the column tiles, so that a CTA meets one
    // column tile in all its tiles (tile mod tiles_n = blockIdx.x mod tiles_n) and keeps that tile's stat_cols = bn
    // columns only (stat_local), leaving the neutral element in the rest of its partial row.
    float *st_lo, *st_hi; double *st_sum;
    int stat_cols, stat_local;
    // Optional tail of the epilogue: per-column normalisation by the Range BN that follows the product (ep_fold:
    // (mean, scale, gamma, beta) per output column, copied to shared memory), ReLU, and the 8-bit codes of the result
    // (parameters *ep_rq) written to ep_q [M x N] with each row's code sum in ep_rowsum (one column tile only).  `out`
    // then receives the transformed value.  Statistics are of the untransformed output and exclude a tail.
    const float4 *ep_fold; int ep_relu;
    const qbp_qparams *ep_rq; int8_t *ep_q; int32_t *ep_rowsum;
    uint32_t stat_span;           // bytes of the statistics region in shared memory (the fold table follows it)
    int grid;                     // CTAs launched
    uint32_t cterm_span;          // bytes of the column-term region in shared memory (the statistics follow it)
    int iter_entries;             // entries of the k-iteration table in shared memory (conv), a multiple of 64
    int b_resident;               // conv: all filter tiles of the CTA's N tile stay in shared memory
    uint32_t b_res_bytes;         // bytes reserved for them at the start of shared memory
    int ncls;                     // rows of the column-term table (1, or 16 border classes)
    int cterm_all;                // the whole table [ncls][N] is kept in shared memory (else one tile's columns)
    int tiles_m, tiles_n, tiles_total;
    // output
    int64_t M, N;                 // rows / columns of the output matrix
    int32_t *acc_out; float *out;
    const int32_t *rowterm;       // [M]
    const int32_t *colterm;       // [ncls][N]
    const qbp_qparams *qa, *qb;
    int *status;
    int kblock;                   // GEMM: reduction elements per k iteration
    // conv geometry (output pixel grid == input pixel grid: stride 1, same padding)
    int H, W, Nimg, pad, S, cchunks, chunk_bytes, Cred;
    int bw_log2, bh_log2, tiles_w, tiles_h;
    FastDiv d_tiles_n, d_tiles_w, d_tiles_h, d_group;
};

struct TileOrigin { int m0, n0, img0, h0, w0; };
struct ColStat { double sum; float lo, hi; };

__device__ __forceinline__ TileOrigin tile_origin(const MmaParams &P, int tile)
{
    TileOrigin o;
    int tile_m, tile_n;
    if (P.mode == MODE_GEMM) {
        // groups of kGroupM tile rows; inside a group the row index moves fastest, so that the CTAs
        // running at one time share few A row-blocks and few B column-blocks (L2 reuse)
        int g, r;
        P.d_group.divmod(tile, g, r);                    // by kGroupM * tiles_n
        const int rows_here = min(kGroupM, P.tiles_m - g * kGroupM);
        if (rows_here == kGroupM) { tile_n = r / kGroupM; tile_m = g * kGroupM + r % kGroupM; }
        else                      { tile_n = r / rows_here; tile_m = g * kGroupM + r % rows_here; }   // the last, ragged group
    } else {
        P.d_tiles_n.divmod(tile, tile_m, tile_n);
    }
    o.n0 = tile_n * P.bn;
    o.m0 = tile_m * 128 * P.msub; o.img0 = 0; o.h0 = 0; o.w0 = 0;
    if (P.mode != MODE_GEMM) {
        int t1, tw, tn, th;
        P.d_tiles_w.divmod(tile_m, t1, tw);
        P.d_tiles_h.divmod(t1, tn, th);
        o.w0 = tw << P.bw_log2;
        o.h0 = th << P.bh_log2;
        o.img0 = tn * (128 >> (P.bw_log2 + P.bh_log2));
    }
    return o;
}

// The MMAs of one pipeline stage, run by the whole MMA warp in step; one elected lane issues.  Every operand is
// plain arithmetic on loop counters and launch constants, and the "overwrite the accumulator" flag is a constant of
// the code path (the first MMAs of a tile are peeled off): the instruction takes its operands from warp-uniform
// registers, and anything looked up per MMA (a table entry, a flag derived from one) costs a transfer each time --
// measured 53 cycles per 128 x 64 x 32 MMA this way against 110 to 130 from a table.  Offsets are in 16-byte units;
// the 14-bit address field of a descriptor cannot carry: shared memory ends below 256 KB.
#define QBP_ISSUE_ONE(d, a_lo, a_hi, b_lo, b_hi, idesc, accumulate)                                                   \
    do {                                                                                                             \
        if (elect_one())                                                                                             \
            mma_i8((d), ((uint64_t)(a_hi) << 32) | (uint64_t)(a_lo), ((uint64_t)(b_hi) << 32) | (uint64_t)(b_lo), (idesc), \
                   (accumulate));                                                                                    \
    } while (0)

// The 9 x MPI MMAs of one halo tile (a 3 x 3 filter over one channel chunk of 32 * MPI bytes, 10-pixel tile rows),
// fully unrolled.  The A operand of a tap is the halo tile read from a shifted start: the shared-memory swizzle is a
// function of the address, so a window that starts any whole number of pixel rows into the tile reads what TMA
// wrote there.  Forward: output (p,q) reads input (p - pad + r, q - pad + t); layer gradient: (h + pad - r,
// w + pad - t); the tile's origin is (h0 - pad, w0 - pad) in both, so the gradient takes the windows in reverse.
// RB = 0: forward, filter tiles K-major; else layer gradient, filter tiles M/N-major with rows of RB bytes.
//
// What is fixed by (MPI, RB) is spelled as constants -- the A offsets, the upper descriptor words, the filter's k
// step -- because the MMA takes its operands from the warp's few uniform registers: with the same values passed in
// at run time next to the per-stage addresses the compiler ran out of them and each MMA cost 130 cycles instead of 40.
constexpr int kHaloW = 10;           // pixels per row of a halo tile: the 8-pixel box row and one border pixel each side
__host__ __device__ constexpr uint32_t swizzle_bits(uint32_t row_bytes) { return row_bytes == 128 ? 2u : row_bytes == 64 ? 4u : 6u; }
// BN: the output columns of the tile when they are one of the common counts (then the filter tile size and the
// instruction descriptor are constants too), 0: taken from the launch parameters.
template <int MPI, int RB, int BN>
__device__ __forceinline__ void issue_halo_3x3(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t b_tile16_rt, uint32_t idesc_rt,
                                               uint32_t first_acc)
{
    constexpr bool FWD = RB == 0;
    constexpr uint32_t cb = 32u * MPI;
    constexpr int px16 = 2 * MPI, row16 = kHaloW * px16;
    constexpr uint32_t a_hi = ((kHaloW * cb) >> 4) | (1u << 14) | (swizzle_bits(cb) << 29);
    constexpr uint32_t b_hi = FWD ? ((8u * cb) >> 4) | (1u << 14) | (swizzle_bits(cb) << 29)
                                  : ((8u * (uint32_t)RB) >> 4) | (1u << 14) | (swizzle_bits((uint32_t)RB) << 29);
    constexpr uint32_t b_kstep = FWD ? 2u : (32u * (uint32_t)RB) >> 4;
    // a filter tile is BN x 32 * MPI bytes either way round; s8 x s8 -> s32, M = 128, N = BN, B M/N-major for the gradient
    const uint32_t b_tile16 = BN ? (uint32_t)(2 * MPI * BN) : b_tile16_rt;
    const uint32_t idesc = BN ? (2u << 4) | (1u << 7) | (1u << 10) | ((FWD ? 0u : 1u) << 16) | (((uint32_t)BN >> 3) << 17) | ((128u >> 4) << 24)
                              : idesc_rt;
#pragma unroll
    for (int i = 0; i < 9 * MPI; ++i) {
        const int tap = i / MPI, kk = i % MPI, r = tap / 3, t = tap % 3;
        const uint32_t ao = (uint32_t)((FWD ? r : 2 - r) * row16 + (FWD ? t : 2 - t) * px16 + kk * 2);
        const uint32_t bo = (uint32_t)tap * b_tile16 + (uint32_t)kk * b_kstep;
        if (elect_one())
            mma_i8(d, ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + ao), ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + bo), idesc,
                   i == 0 ? first_acc : 1u);
    }
}

template <int MPI>
__device__ __forceinline__ void issue_halo_3x3_any(int rb, int bn, uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t b_tile16,
                                                   uint32_t idesc, uint32_t first_acc)
{
    if (rb == 0) {
        if (bn == 64)       issue_halo_3x3<MPI, 0, 64>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
        else if (bn == 128) issue_halo_3x3<MPI, 0, 128>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
        else                issue_halo_3x3<MPI, 0, 0>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
    } else if (rb == 128) {
        if (bn == 128)      issue_halo_3x3<MPI, 128, 128>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
        else                issue_halo_3x3<MPI, 128, 0>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
    } else if (rb == 64) {
        issue_halo_3x3<MPI, 64, 64>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
    } else {
        issue_halo_3x3<MPI, 32, 32>(d, a_lo, b_lo, b_tile16, idesc, first_acc);
    }
}

// The MMA warp's whole loop for the common 3 x 3 case: one halo tile per CTA tile (one channel chunk), the filter resident,
// the output columns one of the common counts.  The general loop below builds each stage's operands from launch
// parameters inside a loop over the stage's halo tiles, which keeps them out of the warp's uniform registers: its
// MMAs then issue every 70 cycles, against the 48 that a 128 x 64 x 32 product takes (measured); here everything but
// the two ring addresses is a constant.  False when a wait ran out.
struct HaloLoopArgs {
    uint64_t *full_bar, *empty_bar, *acc_full, *acc_empty;
    uint32_t tmem, ring, b_lo, a_desc_lo, stage_bytes;
    int stages, nbuf, tiles_total;
};
template <int MPI, int RB, int BN>
__device__ __forceinline__ bool mma_loop_halo1(const HaloLoopArgs &A)
{
    uint32_t s = 0, ph = 0, buf = 0, bph = 1;
    uint32_t stage_addr = A.ring, d = A.tmem;
    for (int tile = blockIdx.x; tile < A.tiles_total; tile += gridDim.x) {
        if (!mbar_wait_uniform(&A.acc_empty[buf], bph)) return false;
        if (!mbar_wait_uniform(&A.full_bar[s], ph)) return false;
        tc_fence_after();
        issue_halo_3x3<MPI, RB, BN>(d, ((stage_addr >> 4) & 0x3FFFu) | A.a_desc_lo, A.b_lo, 0u, 0u, 0u);
        if (elect_one()) mma_commit(&A.empty_bar[s]);
        if (elect_one()) mma_commit(&A.acc_full[buf]);
        stage_addr += A.stage_bytes; d += (uint32_t)BN;
        if (++s == (uint32_t)A.stages) { s = 0; ph ^= 1u; stage_addr = A.ring; }
        if (++buf == (uint32_t)A.nbuf) { buf = 0; bph ^= 1u; d = A.tmem; }
    }
    return true;
}

__device__ __forceinline__ void issue_stage(const MmaParams &P, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                            uint32_t d_tmem, bool first_stage)
{
    const uint32_t a_tile16 = P.a.tile_bytes >> 4, b_tile16 = P.b.tile_bytes >> 4;
    const uint32_t first_acc = first_stage ? 0u : 1u;
    if (!P.halo) {
        // k iteration j, k step kk, sub-tile sub (innermost: consecutive MMAs then write different accumulators
        // and do not wait for one another)
        if (P.msub == 1) {
            QBP_ISSUE_ONE(d_tmem, a_lo, a_hi, b_lo, b_hi, P.idesc, first_acc);
            for (int j = 0; j < P.ips; ++j) {
#pragma unroll 4
                for (int kk = (j == 0 ? 1 : 0); kk < P.mma_per_iter; ++kk)
                    QBP_ISSUE_ONE(d_tmem, a_lo + (uint32_t)kk * P.a.kstep, a_hi, b_lo + (uint32_t)kk * P.b.kstep, b_hi, P.idesc, 1u);
                a_lo += a_tile16; b_lo += b_tile16;
            }
        } else {
            const uint32_t d1 = d_tmem + (uint32_t)P.bn;
            QBP_ISSUE_ONE(d_tmem, a_lo, a_hi, b_lo, b_hi, P.idesc, first_acc);
            QBP_ISSUE_ONE(d1, a_lo + a_tile16, a_hi, b_lo, b_hi, P.idesc, first_acc);
            for (int j = 0; j < P.ips; ++j) {
#pragma unroll 4
                for (int kk = (j == 0 ? 1 : 0); kk < P.mma_per_iter; ++kk) {
                    QBP_ISSUE_ONE(d_tmem, a_lo + (uint32_t)kk * P.a.kstep, a_hi, b_lo + (uint32_t)kk * P.b.kstep, b_hi, P.idesc, 1u);
                    QBP_ISSUE_ONE(d1, a_lo + a_tile16 + (uint32_t)kk * P.a.kstep, a_hi, b_lo + (uint32_t)kk * P.b.kstep, b_hi, P.idesc, 1u);
                }
                a_lo += 2u * a_tile16; b_lo += b_tile16;
            }
        }
    } else {
        const uint32_t b_chunk16 = 9u * b_tile16;             // the nine filter tiles of one channel chunk
        for (int hj = 0; hj < P.ips; ++hj) {
            const uint32_t acc0 = hj == 0 ? first_acc : 1u;
            if (P.mma_per_iter == 4)      issue_halo_3x3_any<4>(P.halo_rb, P.bn, d_tmem, a_lo, b_lo, b_tile16, P.idesc, acc0);
            else if (P.mma_per_iter == 2) issue_halo_3x3_any<2>(P.halo_rb, P.bn, d_tmem, a_lo, b_lo, b_tile16, P.idesc, acc0);
            else                          issue_halo_3x3_any<1>(P.halo_rb, P.bn, d_tmem, a_lo, b_lo, b_tile16, P.idesc, acc0);
            a_lo += a_tile16; b_lo += b_chunk16;
        }
    }
}

// Persistent: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...  The producer runs ahead of
// the MMA warp across tile boundaries through the shared-memory ring.  A CTA tile is msub accumulator
// sub-tiles of 128 rows x bn columns that share the B operand of every stage (256 x 256 halves the
// operand bytes fetched per multiply-add against 128 x 256).  When two sets of accumulators fit in
// tensor memory they are used in turn, so that the epilogues of earlier tiles overlap the MMAs of later ones.
// Epilogue: tcgen05.ld -> zero-point terms -> fp32 -> swizzled staging slab -> TMA store per warp.
// TAIL: the instance with the optional normalise / ReLU / requantise tail of the epilogue (the plain instance, which the
// bandwidth-bound convolutions of a training step use, carries none of it).
template <bool TAIL>
__global__ void __launch_bounds__(kMmaThreads, 1) qbp_mma_kernel(const __grid_constant__ MmaParams P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_full[kMaxAccBufs], acc_empty[kMaxAccBufs], b_full;
    __shared__ uint32_t tmem_slot;

    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t *smem_b = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);     // resident filter tiles (if any)
    uint8_t *smem = smem_b + P.b_res_bytes;                                  // the stage ring
    const uint32_t a_iter = P.a.tile_bytes * (uint32_t)P.msub;               // A bytes of one k iteration
    const uint32_t a_stage = a_iter * (uint32_t)P.ips;
    const uint32_t stage_bytes = a_stage + (P.b_resident ? 0u : P.b.tile_bytes * (uint32_t)P.ips);
    uint8_t *staging = smem + (((size_t)P.stages * stage_bytes + 1023) & ~(size_t)1023);   // slabs of the working epilogue warps, 1024-byte aligned
    int4 *s_iter = reinterpret_cast<int4 *>(staging + P.ewarps * kStageSlab * P.nslab);   // conv: one entry per k iteration
    int32_t *s_cterm = reinterpret_cast<int32_t *>(s_iter + P.iter_entries);             // column terms
    ColStat *s_stat = reinterpret_cast<ColStat *>(reinterpret_cast<uint8_t *>(s_cterm) + P.cterm_span);   // [ewarps][N]
    float4 *s_fold = reinterpret_cast<float4 *>(reinterpret_cast<uint8_t *>(s_stat) + P.stat_span);       // [N]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < P.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        // an accumulator buffer is read by both epilogue groups (msub == 2) or by one of them
        for (int b = 0; b < P.nbuf; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], P.msub == 2 ? 8 : 4); }
        mbar_init(&b_full, 1);
        mbar_fence_init();
        tma_prefetch_desc(&P.mapA);
        tma_prefetch_desc(&P.mapB);
        if (P.out) tma_prefetch_desc(&P.mapC);
    }
    if (warp == 1) { tmem_alloc(&tmem_slot, (uint32_t)P.tmem_cols); tmem_relinquish(); }
    if (P.mode != MODE_GEMM)
        for (int it = threadIdx.x; it < P.k_iters; it += kMmaThreads) {
            // k iteration -> (channel offset, tap column, tap row, filter coordinate of the tap's channel chunk);
            // tap-major, or chunk-major when a stage is a halo tile of one chunk (its filter tiles are then contiguous)
            const int taps = P.k_iters / P.cchunks;
            const int tap = P.halo ? it % taps : it / P.cchunks, cc = P.halo ? it / taps : it % P.cchunks;
            const int c0 = cc * P.chunk_bytes;
            s_iter[it] = make_int4(c0, tap % P.S, tap / P.S, P.mode == MODE_FPROP ? tap * P.Cred + c0 : tap * (int)P.N);
        }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t buf_cols = (uint32_t)(P.msub * P.bn);
    bool timed_out = false;

    if (warp == 0) {
        // ---------------------------------------------------- TMA producer
        // Lane 0 owns the barriers.  Convolution: the `ips` activation tiles of a stage are issued by
        // `ips` lanes at once, each from its own entry of the k-iteration table.
        if (P.b_resident && lane == 0) {
            // the filter is the same for every tile of this CTA: fetch it once
            mbar_expect_tx(&b_full, P.b.tile_bytes * (uint32_t)P.k_iters);
            for (int it = 0; it < P.k_iters; ++it) {
                const int4 e = s_iter[it];
                uint8_t *dst = smem_b + (size_t)it * P.b.tile_bytes;
                if (P.mode == MODE_FPROP) tma_load_2d(dst, &P.mapB, &b_full, e.w, 0);
                else
                    for (int l = 0; l < P.b_loads; ++l)
                        tma_load_2d(dst + (size_t)l * P.b_load_bytes, &P.mapB, &b_full, e.w + l * 128, e.x);
            }
        }
        uint32_t s = 0, ph = 1;                             // ring position and the parity to wait for, across tiles
        const int groups = P.groups;
        for (int tile = blockIdx.x; tile < P.tiles_total && !timed_out; tile += gridDim.x) {
            const TileOrigin o = tile_origin(P, tile);
            if (P.mode == MODE_GEMM) {
                if (lane == 0) {
                    for (int it = 0; it < P.k_iters; ++it) {
                        if (!mbar_wait(&empty_bar[s], ph)) { timed_out = true; break; }
                        uint8_t *sa = smem + (size_t)s * stage_bytes;
                        uint8_t *sb = sa + a_stage;
                        mbar_expect_tx(&full_bar[s], stage_bytes);
                        const int k0 = it * P.kblock;
                        // K-major operands: one box of all rows; M/N-major: one box per 128-byte column chunk
                        if (P.a.major == 0) tma_load_2d(sa, &P.mapA, &full_bar[s], k0, o.m0);
                        else
                            for (int l = 0; l < P.a_loads; ++l)
                                tma_load_2d(sa + (size_t)l * P.a_load_bytes, &P.mapA, &full_bar[s], o.m0 + l * 128, k0);
                        if (P.b.major == 0) tma_load_2d(sb, &P.mapB, &full_bar[s], k0, o.n0);
                        else
                            for (int l = 0; l < P.b_loads; ++l)
                                tma_load_2d(sb + (size_t)l * P.b_load_bytes, &P.mapB, &full_bar[s], o.n0 + l * 128, k0);
                        if (++s == (uint32_t)P.stages) { s = 0; ph ^= 1u; }
                    }
                }
                timed_out = __shfl_sync(0xffffffffu, timed_out ? 1 : 0, 0) != 0;
                continue;
            }
            // convolution: one activation tile per (tap, channel chunk), `ips` of them per stage
            for (int g = 0; g < groups; ++g) {
                int ok = 1;
                if (lane == 0) {
                    ok = mbar_wait(&empty_bar[s], ph) ? 1 : 0;
                    if (ok) mbar_expect_tx(&full_bar[s], P.stage_tx);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { timed_out = true; break; }
                if (P.halo) {
                    // the pixel box with a border of `pad` pixels, one load per channel chunk; outside the image: zeros
                    if (lane < P.ips)
                        tma_load_4d(smem + (size_t)s * stage_bytes + (size_t)lane * P.a.tile_bytes, &P.mapA, &full_bar[s],
                                    (g * P.ips + lane) * P.chunk_bytes, o.w0 - P.pad, o.h0 - P.pad, o.img0);
                } else if (lane < P.ips) {
                    const int4 e = s_iter[g * P.ips + lane];   // (channel offset, tap column, tap row, filter coordinate)
                    uint8_t *sa = smem + (size_t)s * stage_bytes;
                    uint8_t *da = sa + (size_t)lane * P.a.tile_bytes;
                    uint8_t *db = sa + a_stage + (size_t)lane * P.b.tile_bytes;
                    if (P.mode == MODE_FPROP) {
                        // input pixel of output (p,q) under tap (r,t): (p - pad + r, q - pad + t)
                        tma_load_4d(da, &P.mapA, &full_bar[s], e.x, o.w0 - P.pad + e.y, o.h0 - P.pad + e.z, o.img0);
                        // filter as [K rows x (R*S*C) columns]: this tap's channel chunk, K-major
                        if (!P.b_resident) tma_load_2d(db, &P.mapB, &full_bar[s], e.w, o.n0);
                    } else {
                        // gradient pixel feeding input (h,w) under tap (r,t): (h + pad - r, w + pad - t)
                        tma_load_4d(da, &P.mapA, &full_bar[s], e.x, o.w0 + P.pad - e.y, o.h0 + P.pad - e.z, o.img0);
                        // filter rows = output channels (the reduction), columns = this tap's input channels
                        if (!P.b_resident)
                            for (int l = 0; l < P.b_loads; ++l)
                                tma_load_2d(db + (size_t)l * P.b_load_bytes, &P.mapB, &full_bar[s], e.w + o.n0 + l * 128, e.x);
                    }
                }
                __syncwarp();
                if (++s == (uint32_t)P.stages) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------ MMA issuer
        // The whole warp walks the tiles and stages in step, so that ring positions, descriptors and accumulator
        // addresses stay warp-uniform; an elected lane issues the MMAs and the commits.
        if (P.b_resident && !mbar_wait_uniform(&b_full, 0)) timed_out = true;
        const uint32_t bres_addr = smem_u32(smem_b);
        const uint32_t ring_addr = smem_u32(smem);
        const int groups = P.groups;
        uint32_t s = 0, ph = 0;                          // ring position and parity, across tiles
        uint32_t buf = 0, bph = 1;                       // accumulator buffer and the parity of its "empty" barrier
        // the common 3 x 3 case has a loop of its own (one halo tile per CTA tile; see mma_loop_halo1)
        const int fast = (P.halo && P.ips == 1 && groups == 1 && P.msub == 1 && P.b_resident && !timed_out)
                             ? (P.halo_rb == 0 ? (P.mma_per_iter == 2 && P.bn == 64 ? 1 : P.mma_per_iter == 4 && P.bn == 128 ? 2 : 0)
                                               : (P.mma_per_iter == 2 && P.halo_rb == 64 && P.bn == 64 ? 3
                                                  : P.mma_per_iter == 4 && P.halo_rb == 128 && P.bn == 128 ? 4 : 0))
                             : 0;
        if (fast) {
            HaloLoopArgs A;
            A.full_bar = full_bar; A.empty_bar = empty_bar; A.acc_full = acc_full; A.acc_empty = acc_empty;
            A.tmem = tmem_base; A.ring = ring_addr; A.b_lo = ((bres_addr >> 4) & 0x3FFFu) | P.b.desc_lo; A.a_desc_lo = P.a.desc_lo;
            A.stage_bytes = stage_bytes; A.stages = P.stages; A.nbuf = P.nbuf; A.tiles_total = P.tiles_total;
            const bool ok = fast == 1 ? mma_loop_halo1<2, 0, 64>(A) : fast == 2 ? mma_loop_halo1<4, 0, 128>(A)
                          : fast == 3 ? mma_loop_halo1<2, 64, 64>(A) : mma_loop_halo1<4, 128, 128>(A);
            if (!ok) timed_out = true;
        } else
        for (int tile = blockIdx.x; tile < P.tiles_total && !timed_out; tile += gridDim.x) {
            if (!mbar_wait_uniform(&acc_empty[buf], bph)) { timed_out = true; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + buf * buf_cols;
            for (int g = 0; g < groups; ++g) {
                if (!mbar_wait_uniform(&full_bar[s], ph)) { timed_out = true; break; }
                tc_fence_after();
                const uint32_t stage_addr = ring_addr + s * stage_bytes;
                const uint32_t b_addr = P.b_resident ? bres_addr + (uint32_t)(g * P.b_stage_tiles) * P.b.tile_bytes : stage_addr + a_stage;
                issue_stage(P, ((stage_addr >> 4) & 0x3FFFu) | P.a.desc_lo, P.a.desc_hi,
                            ((b_addr >> 4) & 0x3FFFu) | P.b.desc_lo, P.b.desc_hi, d_tmem, g == 0);
                if (elect_one()) mma_commit(&empty_bar[s]);
                if (++s == (uint32_t)P.stages) { s = 0; ph ^= 1u; }
            }
            if (!timed_out && elect_one()) mma_commit(&acc_full[buf]);
            if (++buf == (uint32_t)P.nbuf) { buf = 0; bph ^= 1u; }
        }
    } else if (warp - 2 < P.ewarps) {
        // ------------------------------------------------------- epilogue
        // msub == 2: two groups of four warps work on every tile, one 128-row sub-tile each.
        // msub == 1: the groups take tiles (and accumulator buffers) in turn: a warp's read-out, arithmetic and
        //            store of a tile is one long dependent chain, so the epilogue's throughput is the number of
        //            tiles in flight.
        const int ew = warp - 2;                         // 0 .. P.ewarps-1
        const int quad = warp & 3;                       // the tensor-memory lanes this warp may read
        const int group = ew >> 2;
        const int row = quad * 32 + lane;
        uint8_t *slab0 = staging + (size_t)(ew * P.nslab) * kStageSlab;
        uint32_t slab_i = 0;
        const float scale = __fmul_rn(P.qa->scale, P.qb->scale);
        ColStat *my_stat = s_stat + (size_t)ew * P.stat_cols;
        const int stat_base = P.stat_local ? (int)(blockIdx.x % (unsigned)P.tiles_n) * P.bn : 0;     // first column this CTA keeps
        if (P.st_sum) {
            for (int i = lane; i < P.stat_cols; i += 32) { my_stat[i].sum = 0.0; my_stat[i].lo = INFINITY; my_stat[i].hi = -INFINITY; }
            __syncwarp();
        }
        const int sub = P.msub == 2 ? group : 0;
        const int lt_step = P.msub == 2 ? 1 : P.egroups;
        const int bar_id = P.msub == 2 ? 1 : 1 + group, bar_cnt = P.msub == 2 ? 256 : 128;
        const int gt = P.msub == 2 ? threadIdx.x - 64 : (threadIdx.x - 64) & 127;     // thread index within the barrier group
        int32_t *region = s_cterm + (P.cterm_all || P.msub == 2 ? 0 : group * P.ncls * P.bn);
        if (P.cterm_all || (TAIL && P.ep_fold)) {
            // the whole column-term table fits: fill it once (and the per-column constants of the normalisation)
            if (P.cterm_all)
                for (int i = threadIdx.x - 64; i < P.ncls * (int)P.N; i += 32 * P.ewarps) s_cterm[i] = __ldg(P.colterm + i);
            if (TAIL && P.ep_fold)
                for (int i = threadIdx.x - 64; i < (int)P.N; i += 32 * P.ewarps) s_fold[i] = __ldg(P.ep_fold + i);
            named_barrier(4, 32 * P.ewarps);
        }
        float rq_inv = 0.0f, rq_zp = 0.0f;
        if (TAIL && P.ep_q) { rq_inv = __fdiv_rn(1.0f, P.ep_rq->scale); rq_zp = (float)(P.ep_rq->zero_point + 128); }

        // where this thread's accumulator row of a tile goes
        struct RowInfo { int64_t m; bool valid, slab_in; int cls, sx, sy, sz; };
        auto row_info = [&](const TileOrigin &o) {
            RowInfo ri; ri.cls = 0; ri.sx = ri.sy = ri.sz = 0;
            if (P.mode == MODE_GEMM) {
                ri.m = (int64_t)o.m0 + sub * 128 + row;
                ri.valid = ri.m < P.M;
                ri.slab_in = (int64_t)o.m0 + sub * 128 + quad * 32 < P.M;
            } else {
                const int dw = row & ((1 << P.bw_log2) - 1);
                const int dh = (row >> P.bw_log2) & ((1 << P.bh_log2) - 1);
                const int dn = row >> (P.bw_log2 + P.bh_log2);
                const int n = o.img0 + dn, p = o.h0 + dh, q = o.w0 + dw;
                ri.valid = n < P.Nimg && p < P.H && q < P.W;
                ri.m = ((int64_t)n * P.H + p) * P.W + q;
                ri.cls = (p == 0 ? 1 : 0) | (p == P.H - 1 ? 2 : 0) | (q == 0 ? 4 : 0) | (q == P.W - 1 ? 8 : 0);
                const int r0 = quad * 32;            // this warp's 32 rows are a sub-box of the pixel box
                ri.sx = o.w0 + (r0 & ((1 << P.bw_log2) - 1));
                ri.sy = o.h0 + ((r0 >> P.bw_log2) & ((1 << P.bh_log2) - 1));
                ri.sz = o.img0 + (r0 >> (P.bw_log2 + P.bh_log2));
                ri.slab_in = ri.sx < P.W && ri.sy < P.H && ri.sz < P.Nimg;
            }
            return ri;
        };

        const int tile_step = (int)gridDim.x * lt_step;
        int tile = blockIdx.x + (P.msub == 2 ? 0 : group * (int)gridDim.x);
        // this group's accumulator buffer and the parity of its "full" barrier; msub == 1: buffers of the group's own parity
        uint32_t buf = P.msub == 2 ? 0u : (uint32_t)group, fph = 0;
        TileOrigin o = tile_origin(P, tile < P.tiles_total ? tile : 0);
        RowInfo ri = row_info(o);
        int rterm = (tile < P.tiles_total && ri.valid) ? __ldg(P.rowterm + ri.m) : 0;
        for (; tile < P.tiles_total; tile += tile_step) {
            // the next tile's row term is fetched now, so that its latency hides behind this tile
            const int tile_next = tile + tile_step;
            const TileOrigin o_next = tile_origin(P, tile_next < P.tiles_total ? tile_next : 0);
            const RowInfo ri_next = row_info(o_next);
            const int rterm_next = (tile_next < P.tiles_total && ri_next.valid) ? __ldg(P.rowterm + ri_next.m) : 0;
            if (!P.cterm_all) {
                // column terms of this tile into shared memory (the previous tile's readers are done first)
                named_barrier(bar_id, bar_cnt);
                for (int i = gt; i < P.ncls * P.bn; i += bar_cnt) {
                    const int cls = i / P.bn, n = o.n0 + i % P.bn;
                    region[i] = n < P.N ? __ldg(P.colterm + (int64_t)cls * P.N + n) : 0;
                }
                named_barrier(bar_id, bar_cnt);
            }
            const int32_t *cterm = P.cterm_all ? s_cterm + ri.cls * (int)P.N + o.n0 : region + ri.cls * P.bn;
            const int64_t ncol = P.N - o.n0;                                // columns left in the matrix
            const int nchunks = (int)((ncol < P.bn ? ncol : P.bn) + 31) / 32;
            if (!timed_out && !mbar_wait_warp(&acc_full[buf], fph)) timed_out = true;
            if (!timed_out) {
                tc_fence_after();
                const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * buf_cols + (uint32_t)(sub * P.bn);
                int row_code_sum = 0;                   // of this thread's output row's 8-bit codes (one column tile)
                for (int c = 0; c < nchunks; ++c) {
                    const int c0 = c * 32;
                    uint32_t r[32];
                    tmem_ld_32x32(t_addr + (uint32_t)c0, r);
                    tmem_ld_wait();
                    if (c == nchunks - 1) {
                        // the accumulator has been read out: hand the buffer back to the MMA warp
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty[buf]);
                    }
                    const int lim = (int)(ncol - c0 < 32 ? ncol - c0 : 32);
                    int acc[32];
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int4 ct = *reinterpret_cast<const int4 *>(cterm + c0 + j);
                        acc[j] = (int)r[j] + rterm + ct.x; acc[j + 1] = (int)r[j + 1] + rterm + ct.y;
                        acc[j + 2] = (int)r[j + 2] + rterm + ct.z; acc[j + 3] = (int)r[j + 3] + rterm + ct.w;
                    }
                    if (P.acc_out && ri.valid) {
                        int32_t *dst = P.acc_out + ri.m * P.N + o.n0 + c0;
                        if (lim == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<int4 *>(dst + j) = make_int4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < lim) dst[j] = acc[j];
                        }
                    }
                    // the fp32 value of the row's 32 outputs: dequantised, then (optionally) normalised and rectified
                    float v[TAIL ? 32 : 1];
                    if (TAIL) {
#pragma unroll
                        for (int j = 0; j < (TAIL ? 32 : 1); ++j) v[j] = __fmul_rn((float)acc[j], scale);
                        if (P.ep_fold) {
#pragma unroll
                            for (int j = 0; j < (TAIL ? 32 : 1); ++j) {
                                const float4 f = s_fold[o.n0 + c0 + (j < lim ? j : 0)];       // (mean, scale, gamma, beta)
                                v[j] = bn_y(bn_xhat(v[j], f.x, f.y), f.z, f.w);
                            }
                        }
                        if (P.ep_relu) {
#pragma unroll
                            for (int j = 0; j < (TAIL ? 32 : 1); ++j) v[j] = fmaxf(v[j], 0.0f);
                        }
                        if (P.ep_q) {
                            // 8-bit codes of the row's 32 values: two 16-byte stores (the row's bytes are contiguous)
                            uint32_t w8[8];
#pragma unroll
                            for (int j = 0; j < (TAIL ? 32 : 1); j += 4) {
                                uint32_t c4[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) c4[e] = (uint32_t)quantize_code<false>(v[TAIL ? j + e : 0], rq_inv, rq_zp, 255.0f, 0u);
                                w8[j >> 2] = (c4[0] | (c4[1] << 8) | (c4[2] << 16) | (c4[3] << 24)) ^ 0x80808080u;
                            }
                            if (ri.valid) {
                                int8_t *dst = P.ep_q + ri.m * P.N + o.n0 + c0;
                                if (lim == 32) {
                                    *reinterpret_cast<uint4 *>(dst) = make_uint4(w8[0], w8[1], w8[2], w8[3]);
                                    *reinterpret_cast<uint4 *>(dst + 16) = make_uint4(w8[4], w8[5], w8[6], w8[7]);
#pragma unroll
                                    for (int k = 0; k < 8; ++k) row_code_sum = __dp4a((int)w8[k], 0x01010101, row_code_sum);
                                } else {
                                    // (N is a multiple of 16: a ragged chunk holds 16 columns)
                                    *reinterpret_cast<uint4 *>(dst) = make_uint4(w8[0], w8[1], w8[2], w8[3]);
#pragma unroll
                                    for (int k = 0; k < 4; ++k) row_code_sum = __dp4a((int)w8[k], 0x01010101, row_code_sum);
                                }
                            }
                        }
                    }
                    if (P.st_sum || P.out) {
                        // the store that last used this slab must have read it before it is overwritten
                        uint8_t *slab = slab0 + slab_i * kStageSlab;
                        if (lane == 0) { if (P.nslab == 2) tma_store_wait_read_but_one(); else tma_store_wait_read(); }
                        __syncwarp();
                        if (P.nslab == 2) slab_i ^= 1u;
                        // 128-byte swizzle: the 16-byte group g of row `lane` sits at group g ^ (lane & 7)
                        uint8_t *rowp = slab + lane * 128;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4 *>(rowp + (((j >> 2) ^ (lane & 7)) << 4)) =
                                TAIL ? make_float4(v[TAIL ? j : 0], v[TAIL ? j + 1 : 0], v[TAIL ? j + 2 : 0], v[TAIL ? j + 3 : 0])
                                     : make_float4(__fmul_rn((float)acc[j], scale), __fmul_rn((float)acc[j + 1], scale),
                                                   __fmul_rn((float)acc[j + 2], scale), __fmul_rn((float)acc[j + 3], scale));
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0 && P.out) {
                            if (ri.slab_in) {
                                if (P.mode == MODE_GEMM) tma_store_2d(&P.mapC, slab, o.n0 + c0, o.m0 + sub * 128 + quad * 32);
                                else                     tma_store_4d(&P.mapC, slab, o.n0 + c0, ri.sx, ri.sy, ri.sz);
                            }
                            // a group per chunk, stored or not (a slab outside the matrix): "all but the latest group
                            // have been read" must mean "the other slab's store", or the wait before the next fill lets a
                            // store that is still reading this slab pass
                            tma_store_commit();
                        }
                        if (P.st_sum) {
                            // lane = column of the slab: its 32 rows (the valid ones) read back from shared memory
                            // (a row's 32 floats lie in one 128-byte line whatever the swizzle: no bank conflicts)
                            const unsigned vmask = __ballot_sync(0xffffffffu, ri.valid);
                            float cs = 0.0f, clo = INFINITY, chi = -INFINITY;
                            if (vmask == 0xffffffffu) {
                                // (rows r and r + 8 swizzle alike: eight base addresses, the rest constant offsets)
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const uint8_t *colp = slab + k * 128 + ((((lane >> 2) ^ k) << 4) | ((lane & 3) << 2));
#pragma unroll
                                    for (int r8 = 0; r8 < 4; r8 += 2) {
                                        // (two rows per three-input min / max)
                                        const float v0 = *reinterpret_cast<const float *>(colp + r8 * 1024);
                                        const float v1 = *reinterpret_cast<const float *>(colp + (r8 + 1) * 1024);
                                        cs += v0; cs += v1; clo = fmin3(clo, v0, v1); chi = fmax3(chi, v0, v1);
                                    }
                                }
                            } else {
#pragma unroll 8
                                for (int r = 0; r < 32; ++r) {
                                    if (!((vmask >> r) & 1u)) continue;
                                    const float v = *reinterpret_cast<const float *>(slab + r * 128 + ((((lane >> 2) ^ (r & 7)) << 4) | ((lane & 3) << 2)));
                                    cs += v; clo = fminf(clo, v); chi = fmaxf(chi, v);
                                }
                            }
                            if (lane < lim && vmask) {
                                ColStat &a = my_stat[o.n0 - stat_base + c0 + lane];
                                a.sum += (double)cs; a.lo = fminf(a.lo, clo); a.hi = fmaxf(a.hi, chi);
                            }
                        }
                    }
                }
                if (TAIL && P.ep_rowsum && ri.valid) P.ep_rowsum[ri.m] = row_code_sum;
            }
            o = o_next; ri = ri_next; rterm = rterm_next;
            buf += (uint32_t)lt_step;
            if (buf >= (uint32_t)P.nbuf) { buf -= (uint32_t)P.nbuf; fph ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
        if (P.st_sum) {
            // the CTA's warps together: one partial row per CTA
            named_barrier(5, 32 * P.ewarps);
            const int64_t prow = (int64_t)blockIdx.x * P.N;
            for (int i = ew * 32 + lane; i < (int)P.N; i += 32 * P.ewarps) {
                double sum = 0.0; float lo = INFINITY, hi = -INFINITY;
                const int li = i - stat_base;
                if (li >= 0 && li < P.stat_cols)
                    for (int w = 0; w < P.ewarps; ++w) {
                        const ColStat &a = s_stat[(size_t)w * P.stat_cols + li];
                        sum += a.sum; lo = fminf(lo, a.lo); hi = fmaxf(hi, a.hi);
                    }
                P.st_sum[prow + i] = sum; P.st_lo[prow + i] = lo; P.st_hi[prow + i] = hi;
            }
        }
    }

    if (timed_out) {
        raise_timeout(P.status);
        __nanosleep(1000000);          // let copies already in flight land before the CTA retires
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { __syncwarp(); tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols); }
}

// ================================================= zero-point correction terms
// GEMM: rowterm[m] = -zb * sum_k A[m,k] + K*za*zb ; colterm[n] = -za * sum_k B[k,n].
// The code sums arrive as int32 (sums along stored rows) or int64 (along stored columns).
__global__ void gemm_terms_kernel(const int32_t *ra32, const long long *ra64, const int32_t *cb32, const long long *cb64,
                                  int64_t M, int64_t N, int64_t K, const qbp_qparams *qa, const qbp_qparams *qb,
                                  int32_t *rowterm, int32_t *colterm)
{
    const int za = qa->zero_point, zb = qb->zero_point;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < M) {
        const int ra = ra32 ? ra32[i] : (int)ra64[i];
        rowterm[i] = -zb * ra + (int)K * za * zb;
    }
    if (i < N) {
        const int cb = cb32 ? cb32[i] : (int)cb64[i];
        colterm[i] = -za * cb;
    }
}

// colterm[cls][n] = -z_in * sum over the taps valid for border class cls of the
// filter's code sum for that tap and output column n.  cls bits: 1 first row,
// 2 last row, 4 first column, 8 last column.  wsum32: [n][tap] (forward: sums over
// the input channels); wsum64: [tap][n] (layer gradient: sums over the output channels).
__global__ void conv_colterm_kernel(const int32_t *wsum32, const long long *wsum64, int N, int R, int S, int pad,
                                    int dgrad, const qbp_qparams *q_in, int32_t *colterm)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int cls = blockIdx.y;
    if (n >= N) return;
    const bool top = cls & 1, bottom = cls & 2, left = cls & 4, right = cls & 8;
    long long sum = 0;
    for (int r = 0; r < R; ++r) {
        // forward: tap row r reads input row p - pad + r; layer gradient: gradient row h + pad - r
        const bool low = dgrad ? r > pad : r < pad, high = dgrad ? r < pad : r > pad;
        if ((low && top) || (high && bottom)) continue;
        for (int s = 0; s < S; ++s) {
            const bool lo_c = dgrad ? s > pad : s < pad, hi_c = dgrad ? s < pad : s > pad;
            if ((lo_c && left) || (hi_c && right)) continue;
            const int tap = r * S + s;
            sum += wsum32 ? (long long)wsum32[(int64_t)n * R * S + tap] : wsum64[(int64_t)tap * N + n];
        }
    }
    colterm[cls * N + n] = -q_in->zero_point * (int)sum;
}

// A small filter in one launch (Appendix B's quantiser for the weights, then what the forward convolution's zero-point
// correction needs of them): min / max scan, scale and zero-point, nearest 8-bit codes, the code sums of every
// (output channel, tap) over the input channels, and the forward column terms
//   colterm[cls][k] = -z_in * sum over the taps valid for border class cls of wsum[k][tap].
// One block of 1024 threads; w [K][taps][C] fp32, C a multiple of 4, 16-byte aligned.  The operation order of the
// quantiser is the library's (make_qparams, quantize_code), so the codes are those of qbp_quantize_s8.
__global__ void __launch_bounds__(1024) filter_prep_kernel(const float *__restrict__ w, int K, int taps, int C, int R, int S, int pad,
                                                            const qbp_qparams *__restrict__ q_in, int8_t *__restrict__ codes,
                                                            qbp_qparams *__restrict__ qp_out, int32_t *__restrict__ colterm)
{
    extern __shared__ int s_wsum[];                      // [K * taps]
    __shared__ float s_lo[32], s_hi[32];
    __shared__ float s_inv, s_zp;
    const int n4 = K * taps * C / 4;
    const int rows = K * taps;
    float lo = INFINITY, hi = -INFINITY;
    for (int i = threadIdx.x; i < n4; i += 1024) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(w) + i);
        lo = fminf(fminf(lo, fminf(v.x, v.y)), fminf(v.z, v.w));
        hi = fmaxf(fmaxf(hi, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
    }
    lo = warp_min(lo); hi = warp_max(hi);
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    for (int i = threadIdx.x; i < rows; i += 1024) s_wsum[i] = 0;
    __syncthreads();
    if (threadIdx.x < 32) {
        lo = warp_min(s_lo[threadIdx.x]); hi = warp_max(s_hi[threadIdx.x]);
        if (threadIdx.x == 0) {
            const qbp_qparams qp = make_qparams(lo, hi, 8);
            *qp_out = qp;
            s_inv = __fdiv_rn(1.0f, qp.scale); s_zp = (float)(qp.zero_point + 128);
        }
    }
    __syncthreads();
    const float inv = s_inv, zp_u = s_zp;
    const int c4 = C / 4;                                 // vectors per (k, tap) row
    for (int i = threadIdx.x; i < n4; i += 1024) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(w) + i);
        const uint32_t c0 = (uint32_t)quantize_code<false>(v.x, inv, zp_u, 255.0f, 0u), c1 = (uint32_t)quantize_code<false>(v.y, inv, zp_u, 255.0f, 0u);
        const uint32_t c2 = (uint32_t)quantize_code<false>(v.z, inv, zp_u, 255.0f, 0u), c3 = (uint32_t)quantize_code<false>(v.w, inv, zp_u, 255.0f, 0u);
        const uint32_t packed = (c0 | (c1 << 8) | (c2 << 16) | (c3 << 24)) ^ 0x80808080u;
        reinterpret_cast<uint32_t *>(codes)[i] = packed;
        atomicAdd(&s_wsum[i / c4], __dp4a((int)packed, 0x01010101, 0));
    }
    __syncthreads();
    const int zin = q_in->zero_point;
    for (int i = threadIdx.x; i < 16 * K; i += 1024) {
        const int cls = i / K, k = i - cls * K;
        const bool top = cls & 1, bottom = cls & 2, left = cls & 4, right = cls & 8;
        int sum = 0;
        for (int r = 0; r < R; ++r) {
            if ((r < pad && top) || (r > pad && bottom)) continue;
            for (int t = 0; t < S; ++t) {
                if ((t < pad && left) || (t > pad && right)) continue;
                sum += s_wsum[k * taps + r * S + t];
            }
        }
        colterm[i] = -zin * sum;
    }
}

// The layer-gradient product's column terms from a small filter's codes in one launch: the code sums of every
// (tap, input channel) over the output channels, then
//   colterm[cls][c] = -z_g * sum over the taps valid for border class cls (gradient orientation) of wsum[tap][c].
// One block of 1024 threads; codes [K][taps * C], C a multiple of 4.
__global__ void __launch_bounds__(1024) filter_dgrad_colterm_kernel(const int8_t *__restrict__ codes, int K, int taps, int C, int R,
                                                                     int S, int pad, const qbp_qparams *__restrict__ q_g,
                                                                     int32_t *__restrict__ colterm)
{
    extern __shared__ int s_wsum[];                      // [taps * C]
    const int cols4 = taps * C / 4;
    for (int j = threadIdx.x; j < cols4; j += 1024) {
        int a0 = 0, a1 = 0, a2 = 0, a3 = 0;
        for (int k = 0; k < K; ++k) {
            const int v = (int)__ldg(reinterpret_cast<const uint32_t *>(codes) + (int64_t)k * cols4 + j);
            a0 = __dp4a(v, 0x00000001, a0); a1 = __dp4a(v, 0x00000100, a1); a2 = __dp4a(v, 0x00010000, a2); a3 = __dp4a(v, 0x01000000, a3);
        }
        s_wsum[4 * j] = a0; s_wsum[4 * j + 1] = a1; s_wsum[4 * j + 2] = a2; s_wsum[4 * j + 3] = a3;
    }
    __syncthreads();
    const int zg = q_g->zero_point;
    for (int i = threadIdx.x; i < 16 * C; i += 1024) {
        const int cls = i / C, c = i - cls * C;
        const bool top = cls & 1, bottom = cls & 2, left = cls & 4, right = cls & 8;
        int sum = 0;
        for (int r = 0; r < R; ++r) {
            // gradient row h + pad - r feeds input row h: tap rows below the centre fall off the first row
            if ((r > pad && top) || (r < pad && bottom)) continue;
            for (int t = 0; t < S; ++t) {
                if ((t > pad && left) || (t < pad && right)) continue;
                sum += s_wsum[(r * S + t) * C + c];
            }
        }
        colterm[i] = -zg * sum;
    }
}

// rowterm[pixel] = -z_w * (sum of the input's channel sums over the taps inside the image)
//                   + (taps inside) * Cred * z_in * z_w          (pad is 0 or 1)
// blockIdx.y = image, blockIdx.x * 256 + threadIdx.x = position inside it; the nine taps unrolled under predicates
// and the one division by a multiply-high (with plain divisions and loops this kernel ran 260 instructions per pixel).
__global__ void __launch_bounds__(256) conv_rowterm_kernel(const int32_t *__restrict__ chan_sum, int HW, int H, int W,
                                                           FastDiv dW, int pad, int Cred, const qbp_qparams *q_in,
                                                           const qbp_qparams *q_w, int32_t *__restrict__ rowterm)
{
    const int i = (int)blockIdx.x * 256 + (int)threadIdx.x;
    if (i >= HW) return;
    int p, q;
    dW.divmod(i, p, q);
    const int m = (int)blockIdx.y * HW + i;                  // (fewer than 2^31 positions)
    const bool up = pad && p > 0, down = pad && p + 1 < H, left = pad && q > 0, right = pad && q + 1 < W;
    const int32_t *c = chan_sum + m;
    int box = __ldg(c);
    if (left) box += __ldg(c - 1);
    if (right) box += __ldg(c + 1);
    if (up) {
        box += __ldg(c - W);
        if (left) box += __ldg(c - W - 1);
        if (right) box += __ldg(c - W + 1);
    }
    if (down) {
        box += __ldg(c + W);
        if (left) box += __ldg(c + W - 1);
        if (right) box += __ldg(c + W + 1);
    }
    const int taps = (1 + (up ? 1 : 0) + (down ? 1 : 0)) * (1 + (left ? 1 : 0) + (right ? 1 : 0));
    const int za = q_in->zero_point, zb = q_w->zero_point;
    rowterm[m] = -zb * box + taps * Cred * za * zb;
}

// Per-column sum / min / max from the epilogue warps' partial rows: one block of 128 threads per column.
__global__ void __launch_bounds__(128) colstat_finalize_kernel(const float *__restrict__ part_lo, const float *__restrict__ part_hi,
                                                               const double *__restrict__ part_sum, int rows, int N,
                                                               double *__restrict__ col_sum, float *__restrict__ col_min,
                                                               float *__restrict__ col_max)
{
    const int c = blockIdx.x;
    float lo = INFINITY, hi = -INFINITY;
    double sum = 0.0;
    for (int i = threadIdx.x; i < rows; i += 128) {
        lo = fminf(lo, part_lo[(int64_t)i * N + c]); hi = fmaxf(hi, part_hi[(int64_t)i * N + c]); sum += part_sum[(int64_t)i * N + c];
    }
    lo = warp_min(lo); hi = warp_max(hi);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    __shared__ float s_lo[4], s_hi[4];
    __shared__ double s_sum[4];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; s_sum[threadIdx.x >> 5] = sum; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 4; ++w) { lo = fminf(lo, s_lo[w]); hi = fmaxf(hi, s_hi[w]); sum += s_sum[w]; }
        col_sum[c] = sum; col_min[c] = lo; col_max[c] = hi;
    }
}

int colstat_rows_max() { return sm_count(); }

// Whether filter_prep_kernel takes this filter: small enough for one block and its shared-memory table.
bool filter_prep_supported(const qbp_conv_desc *d, const float *w, const int8_t *codes)
{
    const int64_t elems = (int64_t)d->K * d->R * d->S * d->C;
    // (one block: beyond some 48 K elements the five launches it replaces are faster)
    return d->C % 4 == 0 && elems <= 49152 && (int64_t)d->K * d->R * d->S <= 8192 && aligned16(w) && ((uintptr_t)codes & 3) == 0;
}

int launch_filter_dgrad_colterm(const qbp_conv_desc *d, const int8_t *codes, const qbp_qparams *q_g, int32_t *colterm, cudaStream_t st)
{
    const int taps = d->R * d->S;
    QBP_TRACE_BEGIN(st);
    filter_dgrad_colterm_kernel<<<1, 1024, sizeof(int) * (size_t)taps * d->C, st>>>(codes, d->K, taps, d->C, d->R, d->S, d->pad, q_g, colterm);
    QBP_LAUNCH_OK("filter_dgrad_colterm_kernel");
    return QBP_OK;
}

int launch_filter_prep(const qbp_conv_desc *d, const float *w, const qbp_qparams *q_in, int8_t *codes, qbp_qparams *qw,
                       int32_t *colterm, cudaStream_t st)
{
    const int taps = d->R * d->S;
    QBP_TRACE_BEGIN(st);
    filter_prep_kernel<<<1, 1024, sizeof(int) * (size_t)d->K * taps, st>>>(w, d->K, taps, d->C, d->R, d->S, d->pad, q_in, codes, qw, colterm);
    QBP_LAUNCH_OK("filter_prep_kernel");
    return QBP_OK;
}

// Self-test of the bounded wait (diagnostics): one warp waits on an mbarrier on which nothing ever arrives, with
// the wait wrappers the product kernels use and a limit of `limit` cycles; the wait gives up, the status word is
// raised and the kernel ends through its normal exit.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(long long limit, int *status)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
    __syncwarp();
    bool timed_out = !mbar_wait_uniform(&bar, 0, limit);            // every lane polls (the MMA warps' wait)
    if (!timed_out) timed_out = !mbar_wait_warp(&bar, 0, limit);    // (not reached: the first wait cannot succeed)
    if (timed_out && threadIdx.x == 0) raise_timeout(status);
}

static size_t colstat_ws_bytes(int64_t N, bool conv = false)
{
    if (N > QBP_EPILOGUE_MAX_COLUMNS && !conv) return 0;
    const size_t cells = (size_t)colstat_rows_max() * (size_t)N;
    return align_up(cells * sizeof(float), 256) * 2 + align_up(cells * sizeof(double), 256);
}

// Parameters of the requantisation in a product's epilogue from the caller's clamping values.
__global__ void epilogue_qparams_kernel(const qbp_qparams *__restrict__ range, qbp_qparams *__restrict__ qp8)
{
    *qp8 = make_qparams(range->vmin, range->vmax, 8);
}

// What the caller's epilogue record asks for: column statistics (wanted) and / or the ReLU / requantisation tail.
static int check_epilogue(const char *who, const qbp_epilogue *ep, const float *out, int64_t N, bool &wanted, EpilogueTail &tail,
                          bool &has_tail, int64_t max_stat_cols = QBP_EPILOGUE_MAX_COLUMNS)
{
    wanted = ep && (ep->col_sum || ep->col_min || ep->col_max);
    has_tail = ep && (ep->relu || ep->q_out);
    tail = EpilogueTail{nullptr, 0, nullptr, nullptr, nullptr, 0};
    if (wanted) {
        if (!ep->col_sum || !ep->col_min || !ep->col_max) return fail(QBP_ERR_INVALID_ARG, "%s: the epilogue needs col_sum, col_min and col_max together", who);
        if (!out) return fail(QBP_ERR_INVALID_ARG, "%s: column statistics need the fp32 output", who);
        if (N > max_stat_cols) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "%s: column statistics for at most %lld columns", who, (long long)max_stat_cols);
        if (has_tail) return fail(QBP_ERR_INVALID_ARG, "%s: column statistics and ReLU / requantisation exclude one another", who);
    }
    if (has_tail) {
        if (ep->q_out && (!ep->requant_range || !ep->qp_out)) return fail(QBP_ERR_INVALID_ARG, "%s: requantisation needs requant_range and qp_out", who);
        if (!ep->q_out && !out) return fail(QBP_ERR_INVALID_ARG, "%s: ReLU without an output", who);
        if (ep->q_out && !aligned16(ep->q_out)) return fail(QBP_ERR_INVALID_ARG, "%s: q_out must be 16-byte aligned", who);
        tail.relu = ep->relu ? 1 : 0; tail.rq = ep->qp_out; tail.q = ep->q_out; tail.row_sums = ep->q_out ? ep->row_sums_out : nullptr;
    }
    return QBP_OK;
}

static int launch_epilogue_qparams(const qbp_epilogue *ep, cudaStream_t st)
{
    if (!ep->q_out) return QBP_OK;
    QBP_TRACE_BEGIN(st);
    epilogue_qparams_kernel<<<1, 1, 0, st>>>(ep->requant_range, ep->qp_out);
    QBP_LAUNCH_OK("epilogue_qparams_kernel");
    return QBP_OK;
}

static int finish_epilogue(const qbp_epilogue *ep, const ColStatParts &parts, int64_t N, cudaStream_t st)
{
    QBP_TRACE_BEGIN(st);
    colstat_finalize_kernel<<<(int)N, 128, 0, st>>>(parts.lo, parts.hi, parts.sum, parts.rows, (int)N, ep->col_sum, ep->col_min, ep->col_max);
    QBP_LAUNCH_OK("colstat_finalize_kernel");
    return QBP_OK;
}

// ================================================================== launchers
// Shared memory of the kernel that is not the stage ring or the resident filter: alignment slack, epilogue staging
// slabs, the tables, the column terms (the whole table when it is small, else one tile's columns per epilogue group).
static uint32_t fixed_smem(MmaParams &P)
{
    // several small accumulators let the MMAs run ahead of the epilogue (msub == 1: one per epilogue group in turn)
    P.nbuf = std::min(kMaxAccBufs, 512 / (P.msub * P.bn));
    P.egroups = P.msub == 2 ? 2 : std::min(kEpiWarps / 4, P.nbuf);
    if (P.msub == 1) P.nbuf -= P.nbuf % P.egroups;
    P.ewarps = 4 * P.egroups;
    P.cterm_all = (size_t)P.ncls * P.N * sizeof(int32_t) <= 32u * 1024u ? 1 : 0;
    const size_t cterm_bytes = P.cterm_all ? ((size_t)P.ncls * P.N + 64) * sizeof(int32_t)
                                           : (size_t)(P.msub == 1 ? P.egroups : 1) * P.ncls * P.bn * sizeof(int32_t);
    P.iter_entries = P.mode == MODE_GEMM ? 0 : (int)align_up((size_t)P.k_iters, 64);
    P.cterm_span = (uint32_t)align_up(cterm_bytes, 1024);
    P.stat_local = (P.st_sum && P.N > QBP_EPILOGUE_MAX_COLUMNS) ? 1 : 0;
    P.stat_cols = P.stat_local ? P.bn : (int)P.N;
    P.stat_span = P.st_sum ? (uint32_t)align_up((size_t)P.ewarps * P.stat_cols * sizeof(ColStat), 1024) : 0u;
    const uint32_t fold_bytes = P.ep_fold ? (uint32_t)align_up((size_t)P.N * sizeof(float4), 1024) : 0u;
    return 2048u + (uint32_t)P.ewarps * kStageSlab * (uint32_t)P.nslab + (uint32_t)P.iter_entries * 16u + P.cterm_span +
           P.stat_span + fold_bytes;
}

// Whether a convolution can run from halo tiles: the whole filter resident beside at least three halo tiles.
static bool halo_fits(MmaParams &P, uint32_t halo_tile_bytes)
{
    const uint32_t fixed = fixed_smem(P);
    return P.tiles_n == 1 && fixed + align_up((size_t)P.b.tile_bytes * P.k_iters, 1024) + 3u * halo_tile_bytes <= kSmemBudget;
}

static int launch_mma(MmaParams &P, int tiles_m, bool clear_status, cudaStream_t st)
{
    const uint32_t fixed = fixed_smem(P);
    const uint32_t budget = kSmemBudget - fixed;
    P.ips = 1; P.b_resident = 0; P.b_res_bytes = 0;
    if (P.halo) {
        // one halo tile per channel chunk; as many chunks per stage as leave three stages (a commit per stage
        // drains the MMA pipeline, so fewer and longer stages are better)
        const int taps = P.k_iters / P.cchunks;
        P.b_resident = 1; P.b_res_bytes = (uint32_t)align_up((size_t)P.b.tile_bytes * P.k_iters, 1024);
        for (int c = 1; c <= P.cchunks; ++c)
            if (P.cchunks % c == 0 && c <= 32 && c * taps * P.mma_per_iter <= kMaxStageMmas &&
                3u * (uint32_t)c * P.a.tile_bytes <= budget - P.b_res_bytes) P.ips = c;
        P.groups = P.cchunks / P.ips;
        P.stage_mmas = P.ips * taps * P.mma_per_iter;
        P.b_stage_tiles = P.ips * taps;
        P.stage_tx = (uint32_t)P.ips * (uint32_t)(P.halo_w * ((1 << P.bh_log2) + 2 * P.pad) * P.chunk_bytes);
    } else if (P.mode != MODE_GEMM) {
        // keep the whole filter in shared memory when it fits beside at least three activation stages
        const uint32_t b_all = P.b.tile_bytes * (uint32_t)P.k_iters;
        if (P.tiles_n == 1 && b_all + 3 * P.a.tile_bytes <= budget) { P.b_resident = 1; P.b_res_bytes = (uint32_t)align_up(b_all, 1024); }
        // several operand tiles share one stage: every tcgen05.commit that releases a stage drains the MMA
        // pipeline (some hundred cycles), which short MMAs cannot afford often; two stages must still fit
        const uint32_t per_iter = P.a.tile_bytes + (P.b_resident ? 0u : P.b.tile_bytes);
        for (int c = 1; c <= P.k_iters; ++c)
            if (P.k_iters % c == 0 && c <= 32 && 2u * (uint32_t)c * per_iter <= budget - P.b_res_bytes) P.ips = c;
    }
    const uint32_t stage_bytes = (uint32_t)P.ips * (P.a.tile_bytes * (uint32_t)P.msub + (P.b_resident ? 0u : P.b.tile_bytes));
    if (!P.halo) {
        P.groups = P.k_iters / P.ips;
        P.stage_mmas = P.ips * P.msub * P.mma_per_iter;
        P.b_stage_tiles = P.ips;
        P.stage_tx = stage_bytes;
    }
    int stages = (int)((budget - P.b_res_bytes) / stage_bytes);
    if (stages < 2) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "tensor-core tile does not fit shared memory");
    stages = std::min(stages, kMaxStages);
    P.stages = stages;
    int cols = 32; while (cols < P.nbuf * P.msub * P.bn) cols <<= 1;
    P.tmem_cols = cols;
    P.tiles_m = tiles_m;
    P.tiles_total = tiles_m * P.tiles_n;
    P.d_tiles_n = make_fastdiv(P.tiles_n);
    P.d_group = make_fastdiv(kGroupM * P.tiles_n);
    P.d_tiles_w = make_fastdiv(P.mode == MODE_GEMM ? 1 : P.tiles_w);
    P.d_tiles_h = make_fastdiv(P.mode == MODE_GEMM ? 1 : P.tiles_h);
    const size_t smem = (size_t)fixed + P.b_res_bytes + (size_t)stages * stage_bytes;
    const bool tail = P.ep_fold || P.ep_relu || P.ep_q;
    static PerDeviceOnce configured[2];
    if (tail) QBP_SMEM_OPT_IN(configured[1], qbp_mma_kernel<true>, kSmemBudget);
    else      QBP_SMEM_OPT_IN(configured[0], qbp_mma_kernel<false>, kSmemBudget);
    if (clear_status) QBP_CUDA_OK(cudaMemsetAsync(P.status, 0, sizeof(int), st));
    // one CTA per SM (its shared-memory ring fills the SM), each walking its share of the tiles
    int grid = std::min(P.tiles_total, sm_count());
    if (P.stat_local) {
        // (a CTA then meets one column tile only: its tiles are blockIdx.x + k * grid)
        if (P.mode == MODE_GEMM || P.tiles_n > grid) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "column statistics: too many columns");
        grid -= grid % P.tiles_n;
    }
    P.grid = grid;
    QBP_TRACE_BEGIN(st);
    if (tail) qbp_mma_kernel<true><<<grid, kMmaThreads, smem, st>>>(P);
    else      qbp_mma_kernel<false><<<grid, kMmaThreads, smem, st>>>(P);
    QBP_LAUNCH_OK("qbp_mma_kernel");
    return QBP_OK;
}

static size_t gemm_ws_bytes(int64_t M, int64_t N)
{
    return 256 + align_up(sizeof(int32_t) * M, 256) + align_up(sizeof(int32_t) * N, 256) +
           align_up(sizeof(int64_t) * M, 256) + align_up(sizeof(int64_t) * N, 256) + colstat_ws_bytes(N);
}

bool conv_supported(const qbp_conv_desc *d)
{
    return d->stride == 1 && d->R == d->S && (d->R == 1 || d->R == 3) && d->pad == (d->R - 1) / 2 && d->N > 0 &&
           d->H > 0 && d->W > 0 && d->C > 0 && d->K > 0 && d->C % 16 == 0 && d->K % 16 == 0;
}

// What the product itself carves from the workspace, and with the room for the column statistics' partial rows
// (at its end) that the public entry point may need.
static size_t conv_core_ws_bytes(const qbp_conv_desc *d)
{
    const int64_t pix = (int64_t)d->N * d->H * d->W;
    const int64_t nmax = std::max(d->C, d->K);
    return 256 + align_up(sizeof(int32_t) * pix, 256) * 2 + align_up(sizeof(int32_t) * 16 * nmax, 256) +
           align_up(sizeof(int64_t) * (int64_t)d->R * d->S * nmax, 256);
}
static size_t conv_ws_bytes(const qbp_conv_desc *d)
{
    return conv_core_ws_bytes(d) + std::max(colstat_ws_bytes(d->C, true), colstat_ws_bytes(d->K, true));
}

// Picks the pixel box (bw x bh x bn = 128, powers of two) that wastes the fewest MMA rows.
static void pick_pixel_box(int Nimg, int H, int W, int &bwl, int &bhl)
{
    long long best = -1;
    for (int a = 0; a <= 7; ++a)
        for (int b = 0; a + b <= 7; ++b) {
            const int bw = 1 << a, bh = 1 << b, bn = 128 >> (a + b);
            const long long tiles = (long long)((W + bw - 1) / bw) * ((H + bh - 1) / bh) * ((Nimg + bn - 1) / bn);
            // prefer fewer tiles, then wider rows (longer contiguous runs per TMA row)
            const long long score = tiles * 64 - a * 8 - b;
            if (best < 0 || score < best) { best = score; bwl = a; bhl = b; }
        }
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) int qbp_device_status(const void *ws, void *stream)
{
    if (!ws) return fail(QBP_ERR_INVALID_ARG, "device_status: ws is NULL");
    int word = 0;
    QBP_CUDA_OK(cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    QBP_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    if (word == (int)QBP_ERR_TIMEOUT)
        return fail(QBP_ERR_TIMEOUT, "a bounded device-side wait gave up: the outputs of the calls that used this workspace are invalid");
    if (word != 0) return fail(QBP_ERR_INVALID_ARG, "device_status: the workspace does not start with a status word (found %d)", word);
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) int qbp_selftest_bounded_wait(void *ws, size_t ws_bytes, uint32_t limit_cycles, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (!ws || ws_bytes < sizeof(int)) return fail(QBP_ERR_WORKSPACE, "selftest_bounded_wait: workspace of 4 bytes needed");
    if (limit_cycles == 0 || limit_cycles > 100000000u)
        return fail(QBP_ERR_INVALID_ARG, "selftest_bounded_wait: limit_cycles must be in [1, 1e8]");
    QBP_CUDA_OK(cudaMemsetAsync(ws, 0, sizeof(int), st));
    QBP_TRACE_BEGIN(st);
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>((long long)limit_cycles, static_cast<int *>(ws));
    QBP_LAUNCH_OK("bounded_wait_selftest_kernel");
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) size_t qbp_gemm_s8_workspace_bytes(int64_t M, int64_t N, int64_t K)
{
    (void)K;
    return gemm_ws_bytes(M > 0 ? M : 1, N > 0 ? N : 1);
}

extern "C" __attribute__((visibility("default"))) int qbp_gemm_s8(int transA, int transB, int64_t M, int64_t N, int64_t K, const int8_t *A,
                           const qbp_qparams *qa, const int8_t *B, const qbp_qparams *qb, int32_t *acc_out, float *C,
                           const qbp_epilogue *ep, void *ws, size_t ws_bytes, void *stream)
{
    return gemm_s8_impl(transA, transB, M, N, K, A, qa, B, qb, acc_out, C, ep, nullptr, ws, ws_bytes, (cudaStream_t)stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_gemm_s8_sums(int transA, int transB, int64_t M, int64_t N, int64_t K, const int8_t *A,
                           const qbp_qparams *qa, const int32_t *a_sums, const int8_t *B, const qbp_qparams *qb,
                           const int32_t *b_sums, int32_t *acc_out, float *C, const qbp_epilogue *ep, void *ws,
                           size_t ws_bytes, void *stream)
{
    return gemm_s8_impl(transA, transB, M, N, K, A, qa, B, qb, acc_out, C, ep, nullptr, ws, ws_bytes, (cudaStream_t)stream, a_sums, b_sums);
}

int qbp::gemm_s8_impl(int transA, int transB, int64_t M, int64_t N, int64_t K, const int8_t *A, const qbp_qparams *qa,
                      const int8_t *B, const qbp_qparams *qb, int32_t *acc_out, float *C, const qbp_epilogue *ep,
                      int *ext_status, void *ws, size_t ws_bytes, cudaStream_t st, const int32_t *a_sums, const int32_t *b_sums)
{
    if (M <= 0 || N <= 0 || K <= 0) return fail(QBP_ERR_INVALID_ARG, "gemm_s8: M, N, K must be positive");
    if (M % 16 || N % 16 || K % 16) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "gemm_s8: M, N, K must be multiples of 16");
    if (K > 33025) return fail(QBP_ERR_OVERFLOW_K, "gemm_s8: K = %lld exceeds 33025 (255*255*K must fit int32)", (long long)K);
    if (M > INT32_MAX || N > INT32_MAX) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "gemm_s8: extent too large");
    if (!A || !B || !qa || !qb) return fail(QBP_ERR_INVALID_ARG, "gemm_s8: NULL operand");
    if (!acc_out && !C && !(ep && ep->q_out)) return fail(QBP_ERR_INVALID_ARG, "gemm_s8: acc_out and C are both NULL");
    if (!aligned16(A) || !aligned16(B) || (C && !aligned16(C)) || (acc_out && !aligned16(acc_out)))
        return fail(QBP_ERR_INVALID_ARG, "gemm_s8: operands must be 16-byte aligned");
    if (!ws || ws_bytes < gemm_ws_bytes(M, N))
        return fail(QBP_ERR_WORKSPACE, "gemm_s8: workspace of %zu bytes needed, %zu given", gemm_ws_bytes(M, N), ws_bytes);

    bool stats = false, has_tail = false;
    EpilogueTail tail;
    {
        const int erc = check_epilogue("gemm_s8", ep, C, N, stats, tail, has_tail);
        if (erc) return erc;
        if (!acc_out && !C && !(has_tail && tail.q)) return fail(QBP_ERR_INVALID_ARG, "gemm_s8: no output wanted");
    }
    WsCarver w(ws, ws_bytes);
    int *status = w.take<int>(1);
    if (ext_status) status = ext_status;         // the caller's sticky word: raised here, never cleared
    int32_t *rowterm = w.take<int32_t>(M);
    int32_t *colterm = w.take<int32_t>(N);
    int64_t *tmp_m = w.take<int64_t>(M);
    int64_t *tmp_n = w.take<int64_t>(N);
    ColStatParts parts{nullptr, nullptr, nullptr, 0};
    if (stats) {
        const size_t cells = (size_t)colstat_rows_max() * (size_t)N;
        parts.lo = w.take<float>(cells); parts.hi = w.take<float>(cells); parts.sum = w.take<double>(cells);
    }

    // code sums along the reduction
    int rc = QBP_OK;
    // (sums along stored rows are int32, along stored columns int64; the caller's are int32 either way)
    const bool a32 = a_sums || !transA, b32 = b_sums || transB;
    if (!a_sums) {
        if (!transA) rc = launch_rowsum(A, true, M, K, (int32_t *)tmp_m, st);
        else         rc = launch_colsum(A, true, K, M, tmp_m, st);
        if (rc) return rc;
    }
    if (!b_sums) {
        if (transB) rc = launch_rowsum(B, true, N, K, (int32_t *)tmp_n, st);
        else        rc = launch_colsum(B, true, K, N, tmp_n, st);
        if (rc) return rc;
    }
    const int32_t *ra32 = a_sums ? a_sums : (const int32_t *)tmp_m, *cb32 = b_sums ? b_sums : (const int32_t *)tmp_n;
    const int64_t mx = std::max(M, N);
    QBP_TRACE_BEGIN(st);
    gemm_terms_kernel<<<(int)((mx + 255) / 256), 256, 0, st>>>(
        a32 ? ra32 : nullptr, a32 ? nullptr : (const long long *)tmp_m,
        b32 ? cb32 : nullptr, b32 ? nullptr : (const long long *)tmp_n, M, N, K, qa, qb,
        rowterm, colterm);
    QBP_LAUNCH_OK("gemm_terms_kernel");

    // large products run on CTA pairs (256 x 256 tiles across two SMs); the column statistics are the
    // single-CTA kernel's (at most 256 columns: narrow either way)
    if (gemm2_eligible(M, N, K) && !stats && !has_tail)
        return launch_gemm2(transA, transB, M, N, K, A, qa, B, qb, acc_out, C, rowterm, colterm, status, !ext_status, st);

    MmaParams P{};
    P.mode = MODE_GEMM;
    P.kblock = 128;
    P.k_iters = (int)((K + 127) / 128);
    P.mma_per_iter = 4;
    P.msub = M > 128 ? 2 : 1;            // 256-row CTA tiles halve the operand traffic per multiply-add
    P.ncls = 1; P.nslab = 1;
    // A: stored [M x K] -> K-major rows of 128 reduction bytes; stored [K x M] -> M-major, one box per sub-tile
    if (!transA) {
        P.a = layout_kmajor(128, 128);
        rc = make_map_2d(&P.mapA, A, M, K, 128u * P.msub, 128);
    } else {
        P.a = layout_mnmajor(128, 128, 1, 0);
        P.a_loads = P.msub; P.a_load_bytes = P.a.tile_bytes;
        rc = make_map_2d(&P.mapA, A, K, M, 128, 128);
    }
    if (rc) return rc;
    if (transB) {
        P.bn = (int)std::min<int64_t>(256, N);
        P.b = layout_kmajor((uint32_t)P.bn, 128);
        rc = make_map_2d(&P.mapB, B, N, K, (uint32_t)P.bn, 128);
    } else {
        // N-contiguous operand: one swizzled row holds min(128, N) output columns; two such chunks make 256
        const uint32_t rb = N >= 128 ? 128u : N >= 64 ? 64u : 32u;
        const uint32_t chunks = (rb == 128 && N >= 256) ? 2u : 1u;
        P.bn = (int)(rb * chunks);
        P.b = layout_mnmajor(128, rb, chunks, 128 * rb);
        P.b_loads = (int)chunks; P.b_load_bytes = 128 * rb;
        rc = make_map_2d(&P.mapB, B, K, N, 128, rb);
    }
    if (rc) return rc;
    if (C && (rc = make_map_out_2d(&P.mapC, C, M, N))) return rc;
    P.idesc = make_idesc(true, true, P.a.major, P.b.major, 128, (uint32_t)P.bn);
    P.tiles_n = (int)((N + P.bn - 1) / P.bn);
    P.M = M; P.N = N;
    P.acc_out = acc_out; P.out = C;
    P.rowterm = rowterm; P.colterm = colterm; P.qa = qa; P.qb = qb; P.status = status;
    if (stats) { P.st_lo = parts.lo; P.st_hi = parts.hi; P.st_sum = parts.sum; }
    bool fused_row_sums = false;
    if (has_tail) {
        if ((rc = launch_epilogue_qparams(ep, st))) return rc;
        P.ep_relu = tail.relu; P.ep_rq = tail.rq; P.ep_q = tail.q;
        fused_row_sums = tail.q && tail.row_sums && P.tiles_n == 1;
        if (fused_row_sums) P.ep_rowsum = tail.row_sums;
    }
    if ((rc = launch_mma(P, (int)((M + 128 * P.msub - 1) / (128 * P.msub)), !ext_status, st))) return rc;
    if (stats) { parts.rows = P.grid; return finish_epilogue(ep, parts, N, st); }
    if (has_tail && tail.q && tail.row_sums && !fused_row_sums) return launch_rowsum(tail.q, true, M, N, tail.row_sums, st);
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) size_t qbp_conv_s8_workspace_bytes(int mode, const qbp_conv_desc *d)
{
    (void)mode;
    if (!d || !conv_supported(d)) return 0;
    return conv_ws_bytes(d);
}

extern "C" __attribute__((visibility("default"))) int qbp_conv_s8_implicit(int mode, const qbp_conv_desc *d, const int8_t *in, const qbp_qparams *q_in,
                                    const int8_t *wgt, const qbp_qparams *q_w, int32_t *acc_out, float *out,
                                    const qbp_epilogue *ep, void *ws, size_t ws_bytes, void *stream)
{
    bool stats = false, has_tail = false;
    EpilogueTail tail;
    if (d && ep) {
        const int64_t Nout = mode == QBP_CONV_DGRAD ? d->C : d->K;
        // (a convolution takes the statistics of any number of channels: see MmaParams::stat_local)
        const int erc = check_epilogue("conv_s8", ep, out, Nout, stats, tail, has_tail, INT32_MAX);
        if (erc) return erc;
        if (has_tail) {
            const int rc = launch_epilogue_qparams(ep, (cudaStream_t)stream);
            if (rc) return rc;
            return conv_s8_impl(mode, d, in, q_in, wgt, q_w, acc_out, out, nullptr, nullptr, nullptr, ws, ws_bytes, (cudaStream_t)stream, &tail);
        }
        if (stats) {
            // the partial rows sit at the end of the workspace, behind what the product itself carves
            if (!conv_supported(d))
                return fail(QBP_ERR_UNSUPPORTED_SHAPE, "conv_s8: needs stride 1, R = S in {1,3}, pad = (R-1)/2, C and K multiples of 16");
            const size_t core = conv_core_ws_bytes(d), need = conv_ws_bytes(d);
            if (!ws || ws_bytes < need)
                return fail(QBP_ERR_WORKSPACE, "conv_s8: workspace of %zu bytes needed, %zu given", need, ws_bytes);
            const size_t cells = (size_t)colstat_rows_max() * (size_t)Nout;
            char *base = static_cast<char *>(ws) + core;
            ColStatParts parts;
            parts.lo = reinterpret_cast<float *>(base);
            parts.hi = reinterpret_cast<float *>(base + align_up(cells * sizeof(float), 256));
            parts.sum = reinterpret_cast<double *>(base + 2 * align_up(cells * sizeof(float), 256));
            parts.rows = 0;
            const int rc = conv_s8_impl(mode, d, in, q_in, wgt, q_w, acc_out, out, nullptr, &parts, nullptr, ws, core, (cudaStream_t)stream);
            if (rc) return rc;
            return finish_epilogue(ep, parts, Nout, (cudaStream_t)stream);
        }
    }
    return conv_s8_impl(mode, d, in, q_in, wgt, q_w, acc_out, out, nullptr, nullptr, nullptr, ws, ws_bytes, (cudaStream_t)stream);
}

int qbp::conv_s8_impl(int mode, const qbp_conv_desc *d, const int8_t *in, const qbp_qparams *q_in, const int8_t *wgt,
                      const qbp_qparams *q_w, int32_t *acc_out, float *out, const int32_t *in_chan_sum, ColStatParts *stats,
                      int *ext_status, void *ws, size_t ws_bytes, cudaStream_t st, const EpilogueTail *tail)
{
    if (!d) return fail(QBP_ERR_INVALID_ARG, "conv_s8: descriptor is NULL");
    if (mode != QBP_CONV_FPROP && mode != QBP_CONV_DGRAD) return fail(QBP_ERR_INVALID_ARG, "conv_s8: bad mode");
    if (!conv_supported(d))
        return fail(QBP_ERR_UNSUPPORTED_SHAPE,
                    "conv_s8: needs stride 1, R = S in {1,3}, pad = (R-1)/2, C and K multiples of 16");
    if ((int64_t)d->R * d->S * std::max(d->C, d->K) > 33025)
        return fail(QBP_ERR_OVERFLOW_K, "conv_s8: reduction length exceeds 33025");
    if ((int64_t)d->N * d->H * d->W >= (1ll << 31)) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "conv_s8: 2^31 or more positions");
    if (!in || !wgt || !q_in || !q_w) return fail(QBP_ERR_INVALID_ARG, "conv_s8: NULL operand");
    const bool want_codes = tail && tail->q;
    if (!acc_out && !out && !stats && !want_codes) return fail(QBP_ERR_INVALID_ARG, "conv_s8: no output wanted");
    if (!aligned16(in) || !aligned16(wgt) || (out && !aligned16(out)) || (acc_out && !aligned16(acc_out)))
        return fail(QBP_ERR_INVALID_ARG, "conv_s8: operands must be 16-byte aligned");
    if (!ws || ws_bytes < conv_core_ws_bytes(d))
        return fail(QBP_ERR_WORKSPACE, "conv_s8: workspace of %zu bytes needed, %zu given", conv_ws_bytes(d), ws_bytes);
    if (tail) {
        const int n_out = mode == QBP_CONV_DGRAD ? d->C : d->K;
        if (stats && (tail->fold || tail->relu || tail->q))
            return fail(QBP_ERR_INVALID_ARG, "conv_s8: column statistics are of the plain output (no epilogue tail)");
        if (want_codes && (!tail->rq || !aligned16(tail->q))) return fail(QBP_ERR_INVALID_ARG, "conv_s8: 8-bit output needs parameters and a 16-byte aligned buffer");
        if (tail->fold && n_out > 256)
            return fail(QBP_ERR_UNSUPPORTED_SHAPE, "conv_s8: the fused normalisation takes at most 256 output channels");
    }

    const bool dgrad = mode == QBP_CONV_DGRAD;
    const int Cred = dgrad ? d->K : d->C;        // channels reduced over
    const int Nout = dgrad ? d->C : d->K;        // channels produced
    const int64_t pix = (int64_t)d->N * d->H * d->W;
    const int taps = d->R * d->S;
    const int64_t nmax = std::max(d->C, d->K);

    WsCarver w(ws, ws_bytes);
    int *status = w.take<int>(1);
    if (ext_status) status = ext_status;         // the caller's sticky word: raised here, never cleared
    int32_t *rowterm = w.take<int32_t>(pix);
    int32_t *chan_sum = w.take<int32_t>(pix);
    int32_t *colterm = w.take<int32_t>(16 * nmax);
    int64_t *wsum = w.take<int64_t>((int64_t)taps * nmax);

    int rc = QBP_OK;
    if (!(tail && tail->keep_terms)) {
        if (in_chan_sum) chan_sum = const_cast<int32_t *>(in_chan_sum);
        else if ((rc = launch_rowsum(in, true, pix, Cred, chan_sum, st))) return rc;
        if (!(tail && tail->colterm)) {          // (else: the column terms came with the filter's codes)
            if (!dgrad) rc = launch_rowsum(wgt, true, (int64_t)d->K * taps, d->C, (int32_t *)wsum, st);   // [k][tap]
            else        rc = launch_colsum(wgt, true, d->K, (int64_t)taps * d->C, wsum, st);                    // [tap][c]
            if (rc) return rc;
            QBP_TRACE_BEGIN(st);
            conv_colterm_kernel<<<dim3((Nout + 127) / 128, 16), 128, 0, st>>>(
                dgrad ? nullptr : (const int32_t *)wsum, dgrad ? (const long long *)wsum : nullptr, Nout, d->R, d->S, d->pad,
                dgrad ? 1 : 0, q_in, colterm);
            QBP_LAUNCH_OK("conv_colterm_kernel");
        }
        QBP_TRACE_BEGIN(st);
        conv_rowterm_kernel<<<dim3((unsigned)((d->H * d->W + 255) / 256), (unsigned)d->N), 256, 0, st>>>(
            chan_sum, d->H * d->W, d->H, d->W, make_fastdiv(d->W), d->pad, Cred, q_in, q_w, rowterm);
        QBP_LAUNCH_OK("conv_rowterm_kernel");
    }

    MmaParams P{};
    P.mode = dgrad ? MODE_DGRAD : MODE_FPROP;
    P.msub = 1; P.ncls = 16; P.nslab = 1;
    if (stats) { P.st_lo = stats->lo; P.st_hi = stats->hi; P.st_sum = stats->sum; }
    if (tail) { P.ep_fold = tail->fold; P.ep_relu = tail->relu; P.ep_rq = tail->rq; P.ep_q = tail->q; }
    if (tail && tail->colterm) colterm = const_cast<int32_t *>(tail->colterm);
    P.H = d->H; P.W = d->W; P.Nimg = d->N; P.pad = d->pad; P.S = d->S; P.Cred = Cred;
    const uint32_t cb = Cred % 128 == 0 ? 128u : Cred % 64 == 0 ? 64u : 32u;      // reduction bytes per stage row
    P.chunk_bytes = (int)cb;
    P.cchunks = (Cred + (int)cb - 1) / (int)cb;      // a ragged last chunk is zero-filled by TMA on the activation side
    P.k_iters = taps * P.cchunks;
    P.mma_per_iter = (int)cb / 32;
    if (!dgrad) {
        P.bn = std::min(256, Nout);
        P.b = layout_kmajor((uint32_t)P.bn, cb);
        rc = make_map_2d(&P.mapB, wgt, d->K, (uint64_t)taps * d->C, (uint32_t)P.bn, cb);
    } else {
        const uint32_t rb = Nout >= 128 ? 128u : Nout >= 64 ? 64u : 32u;
        const uint32_t chunks = (rb == 128 && Nout >= 256) ? 2u : 1u;
        P.bn = (int)(rb * chunks);
        P.b = layout_mnmajor(cb, rb, chunks, cb * rb);
        P.b_loads = (int)chunks; P.b_load_bytes = cb * rb;
        rc = make_map_2d(&P.mapB, wgt, d->K, (uint64_t)taps * d->C, cb, rb);
    }
    if (rc) return rc;
    P.tiles_n = (Nout + P.bn - 1) / P.bn;
    P.M = pix; P.N = Nout;

    int bwl = 0, bhl = 0;
    pick_pixel_box(d->N, d->H, d->W, bwl, bhl);
    // 3 x 3: a box of 16 rows x 8 pixels of one image, loaded once with its border; the nine taps are windows of
    // that tile (a ninth of the operand traffic of one load per tap).  Taken when the filter stays resident and the
    // fixed box does not waste many more MMA rows than the free one.
    if (d->R == 3) {
        const uint32_t halo_bytes = (uint32_t)align_up((size_t)18 * 10 * cb, 1024);
        const long long tiles_free = (long long)((d->W + (1 << bwl) - 1) >> bwl) * ((d->H + (1 << bhl) - 1) >> bhl) *
                                     ((d->N + (128 >> (bwl + bhl)) - 1) / (128 >> (bwl + bhl)));
        const long long tiles_halo = (long long)((d->W + 7) / 8) * ((d->H + 15) / 16) * d->N;
        P.nslab = 2;                  // (two slabs per warp: a store is still reading one while the next is filled)
        if (tiles_halo * 2 <= tiles_free * 3 && halo_fits(P, halo_bytes)) {
            P.halo = 1; P.halo_w = kHaloW; bwl = 3; bhl = 4;
            P.halo_rb = dgrad ? (Nout >= 128 ? 128 : Nout >= 64 ? 64 : 32) : 0;
        } else {
            P.nslab = 1;
        }
    }
    P.bw_log2 = bwl; P.bh_log2 = bhl;
    const int bw = 1 << bwl, bh = 1 << bhl, bn_img = 128 >> (bwl + bhl);
    P.tiles_w = (d->W + bw - 1) / bw; P.tiles_h = (d->H + bh - 1) / bh;
    const int tiles_img = (d->N + bn_img - 1) / bn_img;
    if (!P.halo) {
        P.a = layout_kmajor(128, cb);
        rc = make_map_nhwc(&P.mapA, in, d->N, d->H, d->W, Cred, bn_img, bh, bw, cb);
    } else {
        // 8-pixel groups (one image row of the box each) a halo row apart
        P.a = layout_kmajor(128, cb);
        P.a.tile_bytes = (uint32_t)align_up((size_t)(bh + 2) * P.halo_w * cb, 1024);
        P.a.desc_hi = (((uint32_t)P.halo_w * cb) >> 4) | (1u << 14) | (P.a.desc_hi & 0xE0000000u);
        rc = make_map_nhwc(&P.mapA, in, d->N, d->H, d->W, Cred, 1, bh + 2, P.halo_w, cb);
    }
    if (rc) return rc;
    if (out) {
        // a warp's 32 accumulator rows are a sub-box of the 128-pixel box (all extents are powers of two)
        const uint32_t sw = (uint32_t)std::min(bw, 32), sh = (uint32_t)std::min(bh, 32 / (int)sw), sn = 32 / (sw * sh);
        if ((rc = make_map_out_nhwc(&P.mapC, out, d->N, d->H, d->W, Nout, sn, sh, sw))) return rc;
    }
    P.idesc = make_idesc(true, true, P.a.major, P.b.major, 128, (uint32_t)P.bn);
    P.acc_out = acc_out; P.out = out;
    P.rowterm = rowterm; P.colterm = colterm; P.qa = q_in; P.qb = q_w; P.status = status;
    // each row's code sum comes from the epilogue when one column tile holds the whole row, else from a pass over the codes
    const bool fused_row_sums = want_codes && tail->row_sums && P.tiles_n == 1;
    if (fused_row_sums) P.ep_rowsum = tail->row_sums;
    if ((rc = launch_mma(P, P.tiles_w * P.tiles_h * tiles_img, !ext_status, st))) return rc;
    if (stats) stats->rows = P.grid;
    if (want_codes && tail->row_sums && !fused_row_sums) return launch_rowsum(tail->q, true, pix, Nout, tail->row_sums, st);
    return QBP_OK;
}
