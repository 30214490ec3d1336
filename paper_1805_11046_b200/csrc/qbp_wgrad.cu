// Weight gradient g_W = g_l I_{l-1}^T (Eq. (grad_weight)) from the 16-bit copy
// of the layer gradient and the 8-bit layer input (Sections 6, 7), on the
// int8 tensor cores.
//
// The 16-bit code is split into a signed high byte and an unsigned low byte,
// g16 = 256*hi + lo, so that  sum x*g16 = 256 * sum x*hi + sum x*lo  with two
// tcgen05.mma kind::i8 products (s8 x s8 and s8 x u8) into two int32
// accumulators in tensor memory.  The reduction runs over the batch rows
// (batch x spatial positions for a convolution): both operands are therefore
// "M/N-major" in shared memory -- the TMA box is [reduction rows x channels].
// A CTA reduces at most 65536 rows (128*255*65536 < 2^31 bounds the low limb,
// 128*128*65536 the high one) and combines its two accumulators exactly in
// int64.  Integer addition is order-free, so the split of the reduction over
// CTAs does not change the result.
//
// Work split: an item is (group of up to `ma` accumulator tiles of 128 output
// rows, tile of bn output columns); the reduction of an item is cut into
// slices in proportion to the item's cost per reduction step, so that one
// wave of CTAs finishes together.  A CTA that owns a whole reduction applies
// the zero-points and the scale itself; otherwise the CTAs write int64
// partials and a second kernel adds them up.
//
// Convolution: the MMA's 128 rows hold `chunks` filter taps x the input
// channels of one tap (2 taps x 64 channels, or 1 tap x 128 channels); each
// tap is its own TMA load of the input, shifted by the tap offset, padding
// zero-filled.  Zero-points are applied afterwards from per-border-class code
// sums (a tap near the border sees fewer positions).
//
// The TMA-issuing lanes run from a small table built once per CTA (one entry per load of a stage); the MMA warp
// runs whole with an elected issuer and the stage's MMAs fully unrolled for the operand layouts (see
// wg_issue_stage); stages are released in groups: a tcgen05.commit drains the MMA pipeline, which short MMAs
// cannot afford often.
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

constexpr int kWgThreads = 192;
constexpr int kWgFinalizeLanes = 4;   // lanes of the second kernel that share one output element's partials
constexpr int kWgRows = 128;         // reduction rows per pipeline stage: four k steps of 32 (what the MMA warp does
                                     // between stages is a fixed cost, so a stage should hold many MMAs)
constexpr int kWgMaxStages = 16;
constexpr int kWgMaxTiles = 4;       // A tiles (128 accumulator rows each) per CTA: 4 x 2 limbs x 64 columns fill tensor memory
constexpr int kWgMaxLoads = 32;      // TMA loads per stage: one lane each
constexpr uint32_t kWgSmem = 220u * 1024u;

struct WgradParams {
    CUtensorMap mapX, mapHi, mapLo;
    OperandLayout a, b;
    uint32_t idesc_hi, idesc_lo;
    // The low bytes stored as lo - 128 (signed): both limbs have one operand type, and a stage's MMAs take the high
    // and the low tile side by side as one B operand of 2 * bn columns (the x tile is then read from shared memory
    // once instead of once per limb).  g16 - zg = 256 * hi + (lo - 128) - (zg - 128): everything downstream works on
    // those limbs with the zero-point zg - 128.
    int lo_signed;
    uint32_t b2_desc_lo, idesc_fused;
    int tot_g_plain;                 // tot_g holds totals of 256 * hi + lo (left by a quantiser), not of the stored limbs
    // 3 x 3 convolution from halo tiles (with lo_signed): a stage holds the pixel box of x once, with its border of
    // one position (10 positions per box row), instead of one shifted copy per tap; a tap's operand is that tile read
    // from a shifted start (see wg_issue_stage_halo).  halo_bh: box rows per image in a stage (8 or 4; 0: not used).
    int halo_bh;
    uint32_t halo_bytes;             // the tile's room in a stage (1024-byte multiple)
    uint32_t halo_box_bytes;         // bytes one load of it brings
    uint32_t ones_off;               // offset (from the ring's start) of a region of halo_bytes filled with the code 1
    uint32_t a_chunk_bytes;          // bytes of one A chunk (kr rows x rb_a)
    int conv;                        // 0: x [M x K], g [M x N]; 1: NHWC tensors
    int stages, cg, bn, tmem_cols;   // cg: stages released by one commit
    int stages_last, cg_last;        // the ring of the CTAs of the last A group (fewer A tiles: smaller and more stages)
    int kr;                          // reduction rows per pipeline stage
    int a_chunks, rb_a;              // chunks per A tile, bytes (= channels / columns) per chunk row
    int ma;                          // A tiles per CTA (they share the g tiles of a stage)
    int a_tiles;                     // A tiles in all: plain K/128; conv tap groups x channel tiles
    int a_groups;                    // ceil(a_tiles / ma)
    int tiles_c;                     // conv: channel tiles per tap group
    int tiles_b;                     // output-channel (N) tiles of bn
    int iters_total;                 // reduction steps of kr rows each
    int s_full, s_last;              // slices of an item of a full A group / of the last (possibly smaller) group
    int ctas_full;                   // CTAs working on full groups: (a_groups - 1) * tiles_b * s_full
    int direct;                      // every item is one slice: the CTA finishes its outputs itself (plain only)
    // conv geometry
    int H, W, Nimg, pad, R, S, C, taps;
    int bw_log2, bh_log2, tiles_w, tiles_h;
    FastDiv d_tiles_w, d_tiles_h;
    // plain geometry
    int64_t M, N, K;
    long long *part;                 // int64 partials, one block of part_stride values per CTA
    int64_t part_stride;             // ma * 128 * bn, padded
    // direct epilogue (plain): acc = raw + rowterm[k] + colterm[n]
    const long long *rowterm, *colterm;
    const qbp_qparams *qx, *qg;
    long long *acc_out; float *dW;
    int *status;
    // Convolution: per-channel totals of the stored codes over all positions (x: [C]; the 16-bit gradient codes
    // 256 * hi + lo: [N]) that the kernels which wrote the codes left.  The class tables then hold the border classes
    // only, and the interior class is the total minus those.  NULL: the tables hold all sixteen classes.
    const long long *tot_x, *tot_g;
    // ... and those border classes can be taken by this kernel's epilogue warps while the MMAs run (a few percent of
    // the positions: the loads hide behind the main loop): cls_x [16][C], cls_hi / cls_lo [16][N] (zeroed beforehand),
    // the code tensors, and the offset of the CTA's tables in shared memory.  cls_x == NULL: done elsewhere.
    unsigned long long *cls_x, *cls_hi, *cls_lo;
    const uint8_t *codes_x, *codes_hi, *codes_lo;
    uint32_t cls_off;
    // The gradient's per-channel totals from the product itself: when the taps do not fill the last A tile, its first
    // spare chunk is filled with the code 1 once (nothing else writes there), so that the first accumulator row of
    // that chunk is sum over all positions of 1 * g -- MMA rows that were computed and thrown away before.  The
    // epilogue adds that row into ones_tot [N] (zeroed beforehand).  NULL: not used.
    unsigned long long *ones_tot;
};

// Which item and slice a CTA works on.
struct WgItem { int ag, tb, slice, slices; };

__device__ __forceinline__ WgItem wg_item(const WgradParams &P, int bid)
{
    WgItem w;
    int item;
    if (bid < P.ctas_full) { item = bid / P.s_full; w.slice = bid % P.s_full; w.slices = P.s_full; }
    else {
        const int r = bid - P.ctas_full;
        item = P.ctas_full / P.s_full + r / P.s_last; w.slice = r % P.s_last; w.slices = P.s_last;
    }
    w.ag = item / P.tiles_b; w.tb = item % P.tiles_b;
    return w;
}

// ---- MMA issue ------------------------------------------------------------------
// The MMA takes its operands from the warp's few uniform registers.  What the operand layouts (row bytes RBA of the
// x chunks, RBB of the gradient tiles = output columns per tile) and the number NT of A tiles fix is therefore
// spelled as constants and the MMAs of a stage are fully unrolled: descriptors that were looked up per MMA, or
// built from many run-time values, cost 110 to 150 cycles per MMA against 40 to 50 this way.
struct WgMmaArgs {
    uint64_t *full_bar, *empty_bar, *acc_bar;
    uint32_t ring, stage_bytes, a_bytes, tmem;
    int k_iters;
    uint32_t stages, cg;
    uint32_t a_desc_lo, b_desc_lo, idesc_hi;
    // halo tiles: per A tile of the CTA, (start of its first tap in the halo tile) >> 4 | (distance to its second
    // tap) >> 4 << 16, and what multiplies the stage's address (>> 4) before that is added: 1, or 1 - 65536 for the
    // tile whose second chunk is the region of ones (its distance is then counted from the ring's start).
    uint32_t tile_desc[4], tile_mult[4];
};


__host__ __device__ constexpr uint32_t wg_swizzle_bits(uint32_t row_bytes) { return row_bytes == 128 ? 2u : row_bytes == 64 ? 4u : 6u; }

// The 2 * KK * NT MMAs of a stage of kWgRows reduction rows: the limb outermost (switching between the s8 x s8 and s8 x u8
// instruction descriptors stalls the MMA pipe), then the k step, then the A tile, so that consecutive MMAs write
// different accumulators.  FIRST: the stage starts the reduction (its first k step overwrites the accumulators).
// FUSED: both limbs are signed and one MMA takes them side by side (N = 2 * RBB; b_lo then carries the distance
// between the two tiles as its leading byte offset and idesc_hi that N): KK * NT MMAs.
template <int RBA, int RBB, int NT, bool FIRST, bool FUSED>
__device__ __forceinline__ void wg_issue_stage(uint32_t tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc_hi)
{
    constexpr uint32_t a_hi = ((8u * RBA) >> 4) | (1u << 14) | (wg_swizzle_bits(RBA) << 29);
    constexpr uint32_t b_hi = ((8u * RBB) >> 4) | (1u << 14) | (wg_swizzle_bits(RBB) << 29);
    constexpr uint32_t a_kstep = 2u * RBA, b_kstep = 2u * RBB;     // 32 reduction rows, in 16-byte units
    constexpr int KK = kWgRows / 32;                               // k steps per stage
    constexpr uint32_t a_tile16 = (uint32_t)kWgRows * 128u / 16u;  // an A tile: kWgRows rows x 128 bytes
    constexpr uint32_t b_tile16 = (uint32_t)kWgRows * RBB / 16u;   // a limb's tile: kWgRows rows x RBB bytes
    if (FUSED) {
#pragma unroll
        for (int i = 0; i < KK * NT; ++i) {
            const int kk = i / NT, j = i % NT;
            const uint32_t ao = (uint32_t)j * a_tile16 + (uint32_t)kk * a_kstep;
            if (elect_one())
                mma_i8(tmem + (uint32_t)(j * 2 * RBB), ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + ao),
                       ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + (uint32_t)kk * b_kstep), idesc_hi, (FIRST && kk == 0) ? 0u : 1u);
        }
        return;
    }
    const uint32_t idesc_lo = idesc_hi ^ (1u << 10);               // the low limb is unsigned
#pragma unroll
    for (int i = 0; i < 2 * KK * NT; ++i) {
        const int limb = i / (KK * NT), kk = (i / NT) % KK, j = i % NT;
        const uint32_t ao = (uint32_t)j * a_tile16 + (uint32_t)kk * a_kstep;
        const uint32_t bo = (uint32_t)limb * b_tile16 + (uint32_t)kk * b_kstep;
        if (elect_one())
            mma_i8(tmem + (uint32_t)((j * 2 + limb) * RBB), ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + ao),
                   ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + bo), limb ? idesc_lo : idesc_hi, (FIRST && kk == 0) ? 0u : 1u);
    }
}

// The MMA warp's loop over its slice of the reduction.  False when a wait ran out.
template <int RBA, int RBB, int NT, bool FUSED>
__device__ __forceinline__ bool wg_mma_loop(const WgMmaArgs &A)
{
    uint32_t s = 0, ph = 0;
    uint32_t in_group = 0, group = 0;          // stages issued of the current release group, its index (no divisions here:
                                               // what this warp does between two stages leaves the MMA pipe idle)
    uint32_t a_addr = A.ring;
    for (int i = 0; i < A.k_iters; ++i) {
        if (!mbar_wait_uniform(&A.full_bar[s], ph)) return false;
        tc_fence_after();
        const uint32_t a_lo = ((a_addr >> 4) & 0x3FFFu) | A.a_desc_lo;
        const uint32_t b_lo = (((a_addr + A.a_bytes) >> 4) & 0x3FFFu) | A.b_desc_lo;
        if (i == 0) wg_issue_stage<RBA, RBB, NT, true, FUSED>(A.tmem, a_lo, b_lo, A.idesc_hi);
        else        wg_issue_stage<RBA, RBB, NT, false, FUSED>(A.tmem, a_lo, b_lo, A.idesc_hi);
        // release the group of stages this one completes (the commit covers every MMA issued so far)
        if (++in_group == A.cg) {
            if (elect_one()) mma_commit(&A.empty_bar[group]);
            in_group = 0; ++group;
        }
        a_addr += A.stage_bytes;
        if (++s == A.stages) { s = 0; ph ^= 1u; group = 0; a_addr = A.ring; }
    }
    if (elect_one()) mma_commit(A.acc_bar);
    return true;
}

template <int RBA, int RBB, bool FUSED>
__device__ __forceinline__ bool wg_mma_dispatch_nt(int nt, const WgMmaArgs &A)
{
    // (128 output columns per tile leave room for two A tiles in tensor memory)
    if (nt == 1) return wg_mma_loop<RBA, RBB, 1, FUSED>(A);
    if (nt == 2) return wg_mma_loop<RBA, RBB, 2, FUSED>(A);
    if (RBB == 128) return false;
    if (nt == 3) return wg_mma_loop<RBA, RBB, (RBB == 128 ? 1 : 3), FUSED>(A);
    return wg_mma_loop<RBA, RBB, (RBB == 128 ? 1 : 4), FUSED>(A);
}

// ---- the same from halo tiles ---------------------------------------------------
// The x tile of a stage is the pixel box (8 positions wide, BH rows, 16 / BH images) with a border of one position:
// rows of kWgHaloW positions.  The operand of tap (r, s) is the tile read from r * kWgHaloW + s positions in: the
// shared-memory swizzle is a function of the address, so a window that starts any whole number of positions into the
// tile reads what TMA wrote there.  A k step of 32 positions is four box rows: groups of eight positions a tile row
// apart (the stride byte offset), starting at the box row's place in the tile.
constexpr int kWgHaloW = 10;
template <int RBA, int BH>
__host__ __device__ constexpr uint32_t wg_halo_kstep16(int kk)
{
    return (uint32_t)((((kk * 4) / BH) * (BH + 2) * kWgHaloW + ((kk * 4) % BH) * kWgHaloW) * RBA / 16);
}

template <int RBA, int RBB, int NT, bool FIRST, int BH>
__device__ __forceinline__ void wg_issue_stage_halo(uint32_t tmem, const uint32_t (&a_lo)[NT], uint32_t b_lo, uint32_t idesc)
{
    constexpr uint32_t a_hi = (((uint32_t)kWgHaloW * RBA) >> 4) | (1u << 14) | (wg_swizzle_bits(RBA) << 29);
    constexpr uint32_t b_hi = ((8u * RBB) >> 4) | (1u << 14) | (wg_swizzle_bits(RBB) << 29);
    constexpr uint32_t b_kstep = 2u * RBB;
    constexpr int KK = kWgRows / 32;
#pragma unroll
    for (int i = 0; i < KK * NT; ++i) {
        const int kk = i / NT, j = i % NT;
        if (elect_one())
            mma_i8(tmem + (uint32_t)(j * 2 * RBB), ((uint64_t)a_hi << 32) | (uint64_t)(a_lo[j] + wg_halo_kstep16<RBA, BH>(kk)),
                   ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + (uint32_t)kk * b_kstep), idesc, (FIRST && kk == 0) ? 0u : 1u);
    }
}

template <int RBA, int RBB, int NT, int BH>
__device__ __forceinline__ bool wg_mma_loop_halo(const WgMmaArgs &A)
{
    uint32_t s = 0, ph = 0, in_group = 0, group = 0;
    uint32_t a_addr = A.ring;
    for (int i = 0; i < A.k_iters; ++i) {
        if (!mbar_wait_uniform(&A.full_bar[s], ph)) return false;
        tc_fence_after();
        const uint32_t base = (a_addr >> 4) & 0x3FFFu;
        uint32_t a_lo[NT];
#pragma unroll
        for (int j = 0; j < NT; ++j) a_lo[j] = base * A.tile_mult[j] + A.tile_desc[j];
        const uint32_t b_lo = (((a_addr + A.a_bytes) >> 4) & 0x3FFFu) | A.b_desc_lo;
        if (i == 0) wg_issue_stage_halo<RBA, RBB, NT, true, BH>(A.tmem, a_lo, b_lo, A.idesc_hi);
        else        wg_issue_stage_halo<RBA, RBB, NT, false, BH>(A.tmem, a_lo, b_lo, A.idesc_hi);
        if (++in_group == A.cg) {
            if (elect_one()) mma_commit(&A.empty_bar[group]);
            in_group = 0; ++group;
        }
        a_addr += A.stage_bytes;
        if (++s == A.stages) { s = 0; ph ^= 1u; group = 0; a_addr = A.ring; }
    }
    if (elect_one()) mma_commit(A.acc_bar);
    return true;
}

template <int RBA, int RBB>
__device__ __forceinline__ bool wg_mma_dispatch_halo(int nt, int bh, const WgMmaArgs &A)
{
    if (RBA < 64 || nt < 1 || nt > 4 || (RBB == 128 && nt > 2)) return false;
    constexpr int R = RBA < 64 ? 64 : RBA;             // (instances for the layouts that can occur only)
    if (bh == 8) {
        if (nt == 1) return wg_mma_loop_halo<R, RBB, 1, 8>(A);
        if (nt == 2) return wg_mma_loop_halo<R, RBB, 2, 8>(A);
        if (nt == 3) return wg_mma_loop_halo<R, RBB, (RBB == 128 ? 1 : 3), 8>(A);
        return wg_mma_loop_halo<R, RBB, (RBB == 128 ? 1 : 4), 8>(A);
    }
    if (nt == 1) return wg_mma_loop_halo<R, RBB, 1, 4>(A);
    if (nt == 2) return wg_mma_loop_halo<R, RBB, 2, 4>(A);
    if (nt == 3) return wg_mma_loop_halo<R, RBB, (RBB == 128 ? 1 : 3), 4>(A);
    return wg_mma_loop_halo<R, RBB, (RBB == 128 ? 1 : 4), 4>(A);
}

// Sixteen per-channel sums from one 16-byte group of codes (dot products that pick one byte each).
__device__ __forceinline__ void border_add(bool is_signed, const uint4 &v, int *acc)
{
    const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int b = 0; b < 4; ++b)
            acc[k * 4 + b] = is_signed ? __dp4a((int)wd[k], 1 << (8 * b), acc[k * 4 + b])
                                       : (int)__dp4a(wd[k], 1u << (8 * b), (unsigned)acc[k * 4 + b]);
}

// The border classes (first / last row, first / last column, corners; H, W >= 3) of images [img_begin, img_end) of one
// code tensor of C channels (C / 16 = 2, 4 or 8 groups), by 128 threads (t = 0..127), into tbl [16][C] (shared
// memory, zeroed).  Thread = (group, slot): it walks every slots-th position of the four edges, two images at a
// time, with one set of 16 sums per edge in registers.
__device__ __forceinline__ void wg_border_sums(bool is_signed, const uint8_t *__restrict__ q, int C, int H, int W, int img_begin,
                                               int img_end, int *tbl, int t)
{
    const int cv = C >> 4, slots = 128 / cv;
    const int g = t % cv, k = t / cv;
    int top[16], bot[16], lef[16], rig[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) { top[e] = 0; bot[e] = 0; lef[e] = 0; rig[e] = 0; }
    constexpr int U = 2;
    for (int img0 = img_begin; img0 < img_end; img0 += U) {
        const uint4 *base[U];
#pragma unroll
        for (int u = 0; u < U; ++u) base[u] = reinterpret_cast<const uint4 *>(q + (int64_t)min(img0 + u, img_end - 1) * H * W * C) + g;
        for (int w = 1 + k; w < W - 1; w += slots) {
            uint4 a[U], b[U];
#pragma unroll
            for (int u = 0; u < U; ++u) { a[u] = __ldg(base[u] + (int64_t)w * cv); b[u] = __ldg(base[u] + ((int64_t)(H - 1) * W + w) * cv); }
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (img0 + u < img_end) { border_add(is_signed, a[u], top); border_add(is_signed, b[u], bot); }
        }
        for (int h = 1 + k; h < H - 1; h += slots) {
            uint4 a[U], b[U];
#pragma unroll
            for (int u = 0; u < U; ++u) { a[u] = __ldg(base[u] + (int64_t)h * W * cv); b[u] = __ldg(base[u] + ((int64_t)h * W + W - 1) * cv); }
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (img0 + u < img_end) { border_add(is_signed, a[u], lef); border_add(is_signed, b[u], rig); }
        }
        if (k < 4) {
            // the four corners: classes 5, 9 (first row), 6, 10 (last row)
            const int h = k < 2 ? 0 : H - 1, w = (k & 1) ? W - 1 : 0;
            int cor[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) cor[e] = 0;
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (img0 + u < img_end) border_add(is_signed, __ldg(base[u] + ((int64_t)h * W + w) * cv), cor);
            int *dst = tbl + ((k < 2 ? 1 : 2) | ((k & 1) ? 8 : 4)) * C + g * 16;
#pragma unroll
            for (int e = 0; e < 16; ++e)
                if (cor[e]) atomicAdd(dst + e, cor[e]);
        }
    }
    // the lanes of a warp that hold the same group meet by shuffle (cv is 2, 4 or 8), then one lane per group adds
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        int tt = top[e], bb = bot[e], ll = lef[e], rr = rig[e];
        for (int off = cv; off < 32; off <<= 1) {
            tt += __shfl_xor_sync(0xffffffffu, tt, off); bb += __shfl_xor_sync(0xffffffffu, bb, off);
            ll += __shfl_xor_sync(0xffffffffu, ll, off); rr += __shfl_xor_sync(0xffffffffu, rr, off);
        }
        if ((t & 31) < cv) {
            if (tt) atomicAdd(tbl + 1 * C + g * 16 + e, tt);
            if (bb) atomicAdd(tbl + 2 * C + g * 16 + e, bb);
            if (ll) atomicAdd(tbl + 4 * C + g * 16 + e, ll);
            if (rr) atomicAdd(tbl + 8 * C + g * 16 + e, rr);
        }
    }
}

// One instance per pair of operand layouts: RBA = row bytes of the x chunks, RBB = row bytes of the gradient tiles.
template <int RBA, int RBB>
__global__ void __launch_bounds__(kWgThreads, 1) qbp_wgrad_kernel(const __grid_constant__ WgradParams P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kWgMaxStages], empty_bar[kWgMaxStages], acc_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int4 s_load[kWgMaxLoads];      // (destination offset in the stage, 0 x / 1 hi / 2 lo, channel offset, tap dw | dh << 16)
    __shared__ int s_counts[1];               // loads per stage

    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    const uint32_t a_tile_bytes = P.a_chunk_bytes * (uint32_t)P.a_chunks;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WgItem wi = wg_item(P, blockIdx.x);
    const int ag = wi.ag;
    const int n0 = wi.tb * P.bn;
    const int it_begin = (int)((int64_t)P.iters_total * wi.slice / wi.slices);
    const int it_end = (int)((int64_t)P.iters_total * (wi.slice + 1) / wi.slices);
    const int k_iters = it_end - it_begin;
    const int n_tiles = min(P.ma, P.a_tiles - ag * P.ma);        // A tiles this CTA owns
    const uint32_t a_bytes = P.halo_bh ? P.halo_bytes : a_tile_bytes * (uint32_t)n_tiles;
    const uint32_t stage_bytes = a_bytes + 2u * P.b.tile_bytes;
    const bool last_group = ag == P.a_groups - 1;
    const int stages = last_group ? P.stages_last : P.stages, cg = last_group ? P.cg_last : P.cg;
    const int kk_per_iter = P.kr / 32;

    // chunks present in A tile `at`: conv -- taps left in the tap group; plain -- column chunks left in K
    auto chunks_of = [&](int at) {
        if (P.conv) return min(P.a_chunks, P.taps - (at / P.tiles_c) * P.a_chunks);
        return min(P.a_chunks, (int)((P.K - (int64_t)at * 128 + P.rb_a - 1) / P.rb_a));
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&acc_bar, 1);
        mbar_fence_init();
        tma_prefetch_desc(&P.mapX); tma_prefetch_desc(&P.mapHi); tma_prefetch_desc(&P.mapLo);
        // the loads of one stage
        int nl = 0;
        s_load[nl++] = make_int4((int)a_bytes, 1, n0, 0);
        s_load[nl++] = make_int4((int)(a_bytes + P.b.tile_bytes), 2, n0, 0);
        if (P.halo_bh) s_load[nl++] = make_int4(0, 0, 0, ((-P.pad) & 0xFFFF) | ((-P.pad) << 16));     // the box with its border
        for (int j = 0; j < (P.halo_bh ? 0 : n_tiles); ++j) {
            const int at = ag * P.ma + j, nc = chunks_of(at);
            for (int c = 0; c < nc; ++c) {
                const int dst = (int)((uint32_t)j * a_tile_bytes + (uint32_t)c * P.a_chunk_bytes);
                if (!P.conv) s_load[nl++] = make_int4(dst, 0, at * 128 + c * P.rb_a, 0);
                else {
                    const int tap = (at / P.tiles_c) * P.a_chunks + c;
                    const int dh = tap / P.S - P.pad, dw = tap % P.S - P.pad;
                    s_load[nl++] = make_int4(dst, 0, (at % P.tiles_c) * P.rb_a, (dw & 0xFFFF) | (dh << 16));
                }
            }
        }
        s_counts[0] = nl;
    }
    if (warp == 1) { tmem_alloc(&tmem_slot, (uint32_t)P.tmem_cols); tmem_relinquish(); }
    if (P.ones_tot && last_group && P.halo_bh) {
        // halo tiles: the spare chunk of the last A tile is read from a region of its own, filled with the code 1
        uint4 *dst = reinterpret_cast<uint4 *>(smem + P.ones_off);
        for (uint32_t i = threadIdx.x; i < P.halo_bytes / 16; i += kWgThreads) dst[i] = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
        fence_proxy_async();
    } else if (P.ones_tot && last_group) {
        // the spare chunk of the last A tile, in every stage: the code 1 in every byte (whatever the swizzle)
        const int j_last = n_tiles - 1, c_spare = chunks_of(P.a_tiles - 1);
        for (int st_i = 0; st_i < stages; ++st_i) {
            uint4 *dst = reinterpret_cast<uint4 *>(smem + (size_t)st_i * stage_bytes + (size_t)j_last * a_tile_bytes + (size_t)c_spare * P.a_chunk_bytes);
            for (uint32_t i = threadIdx.x; i < P.a_chunk_bytes / 16; i += kWgThreads) dst[i] = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
        }
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    bool timed_out = false;

    if (warp == 0) {
        // ---------------------------------------------------- TMA producer (lane 0 owns the barriers)
        const int n_loads = s_counts[0];
        uint32_t tx_bytes = 2u * P.b.tile_bytes + (P.halo_bh ? P.halo_box_bytes : 0u);
        for (int j = 0; j < (P.halo_bh ? 0 : n_tiles); ++j) tx_bytes += (uint32_t)chunks_of(ag * P.ma + j) * P.a_chunk_bytes;
        const int4 ld = lane < n_loads ? s_load[lane] : make_int4(0, 0, 0, 0);
        const int dw = (int)(short)(ld.w & 0xFFFF), dh = ld.w >> 16;
        const void *map = ld.y == 0 ? (const void *)&P.mapX : ld.y == 1 ? (const void *)&P.mapHi : (const void *)&P.mapLo;
        uint32_t s = 0, gph = 1;                      // stage, parity of the stage group's "empty" barrier
        uint32_t in_group = 0, group = 0;             // position in the release group, the group's index
        for (int i = 0; i < k_iters; ++i) {
            int ok = 1;
            if (lane == 0) {
                if (in_group == 0) ok = mbar_wait(&empty_bar[group], gph) ? 1 : 0;
                if (ok) mbar_expect_tx(&full_bar[s], tx_bytes);
            }
            if (++in_group == (uint32_t)cg) { in_group = 0; ++group; }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) { timed_out = true; break; }
            if (lane < n_loads) {
                uint8_t *dst = smem + (size_t)s * stage_bytes + ld.x;
                const int it = it_begin + i;
                if (!P.conv) tma_load_2d(dst, map, &full_bar[s], ld.z, it * P.kr);
                else {
                    int t1, tw, tn, th;
                    P.d_tiles_w.divmod(it, t1, tw);
                    P.d_tiles_h.divmod(t1, tn, th);
                    const int w0 = tw << P.bw_log2, h0 = th << P.bh_log2;
                    const int img0 = tn * (P.kr >> (P.bw_log2 + P.bh_log2));
                    tma_load_4d(dst, map, &full_bar[s], ld.z, w0 + dw, h0 + dh, img0);
                }
            }
            __syncwarp();
            if (++s == (uint32_t)stages) { s = 0; gph ^= 1u; group = 0; }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------ MMA issuer (the whole warp in step, an elected lane issues)
        WgMmaArgs A;
        A.full_bar = full_bar; A.empty_bar = empty_bar; A.acc_bar = &acc_bar;
        A.ring = smem_u32(smem); A.stage_bytes = stage_bytes; A.a_bytes = a_bytes; A.tmem = tmem_base;
        A.k_iters = k_iters; A.stages = (uint32_t)stages; A.cg = (uint32_t)cg;
        A.a_desc_lo = P.a.desc_lo;
        if (P.halo_bh) {
            // where each A tile's taps start in the halo tile (tap (r, s): r tile rows and s positions in)
            for (int j = 0; j < 4; ++j) {
                const int at = min(ag * P.ma + j, P.a_tiles - 1);
                const int tap0 = at * P.a_chunks, tap1 = tap0 + 1;
                const uint32_t off0 = (uint32_t)((tap0 / P.S) * kWgHaloW + tap0 % P.S) * (uint32_t)P.rb_a >> 4;
                uint32_t lbo = 0, mult = 1u;
                if (P.a_chunks == 2 && tap1 < P.taps)
                    lbo = ((uint32_t)((tap1 / P.S) * kWgHaloW + tap1 % P.S) * (uint32_t)P.rb_a >> 4) - off0;
                else if (P.a_chunks == 2 && P.ones_tot) {
                    // the region of ones, from wherever the stage is: (ones - (stage + off0)) << 16 = (ones - off0) << 16 - (stage << 16)
                    lbo = ((A.ring + P.ones_off) >> 4) - off0;
                    mult = 1u - 65536u;
                }
                A.tile_desc[j] = off0 + (lbo << 16);
                A.tile_mult[j] = mult;
            }
            A.b_desc_lo = P.b2_desc_lo; A.idesc_hi = P.idesc_fused;
            timed_out = !wg_mma_dispatch_halo<RBA, RBB>(n_tiles, P.halo_bh, A);
        } else if (P.lo_signed) {
            A.b_desc_lo = P.b2_desc_lo; A.idesc_hi = P.idesc_fused;
            timed_out = !wg_mma_dispatch_nt<RBA, RBB, true>(n_tiles, A);
        } else {
            A.b_desc_lo = P.b.desc_lo; A.idesc_hi = P.idesc_hi;
            timed_out = !wg_mma_dispatch_nt<RBA, RBB, false>(n_tiles, A);
        }
    } else {
        // ------------------------------------------------------- epilogue
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        if (P.cls_x) {
            // while the MMAs run: the border classes of this CTA's share of the images (by CTA index, whatever its item)
            const int t = threadIdx.x - 64;
            int *tx = reinterpret_cast<int *>(smem + P.cls_off), *th = tx + 16 * P.C, *tl = th + 16 * (int)P.N;
            for (int i = t; i < 16 * (P.C + 2 * (int)P.N); i += 128) tx[i] = 0;
            named_barrier(2, 128);
            const int img_begin = (int)((int64_t)P.Nimg * blockIdx.x / gridDim.x), img_end = (int)((int64_t)P.Nimg * (blockIdx.x + 1) / gridDim.x);
            wg_border_sums(true, P.codes_x, P.C, P.H, P.W, img_begin, img_end, tx, t);
            wg_border_sums(true, P.codes_hi, (int)P.N, P.H, P.W, img_begin, img_end, th, t);
            wg_border_sums(P.lo_signed != 0, P.codes_lo, (int)P.N, P.H, P.W, img_begin, img_end, tl, t);
            named_barrier(2, 128);
            for (int i = t; i < 16 * P.C; i += 128)
                if (tx[i]) atomicAdd(P.cls_x + i, (unsigned long long)(long long)tx[i]);
            for (int i = t; i < 16 * (int)P.N; i += 128) {
                if (th[i]) atomicAdd(P.cls_hi + i, (unsigned long long)(long long)th[i]);
                if (tl[i]) atomicAdd(P.cls_lo + i, (unsigned long long)(long long)tl[i]);
            }
        }
        if (k_iters > 0 && !mbar_wait_warp(&acc_bar, 0)) timed_out = true;
        tc_fence_after();
        if (!timed_out && k_iters > 0) {
            const float scale = P.direct ? __fmul_rn(P.qx->scale, P.qg->scale) : 0.0f;
            long long *part = P.part + (int64_t)blockIdx.x * P.part_stride;
            for (int j = 0; j < n_tiles; ++j) {
                const int at = ag * P.ma + j;
                bool valid = row / P.rb_a < chunks_of(at);
                const int64_t k = (int64_t)at * 128 + row;                  // plain: output row
                if (!P.conv) valid = valid && k < P.K;
                else         valid = valid && (at % P.tiles_c) * P.rb_a + row % P.rb_a < P.C;
                const long long rterm = (P.direct && valid) ? P.rowterm[k] : 0;
                const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(j * 2 * P.bn);
                for (int c0 = 0; c0 < P.bn; c0 += 32) {
                    uint32_t rh[32], rl[32];
                    tmem_ld_32x32(t_addr + (uint32_t)c0, rh);
                    tmem_ld_32x32(t_addr + (uint32_t)(P.bn + c0), rl);
                    tmem_ld_wait();
                    if (P.ones_tot && at == P.a_tiles - 1 && row == P.rb_a * chunks_of(at)) {
                        // the row of ones: this slice's sum of the 16-bit gradient codes, per output channel
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (n0 + c0 + e < P.N)
                                atomicAdd(P.ones_tot + n0 + c0 + e, (unsigned long long)(256ll * (long long)(int)rh[e] + (long long)(int)rl[e]));
                    }
                    if (!valid) continue;
                    if (P.direct) {
                        // the whole reduction is here: zero-points, scale, store
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            const int64_t n = (int64_t)n0 + c0 + e;
                            if (n < P.N) {
                                const long long acc = 256ll * (long long)(int)rh[e] + (long long)(int)rl[e] + rterm + P.colterm[n];
                                if (P.acc_out) P.acc_out[k * P.N + n] = acc;
                                if (P.dW) P.dW[k * P.N + n] = __fmul_rn((float)acc, scale);
                            }
                        }
                    } else if (P.conv) {
                        // partial block [tile][column][row]: a warp's 32 rows are contiguous, and so are the
                        // channels the second kernel reads together
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            part[((int64_t)j * P.bn + c0 + e) * 128 + row] = 256ll * (long long)(int)rh[e] + (long long)(int)rl[e];
                    } else {
                        // partial block [tile][row][column]
                        long long *dst = part + ((int64_t)j * 128 + row) * P.bn + c0;
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            longlong2 v;
                            v.x = 256ll * (long long)(int)rh[e] + (long long)(int)rl[e];
                            v.y = 256ll * (long long)(int)rh[e + 1] + (long long)(int)rl[e + 1];
                            *reinterpret_cast<longlong2 *>(dst + e) = v;
                        }
                    }
                }
            }
        }
    }

    if (timed_out) {
        raise_timeout(P.status);
        __nanosleep(1000000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { __syncwarp(); tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols); }
}

// ------------------------------------------------------------ code sums
// Sums of stored codes per channel and per border class of the pixel the code
// sits at (bit 1: first row, 2: last row, 4: first column, 8: last column).
// sums[cls][c] (int64, zeroed beforehand).
template <bool IS_SIGNED>
__global__ void __launch_bounds__(256) class_sums_kernel(const uint8_t *__restrict__ q, int pixels, int H, int W,
                                                         int C, unsigned long long *__restrict__ sums)
{
    extern __shared__ int s_acc[];                       // [16][C]
    for (int i = threadIdx.x; i < 16 * C; i += 256) s_acc[i] = 0;
    __syncthreads();
    const int cv = C >> 4;                               // 16-byte groups per pixel
    const int tw = cv < 256 ? cv : 256;
    const int rpb = 256 / tw;
    const int tx = threadIdx.x % tw, ty = threadIdx.x / tw;
    constexpr int U = 8;                                 // loads in flight per thread
    if (ty < rpb) {
        const int step = (int)gridDim.x * rpb;
        for (int g = tx; g < cv; g += tw) {
            int interior[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) interior[e] = 0;
            for (int p0 = (int)blockIdx.x * rpb + ty; p0 < pixels; p0 += U * step) {
                uint4 v[U];
                bool ok[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int p = p0 + u * step;
                    ok[u] = p < pixels;
                    if (ok[u]) v[u] = __ldg(reinterpret_cast<const uint4 *>(q + (int64_t)p * C) + g);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (!ok[u]) continue;
                    const unsigned p = (unsigned)(p0 + u * step);
                    const unsigned w = p % (unsigned)W, h = (p / (unsigned)W) % (unsigned)H;
                    const int cls = (h == 0 ? 1 : 0) | (h == (unsigned)H - 1 ? 2 : 0) | (w == 0 ? 4 : 0) | (w == (unsigned)W - 1 ? 8 : 0);
                    const uint32_t wd[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    if (cls == 0) {
                        // one byte per dot product: the selector picks it, sign- or zero-extended
#pragma unroll
                        for (int k = 0; k < 4; ++k)
#pragma unroll
                            for (int b = 0; b < 4; ++b)
                                interior[k * 4 + b] = IS_SIGNED ? __dp4a((int)wd[k], 1 << (8 * b), interior[k * 4 + b])
                                                                : (int)__dp4a(wd[k], 1u << (8 * b), (unsigned)interior[k * 4 + b]);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
#pragma unroll
                            for (int b = 0; b < 4; ++b)
                                atomicAdd(&s_acc[cls * C + g * 16 + k * 4 + b],
                                          IS_SIGNED ? (int)(int8_t)(wd[k] >> (8 * b)) : (int)((wd[k] >> (8 * b)) & 0xFF));
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < 16; ++e) atomicAdd(&s_acc[g * 16 + e], interior[e]);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 16 * C; i += 256)
        if (s_acc[i] != 0) atomicAdd(&sums[i], (unsigned long long)(long long)s_acc[i]);
}

// The same sums, one image row per block step: thread (w, g) owns 16 channels of column w, so its border class
// in the w direction never changes, and the row's class is the same for the whole block.  The sums over all rows
// stay in 16 registers; the first and last row of an image (a few percent of the rows) are added to their row sets
// in shared memory as well.  No division per pixel, and atomics only for those rows.
// gs = 16-channel groups per block (a power of two, W * gs <= 256); blockIdx.y selects the channel slab.
template <bool IS_SIGNED>
__device__ __forceinline__ void row_class_sums_body(const uint8_t *__restrict__ q, int Nimg, int H, int W, int C, int gs,
                                                    unsigned long long *__restrict__ sums)
{
    extern __shared__ int s_acc[];                       // [3 row sets: all, first, last][4 column classes][gs * 16]
    const int cw = gs * 16;
    for (int i = threadIdx.x; i < 12 * cw; i += 256) s_acc[i] = 0;
    __syncthreads();
    const int w = threadIdx.x / gs, gl = threadIdx.x % gs;
    const int g = blockIdx.y * gs + gl;
    const bool active = w < W && g < (C >> 4);
    const int colclass = (w == 0 ? 1 : 0) | (w == W - 1 ? 2 : 0);
    const int lane = threadIdx.x & 31;
    const int64_t row_bytes = (int64_t)W * C;
    const uint8_t *base = q + (int64_t)(active ? w : 0) * C + (int64_t)(active ? g : 0) * 16;
    constexpr int U = 8;                                 // rows in flight per thread

    int acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0;
    const bool interior = active && colclass == 0;
    {
        // (every thread walks the rows, the idle ones without loading: the shuffles below need whole warps)
        const int rows = Nimg * H, step = (int)gridDim.x, hstep = step % H;
        int h = (int)blockIdx.x % H;
        for (int r = (int)blockIdx.x; r < rows; r += U * step) {
            uint4 v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                v[u] = make_uint4(0, 0, 0, 0);
                if (active && r + u * step < rows) v[u] = __ldcs(reinterpret_cast<const uint4 *>(base + (int64_t)(r + u * step) * row_bytes));
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (r + u * step >= rows) break;
                const uint32_t wd[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int b = 0; b < 4; ++b)          // one byte per dot product: the selector picks it, sign- or zero-extended
                        acc[k * 4 + b] = IS_SIGNED ? __dp4a((int)wd[k], 1 << (8 * b), acc[k * 4 + b])
                                                   : (int)__dp4a(wd[k], 1u << (8 * b), (unsigned)acc[k * 4 + b]);
                if (active && H > 1 && (h == 0 || h == H - 1)) {
                    // a first or last row (the same for the whole block, and rare): its codes also go to that row set
                    int *dst = &s_acc[((h == 0 ? 1 : 2) * 4 + colclass) * cw + gl * 16];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            atomicAdd(dst + k * 4 + b, IS_SIGNED ? (int)(int8_t)(wd[k] >> (8 * b)) : (int)((wd[k] >> (8 * b)) & 0xFF));
                }
                h += hstep; if (h >= H) h -= H;
            }
        }
    }
    {
        // all rows, reduced the same way
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            int r = interior ? acc[e] : 0;
            for (int off = gs; off < 32; off <<= 1) r += __shfl_xor_sync(0xffffffffu, r, off);
            const int ch = gl * 16 + e;
            if (lane < gs && r) atomicAdd(&s_acc[0 * cw + ch], r);
            if (active && colclass != 0 && acc[e]) atomicAdd(&s_acc[colclass * cw + ch], acc[e]);
        }
    }
    __syncthreads();
    // exclusive classes (bit 1: first row, 2: last row, 4: first column, 8: last column); a single row is both
    for (int i = threadIdx.x; i < 4 * cw; i += 256) {
        const int cc = i / cw, c = (int)blockIdx.y * cw + i % cw;
        if (c >= C) continue;
        const int colbits = (cc & 1 ? 4 : 0) | (cc & 2 ? 8 : 0);
        const int all = s_acc[(0 * 4 + cc) * cw + i % cw], top = s_acc[(1 * 4 + cc) * cw + i % cw], bot = s_acc[(2 * 4 + cc) * cw + i % cw];
        if (H == 1) {
            if (all) atomicAdd(&sums[(3 | colbits) * C + c], (unsigned long long)(long long)all);
        } else {
            const int mid = all - top - bot;
            if (mid) atomicAdd(&sums[(0 | colbits) * C + c], (unsigned long long)(long long)mid);
            if (top) atomicAdd(&sums[(1 | colbits) * C + c], (unsigned long long)(long long)top);
            if (bot) atomicAdd(&sums[(2 | colbits) * C + c], (unsigned long long)(long long)bot);
        }
    }
}

template <bool IS_SIGNED>
__global__ void __launch_bounds__(256, 3) row_class_sums_kernel(const uint8_t *__restrict__ q, int Nimg, int H, int W,
                                                                int C, int gs, unsigned long long *__restrict__ sums)
{
    row_class_sums_body<IS_SIGNED>(q, Nimg, H, W, C, gs, sums);
}

// The three tensors of a weight gradient with as many input as output channels in one launch (blockIdx.z: the
// layer input, the gradient's signed high bytes, its unsigned low bytes); sums: three tables of 16 * C, one after another.
__global__ void __launch_bounds__(256, 3) row_class_sums3_kernel(const uint8_t *__restrict__ x, const uint8_t *__restrict__ hi,
                                                                 const uint8_t *__restrict__ lo, int Nimg, int H, int W, int C,
                                                                 int gs, unsigned long long *__restrict__ sums, int lo_signed)
{
    if (blockIdx.z == 0)      row_class_sums_body<true>(x, Nimg, H, W, C, gs, sums);
    else if (blockIdx.z == 1) row_class_sums_body<true>(hi, Nimg, H, W, C, gs, sums + 16 * C);
    else if (lo_signed)       row_class_sums_body<true>(lo, Nimg, H, W, C, gs, sums + 32 * C);
    else                      row_class_sums_body<false>(lo, Nimg, H, W, C, gs, sums + 32 * C);
}

// The border classes only (first / last row, first / last column and the four corners; H, W >= 3) of the three code
// tensors of a convolution's weight gradient: a few percent of the positions.  blockIdx.z: the layer input, the
// gradient's signed high bytes, its unsigned low bytes (tables of 16 * Cx / 16 * Cg / 16 * Cg, zeroed beforehand);
// blockIdx.x strides over groups of four images.  Thread = (16-channel group g, slot k): it walks positions k,
// k + slots, ... of each of the four edges (corners excluded) and keeps one set of 16 sums per edge in registers;
// the corners go straight to shared memory.  Few blocks: each ends with one atomic per table entry.
__global__ void __launch_bounds__(256) border_class_sums_kernel(const uint8_t *__restrict__ x, const uint8_t *__restrict__ hi,
                                                                const uint8_t *__restrict__ lo, int Nimg, int H, int W, int Cx,
                                                                int Cg, unsigned long long *__restrict__ sums_x,
                                                                unsigned long long *__restrict__ sums_hi,
                                                                unsigned long long *__restrict__ sums_lo, int lo_signed)
{
    extern __shared__ int s_acc[];                       // [16][C]
    const uint8_t *q = blockIdx.z == 0 ? x : blockIdx.z == 1 ? hi : lo;
    unsigned long long *sums = blockIdx.z == 0 ? sums_x : blockIdx.z == 1 ? sums_hi : sums_lo;
    const int C = blockIdx.z == 0 ? Cx : Cg;
    const bool is_signed = blockIdx.z != 2 || lo_signed;
    for (int i = threadIdx.x; i < 16 * C; i += 256) s_acc[i] = 0;
    __syncthreads();
    const int cv = C >> 4;
    const int slots = 256 / cv;                          // (cv <= 256: C <= 4096)
    const int g = threadIdx.x % cv, k = threadIdx.x / cv;
    int top[16], bot[16], lef[16], rig[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) { top[e] = 0; bot[e] = 0; lef[e] = 0; rig[e] = 0; }
    if (k < slots) {
        // four images at a time, all their loads first: the positions are few and far apart, so latency is what counts
        constexpr int U = 4;
        for (int img0 = blockIdx.x * U; img0 < Nimg; img0 += gridDim.x * U) {
            const uint4 *base[U];
#pragma unroll
            for (int u = 0; u < U; ++u) base[u] = reinterpret_cast<const uint4 *>(q + (int64_t)min(img0 + u, Nimg - 1) * H * W * C) + g;
            for (int w = 1 + k; w < W - 1; w += slots) {
                uint4 a[U], b[U];
#pragma unroll
                for (int u = 0; u < U; ++u) { a[u] = __ldg(base[u] + (int64_t)w * cv); b[u] = __ldg(base[u] + ((int64_t)(H - 1) * W + w) * cv); }
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (img0 + u < Nimg) { border_add(is_signed, a[u], top); border_add(is_signed, b[u], bot); }
            }
            for (int h = 1 + k; h < H - 1; h += slots) {
                uint4 a[U], b[U];
#pragma unroll
                for (int u = 0; u < U; ++u) { a[u] = __ldg(base[u] + (int64_t)h * W * cv); b[u] = __ldg(base[u] + ((int64_t)h * W + W - 1) * cv); }
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (img0 + u < Nimg) { border_add(is_signed, a[u], lef); border_add(is_signed, b[u], rig); }
            }
            if (k < 4) {
                // the four corners: classes 5, 9 (first row), 6, 10 (last row)
                const int h = k < 2 ? 0 : H - 1, w = (k & 1) ? W - 1 : 0;
                int cor[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) cor[e] = 0;
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (img0 + u < Nimg) border_add(is_signed, __ldg(base[u] + ((int64_t)h * W + w) * cv), cor);
                int *dst = s_acc + ((k < 2 ? 1 : 2) | ((k & 1) ? 8 : 4)) * C + g * 16;
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    if (cor[e]) atomicAdd(dst + e, cor[e]);
            }
        }
    }
    // the lanes of a warp that hold the same channel group meet by shuffle (when cv is a power of two below 32: whole
    // warps are then inside `k < slots`), then one lane per group adds to the block's table
    const bool shuffle = cv < 32 && (cv & (cv - 1)) == 0;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        int t = top[e], b = bot[e], l = lef[e], r = rig[e];
        if (shuffle)
            for (int off = cv; off < 32; off <<= 1) {
                t += __shfl_xor_sync(0xffffffffu, t, off); b += __shfl_xor_sync(0xffffffffu, b, off);
                l += __shfl_xor_sync(0xffffffffu, l, off); r += __shfl_xor_sync(0xffffffffu, r, off);
            }
        if (k < slots && (!shuffle || (threadIdx.x & 31) < cv)) {
            if (t) atomicAdd(s_acc + 1 * C + g * 16 + e, t);
            if (b) atomicAdd(s_acc + 2 * C + g * 16 + e, b);
            if (l) atomicAdd(s_acc + 4 * C + g * 16 + e, l);
            if (r) atomicAdd(s_acc + 8 * C + g * 16 + e, r);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 16 * C; i += 256)
        if (s_acc[i] != 0) atomicAdd(&sums[i], (unsigned long long)(long long)s_acc[i]);
}

// Plain product, direct epilogue: rowterm[k] = -zg * SX[k] + M*zx*zg, colterm[n] = -zx * (256*SHI[n] + SLO[n]).
__global__ void wgrad_terms_kernel(const long long *__restrict__ sx, const long long *__restrict__ shi,
                                   const long long *__restrict__ slo, int64_t M, int64_t N, int64_t K,
                                   const qbp_qparams *qx, const qbp_qparams *qg, long long *__restrict__ rowterm,
                                   long long *__restrict__ colterm, int zg_shift)
{
    const long long zx = qx->zero_point, zg = qg->zero_point - zg_shift;      // (signed low bytes: lo - 128 against zg - 128)
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < K) rowterm[i] = -zg * sx[i] + M * zx * zg;
    if (i < N) colterm[i] = -zx * (256 * shi[i] + slo[i]);
}

// Adds the CTAs' partials, applies the zero-points and dequantises:
//   acc = raw - zg * SX - zx * SG + count * zx * zg
// where SX / SG / count are taken over the positions at which the tap is inside
// the image.  Output element e: plain [k][n]; conv [k][tap][c].
__global__ void __launch_bounds__(256) wgrad_finalize_kernel(const WgradParams P, const long long *__restrict__ sx,
                                                             const long long *__restrict__ shi,
                                                             const long long *__restrict__ slo, int64_t total)
{
    // kWgFinalizeLanes lanes per output element share its slices (an element's partials are few hundred bytes each, far apart:
    // one thread walking them alone is bound by latency)
    constexpr int kLanes = kWgFinalizeLanes;
    const int64_t e_raw = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / kLanes;
    const int part_lane = threadIdx.x % kLanes;
    const bool live = e_raw < total;
    const int64_t e = live ? e_raw : total - 1;           // (idle lanes of the last warp compute a duplicate and do not store)
    // (signed low bytes: the limbs hold g16 - 128, against the zero-point zg - 128)
    const long long zx = P.qx->zero_point, zg = P.qg->zero_point - (P.lo_signed ? 128 : 0);
    long long SX = 0, SG = 0, count = 0;
    int at, row, n;                                     // accumulator tile, row in it, output column of g
    if (!P.conv) {
        const int64_t k = e / P.N;
        n = (int)(e % P.N);
        at = (int)(k / 128); row = (int)(k % 128);
        SX = sx[k];
        SG = 256 * shi[n] + slo[n];
        count = P.M;
    } else {
        const int c = (int)(e % P.C);
        const int tap = (int)((e / P.C) % P.taps);
        n = (int)(e / ((int64_t)P.C * P.taps));
        const int r = tap / P.S, s = tap % P.S, pad = P.pad;
        at = (tap / P.a_chunks) * P.tiles_c + c / P.rb_a;
        row = (tap % P.a_chunks) * P.rb_a + c % P.rb_a;
        // positions of g that see this tap: p - pad + r in [0,H)  <=>  not (r<pad and first row), not (r>pad and last row);
        // positions of x that are seen:      h + pad - r in [0,H)  <=>  not (r<pad and last row),  not (r>pad and first row).
        if (P.tot_x) {
            // totals over all positions, less the border classes this tap does not see (the interior always counts)
            SX = P.tot_x[c]; SG = P.tot_g[n];
            if (P.lo_signed && P.tot_g_plain) SG -= 128ll * P.Nimg * P.H * P.W;
            for (int cls = 1; cls < 16; ++cls) {
                const bool top = cls & 1, bottom = cls & 2, left = cls & 4, right = cls & 8;
                const bool g_ok = !((r < pad && top) || (r > pad && bottom) || (s < pad && left) || (s > pad && right));
                const bool x_ok = !((r < pad && bottom) || (r > pad && top) || (s < pad && right) || (s > pad && left));
                if (!g_ok) SG -= 256 * shi[cls * P.N + n] + slo[cls * P.N + n];
                if (!x_ok) SX -= sx[cls * P.C + c];
            }
        } else
        for (int cls = 0; cls < 16; ++cls) {
            const bool top = cls & 1, bottom = cls & 2, left = cls & 4, right = cls & 8;
            const bool g_ok = !((r < pad && top) || (r > pad && bottom) || (s < pad && left) || (s > pad && right));
            const bool x_ok = !((r < pad && bottom) || (r > pad && top) || (s < pad && right) || (s > pad && left));
            if (g_ok) SG += 256 * shi[cls * P.N + n] + slo[cls * P.N + n];
            if (x_ok) SX += sx[cls * P.C + c];
        }
        const long long rows_ok = P.H - (r < pad ? pad - r : r - pad), cols_ok = P.W - (s < pad ? pad - s : s - pad);
        count = (long long)P.Nimg * (rows_ok > 0 ? rows_ok : 0) * (cols_ok > 0 ? cols_ok : 0);
    }
    // the CTAs of this element's item
    const int ag = at / P.ma, j = at % P.ma, tb = n / P.bn, col = n % P.bn;
    const int item = ag * P.tiles_b + tb;
    const int full_items = P.ctas_full / P.s_full;
    const int first = item < full_items ? item * P.s_full : P.ctas_full + (item - full_items) * P.s_last;
    const int slices = item < full_items ? P.s_full : P.s_last;
    const int64_t off = P.conv ? ((int64_t)j * P.bn + col) * 128 + row : ((int64_t)j * 128 + row) * P.bn + col;
    long long raw = 0;
    const long long *src = P.part + (int64_t)first * P.part_stride + off;
    int sl = part_lane;
    for (; sl + 7 * kLanes < slices; sl += 8 * kLanes) {
        long long v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldcs(src + (int64_t)(sl + u * kLanes) * P.part_stride);
#pragma unroll
        for (int u = 0; u < 8; ++u) raw += v[u];
    }
    for (; sl < slices; sl += kLanes) raw += __ldcs(src + (int64_t)sl * P.part_stride);
#pragma unroll
    for (int o = 1; o < kLanes; o <<= 1) raw += __shfl_xor_sync(0xffffffffu, raw, o);
    if (!live || part_lane != 0) return;
    const long long acc = raw - zg * SX - zx * SG + count * zx * zg;
    if (P.acc_out) P.acc_out[e] = acc;
    if (P.dW) P.dW[e] = __fmul_rn((float)acc, __fmul_rn(P.qx->scale, P.qg->scale));
}

// Pixel box of `rows` = bw x bh x bn positions (powers of two) that needs the fewest steps.
static void pick_pixel_box_w(int rows, int Nimg, int H, int W, int &bwl, int &bhl)
{
    long long best = -1;
    int lg = 0; while ((1 << lg) < rows) ++lg;
    for (int a = 0; a <= lg; ++a)
        for (int b = 0; a + b <= lg; ++b) {
            const int bw = 1 << a, bh = 1 << b, bn = rows >> (a + b);
            const long long tiles = (long long)((W + bw - 1) / bw) * ((H + bh - 1) / bh) * ((Nimg + bn - 1) / bn);
            const long long score = tiles * 64 - a * 8 - b;
            if (best < 0 || score < best) { best = score; bwl = a; bhl = b; }
        }
}

bool wgrad_conv_supported(const qbp_conv_desc *d)
{
    return d->stride == 1 && d->R == d->S && (d->R == 1 || d->R == 3) && d->pad == (d->R - 1) / 2 && d->N > 0 &&
           d->H > 0 && d->W > 0 && d->C > 0 && d->K > 0 && d->C % 32 == 0 && d->K % 32 == 0;
}

// Everything of the launch that does not depend on pointers: tiling, split, workspace.
struct WgradPlan {
    WgradParams P;
    int grid;
    size_t smem;
    int bw, bh, bn_img;
};

// Whether the kernel's epilogue warps can take the border classes themselves: a padded convolution whose x and g
// tensors have 32, 64 or 128 channels (a pixel is 2, 4 or 8 sixteen-byte groups) and at least 3 x 3 positions.
static bool wgrad_inline_border(const qbp_conv_desc *d)
{
    auto ok = [](int c) { return c == 32 || c == 64 || c == 128; };
    return d && d->pad > 0 && ok(d->C) && ok(d->K) && d->H >= 3 && d->W >= 3;
}

}  // namespace qbp

// Whether the product can take the gradient's per-channel totals itself (a spare chunk in its last A tile).
bool qbp::wgrad_self_totals(const qbp_conv_desc *d)
{
    if (!d || !wgrad_conv_supported(d)) return false;
    const int rb_a = d->C >= 128 ? 128 : d->C >= 64 ? 64 : 32;
    const int a_chunks = 128 / rb_a;
    return d->C % rb_a == 0 && (d->R * d->S) % a_chunks != 0;
}

namespace qbp {

static void plan_wgrad(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K, WgradPlan &pl, bool lo_signed = false)
{
    WgradParams &P = pl.P;
    P = WgradParams{};
    P.conv = d ? 1 : 0;
    P.M = M; P.N = N; P.K = K;
    // g side: one swizzled row holds bn output channels
    const uint32_t rb_b = N >= 128 ? 128u : N >= 64 ? 64u : 32u;
    P.bn = (int)rb_b;
    P.tiles_b = (int)((N + P.bn - 1) / P.bn);
    // x side: 128 MMA rows = a_chunks chunks of rb_a columns / channels
    const uint32_t rb_a = K >= 128 ? 128u : K >= 64 ? 64u : 32u;
    P.rb_a = (int)rb_a;
    P.a_chunks = 128 / (int)rb_a;
    if (!d) {
        P.a_tiles = (int)((K + 127) / 128);
        P.tiles_c = 1;
    } else {
        P.H = d->H; P.W = d->W; P.Nimg = d->N; P.pad = d->pad; P.R = d->R; P.S = d->S; P.C = d->C;
        P.taps = d->R * d->S;
        P.tiles_c = (d->C + (int)rb_a - 1) / (int)rb_a;
        P.a_tiles = ((P.taps + P.a_chunks - 1) / P.a_chunks) * P.tiles_c;
    }
    // A tiles per CTA: at most what tensor memory holds (two accumulators of bn columns each), spread evenly over
    // the groups that takes (5 tiles: 3 + 2 rather than 4 + 1 -- a stage of few MMAs is bound by its fixed costs)
    const int ma_max = std::max(1, std::min({kWgMaxTiles, 512 / (2 * P.bn), P.a_tiles}));
    P.a_groups = (P.a_tiles + ma_max - 1) / ma_max;
    P.ma = (P.a_tiles + P.a_groups - 1) / P.a_groups;
    int cols = 32; while (cols < P.ma * 2 * P.bn) cols <<= 1;
    P.tmem_cols = cols;
    // reduction rows per stage: kWgRows (the ring is shallower than with 64, but a stage holds twice the MMAs)
    const uint32_t kr = kWgRows;
    P.kr = (int)kr;
    P.a_chunk_bytes = kr * rb_a;
    P.a = layout_mnmajor(kr, rb_a, (uint32_t)P.a_chunks, P.a_chunk_bytes);
    P.b = layout_mnmajor(kr, rb_b, 1, 0);
    P.idesc_hi = make_idesc(true, true, 1, 1, 128, (uint32_t)P.bn);
    P.idesc_lo = make_idesc(true, false, 1, 1, 128, (uint32_t)P.bn);
    P.lo_signed = lo_signed ? 1 : 0;
    P.b2_desc_lo = layout_mnmajor(kr, rb_b, 2, P.b.tile_bytes).desc_lo;      // the low tile follows the high one in a stage
    P.idesc_fused = make_idesc(true, true, 1, 1, 128, 2u * (uint32_t)P.bn);
    if (!d) {
        P.iters_total = (int)((M + kr - 1) / kr);
        pl.bw = pl.bh = pl.bn_img = 0;
    } else {
        int bwl = 0, bhl = 0;
        pick_pixel_box_w((int)kr, d->N, d->H, d->W, bwl, bhl);
        if (lo_signed && d->R == 3 && P.tiles_c == 1 && P.a_chunks <= 2) {
            // halo tiles: boxes 8 positions wide and 8 or 4 rows high, when that costs at most a fifth more steps
            // than the free choice of box
            const long long free_tiles = (long long)((d->W + (1 << bwl) - 1) >> bwl) * ((d->H + (1 << bhl) - 1) >> bhl) *
                                         ((d->N + ((int)kr >> (bwl + bhl)) - 1) / ((int)kr >> (bwl + bhl)));
            long long best = -1;
            for (int bh = 8; bh >= 4; bh >>= 1) {
                const long long t = (long long)((d->W + 7) / 8) * ((d->H + bh - 1) / bh) * ((d->N + 16 / bh - 1) / (16 / bh));
                if (best < 0 || t < best) { best = t; P.halo_bh = bh; }
            }
            if (best * 5 > free_tiles * 6) P.halo_bh = 0;
            if (P.halo_bh) {
                bwl = 3; bhl = P.halo_bh == 8 ? 3 : 2;
                P.halo_box_bytes = (uint32_t)(kWgHaloW * (P.halo_bh + 2) * (16 / P.halo_bh)) * rb_a;
                P.halo_bytes = (uint32_t)align_up((size_t)P.halo_box_bytes, 1024);
            }
        }
        P.bw_log2 = bwl; P.bh_log2 = bhl;
        pl.bw = 1 << bwl; pl.bh = 1 << bhl; pl.bn_img = (int)kr >> (bwl + bhl);
        P.tiles_w = (d->W + pl.bw - 1) / pl.bw; P.tiles_h = (d->H + pl.bh - 1) / pl.bh;
        P.iters_total = P.tiles_w * P.tiles_h * ((d->N + pl.bn_img - 1) / pl.bn_img);
        P.d_tiles_w = make_fastdiv(P.tiles_w); P.d_tiles_h = make_fastdiv(P.tiles_h);
    }
    // pipeline: stages of kr rows; one commit releases `cg` stages (some 24 MMAs between commits while that leaves
    // three groups in the ring).  The CTAs of the last group (fewer A tiles) get a ring of their own shape.
    const int n_last = P.a_tiles - (P.a_groups - 1) * P.ma;                 // A tiles of the last group
    // (the border-class tables of the epilogue warps sit behind the ring)
    // (... and behind those the region of ones of the halo variant)
    const uint32_t cls_only = wgrad_inline_border(d) ? (uint32_t)align_up(sizeof(int) * 16 * (size_t)(K + 2 * N), 1024) : 0u;
    const uint32_t cls_bytes = cls_only + (P.halo_bh ? P.halo_bytes : 0u);
    auto ring = [&](int tiles, int &stages, int &cg) {
        const uint32_t stage_bytes = (P.halo_bh ? P.halo_bytes : P.a_chunk_bytes * P.a_chunks * (uint32_t)tiles) + 2 * P.b.tile_bytes;
        stages = std::max(2, std::min<int>(kWgMaxStages, (int)((kWgSmem - 1024 - cls_bytes) / stage_bytes)));
        const int mmas = tiles * (int)(kr / 32) * 2;       // (in MMAs of bn columns: a fused one counts twice)
        cg = 1;
        while (cg * mmas < 24 && stages / (cg + 1) >= 3) ++cg;
        stages -= stages % cg;
        return (size_t)stages * stage_bytes + 1024;
    };
    const size_t smem_full = ring(P.ma, P.stages, P.cg);
    const size_t smem_last = ring(n_last, P.stages_last, P.cg_last);
    P.cls_off = (uint32_t)(std::max(smem_full, smem_last) - 1024);           // behind the longer of the two rings
    P.ones_off = P.cls_off + cls_only;
    pl.smem = std::max(smem_full, smem_last) + cls_bytes;
    // split of the reductions: at most 65536 rows per CTA; with few items, enough slices to fill the machine
    // once, in proportion to an item's cost per reduction step: a fixed part (waits, the share of a commit)
    // worth about eight MMAs, plus its MMAs
    const int max_iters = 65536 / (int)kr;
    const int min_slices = (P.iters_total + max_iters - 1) / max_iters;
    auto cost = [&](int tiles) { return (int64_t)(8 + tiles * (int)(kr / 32) * 2); };
    const int64_t weight = ((int64_t)(P.a_groups - 1) * cost(P.ma) + cost(n_last)) * P.tiles_b;
    const int T = sm_count();
    auto slices_for = [&](int tiles) {
        int64_t s = (int64_t)T * cost(tiles) / weight;
        s = std::max<int64_t>(s, min_slices);
        s = std::max<int64_t>(1, std::min<int64_t>(s, P.iters_total));
        return (int)s;
    };
    P.s_full = slices_for(P.ma);
    P.s_last = slices_for(n_last);
    P.ctas_full = (P.a_groups - 1) * P.tiles_b * P.s_full;
    pl.grid = P.ctas_full + P.tiles_b * P.s_last;
    P.direct = (!d && P.s_full == 1 && P.s_last == 1) ? 1 : 0;
    // (not a power of two apart: the CTAs write their blocks in step, and equal low address bits pile onto few L2 slices)
    P.part_stride = (int64_t)P.ma * 128 * P.bn + 272;
}

static size_t wgrad_ws_bytes(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K)
{
    const int64_t cx = d ? d->C : K, cg = d ? d->K : N;
    const size_t sums = align_up(sizeof(int64_t) * 16 * cx, 256) + 2 * align_up(sizeof(int64_t) * 16 * cg, 256);
    const size_t terms = align_up(sizeof(int64_t) * cx, 256) + align_up(sizeof(int64_t) * cg, 256);
    // (the split, and with it the partials, may differ between the two forms of the low limb: room for either)
    size_t part = 0;
    for (int lo_signed = 0; lo_signed < 2; ++lo_signed) {
        WgradPlan pl;
        plan_wgrad(d, M, N, K, pl, lo_signed != 0);
        part = std::max(part, pl.P.direct ? (size_t)0 : align_up(sizeof(int64_t) * (size_t)pl.grid * (size_t)pl.P.part_stride, 256));
    }
    return 256 + sums + terms + part;
}

template <bool IS_SIGNED>
static int launch_class_sums(const void *q, int64_t pixels, int H, int W, int C, int64_t *sums, cudaStream_t st)
{
    QBP_CUDA_OK(cudaMemsetAsync(sums, 0, sizeof(int64_t) * 16 * C, st));
    if ((size_t)C * 16 * sizeof(int) > 200 * 1024) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "wgrad: more than 3200 channels");
    const size_t smem = (size_t)C * 16 * sizeof(int);
    static PerDeviceOnce configured;
    if (smem > 48 * 1024) QBP_SMEM_OPT_IN(configured, class_sums_kernel<IS_SIGNED>, 200 * 1024);
    if (pixels >= (1ll << 30)) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "wgrad: more than 2^30 positions");
    if (W <= 256) {
        // a block step is one image row: W columns x gs channel groups of 16
        const int cv = C / 16;
        int gs = 1; while (gs * 2 <= cv && gs * 2 * W <= 256 && gs < 16) gs *= 2;
        const int slabs = (cv + gs - 1) / gs;
        const int64_t rows = pixels / W;
        const int Nimg = (int)(rows / H);
        // int32 registers: a thread sees at most rows / grid * 255 per channel
        int64_t grid_x = std::min<int64_t>(rows, std::max<int64_t>(1, (int64_t)sm_count() * 3 / slabs));
        grid_x = std::max<int64_t>(grid_x, rows / (1 << 22) + 1);
        QBP_TRACE_BEGIN(st);
        row_class_sums_kernel<IS_SIGNED><<<dim3((unsigned)grid_x, (unsigned)slabs), 256, (size_t)12 * gs * 16 * sizeof(int), st>>>(
            (const uint8_t *)q, Nimg, H, W, C, gs, (unsigned long long *)sums);
        QBP_LAUNCH_OK("class_sums_kernel");
        return QBP_OK;
    }
    // int32 partials: a thread sees at most pixels / grid * 255 per channel.  Few blocks (each ends with up to
    // 16*C atomics on the same 16*C sums), eight 16-byte loads in flight per thread.
    const int cv = C / 16, tw = cv < 256 ? cv : 256, rpb = 256 / tw;
    const int bps = std::max(1, std::min(2, (int)((200 * 1024) / std::max<size_t>(smem, 1024))));
    int64_t grid = std::min<int64_t>((pixels + 8 * rpb - 1) / (8 * rpb), (int64_t)sm_count() * bps);
    grid = std::max<int64_t>(grid, pixels / (1 << 22) + 1);
    QBP_TRACE_BEGIN(st);
    class_sums_kernel<IS_SIGNED><<<(unsigned)grid, 256, smem, st>>>((const uint8_t *)q, (int)pixels, H, W, C, (unsigned long long *)sums);
    QBP_LAUNCH_OK("class_sums_kernel");
    return QBP_OK;
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) size_t qbp_wgrad_s16_workspace_bytes(const qbp_conv_desc *d, int64_t M,
                                                                                      int64_t N, int64_t K)
{
    if (d) {
        if (!wgrad_conv_supported(d)) return 0;
        M = (int64_t)d->N * d->H * d->W; N = d->K; K = d->C;
    }
    return wgrad_ws_bytes(d, M > 0 ? M : 1, N > 0 ? N : 1, K > 0 ? K : 1);
}

extern "C" __attribute__((visibility("default"))) int qbp_wgrad_s16(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K,
                                                                   const int8_t *x, const qbp_qparams *qx,
                                                                   const int8_t *g_hi, const uint8_t *g_lo,
                                                                   const qbp_qparams *qg16, int64_t *acc_out, float *dW,
                                                                   void *ws, size_t ws_bytes, void *stream)
{
    return wgrad_s16_impl(d, M, N, K, x, qx, g_hi, g_lo, qg16, acc_out, dW, nullptr, ws, ws_bytes, (cudaStream_t)stream);
}

int qbp::wgrad_s16_impl(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K, const int8_t *x, const qbp_qparams *qx,
                        const int8_t *g_hi, const uint8_t *g_lo, const qbp_qparams *qg16, int64_t *acc_out, float *dW,
                        int *ext_status, void *ws, size_t ws_bytes, cudaStream_t st, const int64_t *tot_x, const int64_t *tot_g16,
                        bool tot_g_filled, bool lo_signed)
{
    if (!x || !g_hi || !g_lo || !qx || !qg16) return fail(QBP_ERR_INVALID_ARG, "wgrad_s16: NULL operand");
    if (!acc_out && !dW) return fail(QBP_ERR_INVALID_ARG, "wgrad_s16: acc_out and dW are both NULL");
    if (!aligned16(x) || !aligned16(g_hi) || !aligned16(g_lo))
        return fail(QBP_ERR_INVALID_ARG, "wgrad_s16: operands must be 16-byte aligned");
    if (d) {
        if (!wgrad_conv_supported(d))
            return fail(QBP_ERR_UNSUPPORTED_SHAPE,
                        "wgrad_s16: needs stride 1, R = S in {1,3}, pad = (R-1)/2, C and K multiples of 32");
        M = (int64_t)d->N * d->H * d->W; N = d->K; K = d->C;
    } else {
        if (M <= 0 || N <= 0 || K <= 0) return fail(QBP_ERR_INVALID_ARG, "wgrad_s16: M, N, K must be positive");
        if (N % 16 || K % 16) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "wgrad_s16: N and K must be multiples of 16");
        if (M > (int64_t)INT32_MAX || N > (int64_t)INT32_MAX || K > (int64_t)INT32_MAX)
            return fail(QBP_ERR_UNSUPPORTED_SHAPE, "wgrad_s16: extent too large");
    }
    if (!ws || ws_bytes < wgrad_ws_bytes(d, M, N, K))
        return fail(QBP_ERR_WORKSPACE, "wgrad_s16: workspace of %zu bytes needed, %zu given", wgrad_ws_bytes(d, M, N, K), ws_bytes);

    WgradPlan pl;
    plan_wgrad(d, M, N, K, pl, lo_signed);
    WgradParams &P = pl.P;
    const int64_t outs = d ? (int64_t)d->K * d->R * d->S * d->C : K * N;
    WsCarver w(ws, ws_bytes);
    int *status = w.take<int>(1);
    if (ext_status) status = ext_status;         // the caller's sticky word: raised here, never cleared
    int64_t *sx = w.take<int64_t>(16 * K);
    int64_t *shi = w.take<int64_t>(16 * N);
    int64_t *slo = w.take<int64_t>(16 * N);
    int64_t *rowterm = w.take<int64_t>(K);
    int64_t *colterm = w.take<int64_t>(N);
    int64_t *part = P.direct ? nullptr : w.take<int64_t>((size_t)pl.grid * (size_t)P.part_stride);

    // large plain products run on CTA pairs (256 x 256 tiles across two SMs, the whole reduction in one pair)
    const bool pair_kernel = !d && wgrad2_eligible(M, N, K);
    // code sums for the zero-point terms: per border class (convolution) or plain column sums
    int rc;
    // (the border tables stay within int32 per block: a block sees at most Nimg * 2 (W + H) border positions)
    const bool from_totals = d && tot_x && tot_g16 && d->H >= 3 && d->W >= 3 && std::max(K, N) <= 1536 &&
                             (int64_t)d->N * 2 * (d->H + d->W) < (1ll << 22) && (tot_g_filled || wgrad_self_totals(d));
    if (from_totals) {
        // the kernels that wrote the codes left their per-channel totals: only the border positions are read again
        QBP_CUDA_OK(cudaMemsetAsync(sx, 0, (size_t)((char *)(slo + 16 * N) - (char *)sx), st));
        if (wgrad_inline_border(d)) {
            // the product kernel's epilogue warps take the border classes while its MMAs run
            P.cls_x = (unsigned long long *)sx; P.cls_hi = (unsigned long long *)shi; P.cls_lo = (unsigned long long *)slo;
            P.codes_x = (const uint8_t *)x; P.codes_hi = (const uint8_t *)g_hi; P.codes_lo = g_lo;
        } else if (d->pad > 0) {         // (without padding every tap sees every position: the totals are all there is)
            static PerDeviceOnce configured;
            QBP_SMEM_OPT_IN(configured, border_class_sums_kernel, 96 * 1024);
            const int gx = (int)std::min<int64_t>((d->N + 3) / 4, 128);      // one group of four images per block when possible
            QBP_TRACE_BEGIN(st);
            border_class_sums_kernel<<<dim3((unsigned)gx, 1, 3), 256, (size_t)std::max(K, N) * 16 * sizeof(int), st>>>(
                (const uint8_t *)x, (const uint8_t *)g_hi, g_lo, d->N, d->H, d->W, (int)K, (int)N, (unsigned long long *)sx,
                (unsigned long long *)shi, (unsigned long long *)slo, lo_signed ? 1 : 0);
            QBP_LAUNCH_OK("border_class_sums_kernel");
        }
        P.tot_x = (const long long *)tot_x; P.tot_g = (const long long *)tot_g16;
        P.tot_g_plain = tot_g_filled ? 1 : 0;
        if (!tot_g_filled) {
            // nobody left the gradient's totals: the product takes them itself (a row of ones in its spare chunk)
            QBP_CUDA_OK(cudaMemsetAsync(const_cast<int64_t *>(tot_g16), 0, sizeof(int64_t) * (size_t)N, st));
            P.ones_tot = (unsigned long long *)const_cast<int64_t *>(tot_g16);
        }
    } else if (d && K == N && d->W <= 256 && M < (1ll << 30) && shi == sx + 16 * K && slo == shi + 16 * N) {
        // as many input as output channels: the three tensors in one launch
        QBP_CUDA_OK(cudaMemsetAsync(sx, 0, sizeof(int64_t) * 48 * K, st));
        const int cv = (int)K / 16;
        int gs = 1; while (gs * 2 <= cv && gs * 2 * d->W <= 256 && gs < 16) gs *= 2;
        const int slabs = (cv + gs - 1) / gs;
        const int64_t rows = M / d->W;
        // one wave of three blocks per SM over the three tensors
        int64_t grid_x = std::min<int64_t>(rows, std::max<int64_t>(1, (int64_t)sm_count() / slabs));
        grid_x = std::max<int64_t>(grid_x, rows / (1 << 22) + 1);
        QBP_TRACE_BEGIN(st);
        row_class_sums3_kernel<<<dim3((unsigned)grid_x, (unsigned)slabs, 3), 256, (size_t)12 * gs * 16 * sizeof(int), st>>>(
            (const uint8_t *)x, (const uint8_t *)g_hi, (const uint8_t *)g_lo, (int)(rows / d->H), d->H, d->W, (int)K, gs,
            (unsigned long long *)sx, lo_signed ? 1 : 0);
        QBP_LAUNCH_OK("class_sums_kernel");
    } else if (d) {
        if ((rc = launch_class_sums<true>(x, M, d->H, d->W, (int)K, sx, st))) return rc;
        if ((rc = launch_class_sums<true>(g_hi, M, d->H, d->W, (int)N, shi, st))) return rc;
        if ((rc = lo_signed ? launch_class_sums<true>(g_lo, M, d->H, d->W, (int)N, slo, st)
                            : launch_class_sums<false>(g_lo, M, d->H, d->W, (int)N, slo, st))) return rc;
    } else {
        if ((rc = launch_colsum(x, true, M, K, sx, st))) return rc;
        if ((rc = launch_colsum(g_hi, true, M, N, shi, st))) return rc;
        if ((rc = launch_colsum(g_lo, lo_signed, M, N, slo, st))) return rc;
        if (P.direct || pair_kernel) {
            const int64_t mx = std::max(K, N);
            QBP_TRACE_BEGIN(st);
            wgrad_terms_kernel<<<(unsigned)((mx + 255) / 256), 256, 0, st>>>((const long long *)sx, (const long long *)shi,
                                                                            (const long long *)slo, M, N, K, qx, qg16,
                                                                            (long long *)rowterm, (long long *)colterm, lo_signed ? 128 : 0);
            QBP_LAUNCH_OK("wgrad_terms_kernel");
        }
    }
    if (!ext_status) QBP_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
    if (pair_kernel)
        return launch_wgrad2(M, N, K, x, qx, g_hi, g_lo, qg16, acc_out, dW, (const long long *)rowterm,
                             (const long long *)colterm, status, st, lo_signed);

    P.part = (long long *)part; P.status = status;
    P.rowterm = (const long long *)rowterm; P.colterm = (const long long *)colterm;
    P.qx = qx; P.qg = qg16; P.acc_out = (long long *)acc_out; P.dW = dW;
    const uint32_t kr = (uint32_t)P.kr, rb_a = (uint32_t)P.rb_a, rb_b = (uint32_t)P.bn;
    if (!d) {
        if ((rc = make_map_2d(&P.mapX, x, M, K, kr, rb_a))) return rc;
        if ((rc = make_map_2d(&P.mapHi, g_hi, M, N, kr, rb_b))) return rc;
        if ((rc = make_map_2d(&P.mapLo, g_lo, M, N, kr, rb_b))) return rc;
    } else {
        if ((rc = P.halo_bh ? make_map_nhwc(&P.mapX, x, d->N, d->H, d->W, d->C, pl.bn_img, pl.bh + 2, kWgHaloW, rb_a)
                            : make_map_nhwc(&P.mapX, x, d->N, d->H, d->W, d->C, pl.bn_img, pl.bh, pl.bw, rb_a))) return rc;
        if ((rc = make_map_nhwc(&P.mapHi, g_hi, d->N, d->H, d->W, d->K, pl.bn_img, pl.bh, pl.bw, rb_b))) return rc;
        if ((rc = make_map_nhwc(&P.mapLo, g_lo, d->N, d->H, d->W, d->K, pl.bn_img, pl.bh, pl.bw, rb_b))) return rc;
    }
    // the kernel instance for this pair of operand layouts
    void (*kernel)(const WgradParams) = nullptr;
    const int layout_id = (rb_a == 128 ? 0 : rb_a == 64 ? 1 : 2) * 3 + (rb_b == 128 ? 0 : rb_b == 64 ? 1 : 2);
    switch (layout_id) {
    case 0: kernel = qbp_wgrad_kernel<128, 128>; break;
    case 1: kernel = qbp_wgrad_kernel<128, 64>; break;
    case 2: kernel = qbp_wgrad_kernel<128, 32>; break;
    case 3: kernel = qbp_wgrad_kernel<64, 128>; break;
    case 4: kernel = qbp_wgrad_kernel<64, 64>; break;
    case 5: kernel = qbp_wgrad_kernel<64, 32>; break;
    case 6: kernel = qbp_wgrad_kernel<32, 128>; break;
    case 7: kernel = qbp_wgrad_kernel<32, 64>; break;
    default: kernel = qbp_wgrad_kernel<32, 32>; break;
    }
    static PerDeviceOnce configured[9];
    QBP_SMEM_OPT_IN(configured[layout_id], kernel, kWgSmem);
    QBP_TRACE_BEGIN(st);
    kernel<<<pl.grid, kWgThreads, pl.smem, st>>>(P);
    QBP_LAUNCH_OK("qbp_wgrad_kernel");
    if (!P.direct) {
        const int blocks = (int)((outs * kWgFinalizeLanes + 255) / 256);
        QBP_TRACE_BEGIN(st);
        wgrad_finalize_kernel<<<blocks, 256, 0, st>>>(P, (const long long *)sx, (const long long *)shi, (const long long *)slo, outs);
        QBP_LAUNCH_OK("wgrad_finalize_kernel");
    }
    return QBP_OK;
}
