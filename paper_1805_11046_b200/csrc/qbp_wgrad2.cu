// The dense weight gradient g_W = g_l I_{l-1}^T (Eq. (grad_weight)) on CTA pairs: tcgen05.mma.cta_group::2.
//
// dW [K x N] = X [M x K]^T G16 [M x N] with the 16-bit gradient as two byte limbs (G16 = 256 * hi + lo): two
// products per pair tile, X^T hi (s8 x s8) and X^T lo (s8 x u8), each into its own int32 accumulator, combined
// exactly in int64 in the epilogue.  The reduction runs over the M rows, so both operands are M/N-major in shared
// memory (TMA boxes [reduction rows x columns]).
//
// Two CTAs of a cluster compute one 256 x 256 output tile: CTA r holds columns [128 r, 128 r + 128) of the X block
// (= output rows) and columns [128 r, 128 r + 128) of both limb blocks, and the accumulators of its 128 output rows
// (256 columns of the high product, 256 of the low one: all 512 columns of its tensor memory).  One thread of the
// leader issues every MMA; against the single-CTA kernel (256 x 128 tiles) each SM fetches a third fewer operand
// bytes per multiply-add and issues half the instructions.  A pair reduces all M rows of its tile, M <= 65536
// (the low limb's int32 bound, 128 * 255 * rows < 2^31), so nothing is split and no second kernel is needed:
// the epilogue applies the zero-point terms, the scale and stores.
//
// Roles per CTA: warp 0 loads this CTA's operand parts by TMA and reports them to the leader's "full" barrier;
// warp 1 allocates tensor memory (both CTAs) and, in the leader, issues the MMAs and releases stages with a commit
// that arrives in both CTAs; warps 2..9 drain this CTA's accumulator rows.  Every wait is bounded; on expiry the
// CTA raises the status word and leaves through the normal exit.  No TMA load here uses cluster multicast.
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

constexpr int kW2Threads = 320;
constexpr int kW2EpiWarps = 8;
constexpr int kW2Stages = 4;                    // of 48 KB: 128 reduction rows x (128 X + 128 hi + 128 lo columns)
constexpr int kW2Cg = 2;                        // stages released per commit
constexpr int kW2GroupM = 8;
constexpr uint32_t kW2Slab = 32 * 128;
constexpr uint32_t kW2StageBytes = 3u * 128u * 128u;
constexpr uint32_t kW2Smem = 1024u + kW2Stages * kW2StageBytes + kW2EpiWarps * kW2Slab;

struct Wgrad2Params {
    CUtensorMap mapX, mapHi, mapLo, mapC;
    uint32_t desc_lo;                // descriptor bits 16..31 of the M/N-major 128 x 128 tiles
    uint32_t idesc_hi;               // s8 x s8, M = 256, N = 256, both operands M/N-major
    uint32_t lo_flip;                // the low limb's descriptor = idesc_hi ^ lo_flip: the B sign bit for unsigned low bytes, 0 for lo - 128
    int k_iters;                     // reduction steps of 128 rows
    int tiles_m, tiles_n, tiles_total, pairs;
    FastDiv d_group;
    int64_t M, N, K;                 // reduction rows; output columns; output rows
    long long *acc_out; float *dW;
    const long long *rowterm, *colterm;
    const qbp_qparams *qx, *qg;
    int *status;
};

__device__ __forceinline__ uint32_t w2_cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void w2_cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t w2_map_to_cta(const void *p, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void w2_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of this CTA's box whose completion is reported to an mbarrier of either CTA of the pair (no multicast)
__device__ __forceinline__ void w2_tma_load_2d(void *dst, const void *map, uint32_t bar_cluster_addr, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void w2_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate));
}
__device__ __forceinline__ void w2_commit(uint64_t *bar)
{
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask)
                 : "memory");
}

// The eight pair MMAs of a stage (128 reduction rows = four k steps per limb), the limb outermost: switching
// between the two instruction descriptors stalls the MMA pipe.  Offsets in 16-byte units: 256 per k step of an
// M/N-major 128-byte-row tile, 1024 per 128 x 128 tile.
template <bool FIRST>
__device__ __forceinline__ void w2_issue_stage(uint32_t tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc_hi, uint32_t lo_flip)
{
    constexpr uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    const uint32_t idesc_lo = idesc_hi ^ lo_flip;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int limb = i >> 2, kk = i & 3;
        if (elect_one())
            w2_mma(tmem + 256u * (uint32_t)limb, ((uint64_t)hi << 32) | (uint64_t)(a_lo + (uint32_t)kk * 256u),
                   ((uint64_t)hi << 32) | (uint64_t)(b_lo + (uint32_t)limb * 1024u + (uint32_t)kk * 256u),
                   limb ? idesc_lo : idesc_hi, (FIRST && kk == 0) ? 0u : 1u);
    }
}

struct W2Tile { int k0, n0; };
__device__ __forceinline__ W2Tile w2_tile(const Wgrad2Params &P, int tile)
{
    int g, r, tile_m, tile_n;
    P.d_group.divmod(tile, g, r);                        // by kW2GroupM * tiles_n
    const int rows_here = min(kW2GroupM, P.tiles_m - g * kW2GroupM);
    if (rows_here == kW2GroupM) { tile_n = r / kW2GroupM; tile_m = g * kW2GroupM + r % kW2GroupM; }
    else                        { tile_n = r / rows_here; tile_m = g * kW2GroupM + r % rows_here; }
    W2Tile t; t.k0 = tile_m * 256; t.n0 = tile_n * 256;
    return t;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kW2Threads, 1) qbp_wgrad2_kernel(const __grid_constant__ Wgrad2Params P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kW2Stages], empty_bar[kW2Stages], acc_full, acc_empty;
    __shared__ uint32_t tmem_slot;

    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    uint8_t *staging = smem + (size_t)kW2Stages * kW2StageBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = w2_cluster_ctarank();
    const int pair = blockIdx.x >> 1;

    if (threadIdx.x == 0) {
        // "full": the leader's arrive + the bytes of both CTAs; "empty": one multicast commit per stage group;
        // "acc_full": one multicast commit per tile; "acc_empty" (the leader's is waited on): 8 warps of each CTA
        for (int s = 0; s < kW2Stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&acc_full, 1); mbar_init(&acc_empty, 2 * kW2EpiWarps);
        mbar_fence_init();
        tma_prefetch_desc(&P.mapX); tma_prefetch_desc(&P.mapHi); tma_prefetch_desc(&P.mapLo);
        if (P.dW) tma_prefetch_desc(&P.mapC);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    w2_cluster_sync();                   // both CTAs' barriers are initialised before either signals the other
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------- TMA producer (both CTAs)
            uint32_t s = 0, gph = 1, in_group = 0, group = 0;
            for (int tile = pair; tile < P.tiles_total && !timed_out; tile += P.pairs) {
                const W2Tile o = w2_tile(P, tile);
                const int k_mine = o.k0 + 128 * (int)rank, n_mine = o.n0 + 128 * (int)rank;
                for (int it = 0; it < P.k_iters; ++it) {
                    if (in_group == 0 && !mbar_wait(&empty_bar[group], gph)) { timed_out = true; break; }
                    if (++in_group == (uint32_t)kW2Cg) { in_group = 0; ++group; }
                    uint8_t *sa = smem + (size_t)s * kW2StageBytes;
                    const uint32_t bar = w2_map_to_cta(&full_bar[s], 0);
                    if (rank == 0) mbar_expect_tx(&full_bar[s], 2u * kW2StageBytes);
                    const int m0 = it * 128;
                    w2_tma_load_2d(sa, &P.mapX, bar, k_mine, m0);
                    w2_tma_load_2d(sa + 16384, &P.mapHi, bar, n_mine, m0);
                    w2_tma_load_2d(sa + 32768, &P.mapLo, bar, n_mine, m0);
                    if (++s == (uint32_t)kW2Stages) { s = 0; gph ^= 1u; group = 0; }
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---------------------------------------------------- MMA issuer (leader CTA only): the whole warp in step
            uint32_t s = 0, ph = 0, in_group = 0, group = 0, eph = 1;
            const uint32_t ring = smem_u32(smem);
            uint32_t a_addr = ring;
            for (int tile = pair; tile < P.tiles_total && !timed_out; tile += P.pairs) {
                if (!mbar_wait_uniform(&acc_empty, eph)) { timed_out = true; break; }
                eph ^= 1u;
                tc_fence_after();
                for (int it = 0; it < P.k_iters; ++it) {
                    if (!mbar_wait_uniform(&full_bar[s], ph)) { timed_out = true; break; }
                    tc_fence_after();
                    const uint32_t a_lo = ((a_addr >> 4) & 0x3FFFu) | P.desc_lo;
                    const uint32_t b_lo = (((a_addr + 16384u) >> 4) & 0x3FFFu) | P.desc_lo;
                    if (it == 0) w2_issue_stage<true>(tmem_base, a_lo, b_lo, P.idesc_hi, P.lo_flip);
                    else         w2_issue_stage<false>(tmem_base, a_lo, b_lo, P.idesc_hi, P.lo_flip);
                    if (++in_group == (uint32_t)kW2Cg) {
                        if (elect_one()) w2_commit(&empty_bar[group]);
                        in_group = 0; ++group;
                    }
                    a_addr += kW2StageBytes;
                    if (++s == (uint32_t)kW2Stages) { s = 0; ph ^= 1u; group = 0; a_addr = ring; }
                }
                if (!timed_out && elect_one()) w2_commit(&acc_full);
            }
        }
    } else {
        // ------------------------------------------------------- epilogue (each CTA drains its own 128 output rows)
        // the two groups of four warps split the eight column chunks of 32
        const int ew = warp - 2, quad = warp & 3, half = ew >> 2;
        const int row = quad * 32 + lane;
        uint8_t *slab = staging + (size_t)ew * kW2Slab;
        const float scale = __fmul_rn(P.qx->scale, P.qg->scale);
        const uint32_t leader_empty = w2_map_to_cta(&acc_empty, 0);
        uint32_t fph = 0;
        for (int tile = pair; tile < P.tiles_total; tile += P.pairs) {
            const W2Tile o = w2_tile(P, tile);
            const int64_t k = (int64_t)o.k0 + 128 * (int)rank + row;                  // output row
            const bool valid = k < P.K;
            const bool slab_in = (int64_t)o.k0 + 128 * (int)rank + quad * 32 < P.K;
            const long long rterm = valid ? P.rowterm[k] : 0;
            const int64_t ncol = P.N - o.n0;
            const int nchunks = (int)((ncol < 256 ? ncol : 256) + 31) / 32;
            if (!timed_out && !mbar_wait_warp(&acc_full, fph)) timed_out = true;
            fph ^= 1u;
            if (!timed_out) {
                tc_fence_after();
                const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
                const int c_begin = half * 4, c_end = min(nchunks, half * 4 + 4);
                if (c_begin >= c_end) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) w2_arrive_cluster(leader_empty);
                }
                for (int c = c_begin; c < c_end; ++c) {
                    const int c0 = c * 32;
                    uint32_t rh[32], rl[32];
                    tmem_ld_32x32(t_addr + (uint32_t)c0, rh);
                    tmem_ld_32x32(t_addr + 256u + (uint32_t)c0, rl);
                    tmem_ld_wait();
                    if (c == c_end - 1) {
                        // this warp has read its part of the accumulators: tell the leader's MMA warp
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) w2_arrive_cluster(leader_empty);
                    }
                    const int lim = (int)(ncol - c0 < 32 ? ncol - c0 : 32);
                    // lane l fetches the column term of column c0 + l; the row's 32 sums take them by shuffle
                    const long long my_cterm = lane < lim ? __ldg(P.colterm + o.n0 + c0 + lane) : 0;
                    if (P.dW) {
                        if (lane == 0) tma_store_wait_read();
                        __syncwarp();
                    }
                    uint8_t *rowp = slab + lane * 128;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        long long a4[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            a4[e] = 256ll * (long long)(int)rh[j + e] + (long long)(int)rl[j + e] + rterm +
                                    __shfl_sync(0xffffffffu, my_cterm, j + e);
                        if (P.acc_out && valid) {
                            long long *dst = P.acc_out + k * P.N + o.n0 + c0 + j;
                            if (j + 4 <= lim) {
                                *reinterpret_cast<longlong2 *>(dst) = make_longlong2(a4[0], a4[1]);
                                *reinterpret_cast<longlong2 *>(dst + 2) = make_longlong2(a4[2], a4[3]);
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (j + e < lim) dst[e] = a4[e];
                            }
                        }
                        if (P.dW)
                            *reinterpret_cast<float4 *>(rowp + (((j >> 2) ^ (lane & 7)) << 4)) =
                                make_float4(__fmul_rn((float)a4[0], scale), __fmul_rn((float)a4[1], scale),
                                            __fmul_rn((float)a4[2], scale), __fmul_rn((float)a4[3], scale));
                    }
                    if (P.dW) {
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0 && slab_in) {
                            tma_store_2d(&P.mapC, slab, o.n0 + c0, o.k0 + 128 * (int)rank + quad * 32);
                            tma_store_commit();
                        }
                    }
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
    }

    if (timed_out) {
        raise_timeout(P.status);
        __nanosleep(1000000);
    }
    tc_fence_before();
    __syncthreads();
    w2_cluster_sync();                   // neither CTA retires while the other may still read its memory or signal it
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// Whether the pair kernel takes this plain product: whole pair tiles in both output directions, a reduction one
// pair can hold in int32 chunks, 16-byte aligned rows.
bool wgrad2_eligible(int64_t M, int64_t N, int64_t K)
{
    return M >= 512 && M <= 65536 && N >= 256 && K >= 256;
}

int launch_wgrad2(int64_t M, int64_t N, int64_t K, const int8_t *x, const qbp_qparams *qx, const int8_t *g_hi,
                  const uint8_t *g_lo, const qbp_qparams *qg16, int64_t *acc_out, float *dW, const long long *rowterm,
                  const long long *colterm, int *status, cudaStream_t st, bool lo_signed)
{
    Wgrad2Params P{};
    int rc;
    // per-CTA operand parts: 128 reduction rows x 128 columns, M/N-major
    const OperandLayout L = layout_mnmajor(128, 128, 1, 0);
    if ((rc = make_map_2d(&P.mapX, x, M, K, 128, 128))) return rc;
    if ((rc = make_map_2d(&P.mapHi, g_hi, M, N, 128, 128))) return rc;
    if ((rc = make_map_2d(&P.mapLo, g_lo, M, N, 128, 128))) return rc;
    if (dW && (rc = make_map_out_2d(&P.mapC, dW, K, N))) return rc;
    P.desc_lo = L.desc_lo;
    P.idesc_hi = make_idesc(true, true, 1, 1, 256, 256);
    P.lo_flip = lo_signed ? 0u : (1u << 10);
    P.k_iters = (int)((M + 127) / 128);
    P.tiles_m = (int)((K + 255) / 256); P.tiles_n = (int)((N + 255) / 256);
    P.tiles_total = P.tiles_m * P.tiles_n;
    P.pairs = std::min(P.tiles_total, sm_count() / 2);
    P.d_group = make_fastdiv(kW2GroupM * P.tiles_n);
    P.M = M; P.N = N; P.K = K;
    P.acc_out = (long long *)acc_out; P.dW = dW;
    P.rowterm = rowterm; P.colterm = colterm; P.qx = qx; P.qg = qg16; P.status = status;
    static PerDeviceOnce configured;
    QBP_SMEM_OPT_IN(configured, qbp_wgrad2_kernel, kW2Smem);
    QBP_TRACE_BEGIN(st);
    qbp_wgrad2_kernel<<<2 * P.pairs, kW2Threads, kW2Smem, st>>>(P);
    QBP_LAUNCH_OK("qbp_wgrad2_kernel");
    return QBP_OK;
}

}  // namespace qbp
