// The dense 8-bit product y = W x (Section 1) on CTA pairs: tcgen05.mma.cta_group::2.
//
// Two CTAs of a cluster (two neighbouring SMs) compute one 256 x 256 output tile: CTA r of the pair holds rows
// [128 r, 128 r + 128) of the A tile and columns [128 r, 128 r + 128) of the B tile in its shared memory and
// the accumulator of its 128 rows (256 columns) in its tensor memory.  One thread of the pair's first CTA (the
// leader) issues every MMA; the tensor cores of both SMs read the B halves of both CTAs.  Against the
// single-CTA kernel this halves the B bytes each SM reads per MMA, halves the instructions and commits per
// multiply-add, and leaves room in tensor memory for a second accumulator, so that the epilogue of a tile
// overlaps the MMAs of the next one.
//
// Roles per CTA: warp 0 loads this CTA's operand halves by TMA and reports them to the leader's "full"
// barrier; warp 1 allocates tensor memory (both CTAs) and, in the leader, issues the MMAs and releases stages
// with a commit that arrives in both CTAs; warps 2..9 drain this CTA's accumulator rows.  Every wait is
// bounded; on expiry the CTA raises the status word and leaves through the normal exit.  No TMA load here
// uses cluster multicast.
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

constexpr int k2Threads = 320;
constexpr int k2EpiWarps = 8;
constexpr int k2MaxStages = 8;
constexpr int k2GroupM = 8;
constexpr uint32_t k2Slab = 32 * 128;
constexpr uint32_t k2Smem = 225u * 1024u;     // dynamic; about 1.2 KB of static shared memory come on top

struct Mma2Params {
    CUtensorMap mapA, mapB, mapC;
    OperandLayout a, b;              // per-CTA halves: A 128 rows, B 128 columns, 128 reduction bytes
    uint32_t idesc;                  // M = 256, N = 256
    int stages, cg;                  // ring stages of one k block; stages released per commit
    int msub;                        // 256-row sub-tiles of the pair tile (2: 512 x 256, one accumulator set)
    int nbuf;                        // accumulator sets in tensor memory (2 when msub == 1)
    int k_iters;
    int tiles_m, tiles_n, tiles_total, pairs;
    FastDiv d_group;
    int64_t M, N;
    int32_t *acc_out; float *out;
    const int32_t *rowterm, *colterm;
    const qbp_qparams *qa, *qb;
    int *status;
};

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(const void *p, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of this CTA's box whose completion is reported to an mbarrier of either CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const void *map, uint32_t bar_cluster_addr, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *slot_in_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate));
}
// Arrive, in both CTAs of the pair, on the mbarrier at this shared-memory offset once every MMA issued so far is done.
__device__ __forceinline__ void mma_commit_pair(uint64_t *bar)
{
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask)
                 : "memory");
}

// ---- MMA issue ------------------------------------------------------------------
// The MMA takes its operands from the warp's few uniform registers: the loop is written for a whole converged warp
// with an elected issuer, its MMAs unrolled with constant offsets, and what the operand layout fixes (the k step:
// 2 sixteen-byte units inside a K-major row, 256 between the 32-row blocks of an M/N-major tile; the upper descriptor
// word: 128-byte swizzle, 8-row groups 1024 bytes apart) is spelled as constants.
struct Pair2MmaArgs {
    uint64_t *full_bar, *empty_bar, *acc_full, *acc_empty;
    uint32_t ring, stage_bytes, a_bytes, tmem, a_desc_lo, b_desc_lo, idesc;
    int k_iters;
    uint32_t stages, cg, nbuf;
    int tile0, tiles_total, tile_step;
};

template <uint32_t AK, uint32_t BK, int MSUB, bool FIRST>
__device__ __forceinline__ void pair_issue_stage(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc)
{
    constexpr uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t a_tile16 = 128u * 128u / 16u;              // a CTA's half of one 256-row sub-tile
#pragma unroll
    for (int i = 0; i < 4 * MSUB; ++i) {
        const int kk = i / MSUB, sub = i % MSUB;
        if (elect_one())
            mma_i8_pair(d_tmem + 256u * (uint32_t)sub, ((uint64_t)hi << 32) | (uint64_t)(a_lo + (uint32_t)sub * a_tile16 + (uint32_t)kk * AK),
                        ((uint64_t)hi << 32) | (uint64_t)(b_lo + (uint32_t)kk * BK), idesc, (FIRST && kk == 0) ? 0u : 1u);
    }
}

// False when a wait ran out.
template <uint32_t AK, uint32_t BK, int MSUB>
__device__ __forceinline__ bool pair_mma_loop(const Pair2MmaArgs &A)
{
    uint32_t s = 0, ph = 0, buf = 0, bph = 1;
    uint32_t in_group = 0, group = 0;              // stages issued of the current release group, its index
    uint32_t a_addr = A.ring;
    for (int tile = A.tile0; tile < A.tiles_total; tile += A.tile_step) {
        if (!mbar_wait_uniform(&A.acc_empty[buf], bph)) return false;
        tc_fence_after();
        const uint32_t d_tmem = A.tmem + buf * 256u;              // MSUB == 2: one set, sub-tile s at column 256 s
        for (int it = 0; it < A.k_iters; ++it) {
            if (!mbar_wait_uniform(&A.full_bar[s], ph)) return false;
            tc_fence_after();
            const uint32_t a_lo = ((a_addr >> 4) & 0x3FFFu) | A.a_desc_lo;
            const uint32_t b_lo = (((a_addr + A.a_bytes) >> 4) & 0x3FFFu) | A.b_desc_lo;
            if (it == 0) pair_issue_stage<AK, BK, MSUB, true>(d_tmem, a_lo, b_lo, A.idesc);
            else         pair_issue_stage<AK, BK, MSUB, false>(d_tmem, a_lo, b_lo, A.idesc);
            // release the group of stages this one completes, in both CTAs (the last group of a tile too: the
            // commit of acc_full below covers the same MMAs, but the producers wait on "empty")
            if (++in_group == A.cg) {
                if (elect_one()) mma_commit_pair(&A.empty_bar[group]);
                in_group = 0; ++group;
            }
            a_addr += A.stage_bytes;
            if (++s == A.stages) { s = 0; ph ^= 1u; group = 0; a_addr = A.ring; }
        }
        if (elect_one()) mma_commit_pair(&A.acc_full[buf]);
        if (++buf == A.nbuf) { buf = 0; bph ^= 1u; }
    }
    return true;
}

struct Tile2 { int m0, n0; };
__device__ __forceinline__ Tile2 tile2_origin(const Mma2Params &P, int tile)
{
    int g, r, tile_m, tile_n;
    P.d_group.divmod(tile, g, r);                        // by k2GroupM * tiles_n
    const int rows_here = min(k2GroupM, P.tiles_m - g * k2GroupM);
    if (rows_here == k2GroupM) { tile_n = r / k2GroupM; tile_m = g * k2GroupM + r % k2GroupM; }
    else                       { tile_n = r / rows_here; tile_m = g * k2GroupM + r % rows_here; }
    Tile2 t; t.m0 = tile_m * 256 * P.msub; t.n0 = tile_n * 256;
    return t;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(k2Threads, 1) qbp_mma2_kernel(const __grid_constant__ Mma2Params P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[k2MaxStages], empty_bar[k2MaxStages], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(16) int32_t s_cterm[256];            // read as int4

    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    const uint32_t a_bytes = P.a.tile_bytes * (uint32_t)P.msub;
    const uint32_t stage_bytes = a_bytes + P.b.tile_bytes;                   // this CTA's halves
    uint8_t *staging = smem + (size_t)P.stages * stage_bytes;                // 1024-aligned: stage_bytes is 32 KB
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                                 // 0: leader of the pair
    const int pair = blockIdx.x >> 1;

    if (threadIdx.x == 0) {
        // "full": the leader's arrive + the bytes of both CTAs; "empty": one multicast commit per stage group;
        // "acc_full": one multicast commit per tile; "acc_empty" (leader's is the one waited on): 8 warps of each CTA
        for (int s = 0; s < P.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 2 * k2EpiWarps); }
        mbar_fence_init();
        tma_prefetch_desc(&P.mapA);
        tma_prefetch_desc(&P.mapB);
        if (P.out) tma_prefetch_desc(&P.mapC);
    }
    if (warp == 1) { tmem_alloc_pair(&tmem_slot, 512); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                  // both CTAs' barriers are initialised before either signals the other
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------- TMA producer (both CTAs)
            const uint32_t cg = (uint32_t)P.cg;
            uint32_t s = 0, gph = 1, in_group = 0, group = 0;
            for (int tile = pair; tile < P.tiles_total && !timed_out; tile += P.pairs) {
                const Tile2 o = tile2_origin(P, tile);
                const int m_mine = o.m0 + 128 * (int)rank, n_mine = o.n0 + 128 * (int)rank;   // sub-tile s: + 256 s rows
                for (int it = 0; it < P.k_iters; ++it) {
                    if (in_group == 0 && !mbar_wait(&empty_bar[group], gph)) { timed_out = true; break; }
                    if (++in_group == cg) { in_group = 0; ++group; }
                    uint8_t *sa = smem + (size_t)s * stage_bytes;
                    uint8_t *sb = sa + a_bytes;
                    const uint32_t bar = map_to_cta(&full_bar[s], 0);
                    if (rank == 0) mbar_expect_tx(&full_bar[s], 2u * stage_bytes);
                    const int k0 = it * 128;
                    for (int sub = 0; sub < P.msub; ++sub) {
                        if (P.a.major == 0) tma_load_2d_pair(sa + sub * P.a.tile_bytes, &P.mapA, bar, k0, m_mine + 256 * sub);
                        else                tma_load_2d_pair(sa + sub * P.a.tile_bytes, &P.mapA, bar, m_mine + 256 * sub, k0);
                    }
                    if (P.b.major == 0) tma_load_2d_pair(sb, &P.mapB, bar, k0, n_mine);
                    else                tma_load_2d_pair(sb, &P.mapB, bar, n_mine, k0);
                    if (++s == (uint32_t)P.stages) { s = 0; gph ^= 1u; group = 0; }
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---------------------------------------------------- MMA issuer (leader CTA only): the whole warp in step,
            // an elected lane issues; one instance of the loop per pair of operand layouts and tile height
            Pair2MmaArgs A;
            A.full_bar = full_bar; A.empty_bar = empty_bar; A.acc_full = acc_full; A.acc_empty = acc_empty;
            A.ring = smem_u32(smem); A.stage_bytes = stage_bytes; A.a_bytes = a_bytes; A.tmem = tmem_base;
            A.a_desc_lo = P.a.desc_lo; A.b_desc_lo = P.b.desc_lo; A.idesc = P.idesc;
            A.k_iters = P.k_iters; A.stages = (uint32_t)P.stages; A.cg = (uint32_t)P.cg; A.nbuf = (uint32_t)P.nbuf;
            A.tile0 = pair; A.tiles_total = P.tiles_total; A.tile_step = P.pairs;
            bool ok;
            if (P.msub == 2) {
                if (P.a.major == 0) ok = P.b.major == 0 ? pair_mma_loop<2, 2, 2>(A) : pair_mma_loop<2, 256, 2>(A);
                else                ok = P.b.major == 0 ? pair_mma_loop<256, 2, 2>(A) : pair_mma_loop<256, 256, 2>(A);
            } else {
                if (P.a.major == 0) ok = P.b.major == 0 ? pair_mma_loop<2, 2, 1>(A) : pair_mma_loop<2, 256, 1>(A);
                else                ok = P.b.major == 0 ? pair_mma_loop<256, 2, 1>(A) : pair_mma_loop<256, 256, 1>(A);
            }
            timed_out = !ok;
        }
    } else {
        // ------------------------------------------------------- epilogue (each CTA drains its own 128 rows)
        // msub == 1: the two groups of four warps split the column chunks (0..3, 4..7); msub == 2: one sub-tile each
        const int ew = warp - 2, quad = warp & 3, half = ew >> 2;
        const int sub = P.msub == 2 ? half : 0;
        const int et = threadIdx.x - 64;
        const int row = quad * 32 + lane;
        uint8_t *slab = staging + (size_t)ew * k2Slab;
        const float scale = __fmul_rn(P.qa->scale, P.qb->scale);
        const uint32_t leader_empty0 = map_to_cta(&acc_empty[0], 0), leader_empty1 = map_to_cta(&acc_empty[1], 0);
        uint32_t buf = 0, fph = 0;
        for (int tile = pair; tile < P.tiles_total; tile += P.pairs) {
            const Tile2 o = tile2_origin(P, tile);
            const int64_t m = (int64_t)o.m0 + 256 * sub + 128 * (int)rank + row;
            const bool valid = m < P.M;
            const bool slab_in = (int64_t)o.m0 + 256 * sub + 128 * (int)rank + quad * 32 < P.M;
            const int rterm = valid ? __ldg(P.rowterm + m) : 0;
            // column terms of this tile (the previous tile's readers are done first)
            named_barrier(1, 32 * k2EpiWarps);
            if (et < 256) s_cterm[et] = o.n0 + et < P.N ? __ldg(P.colterm + o.n0 + et) : 0;
            named_barrier(1, 32 * k2EpiWarps);
            const int64_t ncol = P.N - o.n0;
            const int nchunks = (int)((ncol < 256 ? ncol : 256) + 31) / 32;
            if (!timed_out && !mbar_wait_warp(&acc_full[buf], fph)) timed_out = true;
            if (!timed_out) {
                tc_fence_after();
                const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * 256u + 256u * (uint32_t)sub;
                const int c_begin = P.msub == 2 ? 0 : half * 4, c_end = P.msub == 2 ? nchunks : min(nchunks, half * 4 + 4);
                if (c_begin >= c_end) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(buf ? leader_empty1 : leader_empty0);
                }
                for (int c = c_begin; c < c_end; ++c) {
                    const int c0 = c * 32;
                    uint32_t r[32];
                    tmem_ld_32x32(t_addr + (uint32_t)c0, r);
                    tmem_ld_wait();
                    if (c == c_end - 1) {
                        // this warp has read its part of the accumulator: tell the leader's MMA thread
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(buf ? leader_empty1 : leader_empty0);
                    }
                    const int lim = (int)(ncol - c0 < 32 ? ncol - c0 : 32);
                    int acc[32];
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int4 ct = *reinterpret_cast<const int4 *>(s_cterm + c0 + j);
                        acc[j] = (int)r[j] + rterm + ct.x; acc[j + 1] = (int)r[j + 1] + rterm + ct.y;
                        acc[j + 2] = (int)r[j + 2] + rterm + ct.z; acc[j + 3] = (int)r[j + 3] + rterm + ct.w;
                    }
                    if (P.acc_out && valid) {
                        int32_t *dst = P.acc_out + m * P.N + o.n0 + c0;
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
                    if (P.out) {
                        if (lane == 0) tma_store_wait_read();
                        __syncwarp();
                        uint8_t *rowp = slab + lane * 128;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4 *>(rowp + (((j >> 2) ^ (lane & 7)) << 4)) =
                                make_float4(__fmul_rn((float)acc[j], scale), __fmul_rn((float)acc[j + 1], scale),
                                            __fmul_rn((float)acc[j + 2], scale), __fmul_rn((float)acc[j + 3], scale));
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0 && slab_in) {
                            tma_store_2d(&P.mapC, slab, o.n0 + c0, o.m0 + 256 * sub + 128 * (int)rank + quad * 32);
                            tma_store_commit();
                        }
                    }
                }
            }
            if (++buf == (uint32_t)P.nbuf) { buf = 0; fph ^= 1u; }
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
    cluster_sync_all();                  // neither CTA retires while the other may still read its memory or signal it
    if (warp == 1) { __syncwarp(); tmem_dealloc_pair(tmem_base, 512); }
}

// Whether the pair kernel takes this product: anything with at least one whole pair tile's worth of rows and columns
// (it is the faster kernel from 1024^3 up; the single-CTA kernel keeps the narrow shapes).
bool gemm2_eligible(int64_t M, int64_t N, int64_t K)
{
    return M >= 256 && N >= 256 && K >= 128;
}

int launch_gemm2(int transA, int transB, int64_t M, int64_t N, int64_t K, const int8_t *A, const qbp_qparams *qa,
                 const int8_t *B, const qbp_qparams *qb, int32_t *acc_out, float *C, const int32_t *rowterm,
                 const int32_t *colterm, int *status, bool clear_status, cudaStream_t st)
{
    Mma2Params P{};
    int rc;
    // per-CTA operand halves: 128 rows of A, 128 columns of B, 128 reduction bytes per stage
    if (!transA) { P.a = layout_kmajor(128, 128);        rc = make_map_2d(&P.mapA, A, M, K, 128, 128); }
    else         { P.a = layout_mnmajor(128, 128, 1, 0); rc = make_map_2d(&P.mapA, A, K, M, 128, 128); }
    if (rc) return rc;
    if (transB)  { P.b = layout_kmajor(128, 128);        rc = make_map_2d(&P.mapB, B, N, K, 128, 128); }
    else         { P.b = layout_mnmajor(128, 128, 1, 0); rc = make_map_2d(&P.mapB, B, K, N, 128, 128); }
    if (rc) return rc;
    if (C && (rc = make_map_out_2d(&P.mapC, C, M, N))) return rc;
    P.idesc = make_idesc(true, true, P.a.major, P.b.major, 256, 256);
    P.k_iters = (int)((K + 127) / 128);
    // 512 x 256 pair tiles (two accumulators per CTA fill tensor memory: no second set) cut the operand bytes per
    // multiply-add by a quarter against 256 x 256; worth it once the product is large enough to be fetch-bound
    P.msub = M >= 2048 ? 2 : 1;
    P.nbuf = P.msub == 2 ? 1 : 2;
    P.tiles_m = (int)((M + 256 * P.msub - 1) / (256 * P.msub)); P.tiles_n = (int)((N + 255) / 256);
    P.tiles_total = P.tiles_m * P.tiles_n;
    P.pairs = std::min(P.tiles_total, sm_count() / 2);
    P.d_group = make_fastdiv(k2GroupM * P.tiles_n);
    const uint32_t stage_bytes = P.a.tile_bytes * P.msub + P.b.tile_bytes;  // 32 KB or 48 KB
    int stages = (int)((k2Smem - 1024 - k2EpiWarps * k2Slab) / stage_bytes);
    stages = std::min(stages, k2MaxStages);
    P.cg = 2;                           // sixteen (msub 2) or eight pair MMAs, 1024 cycles or more, between commits
    stages -= stages % P.cg;
    if (stages < 2 * P.cg) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "gemm_s8: the pair kernel's ring does not fit");
    P.stages = stages;
    P.M = M; P.N = N; P.acc_out = acc_out; P.out = C;
    P.rowterm = rowterm; P.colterm = colterm; P.qa = qa; P.qb = qb; P.status = status;
    const size_t smem = 1024 + (size_t)stages * stage_bytes + k2EpiWarps * k2Slab;
    static PerDeviceOnce configured;
    QBP_SMEM_OPT_IN(configured, qbp_mma2_kernel, k2Smem);
    if (clear_status) QBP_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
    QBP_TRACE_BEGIN(st);
    qbp_mma2_kernel<<<2 * P.pairs, k2Threads, smem, st>>>(P);
    QBP_LAUNCH_OK("qbp_mma2_kernel");
    return QBP_OK;
}

}  // namespace qbp
