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
// 128*128*65536 the high one), combines its two accumulators exactly in int64
// and adds them to the int64 result with red.global.add.u64; integer addition
// is order-free, so the split over CTAs does not change the result.
//
// Convolution: the MMA's 128 rows hold `chunks` filter taps x the input
// channels of one tap (2 taps x 64 channels, or 1 tap x 128 channels); each
// tap is its own TMA load of the input, shifted by the tap offset, padding
// zero-filled.  Zero-points are applied afterwards from per-border-class code
// sums (a tap near the border sees fewer positions).
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

constexpr int kWgThreads = 192;
constexpr int kWgMaxStages = 8;
constexpr int kWgMaxTiles = 4;       // A tiles (128 accumulator rows each) per CTA: 4 x 2 limbs x 64 columns fill tensor memory

struct WgradParams {
    CUtensorMap mapX, mapHi, mapLo;
    OperandLayout a, b;
    uint32_t idesc_hi, idesc_lo;
    uint32_t a_chunk_bytes;          // bytes of one A chunk (kr rows x rb_a)
    int conv;                        // 0: x [M x K], g [M x N]; 1: NHWC tensors
    int stages, bn, tmem_cols;
    int kr;                          // reduction rows per pipeline stage (64 or 128)
    int a_chunks, rb_a;              // chunks per A tile, bytes (= channels / columns) per chunk row
    int ma;                          // A tiles per CTA (they share the g tiles of a stage)
    int a_tiles;                     // A tiles in all: plain K/128; conv tap groups x channel tiles
    int a_groups;                    // ceil(a_tiles / ma)
    int tiles_c;                     // conv: channel tiles per tap group
    int tiles_b;                     // output-channel (N) tiles of bn
    int slices, iters_total;         // reduction steps (kr rows each) split into `slices` ranges
    // conv geometry
    int H, W, Nimg, pad, R, S, C, taps;
    int bw_log2, bh_log2, tiles_w, tiles_h;
    // plain geometry
    int64_t M, N, K;
    unsigned long long *raw;         // int64 accumulator, zeroed before launch
    int *status;
};

__global__ void __launch_bounds__(kWgThreads, 1) qbp_wgrad_kernel(const __grid_constant__ WgradParams P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kWgMaxStages], empty_bar[kWgMaxStages], acc_bar;
    __shared__ uint32_t tmem_slot;

    const uint32_t raw_addr = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    const uint32_t a_tile_bytes = P.a_chunk_bytes * (uint32_t)P.a_chunks;
    const uint32_t a_bytes = a_tile_bytes * (uint32_t)P.ma;
    const uint32_t stage_bytes = a_bytes + 2u * P.b.tile_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bid = blockIdx.x;
    const int tb = bid % P.tiles_b; bid /= P.tiles_b;
    const int ag = bid % P.a_groups;
    const int slice = bid / P.a_groups;
    const int n0 = tb * P.bn;
    const int it_begin = (int)((int64_t)P.iters_total * slice / P.slices);
    const int it_end = (int)((int64_t)P.iters_total * (slice + 1) / P.slices);
    const int k_iters = it_end - it_begin;
    const int n_tiles = min(P.ma, P.a_tiles - ag * P.ma);        // A tiles this CTA owns
    const int kk_per_iter = P.kr / 32;

    // chunks present in A tile `at`: conv -- taps left in the tap group; plain -- column chunks left in K
    auto chunks_of = [&](int at) {
        if (P.conv) return min(P.a_chunks, P.taps - (at / P.tiles_c) * P.a_chunks);
        return min(P.a_chunks, (int)((P.K - (int64_t)at * 128 + P.rb_a - 1) / P.rb_a));
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < P.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&acc_bar, 1);
        mbar_fence_init();
        tma_prefetch_desc(&P.mapX); tma_prefetch_desc(&P.mapHi); tma_prefetch_desc(&P.mapLo);
    }
    if (warp == 1) { tmem_alloc(&tmem_slot, (uint32_t)P.tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t tx_bytes = 2u * P.b.tile_bytes;
            for (int j = 0; j < n_tiles; ++j) tx_bytes += (uint32_t)chunks_of(ag * P.ma + j) * P.a_chunk_bytes;
            for (int i = 0; i < k_iters; ++i) {
                const int s = i % P.stages;
                const uint32_t ph = (uint32_t)(i / P.stages) & 1u;
                if (!mbar_wait(&empty_bar[s], ph ^ 1u)) { timed_out = true; break; }
                uint8_t *sa = smem + (size_t)s * stage_bytes;
                uint8_t *shi = sa + a_bytes;
                uint8_t *slo = shi + P.b.tile_bytes;
                mbar_expect_tx(&full_bar[s], tx_bytes);
                const int it = it_begin + i;
                if (!P.conv) {
                    const int row0 = it * P.kr;
                    tma_load_2d(shi, &P.mapHi, &full_bar[s], n0, row0);
                    tma_load_2d(slo, &P.mapLo, &full_bar[s], n0, row0);
                    for (int j = 0; j < n_tiles; ++j) {
                        const int at = ag * P.ma + j, nc = chunks_of(at);
                        for (int c = 0; c < nc; ++c)
                            tma_load_2d(sa + (size_t)j * a_tile_bytes + (size_t)c * P.a_chunk_bytes, &P.mapX, &full_bar[s],
                                        at * 128 + c * P.rb_a, row0);
                    }
                } else {
                    const int tw = it % P.tiles_w;
                    const int th = (it / P.tiles_w) % P.tiles_h;
                    const int tn = it / (P.tiles_w * P.tiles_h);
                    const int w0 = tw << P.bw_log2, h0 = th << P.bh_log2;
                    const int img0 = tn * (P.kr >> (P.bw_log2 + P.bh_log2));
                    tma_load_4d(shi, &P.mapHi, &full_bar[s], n0, w0, h0, img0);
                    tma_load_4d(slo, &P.mapLo, &full_bar[s], n0, w0, h0, img0);
                    for (int j = 0; j < n_tiles; ++j) {
                        const int at = ag * P.ma + j, nc = chunks_of(at);
                        const int group = at / P.tiles_c, tc = at % P.tiles_c;
                        for (int c = 0; c < nc; ++c) {
                            const int tap = group * P.a_chunks + c;
                            const int r = tap / P.S, t = tap % P.S;
                            tma_load_4d(sa + (size_t)j * a_tile_bytes + (size_t)c * P.a_chunk_bytes, &P.mapX, &full_bar[s],
                                        tc * P.rb_a, w0 - P.pad + t, h0 - P.pad + r, img0);
                        }
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            for (int i = 0; i < k_iters; ++i) {
                const int s = i % P.stages;
                const uint32_t ph = (uint32_t)(i / P.stages) & 1u;
                if (!mbar_wait(&full_bar[s], ph)) { timed_out = true; break; }
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t hi_addr = a_addr + a_bytes;
                const uint32_t lo_addr = hi_addr + P.b.tile_bytes;
                const uint32_t bh_lo = ((hi_addr >> 4) & 0x3FFFu) | P.b.desc_lo;
                const uint32_t bl_lo = ((lo_addr >> 4) & 0x3FFFu) | P.b.desc_lo;
                for (int j = 0; j < n_tiles; ++j) {
                    const uint32_t a_lo = (((a_addr + (uint32_t)j * a_tile_bytes) >> 4) & 0x3FFFu) | P.a.desc_lo;
                    const uint32_t d_hi = tmem_base + (uint32_t)(j * 2 * P.bn);
                    for (int kk = 0; kk < kk_per_iter; ++kk) {
                        const uint64_t da = ((uint64_t)P.a.desc_hi << 32) | (uint64_t)(a_lo + kk * P.a.kstep);
                        const uint64_t dh = ((uint64_t)P.b.desc_hi << 32) | (uint64_t)(bh_lo + kk * P.b.kstep);
                        const uint64_t dl = ((uint64_t)P.b.desc_hi << 32) | (uint64_t)(bl_lo + kk * P.b.kstep);
                        const uint32_t accum = (i | kk) != 0 ? 1u : 0u;
                        mma_i8(d_hi, da, dh, P.idesc_hi, accum);
                        mma_i8(d_hi + (uint32_t)P.bn, da, dl, P.idesc_lo, accum);
                    }
                }
                mma_commit(&empty_bar[s]);
            }
            if (!timed_out) mma_commit(&acc_bar);
        }
        __syncwarp();
    } else {
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        if (k_iters > 0) {
            if (!mbar_wait(&acc_bar, 0)) timed_out = true;
            tc_fence_after();
        }
        if (!timed_out && k_iters > 0) {
            for (int j = 0; j < n_tiles; ++j) {
                // row of the accumulator -> (chunk, channel); column -> output channel of g
                const int at = ag * P.ma + j;
                const int chunk = row / P.rb_a, cin = row % P.rb_a;
                bool valid = chunk < chunks_of(at);
                int64_t base, col_stride;
                if (!P.conv) {
                    const int64_t k = (int64_t)at * 128 + row;
                    valid = valid && k < P.K;
                    base = k * P.N; col_stride = 1;
                } else {
                    const int tap = (at / P.tiles_c) * P.a_chunks + chunk;
                    const int c = (at % P.tiles_c) * P.rb_a + cin;
                    valid = valid && c < P.C;
                    base = (int64_t)tap * P.C + c;                          // [k][tap][c]: + k * taps * C
                    col_stride = (int64_t)P.taps * P.C;
                }
                const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(j * 2 * P.bn);
                for (int c0 = 0; c0 < P.bn; c0 += 32) {
                    uint32_t rh[32], rl[32];
                    tmem_ld_32x32(t_addr + (uint32_t)c0, rh);
                    tmem_ld_32x32(t_addr + (uint32_t)(P.bn + c0), rl);
                    tmem_ld_wait();
                    if (!valid) continue;
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int64_t n = (int64_t)n0 + c0 + e;
                        if (n < P.N) {
                            const long long v = 256ll * (long long)(int)rh[e] + (long long)(int)rl[e];
                            atomicAdd(P.raw + base + n * col_stride, (unsigned long long)v);
                        }
                    }
                }
            }
        }
    }

    if (timed_out) {
        atomicExch(P.status, (int)QBP_ERR_TIMEOUT);
        __nanosleep(1000000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
}

// ------------------------------------------------------------ code sums
// Sums of stored codes per channel and per border class of the pixel the code
// sits at (bit 1: first row, 2: last row, 4: first column, 8: last column);
// a plain matrix (plain = 1) keeps every row in class 0.
// sums[cls][c] (int64, zeroed beforehand).
template <bool IS_SIGNED>
__global__ void __launch_bounds__(256) class_sums_kernel(const uint8_t *__restrict__ q, int64_t pixels, int H, int W,
                                                         int C, int plain, unsigned long long *__restrict__ sums)
{
    extern __shared__ int s_acc[];                       // [16][C]
    for (int i = threadIdx.x; i < 16 * C; i += 256) s_acc[i] = 0;
    __syncthreads();
    const int cv = C >> 4;                               // 16-byte groups per pixel
    const int tw = cv < 256 ? cv : 256;
    const int rpb = 256 / tw;
    const int tx = threadIdx.x % tw, ty = threadIdx.x / tw;
    if (ty < rpb) {
        for (int g = tx; g < cv; g += tw) {
            int interior[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) interior[e] = 0;
            for (int64_t p = (int64_t)blockIdx.x * rpb + ty; p < pixels; p += (int64_t)gridDim.x * rpb) {
                const int w = (int)(p % W), h = (int)((p / W) % H);
                // a plain matrix keeps everything in class 0
                const int cls = plain ? 0
                              : (h == 0 ? 1 : 0) | (h == H - 1 ? 2 : 0) | (w == 0 ? 4 : 0) | (w == W - 1 ? 8 : 0);
                uint4 v = __ldg(reinterpret_cast<const uint4 *>(q + p * C) + g);
                const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
                if (cls == 0) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            interior[k * 4 + b] += IS_SIGNED ? (int)(int8_t)(wd[k] >> (8 * b)) : (int)((wd[k] >> (8 * b)) & 0xFF);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            atomicAdd(&s_acc[cls * C + g * 16 + k * 4 + b],
                                      IS_SIGNED ? (int)(int8_t)(wd[k] >> (8 * b)) : (int)((wd[k] >> (8 * b)) & 0xFF));
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

// Applies the zero-points and dequantises:
//   acc = raw - zg * SX - zx * SG + count * zx * zg
// where SX / SG / count are taken over the positions at which the tap is inside
// the image.  Output element e: plain [k][n]; conv [k][tap][c].
__global__ void wgrad_finalize_kernel(const long long *__restrict__ raw, const long long *__restrict__ sx,
                                      const long long *__restrict__ shi, const long long *__restrict__ slo, int conv,
                                      int64_t total, int64_t Mrows, int64_t Nn, int64_t Kk, int Nimg, int H, int W,
                                      int pad, int R, int S, int C, const qbp_qparams *qx, const qbp_qparams *qg,
                                      long long *__restrict__ acc_out, float *__restrict__ dW)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const long long zx = qx->zero_point, zg = qg->zero_point;
    long long SX = 0, SG = 0, count = 0;
    if (!conv) {
        const int64_t k = e / Nn, n = e % Nn;
        for (int cls = 0; cls < 16; ++cls) {
            SX += sx[cls * Kk + k];
            SG += 256 * shi[cls * Nn + n] + slo[cls * Nn + n];
        }
        count = Mrows;
    } else {
        const int c = (int)(e % C);
        const int tap = (int)((e / C) % (R * S));
        const int k = (int)(e / ((int64_t)C * R * S));
        const int r = tap / S, s = tap % S;
        // positions of g that see this tap: p - pad + r in [0,H)  <=>  not (r<pad and first row), not (r>pad and last row);
        // positions of x that are seen:      h + pad - r in [0,H)  <=>  not (r<pad and last row),  not (r>pad and first row).
        for (int cls = 0; cls < 16; ++cls) {
            const bool top = cls & 1, bottom = cls & 2, left = cls & 4, right = cls & 8;
            const bool g_ok = !((r < pad && top) || (r > pad && bottom) || (s < pad && left) || (s > pad && right));
            const bool x_ok = !((r < pad && bottom) || (r > pad && top) || (s < pad && right) || (s > pad && left));
            if (g_ok) SG += 256 * shi[cls * Nn + k] + slo[cls * Nn + k];
            if (x_ok) SX += sx[cls * C + c];
        }
        const long long rows_ok = H - (r < pad ? pad - r : r - pad), cols_ok = W - (s < pad ? pad - s : s - pad);
        count = (long long)Nimg * (rows_ok > 0 ? rows_ok : 0) * (cols_ok > 0 ? cols_ok : 0);
    }
    const long long acc = raw[e] - zg * SX - zx * SG + count * zx * zg;
    if (acc_out) acc_out[e] = acc;
    if (dW) dW[e] = __fmul_rn((float)acc, __fmul_rn(qx->scale, qg->scale));
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

static bool wgrad_conv_supported(const qbp_conv_desc *d)
{
    return d->stride == 1 && d->R == d->S && (d->R == 1 || d->R == 3) && d->pad == (d->R - 1) / 2 && d->N > 0 &&
           d->H > 0 && d->W > 0 && d->C > 0 && d->K > 0 && d->C % 32 == 0 && d->K % 32 == 0;
}

static size_t wgrad_ws_bytes(const qbp_conv_desc *d, int64_t N, int64_t K)
{
    const int64_t outs = d ? (int64_t)d->K * d->R * d->S * d->C : K * N;
    const int64_t cx = d ? d->C : K, cg = d ? d->K : N;
    return 256 + align_up(sizeof(int64_t) * outs, 256) + align_up(sizeof(int64_t) * 16 * cx, 256) +
           2 * align_up(sizeof(int64_t) * 16 * cg, 256);
}

template <bool IS_SIGNED>
static int launch_class_sums(const void *q, int64_t pixels, int H, int W, int C, bool plain, int64_t *sums, cudaStream_t st)
{
    QBP_CUDA_OK(cudaMemsetAsync(sums, 0, sizeof(int64_t) * 16 * C, st));
    if ((size_t)C * 16 * sizeof(int) > 200 * 1024) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "wgrad: more than 3200 channels");
    const size_t smem = (size_t)C * 16 * sizeof(int);
    static thread_local bool configured[2] = {false, false};
    if (smem > 48 * 1024 && !configured[IS_SIGNED]) {
        QBP_CUDA_OK(cudaFuncSetAttribute(class_sums_kernel<IS_SIGNED>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        configured[IS_SIGNED] = true;
    }
    // int32 partials: a thread sees at most pixels / grid * 255 per channel
    const int cv = C / 16, tw = cv < 256 ? cv : 256, rpb = 256 / tw;
    int64_t grid = std::min<int64_t>((pixels + rpb - 1) / rpb, (int64_t)sm_count() * 4);
    grid = std::max<int64_t>(grid, pixels / (1 << 22) + 1);
    QBP_TRACE_BEGIN(st);
    class_sums_kernel<IS_SIGNED><<<(unsigned)grid, 256, smem, st>>>((const uint8_t *)q, pixels, H, W, C, plain ? 1 : 0, (unsigned long long *)sums);
    QBP_LAUNCH_OK("class_sums_kernel");
    return QBP_OK;
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) size_t qbp_wgrad_s16_workspace_bytes(const qbp_conv_desc *d, int64_t M,
                                                                                      int64_t N, int64_t K)
{
    (void)M;
    if (d && !wgrad_conv_supported(d)) return 0;
    return wgrad_ws_bytes(d, N > 0 ? N : 1, K > 0 ? K : 1);
}

extern "C" __attribute__((visibility("default"))) int qbp_wgrad_s16(const qbp_conv_desc *d, int64_t M, int64_t N, int64_t K,
                                                                   const int8_t *x, const qbp_qparams *qx,
                                                                   const int8_t *g_hi, const uint8_t *g_lo,
                                                                   const qbp_qparams *qg16, int64_t *acc_out, float *dW,
                                                                   void *ws, size_t ws_bytes, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
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
    }
    if (!ws || ws_bytes < wgrad_ws_bytes(d, N, K))
        return fail(QBP_ERR_WORKSPACE, "wgrad_s16: workspace of %zu bytes needed, %zu given", wgrad_ws_bytes(d, N, K), ws_bytes);

    const int64_t outs = d ? (int64_t)d->K * d->R * d->S * d->C : K * N;
    WsCarver w(ws, ws_bytes);
    int *status = w.take<int>(1);
    int64_t *raw = w.take<int64_t>(outs);
    int64_t *sx = w.take<int64_t>(16 * K);
    int64_t *shi = w.take<int64_t>(16 * N);
    int64_t *slo = w.take<int64_t>(16 * N);

    const int Hc = d ? d->H : 1, Wc = d ? d->W : 1;
    int rc = launch_class_sums<true>(x, M, Hc, Wc, (int)K, d == nullptr, sx, st);
    if (rc) return rc;
    rc = launch_class_sums<true>(g_hi, M, Hc, Wc, (int)N, d == nullptr, shi, st);
    if (rc) return rc;
    rc = launch_class_sums<false>(g_lo, M, Hc, Wc, (int)N, d == nullptr, slo, st);
    if (rc) return rc;
    QBP_CUDA_OK(cudaMemsetAsync(raw, 0, sizeof(int64_t) * outs, st));
    QBP_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));

    WgradParams P{};
    P.conv = d ? 1 : 0;
    P.M = M; P.N = N; P.K = K;
    P.raw = (unsigned long long *)raw; P.status = status;
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
    // A tiles per CTA: as many as tensor memory holds (two accumulators of bn columns each)
    P.ma = std::max(1, std::min({kWgMaxTiles, 512 / (2 * P.bn), P.a_tiles}));
    P.a_groups = (P.a_tiles + P.ma - 1) / P.ma;
    int cols = 32; while (cols < P.ma * 2 * P.bn) cols <<= 1;
    P.tmem_cols = cols;
    // reduction rows per stage: 128, or 64 when that is what it takes to keep four stages in flight
    uint32_t kr = 128;
    if ((200u * 1024u) / (kr * (rb_a * P.a_chunks * P.ma + 2 * rb_b)) < 4) kr = 64;
    P.kr = (int)kr;
    P.a_chunk_bytes = kr * rb_a;
    P.a = layout_mnmajor(kr, rb_a, (uint32_t)P.a_chunks, P.a_chunk_bytes);
    P.b = layout_mnmajor(kr, rb_b, 1, 0);
    P.idesc_hi = make_idesc(true, true, 1, 1, 128, (uint32_t)P.bn);
    P.idesc_lo = make_idesc(true, false, 1, 1, 128, (uint32_t)P.bn);

    if (!d) {
        P.iters_total = (int)((M + kr - 1) / kr);
        if ((rc = make_map_2d(&P.mapX, x, M, K, kr, rb_a))) return rc;
        if ((rc = make_map_2d(&P.mapHi, g_hi, M, N, kr, rb_b))) return rc;
        if ((rc = make_map_2d(&P.mapLo, g_lo, M, N, kr, rb_b))) return rc;
    } else {
        int bwl = 0, bhl = 0;
        pick_pixel_box_w((int)kr, d->N, d->H, d->W, bwl, bhl);
        P.bw_log2 = bwl; P.bh_log2 = bhl;
        const int bw = 1 << bwl, bh = 1 << bhl, bn_img = (int)kr >> (bwl + bhl);
        P.tiles_w = (d->W + bw - 1) / bw; P.tiles_h = (d->H + bh - 1) / bh;
        P.iters_total = P.tiles_w * P.tiles_h * ((d->N + bn_img - 1) / bn_img);
        if ((rc = make_map_nhwc(&P.mapX, x, d->N, d->H, d->W, d->C, bn_img, bh, bw, rb_a))) return rc;
        if ((rc = make_map_nhwc(&P.mapHi, g_hi, d->N, d->H, d->W, d->K, bn_img, bh, bw, rb_b))) return rc;
        if ((rc = make_map_nhwc(&P.mapLo, g_lo, d->N, d->H, d->W, d->K, bn_img, bh, bw, rb_b))) return rc;
    }
    // split the reduction: at most 65536 rows per CTA, and enough CTAs to fill the machine twice
    const int out_items = P.a_groups * P.tiles_b;
    const int max_iters = 65536 / (int)kr;
    int slices = (P.iters_total + max_iters - 1) / max_iters;
    slices = std::max(slices, std::min(P.iters_total, std::max(1, 2 * sm_count() / out_items)));
    P.slices = std::max(1, slices);

    const uint32_t stage_bytes = P.a_chunk_bytes * P.a_chunks * P.ma + 2 * P.b.tile_bytes;
    int stages = std::max(2, std::min<int>(kWgMaxStages, (200 * 1024) / stage_bytes));
    P.stages = stages;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    static thread_local bool configured = false;
    if (!configured) {
        QBP_CUDA_OK(cudaFuncSetAttribute(qbp_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        configured = true;
    }
    QBP_TRACE_BEGIN(st);
    qbp_wgrad_kernel<<<P.slices * out_items, kWgThreads, smem, st>>>(P);
    QBP_LAUNCH_OK("qbp_wgrad_kernel");

    const int blocks = (int)((outs + 255) / 256);
    QBP_TRACE_BEGIN(st);
    wgrad_finalize_kernel<<<blocks, 256, 0, st>>>((const long long *)raw, (const long long *)sx, (const long long *)shi,
                                                  (const long long *)slo, P.conv, outs, M, N, K, d ? d->N : 0, Hc, Wc,
                                                  d ? d->pad : 0, d ? d->R : 1, d ? d->S : 1, d ? d->C : (int)K, qx, qg16,
                                                  (long long *)acc_out, dW);
    QBP_LAUNCH_OK("wgrad_finalize_kernel");
    return QBP_OK;
}
