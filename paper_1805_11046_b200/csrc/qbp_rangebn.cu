// Range Batch-Normalization (Section 3, Eq. (range)) forward and backward
// (Section 7: derivative of max/min is one where attained).
//
// Both directions are two streaming passes over [n x C] fp32 with the channel
// innermost: a statistics pass (per-channel min, max, sum -- or sum dy,
// sum dy*xhat) and an apply pass, with a one-warp-per-channel combine between
// them.  Sums are carried in fp64 per thread (the fp64 pipe is far from being
// the limit at HBM rate); everything an element's value depends on follows a
// fixed fp32 operation order so that forward and backward agree on which
// outputs the ReLU kept.
#include "qbp_colscan.cuh"
#include "qbp_mma.cuh"

#include <cmath>

namespace qbp {

// ---------------------------------------------------------------- forward
template <int VEC>
__global__ void __launch_bounds__(kScanThreads) bn_stats_kernel(const float *__restrict__ x, int64_t rows, int C, int tw,
                                                                float *__restrict__ part_lo, float *__restrict__ part_hi,
                                                                double *__restrict__ part_sum)
{
    const ScanPos p = scan_pos<VEC>(C, tw);
    const int rpb = kScanThreads / tw;
    float lo[VEC], hi[VEC];
    double sum[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) { lo[e] = INFINITY; hi[e] = -INFINITY; sum[e] = 0.0; }
    if (p.active) {
        const int64_t step = (int64_t)gridDim.x * rpb;
        for (int64_t r0 = (int64_t)blockIdx.x * rpb + p.ty; r0 < rows; r0 += step * kScanUnroll) {
            VecF<VEC> v[kScanUnroll];
            bool ok[kScanUnroll];
#pragma unroll
            for (int u = 0; u < kScanUnroll; ++u) {
                int64_t r = r0 + u * step;
                ok[u] = r < rows;
                if (ok[u]) v[u].load_stream(x + r * C + p.col);
            }
#pragma unroll
            for (int u = 0; u < kScanUnroll; ++u)
                if (ok[u]) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        lo[e] = fminf(lo[e], v[u].v[e]);
                        hi[e] = fmaxf(hi[e], v[u].v[e]);
                        sum[e] += (double)v[u].v[e];
                    }
                }
        }
    }
    __shared__ float s_lo[kScanThreads * VEC], s_hi[kScanThreads * VEC];
    __shared__ double s_sum[kScanThreads * VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        s_lo[threadIdx.x * VEC + e] = lo[e]; s_hi[threadIdx.x * VEC + e] = hi[e]; s_sum[threadIdx.x * VEC + e] = sum[e];
    }
    __syncthreads();
    if (p.ty == 0 && p.active) {
        for (int y = 1; y < rpb; ++y)
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                const int i = (y * tw + p.tx) * VEC + e;
                lo[e] = fminf(lo[e], s_lo[i]); hi[e] = fmaxf(hi[e], s_hi[i]); sum[e] += s_sum[i];
            }
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const int64_t i = (int64_t)blockIdx.x * C + p.col + e;
            part_lo[i] = lo[e]; part_hi[i] = hi[e]; part_sum[i] = sum[e];
        }
    }
}

// One block of 128 threads per channel: mean (or, with sum_out, the raw fp64 sum for a later combination over
// several GPUs), min, max.
__global__ void __launch_bounds__(128) bn_stats_finalize_kernel(const float *__restrict__ part_lo,
                                                                const float *__restrict__ part_hi,
                                                                const double *__restrict__ part_sum, int nparts, int C,
                                                                int64_t n, float *__restrict__ mean,
                                                                float *__restrict__ vmin, float *__restrict__ vmax,
                                                                double *__restrict__ sum_out)
{
    const int c = blockIdx.x;
    float lo = INFINITY, hi = -INFINITY;
    double sum = 0.0;
    for (int i = threadIdx.x; i < nparts; i += 128) {
        lo = fminf(lo, part_lo[(int64_t)i * C + c]);
        hi = fmaxf(hi, part_hi[(int64_t)i * C + c]);
        sum += part_sum[(int64_t)i * C + c];
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
        if (mean) mean[c] = (float)(sum / (double)n);
        if (sum_out) sum_out[c] = sum;
        vmin[c] = lo; vmax[c] = hi;
    }
}

// Mean from a (possibly all-reduced) per-channel sum over n rows; min and max are copied alongside.
__global__ void bn_mean_from_sum_kernel(const double *__restrict__ col_sum, const float *__restrict__ col_min,
                                        const float *__restrict__ col_max, int C, int64_t n, float *__restrict__ mean,
                                        float *__restrict__ vmin, float *__restrict__ vmax)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    mean[c] = (float)(col_sum[c] / (double)n);
    vmin[c] = col_min[c]; vmax[c] = col_max[c];
}

// Requantisation of the output for the next layer (Section 4: the range of an activation that a Range BN produced
// is known from its statistics, so quantising it costs no scan): with rq, the 8-bit codes of y (nearest rounding,
// parameters *rq) are written beside y, or instead of it (y == NULL); rowsum (nullable; rs_group = lanes per row,
// a power of two <= 32 that covers the row) receives each row's sum of stored codes, which the next product's
// zero-point correction needs.
// chansum (nullable, [C], added to with 64-bit atomics): per-channel totals of the stored codes over all rows.
struct BnRequant { const qbp_qparams *rq; int8_t *q; int32_t *rowsum; int rs_group; unsigned long long *chansum; };

template <int VEC, bool RELU, bool REQUANT>
__global__ void __launch_bounds__(kScanThreads) bn_apply_kernel(const float *__restrict__ x, int64_t rows, int C, int tw,
                                                                const float *__restrict__ mean,
                                                                const float *__restrict__ vmin,
                                                                const float *__restrict__ vmax,
                                                                const float *__restrict__ gamma,
                                                                const float *__restrict__ beta, float Cn,
                                                                float *__restrict__ y, BnRequant R, int reverse)
{
    const ScanPos p = scan_pos<VEC>(C, tw);
    // (with row sums the idle threads of a ragged last slab take part in the shuffles: tw <= 32 then, one slab)
    if (!p.active && !(REQUANT && (R.rowsum || R.chansum))) return;
    const int rpb = kScanThreads / tw;
    float mu[VEC], s[VEC], g[VEC], b[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const int c = p.active ? p.col + e : 0;
        mu[e] = mean[c];
        s[e] = bn_scale(vmin[c], vmax[c], Cn);
        g[e] = gamma ? gamma[c] : 1.0f;
        b[e] = beta ? beta[c] : 0.0f;
    }
    float inv = 0.0f, zp_u = 0.0f;
    if (REQUANT) { inv = __fdiv_rn(1.0f, R.rq->scale); zp_u = (float)(R.rq->zero_point + 128); }
    int cs[VEC];                                            // totals of the stored codes of this thread's channels
#pragma unroll
    for (int e = 0; e < VEC; ++e) cs[e] = 0;
    const int64_t step = (int64_t)gridDim.x * rpb;
    // (the loop bound is the same for every thread of the block, so that the shuffles below see whole warps)
    for (int64_t rb = (int64_t)blockIdx.x * rpb; rb < rows; rb += step * kScanUnroll) {
        const int64_t r0 = rb + p.ty;
        VecF<VEC> v[kScanUnroll];
        bool ok[kScanUnroll];
#pragma unroll
        for (int u = 0; u < kScanUnroll; ++u) {
            int64_t r = r0 + u * step;
            ok[u] = p.active && r < rows;
            // (reverse: rows from the last to the first, when the kernel that wrote x ran just before and has left the
            // tail of x in the L2)
            if (ok[u]) v[u].load_stream(x + (reverse ? rows - 1 - r : r) * C + p.col);
        }
#pragma unroll
        for (int u = 0; u < kScanUnroll; ++u) {
            int rs = 0;
            if (ok[u]) {
                uint32_t code[VEC];
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    float yv = bn_y(bn_xhat(v[u].v[e], mu[e], s[e]), g[e], b[e]);
                    v[u].v[e] = RELU ? fmaxf(yv, 0.0f) : yv;
                    if (REQUANT) code[e] = (uint32_t)quantize_code<false>(v[u].v[e], inv, zp_u, 255.0f, 0u);
                }
                const int64_t at = (reverse ? rows - 1 - (r0 + u * step) : r0 + u * step) * C + p.col;
                if (y) v[u].store_stream(y + at);
                if (REQUANT) {
                    if (VEC == 4) {
                        const uint32_t packed = (code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24)) ^ 0x80808080u;
                        *reinterpret_cast<uint32_t *>(R.q + at) = packed;
                        rs = __dp4a((int)packed, 0x01010101, 0);
                        if (R.chansum) {
#pragma unroll
                            for (int e = 0; e < VEC; ++e) cs[e] = __dp4a((int)packed, 1 << (8 * (e & 3)), cs[e]);
                        }
                    } else {
                        R.q[at] = (int8_t)((int)code[0] - 128);
                        rs = (int)code[0] - 128;
                        cs[0] += rs;
                    }
                }
            }
            if (REQUANT && R.rowsum) {
                // a row is rs_group consecutive lanes of one warp (idle lanes add nothing)
                for (int off = 16; off > 0; off >>= 1)
                    if (off < R.rs_group) rs += __shfl_xor_sync(0xffffffffu, rs, off);
                const int64_t r = r0 + u * step;
                if (p.tx == 0 && r < rows) R.rowsum[reverse ? rows - 1 - r : r] = rs;
            }
        }
    }
    if (REQUANT && R.chansum) {
        // the block's threads meet in shared memory (fewer than 2^22 rows: int32 is enough), then one atomic per channel
        __shared__ int s_tot[kScanMaxTw * 4];
        for (int i = threadIdx.x; i < tw * VEC; i += kScanThreads) s_tot[i] = 0;
        __syncthreads();
        if (p.active) {
#pragma unroll
            for (int e = 0; e < VEC; ++e)
                if (cs[e]) atomicAdd(&s_tot[p.tx * VEC + e], cs[e]);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < tw * VEC; i += kScanThreads) {
            const int c = (int)blockIdx.y * tw * VEC + i;
            if (c < C && s_tot[i]) atomicAdd(R.chansum + c, (unsigned long long)(long long)s_tot[i]);
        }
    }
}

// Exact range of y over the whole tensor from the per-channel statistics:
// y is a non-decreasing (gamma >= 0) or non-increasing function of x computed
// with the same rounded operations, so its extremes sit at x = min and x = max.
__global__ void __launch_bounds__(256) bn_out_range_kernel(const float *__restrict__ mean, const float *__restrict__ vmin,
                                                           const float *__restrict__ vmax,
                                                           const float *__restrict__ gamma,
                                                           const float *__restrict__ beta, int C, float Cn, int relu,
                                                           qbp_qparams *__restrict__ out, qbp_qparams *__restrict__ qp8_out,
                                                           float4 *__restrict__ fold)
{
    float lo = INFINITY, hi = -INFINITY;
    for (int c = threadIdx.x; c < C; c += 256) {
        float s = bn_scale(vmin[c], vmax[c], Cn);
        float g = gamma ? gamma[c] : 1.0f, b = beta ? beta[c] : 0.0f;
        if (fold) fold[c] = make_float4(mean[c], s, g, b);      // what a product's epilogue needs to normalise a column
        float a = bn_y(bn_xhat(vmin[c], mean[c], s), g, b);
        float z = bn_y(bn_xhat(vmax[c], mean[c], s), g, b);
        if (relu) { a = fmaxf(a, 0.0f); z = fmaxf(z, 0.0f); }
        lo = fminf(lo, fminf(a, z)); hi = fmaxf(hi, fmaxf(a, z));
    }
    lo = warp_min(lo); hi = warp_max(hi);
    __shared__ float s_lo[8], s_hi[8];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 0; w < 8; ++w) { lo = fminf(lo, s_lo[w]); hi = fmaxf(hi, s_hi[w]); }
        if (out) { out->scale = 0.0f; out->zero_point = 0; out->vmin = lo; out->vmax = hi; }
        if (qp8_out) *qp8_out = make_qparams(lo, hi, 8);
    }
}

// --------------------------------------------------------------- backward
// EXT: also the extremes of the (rectifier-masked) dy of each channel over three sets of positions -- where x is the
// channel's maximum, where it is its minimum, and everywhere else -- as ext [6][blocks][C] (min, max of the ordinary
// positions, then of the maxima, then of the minima).  dx is a monotone function of dy on each set (bn_dx), so the
// finalize kernel knows the exact range of dx from these, before dx is computed.
template <int VEC, bool RELU, bool EXT>
__global__ void __launch_bounds__(kScanThreads) bn_bwd_stats_kernel(const float *__restrict__ dy,
                                                                    const float *__restrict__ x, int64_t rows, int C,
                                                                    int tw, const float *__restrict__ mean,
                                                                    const float *__restrict__ vmin,
                                                                    const float *__restrict__ vmax,
                                                                    const float *__restrict__ gamma,
                                                                    const float *__restrict__ beta, float Cn,
                                                                    double *__restrict__ part_dy,
                                                                    double *__restrict__ part_dyx,
                                                                    float *__restrict__ ext)
{
    const ScanPos p = scan_pos<VEC>(C, tw);
    const int rpb = kScanThreads / tw;
    double sdy[VEC], sdyx[VEC];
    // (the extremes of the ordinary positions in registers; those of the few positions at a channel's maximum or
    // minimum in shared memory, as integers that order like the floats)
    float elo[VEC], ehi[VEC];
    __shared__ int s_tie[EXT ? 4 * kScanThreads * VEC / 4 : 1];      // [min at max, max at max, min at min, max at min][tw * VEC]
#pragma unroll
    for (int e = 0; e < VEC; ++e) { sdy[e] = 0.0; sdyx[e] = 0.0; elo[e] = INFINITY; ehi[e] = -INFINITY; }
    if (EXT) {
        for (int i = threadIdx.x; i < 4 * tw * VEC; i += kScanThreads) s_tie[i] = ((i / (tw * VEC)) & 1) ? float_order(-INFINITY) : float_order(INFINITY);
        __syncthreads();
    }
    if (p.active) {
        float mu[VEC], s[VEC], g[VEC], b[VEC], lo[VEC], hi[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            mu[e] = mean[p.col + e];
            lo[e] = vmin[p.col + e]; hi[e] = vmax[p.col + e];
            s[e] = bn_scale(lo[e], hi[e], Cn);
            g[e] = gamma ? gamma[p.col + e] : 1.0f;
            b[e] = beta ? beta[p.col + e] : 0.0f;
        }
        const int64_t step = (int64_t)gridDim.x * rpb;
        for (int64_t r0 = (int64_t)blockIdx.x * rpb + p.ty; r0 < rows; r0 += step * kScanUnroll) {
            VecF<VEC> vx[kScanUnroll], vd[kScanUnroll];
            bool ok[kScanUnroll];
#pragma unroll
            for (int u = 0; u < kScanUnroll; ++u) {
                int64_t r = r0 + u * step;
                ok[u] = r < rows;
                if (ok[u]) { vx[u].load_stream(x + r * C + p.col); vd[u].load_stream(dy + r * C + p.col); }
            }
            // (the few rows of one step are added in fp32, the steps in fp64: a quarter of the conversions and fp64
            // additions, and an error of a few ulp of four terms)
            float fs[VEC], fp[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) { fs[e] = 0.0f; fp[e] = 0.0f; }
#pragma unroll
            for (int u = 0; u < kScanUnroll; ++u)
                if (ok[u]) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        float xh = bn_xhat(vx[u].v[e], mu[e], s[e]);
                        float d = vd[u].v[e];
                        if (RELU && !(bn_y(xh, g[e], b[e]) > 0.0f)) d = 0.0f;
                        fs[e] += d;
                        fp[e] = fmaf(d, xh, fp[e]);
                        if (EXT) {
                            const bool ih = vx[u].v[e] == hi[e], il = vx[u].v[e] == lo[e];
                            if (ih == il) { elo[e] = fminf(elo[e], d); ehi[e] = fmaxf(ehi[e], d); }
                            else {
                                int *t = s_tie + (ih ? 0 : 2) * tw * VEC + p.tx * VEC + e;
                                atomicMin(t, float_order(d)); atomicMax(t + tw * VEC, float_order(d));
                            }
                        }
                    }
                }
#pragma unroll
            for (int e = 0; e < VEC; ++e) { sdy[e] += (double)fs[e]; sdyx[e] += (double)fp[e]; }
        }
    }
    __shared__ double s_ab[2 * kScanThreads * VEC];
    double *s_a = s_ab, *s_b = s_ab + kScanThreads * VEC;
#pragma unroll
    for (int e = 0; e < VEC; ++e) { s_a[threadIdx.x * VEC + e] = sdy[e]; s_b[threadIdx.x * VEC + e] = sdyx[e]; }
    __syncthreads();
    if (p.ty == 0 && p.active) {
        for (int y = 1; y < rpb; ++y)
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                sdy[e] += s_a[(y * tw + p.tx) * VEC + e];
                sdyx[e] += s_b[(y * tw + p.tx) * VEC + e];
            }
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            part_dy[(int64_t)blockIdx.x * C + p.col + e] = sdy[e];
            part_dyx[(int64_t)blockIdx.x * C + p.col + e] = sdyx[e];
        }
    }
    if (EXT) {
        // the block's rows meet in shared memory (the arrays of the sums, read by now, hold two tables each)
        float *s_f = reinterpret_cast<float *>(s_ab);          // room for four tables of kScanThreads * VEC floats
        static_assert(sizeof(double) == 2 * sizeof(float), "two float tables per double table");
        __syncthreads();
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            s_f[threadIdx.x * VEC + e] = elo[e];
            s_f[(kScanThreads + threadIdx.x) * VEC + e] = ehi[e];
        }
        __syncthreads();
        if (p.ty == 0 && p.active) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                float lo0 = elo[e], hi0 = ehi[e];
                for (int y = 1; y < rpb; ++y) {
                    lo0 = fminf(lo0, s_f[(y * tw + p.tx) * VEC + e]);
                    hi0 = fmaxf(hi0, s_f[(kScanThreads + y * tw + p.tx) * VEC + e]);
                }
                const int64_t at = (int64_t)blockIdx.x * C + p.col + e, tbl = (int64_t)gridDim.x * C;
                ext[at] = lo0; ext[tbl + at] = hi0;
#pragma unroll
                for (int k = 0; k < 4; ++k) ext[(2 + k) * tbl + at] = order_float(s_tie[k * tw * VEC + p.tx * VEC + e]);
            }
        }
    }
}

// One block of 128 threads per channel: dbeta, dgamma, and the two per-channel
// constants of dx: m1 = gamma*dbeta/n, k2 = C(n)*gamma*dgamma.
__global__ void __launch_bounds__(128) bn_bwd_finalize_kernel(const double *__restrict__ part_dy,
                                                              const double *__restrict__ part_dyx, int nparts, int C,
                                                              int64_t n, const float *__restrict__ gamma, double Cn,
                                                              float *__restrict__ dgamma, float *__restrict__ dbeta,
                                                              float2 *__restrict__ coef, double *__restrict__ sum_dy,
                                                              double *__restrict__ sum_dyx,
                                                              const float *__restrict__ ext = nullptr,
                                                              const float *__restrict__ vmin = nullptr,
                                                              const float *__restrict__ vmax = nullptr, float Cn_f = 0.0f,
                                                              float2 *__restrict__ chan_range = nullptr,
                                                              const float *__restrict__ mean = nullptr,
                                                              const float *__restrict__ beta = nullptr,
                                                              float2 *__restrict__ relu_thr = nullptr)
{
    const int c = blockIdx.x;
    double a = 0.0, b = 0.0;
    for (int i = threadIdx.x; i < nparts; i += 128) {
        const double pa_ = part_dy[(int64_t)i * C + c], pb_ = part_dyx[(int64_t)i * C + c];
        a += pa_; b += pb_;
    }
    // ext (see bn_bwd_stats_kernel): the extremes of dy over the three sets of positions, then (below) the exact range
    // of this channel's dx, left in chan_range[c] for the quantiser of the gradient
    float ev[6];
    __shared__ float s_e[6][4];
    if (ext) {
#pragma unroll
        for (int k = 0; k < 6; ++k) ev[k] = (k & 1) ? -INFINITY : INFINITY;
        for (int i = threadIdx.x; i < nparts; i += 128) {
            float o[6];
#pragma unroll
            for (int k = 0; k < 6; ++k) o[k] = ext[((int64_t)k * nparts + i) * C + c];
#pragma unroll
            for (int k = 0; k < 6; ++k) ev[k] = (k & 1) ? fmaxf(ev[k], o[k]) : fminf(ev[k], o[k]);
        }
#pragma unroll
        for (int k = 0; k < 6; ++k) {
            ev[k] = (k & 1) ? warp_max(ev[k]) : warp_min(ev[k]);
            if ((threadIdx.x & 31) == 0) s_e[k][threadIdx.x >> 5] = ev[k];
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    __shared__ double s_a[4], s_b[4];
    if ((threadIdx.x & 31) == 0) { s_a[threadIdx.x >> 5] = a; s_b[threadIdx.x >> 5] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 4; ++w) { a += s_a[w]; b += s_b[w]; }
        if (sum_dy) {                       // raw sums only: combined over several GPUs before the coefficients
            sum_dy[c] = a; sum_dyx[c] = b;
            return;
        }
        const double g = gamma ? (double)gamma[c] : 1.0;
        if (dbeta) dbeta[c] = (float)a;
        if (dgamma) dgamma[c] = (float)b;
        const float m1 = (float)(g * a / (double)n), k2 = (float)(Cn * g * b);
        coef[c] = make_float2(m1, k2);
        if (ext) {
            const float s = bn_scale(vmin[c], vmax[c], Cn_f), gf = gamma ? gamma[c] : 1.0f;
            float rlo = INFINITY, rhi = -INFINITY;
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                float lo = ev[2 * k], hi = ev[2 * k + 1];
                for (int w = 1; w < 4; ++w) { lo = fminf(lo, s_e[2 * k][w]); hi = fmaxf(hi, s_e[2 * k + 1][w]); }
                if (lo <= hi) {              // (a set with no position keeps +inf, -inf)
                    const float ind = k == 0 ? 0.0f : k == 1 ? 1.0f : -1.0f;
                    const float v0 = bn_dx(lo, ind, s, gf, m1, k2), v1 = bn_dx(hi, ind, s, gf, m1, k2);
                    rlo = fminf(rlo, fminf(v0, v1)); rhi = fmaxf(rhi, fmaxf(v0, v1));
                }
            }
            chan_range[c] = make_float2(rlo, rhi);
            // (the rectifier's mask of this channel as a threshold on x, for the pass that follows)
            if (relu_thr) relu_thr[c] = relu_threshold(mean[c], s, gf, beta ? beta[c] : 0.0f);
        }
    }
}

// The Range BN backward apply pass and the bifurcation of the gradient it computes (Sections 3 and 6) in one pass:
// dx goes from registers into its 8-bit copy (stochastic rounding), the two limbs of its 16-bit copy and each row's
// 8-bit code sum; the fp32 dx itself is written only when the caller keeps it (g_out).  The parameters of both copies
// are known beforehand (bn_bwd_finalize_kernel + the range finalize).  Element i of the [rows x C] tensor draws from
// Philox block i / 4 as in quantize_kernel: a thread's four channels are one block.  rowsum8: a row's lanes
// of one warp add up by shuffles; when a row spans several warps or blocks (tw > 32 or several slabs) the pieces are added
// to rowsum8 [rows], zeroed beforehand.
// TOTALS: also each channel's total of the stored 16-bit codes (256 * hi + lo with lo unsigned, whatever lo_flip) over
// all rows, added to chansum16 [C] (zeroed beforehand): a thread keeps its four channels for its whole life, a block
// adds its threads' totals in shared memory and ends with one 64-bit atomic per channel.
// The pass is bound by arithmetic (Philox), and a thread that computes has no load in flight: the operands come through a
// ring in shared memory, filled by each thread's own asynchronous copies kBabSlots - 1 steps ahead of the step it
// computes (a thread reads back only what it copied itself: no barrier), so the memory system always has work.
constexpr int kBabUnroll = 2;     // rows per thread and step (two operands each)
constexpr int kBabSlots = 3;      // ring depth in steps
constexpr size_t kBabRingBytes = (size_t)kBabSlots * kBabUnroll * 2 * kScanThreads * sizeof(float4);
template <bool RELU, bool STORE_G, bool TOTALS>
__global__ void __launch_bounds__(kScanThreads, 3) bn_bwd_apply_bifurcate_kernel(
    const float *__restrict__ dy, const float *__restrict__ x, int64_t rows, int C, int tw, const float *__restrict__ mean,
    const float *__restrict__ vmin, const float *__restrict__ vmax, const float *__restrict__ gamma,
    const float *__restrict__ beta, float Cn, const float2 *__restrict__ coef, float *__restrict__ g_out,
    const qbp_qparams *__restrict__ qp8, const qbp_qparams *__restrict__ qp16, uint32_t id8, uint32_t id16,
    const __grid_constant__ PhiloxKeys keys, uint32_t *__restrict__ q8, uint32_t *__restrict__ q_hi, uint32_t *__restrict__ q_lo,
    uint32_t lo_flip, int32_t *__restrict__ rowsum8, unsigned long long *__restrict__ chansum16,
    const float2 *__restrict__ relu_thr)
{
    const bool rowsum_pieces = tw > 32 || gridDim.y > 1;
    const ScanPos p = scan_pos<4>(C, tw);
    uint32_t cs16[4] = {0u, 0u, 0u, 0u};          // unsigned codes of this thread's rows (fewer than 65536 rows)
    int mine = 0;
    const int rpb = kScanThreads / tw;
    float s[4], g[4], lo[4], hi[4], m1[4], k2[4], thr[4], tsg[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int c = p.active ? p.col + e : 0;
        lo[e] = vmin[c]; hi[e] = vmax[c];
        s[e] = bn_scale(lo[e], hi[e], Cn);
        g[e] = gamma ? gamma[c] : 1.0f;
        const float2 cf = coef[c];
        m1[e] = cf.x; k2[e] = cf.y;
        const float2 th = RELU ? relu_thr[c] : make_float2(0.0f, 1.0f);   // (the mask y > 0 as sgn * x >= threshold)
        thr[e] = th.x; tsg[e] = th.y;
    }
    // both codes in fixed point with 16 fraction bits (quantize_sr8_byte2 / quantize_sr16_top_half)
    const float inv8 = __fdiv_rn(1.0f, qp8->scale) * 65536.0f, zp8 = (float)(qp8->zero_point + 128) * 65536.0f;
    const float inv16 = __fdiv_rn(1.0f, qp16->scale) * 65536.0f, zp16 = (float)(qp16->zero_point + 32768) * 65536.0f;
    const bool one_block = id8 == id16;
    const int64_t step = (int64_t)gridDim.x * rpb;
    // (the loop bound is the block's: every lane takes part in the row-sum shuffles)
    extern __shared__ __align__(16) float4 bab_ring[];         // [slot][row of the step][x | dy][thread]
    float4 *const mine_ring = bab_ring + threadIdx.x;
    const int64_t stride = step * kBabUnroll;
    auto fetch = [&](int64_t base, int slot) {
#pragma unroll
        for (int u = 0; u < kBabUnroll; ++u) {
            const int64_t r = base + p.ty + u * step;
            if (p.active && r < rows) {
                cp_async16(mine_ring + ((slot * kBabUnroll + u) * 2 + 0) * kScanThreads, x + r * C + p.col);
                cp_async16(mine_ring + ((slot * kBabUnroll + u) * 2 + 1) * kScanThreads, dy + r * C + p.col);
            }
        }
        cp_async_commit();                                     // (a group per step, empty past the end: the count below is uniform)
    };
#pragma unroll
    for (int k = 0; k < kBabSlots - 1; ++k) fetch((int64_t)blockIdx.x * rpb + k * stride, k);
    int slot = 0;
    for (int64_t base = (int64_t)blockIdx.x * rpb; base < rows; base += stride) {
        const int64_t r0 = base + p.ty;
        // the slot this thread emptied in the step before takes the step kBabSlots - 1 ahead; then this step's data is in
        fetch(base + (kBabSlots - 1) * stride, slot == 0 ? kBabSlots - 1 : slot - 1);
        cp_async_wait<kBabSlots - 1>();
#pragma unroll
        for (int u = 0; u < kBabUnroll; ++u) {
            const int64_t r = r0 + u * step;
            const bool ok_u = p.active && r < rows;
            int rs = 0;
            if (ok_u) {
                const float4 fx = mine_ring[((slot * kBabUnroll + u) * 2 + 0) * kScanThreads];
                const float4 fd = mine_ring[((slot * kBabUnroll + u) * 2 + 1) * kScanThreads];
                const float ax[4] = {fx.x, fx.y, fx.z, fx.w}, ad[4] = {fd.x, fd.y, fd.z, fd.w};
                float v[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float xv = ax[e];
                    float d = ad[e];
                    if (RELU && !(__fmul_rn(tsg[e], xv) >= thr[e])) d = 0.0f;
                    const float ind = (xv == hi[e] ? 1.0f : 0.0f) - (xv == lo[e] ? 1.0f : 0.0f);
                    v[e] = bn_dx(d, ind, s[e], g[e], m1[e], k2[e]);
                }
                const int64_t j = (r * C + p.col) >> 2;                 // the thread's Philox block = its float4's index
                if (STORE_G) __stcs(reinterpret_cast<float4 *>(g_out) + j, make_float4(v[0], v[1], v[2], v[3]));
                const uint4 r8 = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)((uint64_t)j >> 32), id8, 0u), keys);
                const uint4 r16 = one_block ? r8 : philox4x32_10(make_uint4((uint32_t)j, (uint32_t)((uint64_t)j >> 32), id16, 0u), keys);
                const uint32_t w8[4] = {r8.x, r8.y, r8.z, r8.w}, w16[4] = {r16.x, r16.y, r16.z, r16.w};
                uint32_t c8[4], c16[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    c8[e] = quantize_sr8_byte2(v[e], inv8, zp8, w8[e]);
                    c16[e] = quantize_sr16_top_half(v[e], inv16, zp16, w16[e]);
                }
                // the 8-bit codes are byte 2 of each word; the 16-bit codes bytes 3 (high) and 2 (low)
                const uint32_t packed = __byte_perm(__byte_perm(c8[0], c8[1], 0x0062), __byte_perm(c8[2], c8[3], 0x0062), 0x5410) ^ 0x80808080u;
                q8[j] = packed;
                const uint32_t t01 = __byte_perm(c16[0], c16[1], 0x7362), t23 = __byte_perm(c16[2], c16[3], 0x7362);
                q_hi[j] = __byte_perm(t01, t23, 0x7632) ^ 0x80808080u;
                q_lo[j] = __byte_perm(t01, t23, 0x5410) ^ lo_flip;
                rs = __dp4a((int)packed, 0x01010101, 0);
                if (TOTALS) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) cs16[e] += c16[e] >> 16;
                    ++mine;
                }
            }
            if (rowsum8) {
                for (int off = 16; off > 0; off >>= 1)
                    if (off < tw) rs += __shfl_xor_sync(0xffffffffu, rs, off);
                // (a row wider than a warp's lanes, or than the block: each piece is added to the zeroed sum)
                if (ok_u && (p.tx & 31) == 0) {
                    if (rowsum_pieces) atomicAdd(rowsum8 + r, rs);
                    else rowsum8[r] = rs;
                }
            }
        }
        slot = slot + 1 == kBabSlots ? 0 : slot + 1;
    }
    cp_async_wait<0>();
    if (TOTALS) {
        __shared__ int s_tot[kScanMaxTw * 4];
        for (int i = threadIdx.x; i < tw * 4; i += kScanThreads) s_tot[i] = 0;
        __syncthreads();
        if (p.active && mine) {
#pragma unroll
            for (int e = 0; e < 4; ++e) atomicAdd(&s_tot[p.tx * 4 + e], (int)((long long)cs16[e] - (long long)mine * 32768));
        }
        __syncthreads();
        for (int i = threadIdx.x; i < tw * 4; i += kScanThreads) {
            const int c = blockIdx.y * tw * 4 + i;
            if (c < C && s_tot[i]) atomicAdd(chansum16 + c, (unsigned long long)(long long)s_tot[i]);
        }
    }
}

// The same coefficients from per-channel sums that are already complete (n: the rows they were taken over).
__global__ void bn_bwd_coef_kernel(const double *__restrict__ sum_dy, const double *__restrict__ sum_dyx, int C, int64_t n,
                                   const float *__restrict__ gamma, double Cn, float *__restrict__ dgamma,
                                   float *__restrict__ dbeta, float2 *__restrict__ coef)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    const double a = sum_dy[c], b = sum_dyx[c];
    const double g = gamma ? (double)gamma[c] : 1.0;
    if (dbeta) dbeta[c] = (float)a;
    if (dgamma) dgamma[c] = (float)b;
    coef[c] = make_float2((float)(g * a / (double)n), (float)(Cn * g * b));
}

// RANGE: also leave the block's (min, max) of the dx values it wrote in range_parts[block], so that the
// quantiser that follows needs no scan of its own (Section 4: the range comes for free).
template <int VEC, bool RELU, bool RANGE>
__global__ void __launch_bounds__(kScanThreads) bn_bwd_apply_kernel(const float *__restrict__ dy,
                                                                    const float *__restrict__ x, int64_t rows, int C,
                                                                    int tw, const float *__restrict__ mean,
                                                                    const float *__restrict__ vmin,
                                                                    const float *__restrict__ vmax,
                                                                    const float *__restrict__ gamma,
                                                                    const float *__restrict__ beta, float Cn,
                                                                    const float2 *__restrict__ coef,
                                                                    float *__restrict__ dx,
                                                                    float2 *__restrict__ range_parts)
{
    const ScanPos p = scan_pos<VEC>(C, tw);
    float rlo = INFINITY, rhi = -INFINITY;
    if (p.active) {
    const int rpb = kScanThreads / tw;
    float mu[VEC], s[VEC], g[VEC], b[VEC], lo[VEC], hi[VEC], m1[VEC], k2[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        mu[e] = mean[p.col + e];
        lo[e] = vmin[p.col + e]; hi[e] = vmax[p.col + e];
        s[e] = bn_scale(lo[e], hi[e], Cn);
        g[e] = gamma ? gamma[p.col + e] : 1.0f;
        b[e] = beta ? beta[p.col + e] : 0.0f;
        float2 cf = coef[p.col + e];
        m1[e] = cf.x; k2[e] = cf.y;
    }
    const int64_t step = (int64_t)gridDim.x * rpb;
    for (int64_t r0 = (int64_t)blockIdx.x * rpb + p.ty; r0 < rows; r0 += step * kScanUnroll) {
        VecF<VEC> vx[kScanUnroll], vd[kScanUnroll];
        bool ok[kScanUnroll];
#pragma unroll
        for (int u = 0; u < kScanUnroll; ++u) {
            int64_t r = r0 + u * step;
            ok[u] = r < rows;
            if (ok[u]) { vx[u].load(x + r * C + p.col); vd[u].load(dy + r * C + p.col); }
        }
#pragma unroll
        for (int u = 0; u < kScanUnroll; ++u)
            if (ok[u]) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const float xv = vx[u].v[e];
                    float d = vd[u].v[e];
                    if (RELU && !(bn_y(bn_xhat(xv, mu[e], s[e]), g[e], b[e]) > 0.0f)) d = 0.0f;
                    const float ind = (xv == hi[e] ? 1.0f : 0.0f) - (xv == lo[e] ? 1.0f : 0.0f);
                    vd[u].v[e] = bn_dx(d, ind, s[e], g[e], m1[e], k2[e]);
                    if (RANGE) { rlo = fminf(rlo, vd[u].v[e]); rhi = fmaxf(rhi, vd[u].v[e]); }
                }
                vd[u].store(dx + (r0 + u * step) * C + p.col);
            }
    }
    }
    if (RANGE) {
        rlo = warp_min(rlo); rhi = warp_max(rhi);
        __shared__ float s_lo[kScanThreads / 32], s_hi[kScanThreads / 32];
        if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = rlo; s_hi[threadIdx.x >> 5] = rhi; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kScanThreads / 32; ++w) { rlo = fminf(rlo, s_lo[w]); rhi = fmaxf(rhi, s_hi[w]); }
            range_parts[blockIdx.y * gridDim.x + blockIdx.x] = make_float2(rlo, rhi);
        }
    }
}

static size_t bn_ws_bytes(int64_t C)
{
    // forward: lo, hi (float) + sum (double) partials; backward: two double partials + coefficients
    // (... and, for the backward pass that also bifurcates, six float tables of dy extremes and the channels' ranges)
    size_t per = (size_t)kScanMaxStrips * (size_t)C;
    return 2 * align_up(per * sizeof(double), 256) + 2 * align_up(per * sizeof(float), 256) +
           align_up((size_t)C * sizeof(float2), 256) + 256 + align_up(6 * per * sizeof(float), 256) +
           2 * align_up((size_t)C * sizeof(float2), 256);
}

static int check_bn(const char *who, const void *a, const void *b, int64_t n, int64_t C, const void *ws, size_t ws_bytes)
{
    if (n < 2) return fail(QBP_ERR_INVALID_ARG, "%s: n must be at least 2 (C(1) is infinite)", who);
    if (C <= 0) return fail(QBP_ERR_INVALID_ARG, "%s: C must be positive", who);
    if (!a || !b) return fail(QBP_ERR_INVALID_ARG, "%s: NULL tensor", who);
    if (!ws || ws_bytes < bn_ws_bytes(C))
        return fail(QBP_ERR_WORKSPACE, "%s: workspace of %zu bytes needed, %zu given", who, bn_ws_bytes(C), ws_bytes);
    return QBP_OK;
}

// Upper bound on the (min, max) partials rangebn_bwd_impl writes: row strips x column slabs of the apply grid.
size_t rangebn_range_parts_capacity(int64_t C)
{
    // (vector columns may be single floats: C columns in slabs of kScanMaxTw)
    return (size_t)kScanMaxStrips * (size_t)((C + kScanMaxTw - 1) / kScanMaxTw + 1);
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) size_t qbp_rangebn_workspace_bytes(int64_t n, int64_t C)
{
    (void)n;
    return bn_ws_bytes(C > 0 ? C : 1);
}

namespace qbp {

// The apply pass (and what hangs on it) from per-channel mean / min / max that are already in save_*:
// the exact range of y and the next layer's 8-bit parameters when asked for, y and / or its 8-bit codes.
// n_stat: the rows the statistics were taken over (more than n_rows when several GPUs share a minibatch).
static int bn_fwd_apply_launch(const float *x, int64_t n_rows, int64_t n_stat, int64_t C, const float *gamma,
                               const float *beta, int relu, float *y, const float *save_mean, const float *save_min,
                               const float *save_max, qbp_qparams *out_range, const qbp_requant *rq, cudaStream_t st,
                               bool reverse = false)
{
    const bool requant = rq != nullptr;
    if (requant && (!rq->q || !rq->qp)) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: the requantisation record needs q and qp");
    if (!y && !requant) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: neither y nor 8-bit codes wanted");
    const bool al = aligned16(x) && (!y || aligned16(y)) && (!requant || ((uintptr_t)rq->q & 3) == 0);
    const bool v4 = al && C % 4 == 0;
    const int bps = v4 ? (requant ? (relu ? blocks_per_sm(bn_apply_kernel<4, true, true>, kScanThreads)
                                          : blocks_per_sm(bn_apply_kernel<4, false, true>, kScanThreads))
                                  : (relu ? blocks_per_sm(bn_apply_kernel<4, true, false>, kScanThreads)
                                          : blocks_per_sm(bn_apply_kernel<4, false, false>, kScanThreads)))
                       : blocks_per_sm(bn_apply_kernel<1, true, true>, kScanThreads);
    const ScanGeom ga = scan_geom(n_rows, C, al, bps);
    const dim3 grid_apply(ga.nbx, ga.slabs);
    const float Cn = (float)(1.0 / std::sqrt(2.0 * std::log((double)n_stat)));
    if (out_range || requant) {
        QBP_TRACE_BEGIN(st);
        bn_out_range_kernel<<<1, 256, 0, st>>>(save_mean, save_min, save_max, gamma, beta, (int)C, Cn, relu, out_range,
                                               requant ? rq->qp : nullptr, nullptr);
        QBP_LAUNCH_OK("bn_out_range_kernel");
    }
    BnRequant R{nullptr, nullptr, nullptr, 1, nullptr};
    bool fused_rowsum = false;
    if (requant) {
        R.rq = rq->qp; R.q = rq->q;
        // the row's lanes sit in one warp when the block is at most 32 vectors wide and one slab covers the row
        fused_rowsum = rq->row_sums && ga.tw <= 32 && ga.slabs == 1;
        if (fused_rowsum) { R.rowsum = rq->row_sums; R.rs_group = ga.tw; }
        if (rq->chan_sums) {
            if (n_rows >= (1ll << 22)) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "rangebn_fwd: per-channel code totals for fewer than 2^22 rows");
            QBP_CUDA_OK(cudaMemsetAsync(rq->chan_sums, 0, sizeof(int64_t) * (size_t)C, st));
            R.chansum = reinterpret_cast<unsigned long long *>(rq->chan_sums);
        }
    }
    QBP_TRACE_BEGIN(st);
#define QBP_BN_APPLY(V, RL, RQ) bn_apply_kernel<V, RL, RQ><<<grid_apply, kScanThreads, 0, st>>>(x, n_rows, (int)C, ga.tw, save_mean, save_min, save_max, gamma, beta, Cn, y, R, reverse ? 1 : 0)
    if (ga.vec == 4) {
        if (requant) { if (relu) QBP_BN_APPLY(4, true, true); else QBP_BN_APPLY(4, false, true); }
        else         { if (relu) QBP_BN_APPLY(4, true, false); else QBP_BN_APPLY(4, false, false); }
    } else {
        if (requant) { if (relu) QBP_BN_APPLY(1, true, true); else QBP_BN_APPLY(1, false, true); }
        else         { if (relu) QBP_BN_APPLY(1, true, false); else QBP_BN_APPLY(1, false, false); }
    }
#undef QBP_BN_APPLY
    QBP_LAUNCH_OK("bn_apply_kernel");
    if (requant && rq->row_sums && !fused_rowsum) return launch_rowsum(rq->q, true, n_rows, C, rq->row_sums, st);
    return QBP_OK;
}

// The statistics pass: partials per strip, then either mean / min / max (mean != NULL) or the raw sum / min / max.
static int bn_fwd_stats_launch(const float *x, int64_t n, int64_t C, float *mean, float *vmin, float *vmax, double *sum_out,
                               void *ws, size_t ws_bytes, cudaStream_t st)
{
    WsCarver w(ws, ws_bytes);
    double *psum = w.take<double>((size_t)kScanMaxStrips * C);
    w.take<double>((size_t)kScanMaxStrips * C);
    float *plo = w.take<float>((size_t)kScanMaxStrips * C);
    float *phi = w.take<float>((size_t)kScanMaxStrips * C);
    const bool al = aligned16(x);
    const bool v4 = al && C % 4 == 0;
    const ScanGeom g = scan_geom(n, C, al, v4 ? blocks_per_sm(bn_stats_kernel<4>, kScanThreads)
                                              : blocks_per_sm(bn_stats_kernel<1>, kScanThreads));
    const dim3 grid(g.nbx, g.slabs);
    QBP_TRACE_BEGIN(st);
    if (g.vec == 4) bn_stats_kernel<4><<<grid, kScanThreads, 0, st>>>(x, n, (int)C, g.tw, plo, phi, psum);
    else            bn_stats_kernel<1><<<grid, kScanThreads, 0, st>>>(x, n, (int)C, g.tw, plo, phi, psum);
    QBP_LAUNCH_OK("bn_stats_kernel");
    QBP_TRACE_BEGIN(st);
    bn_stats_finalize_kernel<<<(int)C, 128, 0, st>>>(plo, phi, psum, g.nbx, (int)C, n, mean, vmin, vmax, sum_out);
    QBP_LAUNCH_OK("bn_stats_finalize_kernel");
    return QBP_OK;
}

}  // namespace qbp

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_fwd_q8(const float *x, int64_t n, int64_t C, const float *gamma, const float *beta, int relu,
                               float *y, float *save_mean, float *save_min, float *save_max, qbp_qparams *out_range,
                               const qbp_requant *rq, void *ws, size_t ws_bytes, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    int rc = check_bn("rangebn_fwd", x, x, n, C, ws, ws_bytes);
    if (rc) return rc;
    if (!y && !rq) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: NULL tensor");
    if (!save_mean || !save_min || !save_max) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: NULL statistics buffer");
    if ((rc = bn_fwd_stats_launch(x, n, C, save_mean, save_min, save_max, nullptr, ws, ws_bytes, st))) return rc;
    return bn_fwd_apply_launch(x, n, n, C, gamma, beta, relu, y, save_mean, save_min, save_max, out_range, rq, st);
}

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_fwd(const float *x, int64_t n, int64_t C, const float *gamma, const float *beta, int relu,
                               float *y, float *save_mean, float *save_min, float *save_max, qbp_qparams *out_range,
                               void *ws, size_t ws_bytes, void *stream)
{
    if (!y) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: NULL tensor");
    return qbp_rangebn_fwd_q8(x, n, C, gamma, beta, relu, y, save_mean, save_min, save_max, out_range, nullptr, ws, ws_bytes, stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_fwd_stats(const float *x, int64_t n, int64_t C, double *col_sum, float *col_min,
                               float *col_max, void *ws, size_t ws_bytes, void *stream)
{
    // (n = 1 is a valid share of a larger minibatch: the n >= 2 rule applies to n_stat of the apply call)
    if (n < 1 || C <= 0) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd_stats: n and C must be positive");
    if (!x || !col_sum || !col_min || !col_max) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd_stats: NULL argument");
    if (!ws || ws_bytes < bn_ws_bytes(C))
        return fail(QBP_ERR_WORKSPACE, "rangebn_fwd_stats: workspace of %zu bytes needed, %zu given", bn_ws_bytes(C), ws_bytes);
    return bn_fwd_stats_launch(x, n, C, nullptr, col_min, col_max, col_sum, ws, ws_bytes, (cudaStream_t)stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_fwd_apply(const float *x, int64_t n_rows, int64_t n_stat, int64_t C, const double *col_sum,
                               const float *col_min, const float *col_max, const float *gamma, const float *beta, int relu,
                               float *y, float *save_mean, float *save_min, float *save_max, qbp_qparams *out_range,
                               const qbp_requant *rq, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (n_rows < 1 || n_stat < n_rows || C <= 0) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd_apply: needs 1 <= n_rows <= n_stat, C > 0");
    if (n_stat < 2) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd_apply: n_stat must be at least 2 (C(1) is infinite)");
    if (!x || !col_sum || !col_min || !col_max || !save_mean || !save_min || !save_max)
        return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd_apply: NULL argument");
    QBP_TRACE_BEGIN(st);
    bn_mean_from_sum_kernel<<<(int)((C + 255) / 256), 256, 0, st>>>(col_sum, col_min, col_max, (int)C, n_stat, save_mean, save_min, save_max);
    QBP_LAUNCH_OK("bn_mean_from_sum_kernel");
    return bn_fwd_apply_launch(x, n_rows, n_stat, C, gamma, beta, relu, y, save_mean, save_min, save_max, out_range, rq, st);
}

// The statistics half of the recompute fusion (a convolution run twice: once for the statistics, once to write
// the normalised output as 8-bit codes): from the partials the first run left, the saved statistics, the 8-bit
// parameters of the output and, per channel, (mean, scale, gamma, beta) for the second run's epilogue.
int qbp::rangebn_fold_from_parts(int64_t n, int64_t C, const float *gamma, const float *beta, int relu, float *save_mean,
                                 float *save_min, float *save_max, const ColStatParts &parts, qbp_qparams *qp8_out,
                                 float4 *fold, cudaStream_t st)
{
    if (!save_mean || !save_min || !save_max || !parts.lo || !parts.hi || !parts.sum || parts.rows <= 0 || !qp8_out || !fold)
        return fail(QBP_ERR_INVALID_ARG, "rangebn: NULL argument");
    if (n < 2 || C <= 0) return fail(QBP_ERR_INVALID_ARG, "rangebn: needs n >= 2 rows");
    const float Cn = (float)(1.0 / std::sqrt(2.0 * std::log((double)n)));
    QBP_TRACE_BEGIN(st);
    bn_stats_finalize_kernel<<<(int)C, 128, 0, st>>>(parts.lo, parts.hi, parts.sum, parts.rows, (int)C, n, save_mean, save_min, save_max, nullptr);
    QBP_LAUNCH_OK("bn_stats_finalize_kernel");
    QBP_TRACE_BEGIN(st);
    bn_out_range_kernel<<<1, 256, 0, st>>>(save_mean, save_min, save_max, gamma, beta, (int)C, Cn, relu, nullptr, qp8_out, fold);
    QBP_LAUNCH_OK("bn_out_range_kernel");
    return QBP_OK;
}

// Forward from per-column partials of x that its producer left (rows of [C]: sum, min, max), without a statistics
// pass over x: finalize, then the apply pass.
int qbp::rangebn_fwd_from_parts(const float *x, int64_t n, int64_t C, const float *gamma, const float *beta, int relu,
                                float *y, float *save_mean, float *save_min, float *save_max, const ColStatParts &parts,
                                qbp_qparams *out_range, const qbp_requant *rq, cudaStream_t st)
{
    if (!x || !save_mean || !save_min || !save_max || !parts.lo || !parts.hi || !parts.sum || parts.rows <= 0)
        return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: NULL tensor");
    if (n < 2 || C <= 0) return fail(QBP_ERR_INVALID_ARG, "rangebn_fwd: needs n >= 2 rows");
    QBP_TRACE_BEGIN(st);
    bn_stats_finalize_kernel<<<(int)C, 128, 0, st>>>(parts.lo, parts.hi, parts.sum, parts.rows, (int)C, n, save_mean, save_min, save_max, nullptr);
    QBP_LAUNCH_OK("bn_stats_finalize_kernel");
    // (the product that left the statistics has just written x: its tail is in the L2)
    return bn_fwd_apply_launch(x, n, n, C, gamma, beta, relu, y, save_mean, save_min, save_max, out_range, rq, st, true);
}

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_bwd(const float *dy, const float *x, int64_t n, int64_t C, const float *gamma,
                               const float *beta, int relu, const float *save_mean, const float *save_min,
                               const float *save_max, float *dx, float *dgamma, float *dbeta, void *ws,
                               size_t ws_bytes, void *stream)
{
    return rangebn_bwd_impl(dy, x, n, C, gamma, beta, relu, save_mean, save_min, save_max, dx, dgamma, dbeta, ws, ws_bytes,
                            nullptr, nullptr, (cudaStream_t)stream);
}

namespace qbp {

static int bn_bwd_stats_launch(const float *dy, const float *x, int64_t n_rows, int64_t n_stat, int64_t C, const float *gamma,
                               const float *beta, int relu, const float *save_mean, const float *save_min,
                               const float *save_max, float *dgamma, float *dbeta, float2 *coef, double *sum_dy,
                               double *sum_dyx, double *pa, double *pb, cudaStream_t st, float *ext = nullptr,
                               float2 *chan_range = nullptr, float2 *relu_thr = nullptr)
{
    const bool al = aligned16(x) && aligned16(dy);
    const bool v4 = al && C % 4 == 0;
    const ScanGeom g = scan_geom(n_rows, C, al, v4 ? (ext ? blocks_per_sm(bn_bwd_stats_kernel<4, true, true>, kScanThreads)
                                                          : relu ? blocks_per_sm(bn_bwd_stats_kernel<4, true, false>, kScanThreads)
                                                                 : blocks_per_sm(bn_bwd_stats_kernel<4, false, false>, kScanThreads))
                                                   : blocks_per_sm(bn_bwd_stats_kernel<1, true, false>, kScanThreads));
    const dim3 grid(g.nbx, g.slabs);
    const double Cnd = 1.0 / std::sqrt(2.0 * std::log((double)n_stat));
    const float Cn = (float)Cnd;
    QBP_TRACE_BEGIN(st);
#define QBP_BN_BSTATS(V, R, E) bn_bwd_stats_kernel<V, R, E><<<grid, kScanThreads, 0, st>>>(dy, x, n_rows, (int)C, g.tw, save_mean, save_min, save_max, gamma, beta, Cn, pa, pb, ext)
    if (ext) {
        if (g.vec != 4) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "rangebn_bwd: the pass with dy extremes needs aligned tensors and C a multiple of 4");
        if (relu) QBP_BN_BSTATS(4, true, true); else QBP_BN_BSTATS(4, false, true);
    } else if (g.vec == 4) { if (relu) QBP_BN_BSTATS(4, true, false); else QBP_BN_BSTATS(4, false, false); }
    else                   { if (relu) QBP_BN_BSTATS(1, true, false); else QBP_BN_BSTATS(1, false, false); }
#undef QBP_BN_BSTATS
    QBP_LAUNCH_OK("bn_bwd_stats_kernel");
    QBP_TRACE_BEGIN(st);
    bn_bwd_finalize_kernel<<<(int)C, 128, 0, st>>>(pa, pb, g.nbx, (int)C, n_stat, gamma, Cnd, dgamma, dbeta, coef, sum_dy, sum_dyx,
                                                   ext, save_min, save_max, Cn, chan_range, save_mean, beta, relu_thr);
    QBP_LAUNCH_OK("bn_bwd_finalize_kernel");
    return QBP_OK;
}

static int bn_bwd_apply_launch(const float *dy, const float *x, int64_t n_rows, int64_t n_stat, int64_t C, const float *gamma,
                               const float *beta, int relu, const float *save_mean, const float *save_min,
                               const float *save_max, const float2 *coef, float *dx, float2 *range_parts, int *nparts,
                               cudaStream_t st)
{
    const bool al = aligned16(x) && aligned16(dy) && aligned16(dx);
    const bool v4 = al && C % 4 == 0;
    const ScanGeom ga = scan_geom(n_rows, C, al, v4 ? (relu ? blocks_per_sm(bn_bwd_apply_kernel<4, true, true>, kScanThreads)
                                                            : blocks_per_sm(bn_bwd_apply_kernel<4, false, true>, kScanThreads))
                                                    : blocks_per_sm(bn_bwd_apply_kernel<1, true, true>, kScanThreads));
    const dim3 grid_apply(ga.nbx, ga.slabs);
    const float Cn = (float)(1.0 / std::sqrt(2.0 * std::log((double)n_stat)));
    QBP_TRACE_BEGIN(st);
#define QBP_BN_BAPPLY(V, R, G) bn_bwd_apply_kernel<V, R, G><<<grid_apply, kScanThreads, 0, st>>>(dy, x, n_rows, (int)C, ga.tw, save_mean, save_min, save_max, gamma, beta, Cn, coef, dx, range_parts)
    if (range_parts) {
        if (ga.vec == 4) { if (relu) QBP_BN_BAPPLY(4, true, true); else QBP_BN_BAPPLY(4, false, true); }
        else             { if (relu) QBP_BN_BAPPLY(1, true, true); else QBP_BN_BAPPLY(1, false, true); }
        if (nparts) *nparts = (int)(grid_apply.x * grid_apply.y);
    } else {
        if (ga.vec == 4) { if (relu) QBP_BN_BAPPLY(4, true, false); else QBP_BN_BAPPLY(4, false, false); }
        else             { if (relu) QBP_BN_BAPPLY(1, true, false); else QBP_BN_BAPPLY(1, false, false); }
    }
#undef QBP_BN_BAPPLY
    QBP_LAUNCH_OK("bn_bwd_apply_kernel");
    return QBP_OK;
}

// Whether rangebn_bwd_bifurcate_impl takes a tensor of C channels (row_sums: each row's 8-bit code sum is wanted).
bool rangebn_bwd_bifurcate_supported(const float *dy, const float *x, const float *g_out, int64_t n, int64_t C, bool row_sums)
{
    if (!aligned16(x) || !aligned16(dy) || (g_out && !aligned16(g_out)) || C % 4 || n < 2 || n * C >= (1ll << 40)) return false;
    (void)row_sums;      // (any row width: rows wider than a warp's lanes are added up from their pieces)
    return true;
}

// Range BN backward and the bifurcation of its result in two passes over (dy, x): statistics with the extremes of dy
// (from which the exact range of the gradient follows), then the pass that computes the gradient and writes its 8-bit
// copy, the limbs of its 16-bit copy and the rows' code sums -- and the fp32 gradient only when g_out is given.
int rangebn_bwd_bifurcate_impl(const float *dy, const float *x, int64_t n, int64_t C, const float *gamma, const float *beta,
                               int relu, const float *save_mean, const float *save_min, const float *save_max, float *g_out,
                               float *dgamma, float *dbeta, uint64_t seed, uint32_t id8, uint32_t id16, int8_t *q8,
                               qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi, uint8_t *lo, qbp_qparams *qp16, bool lo_signed,
                               void *ws, size_t ws_bytes, cudaStream_t st, cudaEvent_t after_range, int64_t *tot16)
{
    int rc = check_bn("rangebn_bwd", dy, x, n, C, ws, ws_bytes);
    if (rc) return rc;
    if (!rangebn_bwd_bifurcate_supported(dy, x, g_out, n, C, row_sums8 != nullptr) || ((uintptr_t)q8 & 3) || ((uintptr_t)hi & 3) || ((uintptr_t)lo & 3))
        return fail(QBP_ERR_UNSUPPORTED_SHAPE, "rangebn_bwd (bifurcating): shape or alignment not taken");
    WsCarver w(ws, ws_bytes);
    double *pa = w.take<double>((size_t)kScanMaxStrips * C);
    double *pb = w.take<double>((size_t)kScanMaxStrips * C);
    w.take<float>((size_t)kScanMaxStrips * C);
    w.take<float>((size_t)kScanMaxStrips * C);
    float2 *coef = w.take<float2>((size_t)C);
    w.take<char>(256);
    float *ext = w.take<float>(6 * (size_t)kScanMaxStrips * C);
    float2 *chan_range = w.take<float2>((size_t)C);
    float2 *relu_thr = w.take<float2>((size_t)C);
    if ((rc = bn_bwd_stats_launch(dy, x, n, n, C, gamma, beta, relu, save_mean, save_min, save_max, dgamma, dbeta, coef, nullptr,
                                  nullptr, pa, pb, st, ext, chan_range, relu ? relu_thr : nullptr)))
        return rc;
    if ((rc = launch_range_finalize(chan_range, (int)C, qp8, qp16, st, after_range))) return rc;
    if (tot16) QBP_CUDA_OK(cudaMemsetAsync(tot16, 0, sizeof(int64_t) * (size_t)C, st));
    // (three resident blocks per SM by the kernel's launch bounds, whatever the instance)
    const ScanGeom ga = scan_geom(n, C, true, blocks_per_sm(bn_bwd_apply_bifurcate_kernel<true, true, true>, kScanThreads));
    const dim3 grid(ga.nbx, ga.slabs);
    const float Cn = (float)(1.0 / std::sqrt(2.0 * std::log((double)n)));
    const PhiloxKeys keys = philox_keys_host(seed);
    const uint32_t flip = lo_signed ? 0x80808080u : 0u;
    // each row's code sum by shuffles over the row's lanes of a warp; a row that spans several warps or blocks is
    // added up from its pieces (integer atomics on the zeroed sums: the result does not depend on the order)
    int32_t *row_sums_arg = row_sums8;
    if (row_sums8 && (ga.tw > 32 || ga.slabs > 1)) QBP_CUDA_OK(cudaMemsetAsync(row_sums8, 0, sizeof(int32_t) * (size_t)n, st));
    QBP_TRACE_BEGIN(st);
#define QBP_BN_BAB(R, G, T) do { static PerDeviceOnce once_; QBP_SMEM_OPT_IN(once_, (bn_bwd_apply_bifurcate_kernel<R, G, T>), kBabRingBytes); bn_bwd_apply_bifurcate_kernel<R, G, T><<<grid, kScanThreads, kBabRingBytes, st>>>(dy, x, n, (int)C, ga.tw, save_mean, save_min, save_max, gamma, beta, Cn, coef, g_out, qp8, qp16, id8, id16, keys, reinterpret_cast<uint32_t *>(q8), reinterpret_cast<uint32_t *>(hi), reinterpret_cast<uint32_t *>(lo), flip, row_sums_arg, reinterpret_cast<unsigned long long *>(tot16), relu_thr); } while (0)
#define QBP_BN_BAB2(R, G) do { if (tot16) QBP_BN_BAB(R, G, true); else QBP_BN_BAB(R, G, false); } while (0)
    if (g_out) { if (relu) QBP_BN_BAB2(true, true); else QBP_BN_BAB2(false, true); }
    else       { if (relu) QBP_BN_BAB2(true, false); else QBP_BN_BAB2(false, false); }
#undef QBP_BN_BAB2
#undef QBP_BN_BAB
    QBP_LAUNCH_OK("bn_bwd_apply_bifurcate_kernel");
    return QBP_OK;
}

}  // namespace qbp

// range_parts (nullable, room for rangebn_range_parts_capacity(C) entries) receives one (min, max) of dx per
// block of the apply pass; *nparts their count.
int qbp::rangebn_bwd_impl(const float *dy, const float *x, int64_t n, int64_t C, const float *gamma, const float *beta,
                          int relu, const float *save_mean, const float *save_min, const float *save_max, float *dx,
                          float *dgamma, float *dbeta, void *ws, size_t ws_bytes, float2 *range_parts, int *nparts,
                          cudaStream_t st)
{
    int rc = check_bn("rangebn_bwd", x, dy, n, C, ws, ws_bytes);
    if (rc) return rc;
    if (!dx || !save_mean || !save_min || !save_max) return fail(QBP_ERR_INVALID_ARG, "rangebn_bwd: NULL tensor");
    WsCarver w(ws, ws_bytes);
    double *pa = w.take<double>((size_t)kScanMaxStrips * C);
    double *pb = w.take<double>((size_t)kScanMaxStrips * C);
    w.take<float>((size_t)kScanMaxStrips * C);
    w.take<float>((size_t)kScanMaxStrips * C);
    float2 *coef = w.take<float2>((size_t)C);
    if ((rc = bn_bwd_stats_launch(dy, x, n, n, C, gamma, beta, relu, save_mean, save_min, save_max, dgamma, dbeta, coef,
                                  nullptr, nullptr, pa, pb, st)))
        return rc;
    return bn_bwd_apply_launch(dy, x, n, n, C, gamma, beta, relu, save_mean, save_min, save_max, coef, dx, range_parts, nparts, st);
}

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_bwd_stats(const float *dy, const float *x, int64_t n_rows, int64_t n_stat, int64_t C,
                               const float *gamma, const float *beta, int relu, const float *save_mean,
                               const float *save_min, const float *save_max, double *sum_dy, double *sum_dyxhat,
                               void *ws, size_t ws_bytes, void *stream)
{
    if (n_rows < 1 || n_stat < n_rows || n_stat < 2 || C <= 0)
        return fail(QBP_ERR_INVALID_ARG, "rangebn_bwd_stats: needs 1 <= n_rows <= n_stat, n_stat >= 2, C > 0");
    if (!dy || !x || !save_mean || !save_min || !save_max || !sum_dy || !sum_dyxhat)
        return fail(QBP_ERR_INVALID_ARG, "rangebn_bwd_stats: NULL argument");
    if (!ws || ws_bytes < bn_ws_bytes(C))
        return fail(QBP_ERR_WORKSPACE, "rangebn_bwd_stats: workspace of %zu bytes needed, %zu given", bn_ws_bytes(C), ws_bytes);
    WsCarver w(ws, ws_bytes);
    double *pa = w.take<double>((size_t)kScanMaxStrips * C);
    double *pb = w.take<double>((size_t)kScanMaxStrips * C);
    return bn_bwd_stats_launch(dy, x, n_rows, n_stat, C, gamma, beta, relu, save_mean, save_min, save_max, nullptr, nullptr,
                               nullptr, sum_dy, sum_dyxhat, pa, pb, (cudaStream_t)stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_rangebn_bwd_apply(const float *dy, const float *x, int64_t n_rows, int64_t n_stat, int64_t C,
                               const float *gamma, const float *beta, int relu, const float *save_mean,
                               const float *save_min, const float *save_max, const double *sum_dy,
                               const double *sum_dyxhat, float *dx, float *dgamma, float *dbeta, void *ws,
                               size_t ws_bytes, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (n_rows < 1 || n_stat < n_rows || n_stat < 2 || C <= 0)
        return fail(QBP_ERR_INVALID_ARG, "rangebn_bwd_apply: needs 1 <= n_rows <= n_stat, n_stat >= 2, C > 0");
    if (!dy || !x || !dx || !save_mean || !save_min || !save_max || !sum_dy || !sum_dyxhat)
        return fail(QBP_ERR_INVALID_ARG, "rangebn_bwd_apply: NULL argument");
    if (!ws || ws_bytes < bn_ws_bytes(C))
        return fail(QBP_ERR_WORKSPACE, "rangebn_bwd_apply: workspace of %zu bytes needed, %zu given", bn_ws_bytes(C), ws_bytes);
    WsCarver w(ws, ws_bytes);
    w.take<double>((size_t)kScanMaxStrips * C);
    w.take<double>((size_t)kScanMaxStrips * C);
    w.take<float>((size_t)kScanMaxStrips * C);
    w.take<float>((size_t)kScanMaxStrips * C);
    float2 *coef = w.take<float2>((size_t)C);
    const double Cnd = 1.0 / std::sqrt(2.0 * std::log((double)n_stat));
    QBP_TRACE_BEGIN(st);
    bn_bwd_coef_kernel<<<(int)((C + 255) / 256), 256, 0, st>>>(sum_dy, sum_dyxhat, (int)C, n_stat, gamma, Cnd, dgamma, dbeta, coef);
    QBP_LAUNCH_OK("bn_bwd_coef_kernel");
    return bn_bwd_apply_launch(dy, x, n_rows, n_stat, C, gamma, beta, relu, save_mean, save_min, save_max, coef, dx, nullptr, nullptr, st);
}
