// Appendix C, Ternarized Back-Propagation: 1-bit weights and activations, stochastically ternarised gradients, and
// Algorithm 1 (multiple stochastic ternarisation sampling for the weight gradient).
//
// The operands stay bytes: "XNOR and population count" is the dot product of +-1 values, and on this GPU the int8
// tensor cores run that product about ten times faster than popcount instructions on the CUDA cores (16 per clock and
// SM), so binary and ternary tensors are written as int8 codes with zero-point 0 and the products are the library's
// own (qbp_gemm_s8, qbp_conv_s8_implicit, qbp_wgrad_s16); their integer accumulators are the XNOR-popcount results.
//
// Algorithm 1 adds S products of one ternary sample each and divides by S; a product is linear in the sample, so the
// S samples of an element are added first (at most S <= 127 in magnitude: a byte) and one product is run.
#include "qbp_mma.cuh"

#include <algorithm>

namespace qbp {

constexpr int kTbpThreads = 256;

// b(x) = +1 for x >= 0 (so for -0.0), else -1.  VEC = 4: 16-byte loads, one packed word per thread and step.
template <int VEC>
__global__ void __launch_bounds__(kTbpThreads) binarize_kernel(const float *__restrict__ x, int64_t n, int8_t *__restrict__ q,
                                                               qbp_qparams *__restrict__ qp_out)
{
    if (qp_out && blockIdx.x == 0 && threadIdx.x == 0) {
        qbp_qparams r; r.scale = 1.0f; r.zero_point = 0; r.vmin = -1.0f; r.vmax = 1.0f;
        *qp_out = r;
    }
    const int64_t stride = (int64_t)gridDim.x * kTbpThreads;
    if (VEC == 4) {
        const int64_t nv = n >> 2;
        for (int64_t j = (int64_t)blockIdx.x * kTbpThreads + threadIdx.x; j < nv; j += stride) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(x) + j);
            const uint32_t c0 = v.x >= 0.0f ? 0x01u : 0xFFu, c1 = v.y >= 0.0f ? 0x01u : 0xFFu;
            const uint32_t c2 = v.z >= 0.0f ? 0x01u : 0xFFu, c3 = v.w >= 0.0f ? 0x01u : 0xFFu;
            reinterpret_cast<uint32_t *>(q)[j] = c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0)
            for (int64_t i = nv << 2; i < n; ++i) q[i] = x[i] >= 0.0f ? 1 : -1;
    } else {
        for (int64_t i = (int64_t)blockIdx.x * kTbpThreads + threadIdx.x; i < n; i += stride) q[i] = x[i] >= 0.0f ? 1 : -1;
    }
}

// One element: how many of its `samples` draws keep it.  A draw u = (word >> 8) * 2^-24 keeps the element when
// u * s < |g| (one fp32 product, rounded to nearest; with s = 0 nothing is kept); the words of sample k are Philox
// block (j, id, k).
__device__ __forceinline__ int tern_keep(uint32_t word, float s, float a)
{
    return __fmul_rn(__fmul_rn((float)(word >> 8), 0x1p-24f), s) < a ? 1 : 0;
}

// Sum over `samples` stochastic ternarisations of g: code = sign(g) * (number of samples that keep the element), as
// int8 (q), and / or as the two byte limbs of the same value as a 16-bit code (hi: 0 or -1, lo: the low byte), which
// is what the weight-gradient product takes.  *rng holds the tensor's range (s = max(-vmin, vmax)); *qp_out receives
// scale = s / samples, zero-point 0, so that scale * code estimates g.
template <int VEC>
__global__ void __launch_bounds__(kTbpThreads) stc_ternarize_kernel(const float *__restrict__ g, int64_t n,
                                                                    const qbp_qparams *__restrict__ rng, int samples,
                                                                    uint32_t tensor_id, const __grid_constant__ PhiloxKeys keys,
                                                                    int8_t *__restrict__ q, int8_t *__restrict__ hi,
                                                                    uint8_t *__restrict__ lo, qbp_qparams *__restrict__ qp_out)
{
    const float s = fmaxf(-rng->vmin, rng->vmax);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        qbp_qparams r;
        r.scale = s > 0.0f ? __fdiv_rn(s, (float)samples) : 1.0f;
        r.zero_point = 0; r.vmin = -s; r.vmax = s;
        *qp_out = r;
    }
    const int64_t stride = (int64_t)gridDim.x * kTbpThreads;
    if (VEC == 4) {
        const int64_t nv = n >> 2;
        for (int64_t j = (int64_t)blockIdx.x * kTbpThreads + threadIdx.x; j < nv; j += stride) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(g) + j);
            const float xs[4] = {v.x, v.y, v.z, v.w};
            float p[4]; int cnt[4] = {0, 0, 0, 0};
#pragma unroll
            for (int e = 0; e < 4; ++e) p[e] = fabsf(xs[e]);
            for (int k = 0; k < samples; ++k) {
                const uint4 b = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)((uint64_t)j >> 32), tensor_id, (uint32_t)k), keys);
                cnt[0] += tern_keep(b.x, s, p[0]); cnt[1] += tern_keep(b.y, s, p[1]);
                cnt[2] += tern_keep(b.z, s, p[2]); cnt[3] += tern_keep(b.w, s, p[3]);
            }
            uint32_t w8 = 0, whi = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = xs[e] > 0.0f ? cnt[e] : -cnt[e];
                w8 |= ((uint32_t)c & 0xFFu) << (8 * e);
                whi |= (c < 0 ? 0xFFu : 0u) << (8 * e);
            }
            if (q) reinterpret_cast<uint32_t *>(q)[j] = w8;
            if (hi) reinterpret_cast<uint32_t *>(hi)[j] = whi;
            if (lo) reinterpret_cast<uint32_t *>(lo)[j] = w8;
        }
    }
    // elements the vector loop leaves (all of them when VEC == 1)
    const int64_t first = VEC == 4 ? (n >> 2) << 2 : 0;
    for (int64_t i = first + (int64_t)blockIdx.x * kTbpThreads + threadIdx.x; i < n; i += stride) {
        const float p = fabsf(g[i]);
        const int64_t j = i >> 2;
        int cnt = 0;
        for (int k = 0; k < samples; ++k) {
            const uint4 b = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)((uint64_t)j >> 32), tensor_id, (uint32_t)k), keys);
            const uint32_t w[4] = {b.x, b.y, b.z, b.w};
            cnt += tern_keep(w[i & 3], s, p);
        }
        const int c = g[i] > 0.0f ? cnt : -cnt;
        if (q) q[i] = (int8_t)c;
        if (hi) hi[i] = (int8_t)(c < 0 ? -1 : 0);
        if (lo) lo[i] = (uint8_t)(c & 0xFF);
    }
}

static size_t tern_ws_bytes() { return range_scan_ws_bytes() + 256; }

static int stc_ternarize_impl(const float *g, int64_t n, int samples, uint64_t seed, uint32_t tensor_id, int8_t *q, int8_t *hi,
                              uint8_t *lo, qbp_qparams *qp_out, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (n < 0 || samples < 1 || samples > 127) return fail(QBP_ERR_INVALID_ARG, "stc_ternarize: needs n >= 0 and 1 <= samples <= 127");
    if (!qp_out || (n > 0 && (!g || (!q && !hi && !lo)))) return fail(QBP_ERR_INVALID_ARG, "stc_ternarize: NULL argument");
    if (((uintptr_t)g & 3) != 0) return fail(QBP_ERR_INVALID_ARG, "stc_ternarize: g is not 4-byte aligned");
    if (!ws || ws_bytes < tern_ws_bytes())
        return fail(QBP_ERR_WORKSPACE, "stc_ternarize: workspace of %zu bytes needed, %zu given", tern_ws_bytes(), ws_bytes);
    qbp_qparams *rng = reinterpret_cast<qbp_qparams *>(static_cast<char *>(ws) + range_scan_ws_bytes());
    int rc = range_scan(g, n, ws, range_scan_ws_bytes(), rng, st);
    if (rc) return rc;
    const bool vec = aligned16(g) && (!q || ((uintptr_t)q & 3) == 0) && (!hi || ((uintptr_t)hi & 3) == 0) && (!lo || ((uintptr_t)lo & 3) == 0);
    const int64_t items = vec ? (n + 3) / 4 : n;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((items + kTbpThreads - 1) / kTbpThreads, (int64_t)sm_count() * 8));
    const PhiloxKeys keys = philox_keys_host(seed);
    QBP_TRACE_BEGIN(st);
    if (vec) stc_ternarize_kernel<4><<<grid, kTbpThreads, 0, st>>>(g, n, rng, samples, tensor_id, keys, q, hi, lo, qp_out);
    else     stc_ternarize_kernel<1><<<grid, kTbpThreads, 0, st>>>(g, n, rng, samples, tensor_id, keys, q, hi, lo, qp_out);
    QBP_LAUNCH_OK("stc_ternarize_kernel");
    return QBP_OK;
}

// ---------------------------------------------------------------- bit rows and the literal XNOR + popcount products
// [rows x cols] codes to bit rows: element c of a row is bit c % 32 of word c / 32 (1 for a code > 0, or for a code
// != 0 with `mask`), ceil(cols / 32) words per row, spare bits 0.  One warp per word (a ballot).
__global__ void __launch_bounds__(256) pack_bits_kernel(const int8_t *__restrict__ codes, int64_t rows, int64_t cols, int mask,
                                                        uint32_t *__restrict__ words)
{
    const int64_t wpr = (cols + 31) / 32;
    const int lane = threadIdx.x & 31;
    for (int64_t word = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); word < rows * wpr; word += (int64_t)gridDim.x * 8) {
        const int64_t r = word / wpr, c = (word - r * wpr) * 32 + lane;
        const int v = c < cols ? (int)codes[r * cols + c] : 0;
        const uint32_t bits = __ballot_sync(0xffffffffu, mask ? v != 0 : v > 0);
        if (lane == 0) words[word] = bits;
    }
}

// C [M x N] from bit rows of K bits (wpr words each): 64 x 64 outputs per block, 4 x 4 per thread, 32 words of every
// row staged in shared memory per step (rows padded to 33 words: the threads of a warp read 16 different banks).
//   plain:  C = K - 2 popcount(a xor b)                                   (the +-1 dot product, Appendix C)
//   GATED:  C = popcount(nz & ~(sg xor b)) - popcount(nz & (sg xor b))    (ternary a as non-zero and sign planes)
// The popcount unit retires 16 results per clock and SM, which bounds this form at about 0.15 P bit-products/s; the
// products of the layer path run on the int8 tensor cores instead (qbp_gemm_s8 on +-1 bytes).  This kernel is the
// form for operands kept as bit rows (an eighth of the bytes).
template <bool GATED>
__global__ void __launch_bounds__(256) xnor_gemm_bits_kernel(int M, int N, int K, int wpr, const uint32_t *__restrict__ A,
                                                             const uint32_t *__restrict__ S, const uint32_t *__restrict__ B,
                                                             int32_t *__restrict__ C)
{
    __shared__ uint32_t sA[64][33], sB[64][33], sS[GATED ? 64 : 1][33];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    int acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;
    for (int w0 = 0; w0 < wpr; w0 += 32) {
        // (thread t: word t % 32 of rows t / 32, t / 32 + 8, ...: 128-byte segments)
        const int lw = threadIdx.x & 31, w = w0 + lw;
#pragma unroll
        for (int r = threadIdx.x >> 5; r < 64; r += 8) {
            const bool in_a = m0 + r < M && w < wpr, in_b = n0 + r < N && w < wpr;
            sA[r][lw] = in_a ? A[(int64_t)(m0 + r) * wpr + w] : 0u;
            if (GATED) sS[r][lw] = in_a ? S[(int64_t)(m0 + r) * wpr + w] : 0u;
            sB[r][lw] = in_b ? B[(int64_t)(n0 + r) * wpr + w] : 0u;
        }
        __syncthreads();
#pragma unroll 4
        for (int k = 0; k < 32; ++k) {
            uint32_t a[4], sg[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sA[ty + 16 * i][k]; sg[i] = GATED ? sS[ty + 16 * i][k] : 0u; b[i] = sB[tx + 16 * i][k]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (GATED) { const uint32_t d = sg[i] ^ b[j]; acc[i][j] += __popc(a[i] & ~d) - __popc(a[i] & d); }
                    else acc[i][j] += __popc(a[i] ^ b[j]);
                }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + ty + 16 * i, n = n0 + tx + 16 * j;
            if (m < M && n < N) C[(int64_t)m * N + n] = GATED ? acc[i][j] : K - 2 * acc[i][j];
        }
}

static int xnor_bits_launch(bool gated, int64_t M, int64_t N, int64_t K, const uint32_t *A, const uint32_t *S, const uint32_t *B,
                            int32_t *C, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0 || M > INT32_MAX || N > INT32_MAX || K > INT32_MAX)
        return fail(QBP_ERR_INVALID_ARG, "xnor_gemm_bits: M, N, K must be positive and fit int32");
    if (!A || !B || !C || (gated && !S)) return fail(QBP_ERR_INVALID_ARG, "xnor_gemm_bits: NULL argument");
    if ((N + 63) / 64 > 2147483647ll || (M + 63) / 64 > 65535) return fail(QBP_ERR_UNSUPPORTED_SHAPE, "xnor_gemm_bits: at most 4 M rows");
    const dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
    const int wpr = (int)((K + 31) / 32);
    QBP_TRACE_BEGIN(st);
    if (gated) xnor_gemm_bits_kernel<true><<<grid, 256, 0, st>>>((int)M, (int)N, (int)K, wpr, A, S, B, C);
    else       xnor_gemm_bits_kernel<false><<<grid, 256, 0, st>>>((int)M, (int)N, (int)K, wpr, A, nullptr, B, C);
    QBP_LAUNCH_OK("xnor_gemm_bits_kernel");
    return QBP_OK;
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) int qbp_pack_bits(const int8_t *codes, int64_t rows, int64_t cols, int mask, uint32_t *words, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (rows < 0 || cols <= 0) return fail(QBP_ERR_INVALID_ARG, "pack_bits: rows must be >= 0 and cols > 0");
    if (rows == 0) return QBP_OK;
    if (!codes || !words) return fail(QBP_ERR_INVALID_ARG, "pack_bits: NULL argument");
    const int64_t total = rows * ((cols + 31) / 32);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((total + 7) / 8, (int64_t)sm_count() * 16));
    QBP_TRACE_BEGIN(st);
    pack_bits_kernel<<<grid, 256, 0, st>>>(codes, rows, cols, mask, words);
    QBP_LAUNCH_OK("pack_bits_kernel");
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) int qbp_xnor_gemm_bits(int64_t M, int64_t N, int64_t K, const uint32_t *A_bits, const uint32_t *B_bits,
                                                                         int32_t *C, void *stream)
{
    return xnor_bits_launch(false, M, N, K, A_bits, nullptr, B_bits, C, (cudaStream_t)stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_gated_xnor_gemm_bits(int64_t M, int64_t N, int64_t K, const uint32_t *nz_bits,
                                                                               const uint32_t *sign_bits, const uint32_t *B_bits, int32_t *C,
                                                                               void *stream)
{
    return xnor_bits_launch(true, M, N, K, nz_bits, sign_bits, B_bits, C, (cudaStream_t)stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_binarize_s8(const float *x, int64_t n, int8_t *q, qbp_qparams *qp_out, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (n < 0 || (n > 0 && (!x || !q))) return fail(QBP_ERR_INVALID_ARG, "binarize_s8: NULL tensor or negative size");
    if (((uintptr_t)x & 3) != 0) return fail(QBP_ERR_INVALID_ARG, "binarize_s8: x is not 4-byte aligned");
    const bool vec = aligned16(x) && ((uintptr_t)q & 3) == 0;
    const int64_t items = vec ? (n + 3) / 4 : n;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((items + kTbpThreads - 1) / kTbpThreads, (int64_t)sm_count() * 8));
    QBP_TRACE_BEGIN(st);
    if (vec) binarize_kernel<4><<<grid, kTbpThreads, 0, st>>>(x, n, q, qp_out);
    else     binarize_kernel<1><<<grid, kTbpThreads, 0, st>>>(x, n, q, qp_out);
    QBP_LAUNCH_OK("binarize_kernel");
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) size_t qbp_stc_ternarize_workspace_bytes(void) { return tern_ws_bytes(); }

extern "C" __attribute__((visibility("default"))) int qbp_stc_ternarize_s8(const float *g, int64_t n, int samples, uint64_t seed, uint32_t tensor_id,
                                                                           int8_t *q, qbp_qparams *qp_out, void *ws, size_t ws_bytes, void *stream)
{
    if (n > 0 && !q) return fail(QBP_ERR_INVALID_ARG, "stc_ternarize_s8: q is NULL");
    return stc_ternarize_impl(g, n, samples, seed, tensor_id, q, nullptr, nullptr, qp_out, ws, ws_bytes, (cudaStream_t)stream);
}

// Algorithm 1: the weight gradient of a binarised layer from `samples` stochastic ternarisations of the gradient at
// its output.  The samples of an element are added up (stc_ternarize_kernel), the sum goes through the library's
// 16-bit x 8-bit weight-gradient product as the limbs (t_hi, t_lo) of a 16-bit code, against the +-1 activations.
extern "C" __attribute__((visibility("default"))) size_t qbp_tbp_weight_gradient_workspace_bytes(const qbp_conv_desc *d, int64_t rows, int64_t N, int64_t K)
{
    return align_up(tern_ws_bytes(), 256) + qbp_wgrad_s16_workspace_bytes(d, rows, N, K);
}

extern "C" __attribute__((visibility("default"))) int qbp_tbp_weight_gradient(const qbp_conv_desc *d, int64_t rows, int64_t N, int64_t K,
                                                                              const int8_t *a_codes, const qbp_qparams *qa, const float *g,
                                                                              int samples, uint64_t seed, uint32_t tensor_id, int8_t *t_hi,
                                                                              uint8_t *t_lo, qbp_qparams *qp_t, int64_t *acc_out, float *gW,
                                                                              void *ws, size_t ws_bytes, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (d) { rows = (int64_t)d->N * d->H * d->W; N = d->K; K = d->C; }
    if (rows <= 0 || N <= 0 || K <= 0) return fail(QBP_ERR_INVALID_ARG, "tbp_weight_gradient: sizes must be positive");
    if (!a_codes || !qa || !g || !t_hi || !t_lo || !qp_t) return fail(QBP_ERR_INVALID_ARG, "tbp_weight_gradient: NULL argument");
    // (everything the product would refuse is refused here, before the ternariser is launched)
    if (d ? !wgrad_conv_supported(d) : (N % 16 != 0 || K % 16 != 0))
        return fail(QBP_ERR_UNSUPPORTED_SHAPE, "tbp_weight_gradient: shape outside what qbp_wgrad_s16 takes");
    if (!aligned16(a_codes) || !aligned16(t_hi) || !aligned16(t_lo) || ((uintptr_t)g & 3) != 0)
        return fail(QBP_ERR_INVALID_ARG, "tbp_weight_gradient: a_codes, t_hi, t_lo must be 16-byte aligned, g 4-byte aligned");
    if (!acc_out && !gW) return fail(QBP_ERR_INVALID_ARG, "tbp_weight_gradient: acc_out and gW are both NULL");
    if (samples < 1 || samples > 127) return fail(QBP_ERR_INVALID_ARG, "tbp_weight_gradient: needs 1 <= samples <= 127");
    const size_t head = align_up(tern_ws_bytes(), 256);
    const size_t need = qbp_tbp_weight_gradient_workspace_bytes(d, rows, N, K);
    if (!ws || ws_bytes < need) return fail(QBP_ERR_WORKSPACE, "tbp_weight_gradient: workspace of %zu bytes needed, %zu given", need, ws_bytes);
    int rc = stc_ternarize_impl(g, rows * N, samples, seed, tensor_id, nullptr, t_hi, t_lo, qp_t, ws, head, st);
    if (rc) return rc;
    return wgrad_s16_impl(d, rows, N, K, a_codes, qa, t_hi, t_lo, qp_t, acc_out, gW, nullptr, static_cast<char *>(ws) + head, ws_bytes - head, st);
}
