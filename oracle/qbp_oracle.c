/*
 * qbp_oracle.c -- plain, slow CPU statement of the 8-bit training hot path
 * (Quantized Back-Propagation with Gradients Bifurcation + Range BatchNorm).
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may include, link,
 * import or execute this file: only the tests, the smoke check and the
 * cpu-baseline leg of the benchmark do.  It shares no code, header, table or
 * constant generator with the CUDA library.
 *
 * Every function follows the paper's definitions step by step, scalar loops,
 * no blocking or fusion; OpenMP is used only across independent outputs.
 *
 * Precision:
 *   - the quantiser works in IEEE fp32 with a fixed operation order, because
 *     its result is an integer code that must be reproducible bit for bit;
 *   - integer products accumulate in int64 and are checked against int32;
 *   - Range BN arithmetic is fp64, except the ReLU on/off decision of the
 *     backward pass, which is a boolean and is therefore taken in fp32 with
 *     the same operation order as the forward output.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 *
 * Pin status (tests marked "not gpu"):
 *   qbo_philox4x32_10     published known-answer vectors of Philox4x32-10
 *   qbo_quantize          error bound scale/2, end codes, exact zero, integer
 *                         grid special case, monotonicity, unbiasedness of
 *                         stochastic rounding, the Gaussian cosine bound
 *   qbo_limb_split        exhaustive over all 65536 codes
 *   qbo_gemm_s8/_s16s8    brute force in Python integers, fp64 matmul
 *   qbo_conv_*            im2col + matmul, 1x1 conv == GEMM, adjoint identities
 *   qbo_rangebn_fwd       output range == sqrt(2 ln n), affine invariance,
 *                         C(n) closed form and the paper's worked number
 *   qbo_rangebn_bwd       central finite differences in fp64, sum identities
 *   qbo_binarize/_pack    sign convention on hand-written values, bit order
 *   qbo_xnor_gemm         the +-1 dot product written as a plain integer loop
 *   qbo_stc_tern          exact cases (|g| = max, g = 0), unbiasedness within
 *                         the binomial bound over many samples, sample index
 *                         in the Philox counter
 *   qbo_gated_xnor_gemm   the ternary x binary dot product as a plain loop
 *   qbo_tbp_update        one sample == one product; the mean over many
 *                         samples approaches the exact product g^T a
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1,2,3") */
/* ------------------------------------------------------------------------ */

void qbo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Random word of element i of tensor `tensor_id` under `seed`:
 * key = (lo32 seed, hi32 seed), counter = (lo32 j, hi32 j, tensor_id, 0) with
 * j = i / 4, and element i takes output word i % 4. */
uint32_t qbo_random_word(uint64_t seed, uint32_t tensor_id, uint64_t i)
{
    uint64_t j = i >> 2;
    uint32_t ctr[4] = { (uint32_t)j, (uint32_t)(j >> 32), tensor_id, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    qbo_philox4x32_10(ctr, key, out);
    return out[i & 3];
}

/* ------------------------------------------------------------------------ */
/* Min/max range quantiser (Section 4 "Quantization methods", Appendix B)    */
/* ------------------------------------------------------------------------ */

/* Clamping values = the tensor's own minimum and maximum (Appendix B).
 * per_channel: one pair per innermost index (cols). */
void qbo_range(const float *x, int64_t rows, int64_t cols, int per_channel,
               float *vmin, float *vmax)
{
    if (!per_channel) {
        float lo = INFINITY, hi = -INFINITY;
        for (int64_t i = 0; i < rows * cols; ++i) {
            if (x[i] < lo) lo = x[i];
            if (x[i] > hi) hi = x[i];
        }
        vmin[0] = lo; vmax[0] = hi;
        return;
    }
    for (int64_t c = 0; c < cols; ++c) { vmin[c] = INFINITY; vmax[c] = -INFINITY; }
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float v = x[r * cols + c];
            if (v < vmin[c]) vmin[c] = v;
            if (v > vmax[c]) vmax[c] = v;
        }
}

/* Clamping values of an activation tensor as Appendix B defines them for the
 * high dynamic range of activations: the tensor is cut into `chunks` equal,
 * contiguous groups of rows (rows must be a multiple of chunks); vmax is the
 * average of the groups' maxima and vmin the average of their minima
 * (accumulated in double, returned in fp32).  Values beyond them saturate at
 * the end codes in qbo_quantize.  chunks = 1 is qbo_range per tensor. */
void qbo_range_chunked(const float *x, int64_t rows, int64_t cols, int64_t chunks,
                       float *vmin, float *vmax)
{
    const int64_t per = rows / chunks;
    double slo = 0.0, shi = 0.0;
    for (int64_t k = 0; k < chunks; ++k) {
        float lo = INFINITY, hi = -INFINITY;
        for (int64_t i = k * per * cols; i < (k + 1) * per * cols; ++i) {
            if (x[i] < lo) lo = x[i];
            if (x[i] > hi) hi = x[i];
        }
        slo += (double)lo; shi += (double)hi;
    }
    vmin[0] = (float)(slo / (double)chunks);
    vmax[0] = (float)(shi / (double)chunks);
}

/* Appendix B: scale and zero-point from the clamping values, M bits.
 * Readings: the code grid has L = 2^M - 1 steps so that vmax maps to the top
 * M-bit code; the interval is widened to contain 0 so that real zero is a
 * code; a zero-width interval takes scale 1.  zp_u is the unsigned code of
 * real zero; the stored zero-point is zp_u - 2^(M-1) (codes are kept signed). */
void qbo_qparams(float vmin, float vmax, int bits,
                 float *scale, int32_t *zero_point, float *vmin_used, float *vmax_used)
{
    const int32_t L = (1 << bits) - 1;
    if (vmin > 0.0f) vmin = 0.0f;
    if (vmax < 0.0f) vmax = 0.0f;
    float range = vmax - vmin;
    float s = (range == 0.0f) ? 1.0f : range / (float)L;
    float z = rintf(-vmin / s);
    if (z < 0.0f) z = 0.0f;
    if (z > (float)L) z = (float)L;
    *scale = s;
    *zero_point = (int32_t)z - (1 << (bits - 1));
    *vmin_used = vmin;
    *vmax_used = vmax;
}

/* One element: output = round(x/scale + zero-point), Appendix B, taken as
 * t = fma(x, 1/scale, zp_u) in fp32.  rounding 0: nearest, ties to even.
 * rounding 1: stochastic -- up with probability frac(t).  Section 4 names
 * stochastic rounding for the gradients and gives no formula for the draw;
 * reading: a 16-bit uniform draw cut from the element's Philox word, the high
 * half-word for an 8-bit code and the low half-word for a 16-bit code.  The
 * two copies of one gradient tensor (Gradients Bifurcation: same seed, same
 * tensor id, same element index, hence the same word) then draw from
 * disjoint bits of that word, i.e. independently. */
static int32_t quantize_one(float x, float inv_scale, int32_t zp_u, int32_t L,
                            int rounding, uint32_t rnd)
{
    float t = fmaf(x, inv_scale, (float)zp_u);
    float c;
    if (rounding == 0) {
        c = rintf(t);
    } else {
        float f = floorf(t);
        float frac = t - f;
        uint32_t draw = (L == 255) ? (rnd >> 16) : (rnd & 0xFFFFu);
        float u = (float)draw * 0x1p-16f;
        c = f + ((u < frac) ? 1.0f : 0.0f);
    }
    if (c < 0.0f) c = 0.0f;
    if (c > (float)L) c = (float)L;
    return (int32_t)c;
}

/* Quantise x[rows x cols] (cols innermost) to `bits` in {8,16}.
 * range_in (nullable): clamping values supplied by the caller, e.g. by the
 * preceding Range BN: [vmin, vmax] per tensor, or vmin[cols] then vmax[cols].
 * Outputs: signed stored codes (q8 for bits=8, q16 for bits=16), and per
 * tensor (or per channel) scale, stored zero-point, vmin, vmax as used. */
void qbo_quantize_at(const float *x, int64_t rows, int64_t cols, int bits,
                     int per_channel, int rounding, uint64_t seed, uint32_t tensor_id,
                     uint64_t index_base, const float *range_in,
                     int8_t *q8, int16_t *q16,
                     float *scale, int32_t *zero_point, float *vmin, float *vmax);

void qbo_quantize(const float *x, int64_t rows, int64_t cols, int bits,
                  int per_channel, int rounding, uint64_t seed, uint32_t tensor_id,
                  const float *range_in,
                  int8_t *q8, int16_t *q16,
                  float *scale, int32_t *zero_point, float *vmin, float *vmax)
{
    qbo_quantize_at(x, rows, cols, bits, per_channel, rounding, seed, tensor_id, 0, range_in,
                    q8, q16, scale, zero_point, vmin, vmax);
}

/* The same for a block of rows cut out of a larger tensor: index_base is the
 * flat index of x[0] in that tensor, so that element i draws the random word
 * of position index_base + i (the data-parallel case: each GPU holds some of
 * the rows of one gradient tensor). */
void qbo_quantize_at(const float *x, int64_t rows, int64_t cols, int bits,
                     int per_channel, int rounding, uint64_t seed, uint32_t tensor_id,
                     uint64_t index_base, const float *range_in,
                     int8_t *q8, int16_t *q16,
                     float *scale, int32_t *zero_point, float *vmin, float *vmax)
{
    const int64_t nq = per_channel ? cols : 1;
    const int32_t L = (1 << bits) - 1;
    const int32_t half = 1 << (bits - 1);
    float *lo = (float *)malloc(sizeof(float) * (size_t)nq);
    float *hi = (float *)malloc(sizeof(float) * (size_t)nq);
    if (range_in) {
        memcpy(lo, range_in, sizeof(float) * (size_t)nq);
        memcpy(hi, range_in + nq, sizeof(float) * (size_t)nq);
    } else {
        qbo_range(x, rows, cols, per_channel, lo, hi);
    }
    for (int64_t c = 0; c < nq; ++c)
        qbo_qparams(lo[c], hi[c], bits, &scale[c], &zero_point[c], &vmin[c], &vmax[c]);
    free(lo); free(hi);

    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t c = 0; c < cols; ++c) {
            int64_t i = r * cols + c;
            int64_t p = per_channel ? c : 0;
            float inv = 1.0f / scale[p];
            int32_t zp_u = zero_point[p] + half;
            uint32_t rnd = rounding ? qbo_random_word(seed, tensor_id, index_base + (uint64_t)i) : 0u;
            int32_t code = quantize_one(x[i], inv, zp_u, L, rounding, rnd) - half;
            if (bits == 8) q8[i] = (int8_t)code; else q16[i] = (int16_t)code;
        }
    }
}

/* x~ = scale * (q - zero_point) */
void qbo_dequantize_s8(const int8_t *q, int64_t n, float scale, int32_t zp, float *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = scale * (float)((int32_t)q[i] - zp);
}
void qbo_dequantize_s16(const int16_t *q, int64_t n, float scale, int32_t zp, float *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = scale * (float)((int32_t)q[i] - zp);
}

/* 16-bit code -> signed high byte and unsigned low byte, q = 256*hi + lo. */
void qbo_limb_split(const int16_t *q, int64_t n, int8_t *hi, uint8_t *lo)
{
    for (int64_t i = 0; i < n; ++i) {
        int32_t v = q[i];
        int32_t l = v & 0xFF;
        hi[i] = (int8_t)((v - l) / 256);
        lo[i] = (uint8_t)l;
    }
}

/* ------------------------------------------------------------------------ */
/* Integer products (Section 4: y = W x, Eq. grad_layer, Eq. grad_weight)    */
/* ------------------------------------------------------------------------ */

/* acc[m,n] = sum_k (A[m,k]-za)(B[k,n]-zb); A, B addressed by (row stride,
 * col stride) in elements so that either may be a transposed view.
 * out (nullable) = (float)acc * (sa*sb).  Returns the number of outputs whose
 * exact value does not fit int32 (0 when all fit). */
int64_t qbo_gemm_s8(int64_t M, int64_t N, int64_t K,
                    const int8_t *A, int64_t a_rs, int64_t a_cs, int32_t za,
                    const int8_t *B, int64_t b_rs, int64_t b_cs, int32_t zb,
                    int32_t *acc, float sa, float sb, float *out)
{
    int64_t bad = 0;
    const float s = sa * sb;
    #pragma omp parallel for schedule(static) reduction(+:bad)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int64_t sum = 0;
            for (int64_t k = 0; k < K; ++k)
                sum += (int64_t)((int32_t)A[m * a_rs + k * a_cs] - za) *
                       (int64_t)((int32_t)B[k * b_rs + n * b_cs] - zb);
            if (sum > INT32_MAX || sum < INT32_MIN) ++bad;
            if (acc) acc[m * N + n] = (int32_t)sum;
            if (out) out[m * N + n] = (float)(int32_t)sum * s;
        }
    return bad;
}

/* Weight gradient of a linear layer, Eq. grad_weight: 8-bit layer input
 * times the 16-bit copy of the gradient, reduced over the batch rows:
 * acc[k,n] = sum_m (X[m,k]-zx)(G[m,n]-zg), int64.  out = (float)acc*(sx*sg). */
void qbo_gemm_s16s8(int64_t M, int64_t N, int64_t K,
                    const int8_t *X, int32_t zx, const int16_t *G, int32_t zg,
                    int64_t *acc, float sx, float sg, float *out)
{
    const float s = sx * sg;
    #pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < K; ++k)
        for (int64_t n = 0; n < N; ++n) {
            int64_t sum = 0;
            for (int64_t m = 0; m < M; ++m)
                sum += (int64_t)((int32_t)X[m * K + k] - zx) *
                       (int64_t)((int32_t)G[m * N + n] - zg);
            if (acc) acc[k * N + n] = sum;
            if (out) out[k * N + n] = (float)sum * s;
        }
}

/* The same product written with the two byte limbs of G (q = 256*hi + lo):
 * 256*sum(x*hi) + sum(x*lo), zero-points applied to the recombined value. */
void qbo_gemm_limbs(int64_t M, int64_t N, int64_t K,
                    const int8_t *X, int32_t zx, const int8_t *Ghi, const uint8_t *Glo,
                    int32_t zg, int64_t *acc)
{
    for (int64_t k = 0; k < K; ++k)
        for (int64_t n = 0; n < N; ++n) {
            int64_t phi = 0, plo = 0, sx = 0, sg = 0;
            for (int64_t m = 0; m < M; ++m) {
                int64_t xv = X[m * K + k];
                phi += xv * Ghi[m * N + n];
                plo += xv * Glo[m * N + n];
                sx += xv;
                sg += 256 * (int64_t)Ghi[m * N + n] + Glo[m * N + n];
            }
            acc[k * N + n] = 256 * phi + plo - (int64_t)zg * sx - (int64_t)zx * sg
                             + M * (int64_t)zx * zg;
        }
}

/* ------------------------------------------------------------------------ */
/* Convolution as the same three products (activations NHWC, filters KRSC)   */
/* ------------------------------------------------------------------------ */

typedef struct {
    int64_t N, H, W, C;      /* input  [N,H,W,C]            */
    int64_t K, R, S;         /* filter [K,R,S,C]            */
    int64_t stride, pad;
    int64_t P, Q;            /* output [N,P,Q,K]            */
} qbo_conv_desc;

/* Forward: acc[n,p,q,k] = sum over in-bounds taps (r,s) and c of
 * (x[n,p*st-pad+r,q*st-pad+s,c]-zx)(w[k,r,s,c]-zw).  Padding is real zero. */
static int64_t conv_fprop_one(const qbo_conv_desc *d, const int8_t *x, int32_t zx,
                              const int8_t *w, int32_t zw, int64_t o)
{
    int64_t k = o % d->K; int64_t t = o / d->K;
    int64_t q = t % d->Q; t /= d->Q;
    int64_t p = t % d->P; int64_t n = t / d->P;
    int64_t sum = 0;
    for (int64_t r = 0; r < d->R; ++r) {
        int64_t h = p * d->stride - d->pad + r;
        if (h < 0 || h >= d->H) continue;
        for (int64_t s = 0; s < d->S; ++s) {
            int64_t ww = q * d->stride - d->pad + s;
            if (ww < 0 || ww >= d->W) continue;
            const int8_t *xp = x + ((n * d->H + h) * d->W + ww) * d->C;
            const int8_t *wp = w + ((k * d->R + r) * d->S + s) * d->C;
            for (int64_t c = 0; c < d->C; ++c)
                sum += (int64_t)((int32_t)xp[c] - zx) * (int64_t)((int32_t)wp[c] - zw);
        }
    }
    return sum;
}

/* Layer gradient (Eq. grad_layer): acc[n,h,w,c] = sum over (k,r,s) and the
 * output positions (p,q) with p*st-pad+r = h, q*st-pad+s = w of
 * (g[n,p,q,k]-zg)(w[k,r,s,c]-zw). */
static int64_t conv_dgrad_one(const qbo_conv_desc *d, const int8_t *g, int32_t zg,
                              const int8_t *w, int32_t zw, int64_t o)
{
    int64_t c = o % d->C; int64_t t = o / d->C;
    int64_t ww = t % d->W; t /= d->W;
    int64_t h = t % d->H; int64_t n = t / d->H;
    int64_t sum = 0;
    for (int64_t r = 0; r < d->R; ++r) {
        int64_t ph = h + d->pad - r;
        if (ph < 0 || ph % d->stride) continue;
        int64_t p = ph / d->stride;
        if (p >= d->P) continue;
        for (int64_t s = 0; s < d->S; ++s) {
            int64_t qw = ww + d->pad - s;
            if (qw < 0 || qw % d->stride) continue;
            int64_t q = qw / d->stride;
            if (q >= d->Q) continue;
            const int8_t *gp = g + ((n * d->P + p) * d->Q + q) * d->K;
            for (int64_t k = 0; k < d->K; ++k)
                sum += (int64_t)((int32_t)gp[k] - zg) *
                       (int64_t)((int32_t)w[((k * d->R + r) * d->S + s) * d->C + c] - zw);
        }
    }
    return sum;
}

/* Weight gradient (Eq. grad_weight): acc[k,r,s,c] = sum over (n,p,q) whose
 * tap is in bounds of (g16[n,p,q,k]-zg)(x[n,p*st-pad+r,q*st-pad+s,c]-zx). */
static int64_t conv_wgrad_one(const qbo_conv_desc *d, const int8_t *x, int32_t zx,
                              const int16_t *g, int32_t zg, int64_t o)
{
    int64_t c = o % d->C; int64_t t = o / d->C;
    int64_t s = t % d->S; t /= d->S;
    int64_t r = t % d->R; int64_t k = t / d->R;
    int64_t sum = 0;
    for (int64_t n = 0; n < d->N; ++n)
        for (int64_t p = 0; p < d->P; ++p) {
            int64_t h = p * d->stride - d->pad + r;
            if (h < 0 || h >= d->H) continue;
            for (int64_t q = 0; q < d->Q; ++q) {
                int64_t ww = q * d->stride - d->pad + s;
                if (ww < 0 || ww >= d->W) continue;
                sum += (int64_t)((int32_t)g[((n * d->P + p) * d->Q + q) * d->K + k] - zg) *
                       (int64_t)((int32_t)x[((n * d->H + h) * d->W + ww) * d->C + c] - zx);
            }
        }
    return sum;
}

/* mode 0 forward, 1 layer gradient.  idx (nullable): flat output indices to
 * evaluate (count outputs); NULL evaluates outputs 0..count-1 in order.
 * Returns how many evaluated outputs do not fit int32. */
int64_t qbo_conv_s8(int mode, const qbo_conv_desc *d,
                    const int8_t *in, int32_t z_in, const int8_t *w, int32_t zw,
                    const int64_t *idx, int64_t count,
                    int32_t *acc, float s_in, float s_w, float *out)
{
    int64_t bad = 0;
    const float s = s_in * s_w;
    #pragma omp parallel for schedule(dynamic, 256) reduction(+:bad)
    for (int64_t i = 0; i < count; ++i) {
        int64_t o = idx ? idx[i] : i;
        int64_t sum = mode == 0 ? conv_fprop_one(d, in, z_in, w, zw, o)
                                : conv_dgrad_one(d, in, z_in, w, zw, o);
        if (sum > INT32_MAX || sum < INT32_MIN) ++bad;
        if (acc) acc[i] = (int32_t)sum;
        if (out) out[i] = (float)(int32_t)sum * s;
    }
    return bad;
}

void qbo_conv_wgrad_s16(const qbo_conv_desc *d,
                        const int8_t *x, int32_t zx, const int16_t *g, int32_t zg,
                        const int64_t *idx, int64_t count,
                        int64_t *acc, float sx, float sg, float *out)
{
    const float s = sx * sg;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < count; ++i) {
        int64_t o = idx ? idx[i] : i;
        int64_t sum = conv_wgrad_one(d, x, zx, g, zg, o);
        if (acc) acc[i] = sum;
        if (out) out[i] = (float)sum * s;
    }
}

/* ------------------------------------------------------------------------ */
/* Range Batch-Normalization (Section 3, Eq. range; backward: Section 7)     */
/* ------------------------------------------------------------------------ */

/* C(n) = 1 / sqrt(2 ln n) */
double qbo_rangebn_C(int64_t n) { return 1.0 / sqrt(2.0 * log((double)n)); }

/* x [n x C] (channel innermost).  Per channel: mu = mean, range = max - min
 * (the range of x - mu equals the range of x), xhat = (x-mu)/(C(n)*range),
 * y = gamma*xhat + beta (NULL gamma/beta: 1, 0), optional ReLU.
 * A channel of zero range gives xhat = 0. */
void qbo_rangebn_fwd(const float *x, int64_t n, int64_t C,
                     const float *gamma, const float *beta, int relu,
                     double *y, double *mean, float *vmin, float *vmax)
{
    const double Cn = qbo_rangebn_C(n);
    #pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < C; ++c) {
        double sum = 0.0; float lo = INFINITY, hi = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            float v = x[i * C + c];
            sum += (double)v;
            if (v < lo) lo = v;
            if (v > hi) hi = v;
        }
        double mu = sum / (double)n;
        double r = (double)hi - (double)lo;
        double s = (r > 0.0) ? 1.0 / (Cn * r) : 0.0;
        double g = gamma ? (double)gamma[c] : 1.0, b = beta ? (double)beta[c] : 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double v = g * (((double)x[i * C + c] - mu) * s) + b;
            if (relu && v < 0.0) v = 0.0;
            y[i * C + c] = v;
        }
        mean[c] = mu; vmin[c] = lo; vmax[c] = hi;
    }
}

/* Backward.  Ordinary chain rule where d max/dx (d min/dx) is 1 at every
 * coordinate attaining the maximum (minimum) and 0 elsewhere:
 *   s = 1/(C(n) r), dbeta = sum dy, dgamma = sum dy*xhat,
 *   dx_j = s*( gamma*dy_j - gamma*dbeta/n - C(n)*gamma*dgamma*([x_j==max]-[x_j==min]) ).
 * save_mean/min/max are the forward's saved per-channel statistics (fp32).
 * With ReLU, dy_j is first zeroed where the forward output was not positive;
 * that on/off decision is evaluated in fp32 as fl(fl(gamma*fl(fl(x-mu)*s32))+beta) > 0
 * with s32 = 1.0f / fl((float)C(n) * r), the forward kernel's sequence. */
void qbo_rangebn_bwd(const float *dy, const float *x, int64_t n, int64_t C,
                     const float *gamma, const float *beta, int relu,
                     const float *save_mean, const float *save_min, const float *save_max,
                     double *dx, double *dgamma, double *dbeta)
{
    const double Cn = qbo_rangebn_C(n);
    const float Cn32 = (float)Cn;
    #pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < C; ++c) {
        float mu32 = save_mean[c], lo = save_min[c], hi = save_max[c];
        float r32 = hi - lo;
        float s32 = (r32 > 0.0f) ? 1.0f / (Cn32 * r32) : 0.0f;
        float g32 = gamma ? gamma[c] : 1.0f, b32 = beta ? beta[c] : 0.0f;
        double mu = (double)mu32;
        double r = (double)hi - (double)lo;
        double s = (r > 0.0) ? 1.0 / (Cn * r) : 0.0;
        double g = (double)g32;
        double sdy = 0.0, sdyx = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            float xv = x[i * C + c];
            double d = (double)dy[i * C + c];
            if (relu) {
                float xh = (xv - mu32) * s32;
                float yv = g32 * xh;
                yv = yv + b32;
                if (!(yv > 0.0f)) d = 0.0;
            }
            sdy += d;
            sdyx += d * (((double)xv - mu) * s);
        }
        double m1 = g * sdy / (double)n;
        double m2 = g * sdyx;
        for (int64_t i = 0; i < n; ++i) {
            float xv = x[i * C + c];
            double d = (double)dy[i * C + c];
            if (relu) {
                float xh = (xv - mu32) * s32;
                float yv = g32 * xh;
                yv = yv + b32;
                if (!(yv > 0.0f)) d = 0.0;
            }
            double ind = (xv == hi ? 1.0 : 0.0) - (xv == lo ? 1.0 : 0.0);
            dx[i * C + c] = s * (g * d - m1 - Cn * m2 * ind);
        }
        dgamma[c] = sdyx; dbeta[c] = sdy;
    }
}

/* ------------------------------------------------------------------------ */
/* fp32 weight update (Section 6: the updates are kept in float32)           */
/* ------------------------------------------------------------------------ */

/* g = dw + wd*w;  v = mu*v + g (when a momentum buffer is kept);  w = w - lr*v.
 * The paper fixes the precision (float32), so this is float arithmetic, every
 * operation rounded on its own in this order (no contraction). */
void qbo_sgd_update(float *w, const float *dw, float *vbuf, int64_t n, float lr, float mu, float wd)
{
    for (int64_t i = 0; i < n; ++i) {
        float t = wd * w[i];
        float g = dw[i] + t;
        if (vbuf) {
            float m = mu * vbuf[i];
            g = m + g;
            vbuf[i] = g;
        }
        float step = lr * g;
        w[i] = w[i] - step;
    }
}

/* ------------------------------------------------------------------------ */
/* Appendix C: Ternarized Back-Propagation (1-bit weights and activations,   */
/* ternary gradients, XNOR + popcount products) and Algorithm 1              */
/* ------------------------------------------------------------------------ */

/* 1-bit weights / activations: b(x) = +1 for x >= 0, else -1 (the
 * deterministic sign of the binarised networks Appendix C builds on). */
void qbo_binarize(const float *x, int64_t n, int8_t *b)
{
    for (int64_t i = 0; i < n; ++i) b[i] = (x[i] >= 0.0f) ? 1 : -1;
}

/* [rows x cols] codes of +-1 (or a 0/1 mask when `mask`) to bit rows: element
 * c of a row is bit c % 32 of word c / 32 (1 = "+1" or "set"); a row takes
 * ceil(cols / 32) words, the spare bits of the last word are 0. */
void qbo_pack_bits(const int8_t *b, int64_t rows, int64_t cols, int mask, uint32_t *words)
{
    int64_t wpr = (cols + 31) / 32;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t w = 0; w < wpr; ++w) {
            uint32_t v = 0;
            for (int64_t c = w * 32; c < cols && c < w * 32 + 32; ++c) {
                int on = mask ? (b[r * cols + c] != 0) : (b[r * cols + c] > 0);
                if (on) v |= 1u << (c - w * 32);
            }
            words[r * wpr + w] = v;
        }
}

static int popcount32(uint32_t v) { int n = 0; while (v) { n += (int)(v & 1u); v >>= 1; } return n; }

/* Forward product of a binarised layer (Appendix C: every MAC replaced by
 * XNOR and population count): A [M x K bits], B [N x K bits], both as rows
 * of ceil(K/32) words; C[m][n] = sum_k a*b over +-1 values
 *   = (#equal bits) - (#different bits) = K - 2 popcount(a xor b). */
void qbo_xnor_gemm(int64_t M, int64_t N, int64_t K, const uint32_t *A, const uint32_t *B, int32_t *C)
{
    int64_t wpr = (K + 31) / 32;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int diff = 0;
            for (int64_t w = 0; w < wpr; ++w) diff += popcount32(A[m * wpr + w] ^ B[n * wpr + w]);
            C[m * N + n] = (int32_t)(K - 2 * diff);      /* (spare bits are 0 in both: they never differ) */
        }
}

/* Random word of element i for sample `sample`: as qbo_random_word, with the
 * sample index in the last counter word. */
uint32_t qbo_random_word_sample(uint64_t seed, uint32_t tensor_id, uint64_t i, uint32_t sample)
{
    uint64_t j = i >> 2;
    uint32_t ctr[4] = { (uint32_t)j, (uint32_t)(j >> 32), tensor_id, sample };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    qbo_philox4x32_10(ctr, key, out);
    return out[i & 3];
}

/* Stochastic ternarisation StcTern (Appendix C; the paper names it without a
 * formula -- the reading taken is the one of the ternary-gradient work it
 * cites): s = max |g| over the tensor, t_i = sign(g_i) with probability
 * |g_i| / s, else 0, so that E[s t_i] = g_i.  The draw decides an integer, so
 * it is taken in fp32 in a fixed order: u = (word >> 8) * 2^-24 (exact),
 * t_i != 0 iff u * s < |g_i| (one fp32 product, rounded to nearest: for
 * |g_i| = s it is always below s, so the largest element is always kept).
 * Returns s. */
float qbo_stc_tern(const float *g, int64_t n, uint64_t seed, uint32_t tensor_id, uint32_t sample, int8_t *t)
{
    float s = 0.0f;
    for (int64_t i = 0; i < n; ++i) { float a = fabsf(g[i]); if (a > s) s = a; }
    for (int64_t i = 0; i < n; ++i) {
        int8_t v = 0;
        if (s > 0.0f) {
            float u = (float)(qbo_random_word_sample(seed, tensor_id, (uint64_t)i, sample) >> 8) * 0x1p-24f;
            float us = u * s;
            if (us < fabsf(g[i])) v = (g[i] > 0.0f) ? 1 : -1;
        }
        t[i] = v;
    }
    return s;
}

/* Backward product with ternary gradients and binary weights (the "gated
 * XNOR"): T [M x K] ternary as two bit planes (nz: t != 0, sg: t > 0),
 * B [N x K bits]; C[m][n] = sum_k t*b = popcount(nz & ~(sg ^ b)) -
 * popcount(nz & (sg ^ b)): where t is non-zero, equal signs add one and
 * different signs take one away. */
void qbo_gated_xnor_gemm(int64_t M, int64_t N, int64_t K, const uint32_t *nz, const uint32_t *sg,
                         const uint32_t *B, int32_t *C)
{
    int64_t wpr = (K + 31) / 32;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int acc = 0;
            for (int64_t w = 0; w < wpr; ++w) {
                uint32_t z = nz[m * wpr + w], d = sg[m * wpr + w] ^ B[n * wpr + w];
                acc += popcount32(z & ~d) - popcount32(z & d);
            }
            C[m * N + n] = acc;
        }
}

/* Algorithm 1 (multiple stochastic ternarisation sampling for the update
 * phase): g [rows x N] gradients at the layer's output, a [rows x K] binarised
 * activations (+-1); for every sample: ternarise g, add the product of the
 * ternary tensor with the activations to the accumulator; return the
 * accumulator over the number of samples.  gW [K x N], in units of g: the
 * ternary values stand for s t.  The products are integers: they are
 * accumulated exactly (int64) and scaled once at the end. */
void qbo_tbp_update(const float *g, const int8_t *a, int64_t rows, int64_t N, int64_t K, int samples,
                    uint64_t seed, uint32_t tensor_id, double *gW)
{
    int8_t *t = (int8_t *)malloc((size_t)(rows * N));
    int64_t *acc = (int64_t *)calloc((size_t)(K * N), sizeof(int64_t));
    float s = 0.0f;
    for (int k = 0; k < samples; ++k) {
        s = qbo_stc_tern(g, rows * N, seed, tensor_id, (uint32_t)k, t);
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t c = 0; c < K; ++c)
                for (int64_t n = 0; n < N; ++n)
                    acc[c * N + n] += (int64_t)a[r * K + c] * (int64_t)t[r * N + n];
    }
    for (int64_t i = 0; i < K * N; ++i) gW[i] = (double)s * (double)acc[i] / (double)samples;
    free(t); free(acc);
}
