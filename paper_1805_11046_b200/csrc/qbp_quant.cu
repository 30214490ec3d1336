// Range quantiser kernels (Section 4 "Quantization methods", Appendix B):
// min/max range scan, scale / zero-point, nearest and stochastic rounding to
// 8 and 16 bits, byte-limb split of the 16-bit codes, and the fused
// "bifurcation" that writes the 8-bit and 16-bit copies of a gradient from
// one read.  All of it is HBM-bound streaming work: 16-byte loads, 4 loads in
// flight per thread, warp-shuffle + shared-memory reductions, grids sized to
// fill every SM.  Also hosts the library's error-reporting state.
#include "qbp_colscan.cuh"

#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>

namespace qbp {

// ------------------------------------------------------------ error state
static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap; va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}
int fail(int status, const char *fmt, ...)
{
    va_list ap; va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return status;
}
int sm_count()
{
    static thread_local int cached_dev = -1, cached = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) cached = n;
        else cudaGetLastError();
        cached_dev = dev;
    }
    return cached;
}

// ------------------------------------------------------------ launch tracing
struct TraceRec { const char *name; cudaEvent_t a, b; };
static bool g_trace_on = false;
static std::vector<TraceRec> g_trace;
static std::vector<cudaEvent_t> g_event_pool;

static cudaEvent_t pool_event()
{
    if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}
void trace_begin(cudaStream_t st)
{
    if (!g_trace_on) return;
    TraceRec r{nullptr, pool_event(), pool_event()};
    cudaEventRecord(r.a, st);
    g_trace.push_back(r);
}
void trace_end(const char *name, cudaStream_t st)
{
    if (!g_trace_on || g_trace.empty() || g_trace.back().name) return;
    g_trace.back().name = name;
    cudaEventRecord(g_trace.back().b, st);
}

constexpr int kThreads = 256;
constexpr int kUnroll = 4;
constexpr int kRangeUnroll = 8;          // loads in flight per thread of the read-only range scan
constexpr int kMaxParts = 4096;          // upper bound on per-tensor scan blocks

// ------------------------------------------------------- per-tensor range
// keep_rev: the tensor is walked from its end with loads that leave the lines in the L2 -- for the layer's input, whose
// quantiser follows from the front and so finds the first 100 MB there (scan +3 us, quantiser -3 us, step -2.5 us).
template <int VEC>
__global__ void __launch_bounds__(kThreads) range_partial_kernel(const float *__restrict__ x, int64_t n,
                                                                 float2 *__restrict__ partials, int keep_rev)
{
    float lo = INFINITY, hi = -INFINITY;
    const int64_t nv = n / VEC;
    const int64_t stride = (int64_t)gridDim.x * kThreads * kRangeUnroll;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * kRangeUnroll; base < nv; base += stride) {
        VecF<VEC> v[kRangeUnroll];
        bool ok[kRangeUnroll];
#pragma unroll
        for (int u = 0; u < kRangeUnroll; ++u) {
            int64_t i = base + u * kThreads + threadIdx.x;
            ok[u] = i < nv;
            if (ok[u]) { if (keep_rev) v[u].load(x + (nv - 1 - i) * VEC); else v[u].load_stream(x + i * VEC); }
        }
#pragma unroll
        for (int u = 0; u < kRangeUnroll; ++u)
            if (ok[u]) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) { lo = fminf(lo, v[u].v[e]); hi = fmaxf(hi, v[u].v[e]); }
            }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (int64_t i = nv * VEC; i < n; ++i) { lo = fminf(lo, x[i]); hi = fmaxf(hi, x[i]); }
    lo = warp_min(lo); hi = warp_max(hi);
    __shared__ float s_lo[kThreads / 32], s_hi[kThreads / 32];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x < 32) {
        lo = threadIdx.x < kThreads / 32 ? s_lo[threadIdx.x] : INFINITY;
        hi = threadIdx.x < kThreads / 32 ? s_hi[threadIdx.x] : -INFINITY;
        lo = warp_min(lo); hi = warp_max(hi);
        if (threadIdx.x == 0) partials[blockIdx.x] = make_float2(lo, hi);
    }
}

// One block: combine the partial ranges, emit the parameters for 8 and/or 16 bits.
__global__ void __launch_bounds__(kThreads) range_finalize_kernel(const float2 *__restrict__ partials, int nparts,
                                                                  qbp_qparams *qp8, qbp_qparams *qp16)
{
    float lo = INFINITY, hi = -INFINITY;
    for (int i = threadIdx.x; i < nparts; i += kThreads) {
        float2 p = partials[i];
        lo = fminf(lo, p.x); hi = fmaxf(hi, p.y);
    }
    lo = warp_min(lo); hi = warp_max(hi);
    __shared__ float s_lo[kThreads / 32], s_hi[kThreads / 32];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 0; w < kThreads / 32; ++w) { lo = fminf(lo, s_lo[w]); hi = fmaxf(hi, s_hi[w]); }
        if (qp8) *qp8 = make_qparams(lo, hi, 8);
        if (qp16) *qp16 = make_qparams(lo, hi, 16);
    }
}

// ---------------------------------------------- chunk-averaged clamping values
// Appendix B, activations: the clamping values are the averages, over K chunks of the tensor, of the chunks'
// minima and maxima.  blockIdx.y = chunk (equal contiguous runs of n_chunk elements), blockIdx.x = block inside it.
template <int VEC>
__global__ void __launch_bounds__(kThreads) chunk_range_partial_kernel(const float *__restrict__ x, int64_t n_chunk,
                                                                       float2 *__restrict__ partials)
{
    x += (int64_t)blockIdx.y * n_chunk;
    float lo = INFINITY, hi = -INFINITY;
    const int64_t nv = n_chunk / VEC;              // (VEC = 4 only when n_chunk is a multiple of 4)
    const int64_t stride = (int64_t)gridDim.x * kThreads * kRangeUnroll;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * kRangeUnroll; base < nv; base += stride) {
        VecF<VEC> v[kRangeUnroll];
        bool ok[kRangeUnroll];
#pragma unroll
        for (int u = 0; u < kRangeUnroll; ++u) {
            int64_t i = base + u * kThreads + threadIdx.x;
            ok[u] = i < nv;
            if (ok[u]) v[u].load_stream(x + i * VEC);
        }
#pragma unroll
        for (int u = 0; u < kRangeUnroll; ++u)
            if (ok[u]) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) { lo = fminf(lo, v[u].v[e]); hi = fmaxf(hi, v[u].v[e]); }
            }
    }
    lo = warp_min(lo); hi = warp_max(hi);
    __shared__ float s_lo[kThreads / 32], s_hi[kThreads / 32];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x < 32) {
        lo = threadIdx.x < kThreads / 32 ? s_lo[threadIdx.x] : INFINITY;
        hi = threadIdx.x < kThreads / 32 ? s_hi[threadIdx.x] : -INFINITY;
        lo = warp_min(lo); hi = warp_max(hi);
        if (threadIdx.x == 0) partials[(int64_t)blockIdx.y * gridDim.x + blockIdx.x] = make_float2(lo, hi);
    }
}

// One block: every chunk's (min, max) from its blocks' partials (a warp per chunk, the lanes stride over the
// chunk's blocks), then the two averages, added up in chunk order in double by one thread (the order is part of
// the result: the result depends on it, and the CPU check adds them up the same way).
__global__ void __launch_bounds__(kThreads) chunk_range_finalize_kernel(const float2 *__restrict__ partials, int chunks,
                                                                        int blocks_per_chunk, float2 *__restrict__ per_chunk,
                                                                        qbp_qparams *__restrict__ out)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int k = warp; k < chunks; k += kThreads / 32) {
        float lo = INFINITY, hi = -INFINITY;
        for (int b = lane; b < blocks_per_chunk; b += 32) {
            const float2 p = partials[(int64_t)k * blocks_per_chunk + b];
            lo = fminf(lo, p.x); hi = fmaxf(hi, p.y);
        }
        lo = warp_min(lo); hi = warp_max(hi);
        if (lane == 0) per_chunk[k] = make_float2(lo, hi);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double slo = 0.0, shi = 0.0;
        for (int k = 0; k < chunks; ++k) { slo += (double)per_chunk[k].x; shi += (double)per_chunk[k].y; }
        qbp_qparams r;
        r.scale = 0.0f; r.zero_point = 0;
        r.vmin = (float)(slo / (double)chunks); r.vmax = (float)(shi / (double)chunks);
        *out = r;
    }
}

// Parameters from clamping values the caller already has (one thread each).
__global__ void qparams_from_range_kernel(const qbp_qparams *__restrict__ in, int count, int bits,
                                          qbp_qparams *__restrict__ out)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) out[i] = make_qparams(in[i].vmin, in[i].vmax, bits);
}

// ------------------------------------------------------ per-channel range
template <int VEC>
__global__ void __launch_bounds__(kScanThreads) chan_range_partial_kernel(const float *__restrict__ x, int64_t rows,
                                                                          int C, int tw, float *__restrict__ part_lo,
                                                                          float *__restrict__ part_hi)
{
    const ScanPos p = scan_pos<VEC>(C, tw);
    const int rpb = kScanThreads / tw;
    float lo[VEC], hi[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) { lo[e] = INFINITY; hi[e] = -INFINITY; }
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
                    for (int e = 0; e < VEC; ++e) { lo[e] = fminf(lo[e], v[u].v[e]); hi[e] = fmaxf(hi[e], v[u].v[e]); }
                }
        }
    }
    __shared__ float s_lo[kScanThreads * VEC], s_hi[kScanThreads * VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) { s_lo[threadIdx.x * VEC + e] = lo[e]; s_hi[threadIdx.x * VEC + e] = hi[e]; }
    __syncthreads();
    if (p.ty == 0 && p.active) {
        for (int y = 1; y < rpb; ++y)
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                lo[e] = fminf(lo[e], s_lo[(y * tw + p.tx) * VEC + e]);
                hi[e] = fmaxf(hi[e], s_hi[(y * tw + p.tx) * VEC + e]);
            }
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            part_lo[(int64_t)blockIdx.x * C + p.col + e] = lo[e];
            part_hi[(int64_t)blockIdx.x * C + p.col + e] = hi[e];
        }
    }
}

// One warp per channel over the strip partials.
__global__ void __launch_bounds__(kThreads) chan_range_finalize_kernel(const float *__restrict__ part_lo,
                                                                       const float *__restrict__ part_hi, int nparts,
                                                                       int C, int bits, qbp_qparams *__restrict__ qp)
{
    int c = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (c >= C) return;
    float lo = INFINITY, hi = -INFINITY;
    for (int i = threadIdx.x & 31; i < nparts; i += 32) {
        lo = fminf(lo, part_lo[(int64_t)i * C + c]);
        hi = fmaxf(hi, part_hi[(int64_t)i * C + c]);
    }
    lo = warp_min(lo); hi = warp_max(hi);
    if ((threadIdx.x & 31) == 0) qp[c] = make_qparams(lo, hi, bits);
}

// ------------------------------------------------------------ quantisation
struct QuantOut {
    int8_t *q8;      // 8-bit codes (nullable)
    int16_t *q16;    // 16-bit codes (nullable)
    int8_t *hi;      // high byte of the 16-bit code (nullable)
    uint8_t *lo;     // low byte (nullable)
    int32_t *rowsum8;   // sums of the stored 8-bit codes over each row of `cols` (nullable; vector path only)
    int rs_group;       // lanes that share a row: cols / 4, a power of two <= 32
    int rs_shift;       // log2(rs_group)
    // Per-channel totals of the stored codes over all rows, added (64-bit atomics) to chansum8 [cols] / chansum16
    // [cols] (nullable; vector path, per tensor, cols / 4 a power of two <= 256: a thread then keeps its four
    // channels for its whole life).  The weight gradient's zero-point terms are built from such totals.
    unsigned long long *chansum8, *chansum16;
    // 0x80808080: the low bytes are stored with their top bit flipped, i.e. as the signed bytes lo - 128 (the weight
    // gradient then runs both limbs as one s8 x s8 product); 0: plain unsigned low bytes.
    uint32_t lo_flip;
};

struct QParamsReg { float inv, zp_u; };

__device__ __forceinline__ QParamsReg load_qp(const qbp_qparams *qp, int bits)
{
    QParamsReg r;
    r.inv = __fdiv_rn(1.0f, qp->scale);
    r.zp_u = (float)(qp->zero_point + (1 << (bits - 1)));
    return r;
}

// Scalar path: unaligned tensors, per-element tails.  One Philox block per element.
template <bool SR>
__device__ __forceinline__ void quantize_scalar(const float *x, int64_t i, int cols, bool perch,
                                                const qbp_qparams *qp8, uint32_t id8, const qbp_qparams *qp16,
                                                uint32_t id16, const PhiloxKeys &key, const QuantOut &o, uint64_t index_base)
{
    const int c = perch ? (int)(i % cols) : 0;
    const float v = x[i];
    const uint64_t j = ((uint64_t)i + index_base) >> 2;          // (index_base is a multiple of 4: word i & 3 is unchanged)
    if (o.q8) {
        QParamsReg p = load_qp(qp8 + c, 8);
        uint32_t rnd = 0;
        if (SR) {
            uint4 b = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)(j >> 32), id8, 0u), key);
            const uint32_t w[4] = {b.x, b.y, b.z, b.w};
            rnd = w[i & 3];
        }
        o.q8[i] = (int8_t)(quantize_code<SR>(v, p.inv, p.zp_u, 255.0f, rnd) - 128);
    }
    if (o.q16 || o.hi || o.lo) {
        QParamsReg p = load_qp(qp16 + c, 16);
        uint32_t rnd = 0;
        if (SR) {
            uint4 b = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)(j >> 32), id16, 0u), key);
            const uint32_t w[4] = {b.x, b.y, b.z, b.w};
            rnd = w[i & 3];
        }
        int s = quantize_code<SR>(v, p.inv, p.zp_u, 65535.0f, rnd) - 32768;
        if (o.q16) o.q16[i] = (int16_t)s;
        if (o.hi) o.hi[i] = (int8_t)(s >> 8);
        if (o.lo) o.lo[i] = (uint8_t)((s & 0xFF) ^ (o.lo_flip & 0xFF));
    }
}

// Four codes (low bytes of c[0..3]) into one word.
__device__ __forceinline__ uint32_t pack_bytes0(const uint32_t (&c)[4])
{
    return __byte_perm(__byte_perm(c[0], c[1], 0x0040), __byte_perm(c[2], c[3], 0x0040), 0x5410);
}
// The top bytes of c[0..3] into one word.
__device__ __forceinline__ uint32_t pack_bytes3(const uint32_t (&c)[4])
{
    return __byte_perm(__byte_perm(c[0], c[1], 0x0073), __byte_perm(c[2], c[3], 0x0073), 0x5410);
}
// The second bytes of c[0..3] into one word.
__device__ __forceinline__ uint32_t pack_bytes1(const uint32_t (&c)[4])
{
    return __byte_perm(__byte_perm(c[0], c[1], 0x0051), __byte_perm(c[2], c[3], 0x0051), 0x5410);
}
// The third bytes of c[0..3] into one word.
__device__ __forceinline__ uint32_t pack_bytes2(const uint32_t (&c)[4])
{
    return __byte_perm(__byte_perm(c[0], c[1], 0x0062), __byte_perm(c[2], c[3], 0x0062), 0x5410);
}

// PERCH is a template parameter so that the per-tensor instance (the hot one: it is bound by its instruction
// count when rounding stochastically) carries none of the per-channel parameter handling.
// TOTALS: the instance that also leaves the per-channel totals (the others carry none of that work).
template <bool SR, int VEC, bool PERCH, bool TOTALS>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const float *__restrict__ x, int64_t n, int cols,
                                                            const qbp_qparams *__restrict__ qp8,
                                                            uint32_t id8, const qbp_qparams *__restrict__ qp16,
                                                            uint32_t id16, const __grid_constant__ PhiloxKeys keys,
                                                            QuantOut o, int smem_cols, uint64_t index_base)
{
    if (VEC == 1) {
        const int64_t stride = (int64_t)gridDim.x * kThreads;
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride)
            quantize_scalar<SR>(x, i, cols, PERCH, qp8, id8, qp16, id16, keys, o, index_base);
        return;
    }
    const bool want8 = o.q8 != nullptr, want16 = o.q16 || o.hi || o.lo;
    QParamsReg p8 = {0, 0}, p16 = {0, 0};
    // per channel: (1/scale, zero-point) of every channel once per block in shared memory (when the launcher
    // gave it room), instead of a division per element
    extern __shared__ float2 s_qp[];                         // [cols] for 8 bits, then [cols] for 16 bits
    const bool table = PERCH && smem_cols > 0;
    if (table) {
        for (int c = threadIdx.x; c < cols; c += kThreads) {
            if (want8)  { QParamsReg t = load_qp(qp8 + c, 8);   s_qp[c] = make_float2(t.inv, t.zp_u); }
            if (want16) { QParamsReg t = load_qp(qp16 + c, 16); s_qp[cols + c] = make_float2(t.inv, t.zp_u); }
        }
        __syncthreads();
    }
    if (!PERCH) {
        if (want8) p8 = load_qp(qp8, 8);
        if (want16) p16 = load_qp(qp16, 16);
        // the stochastic codes are taken in fixed point with 16 fraction bits: fold the factor into the parameters
        if (SR) { p8.inv *= 65536.0f; p8.zp_u *= 65536.0f; p16.inv *= 65536.0f; p16.zp_u *= 65536.0f; }
    }
    // both copies of a gradient under one tensor id: one Philox block serves the two (disjoint halves of each word)
    const bool one_block = want8 && want16 && id8 == id16;
    int cs8[4] = {0, 0, 0, 0};                               // this thread's channels: totals of the stored 8-bit codes
    unsigned cs16[4] = {0, 0, 0, 0};                         // ... and of the unsigned 16-bit codes (fewer than 65536 per thread)
    const int64_t nv = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * kThreads * kUnroll;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * kUnroll; base < nv; base += stride) {
        float4 v[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            int64_t j = base + u * kThreads + threadIdx.x;
            ok[u] = j < nv;
            // nearest rounding follows a range scan of the same (large) tensor and is bound by HBM: evict-first loads;
            // the stochastic instance is bound by arithmetic and often finds the tail of its input in the L2
            if (ok[u]) v[u] = SR ? __ldg(reinterpret_cast<const float4 *>(x) + j) : __ldcs(reinterpret_cast<const float4 *>(x) + j);
        }
        int rs[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) rs[u] = 0;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (!ok[u]) continue;
            const int64_t j = base + u * kThreads + threadIdx.x;
            const float xs[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            const int c0 = PERCH ? (int)((j << 2) % cols) : 0;
            uint4 b8 = make_uint4(0, 0, 0, 0), b16 = b8;
            if (SR) {
                // counter = the block's index in the whole tensor (a shard of a larger tensor starts at index_base)
                const uint64_t jb = (uint64_t)j + (index_base >> 2);
                if (want8) b8 = philox4x32_10(make_uint4((uint32_t)jb, (uint32_t)(jb >> 32), id8, 0u), keys);
                if (want16) b16 = one_block ? b8 : philox4x32_10(make_uint4((uint32_t)jb, (uint32_t)(jb >> 32), id16, 0u), keys);
            }
            if (want8) {
                const uint32_t r[4] = {b8.x, b8.y, b8.z, b8.w};
                uint32_t c[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (PERCH) {
                        if (table) { const float2 t = s_qp[c0 + e]; p8.inv = t.x; p8.zp_u = t.y; }
                        else p8 = load_qp(qp8 + c0 + e, 8);
                        if (SR) { p8.inv *= 65536.0f; p8.zp_u *= 65536.0f; }
                    }
                    c[e] = SR ? quantize_sr8_byte2(xs[e], p8.inv, p8.zp_u, r[e])
                              : (uint32_t)quantize_code<SR>(xs[e], p8.inv, p8.zp_u, 255.0f, r[e]);
                }
                const uint32_t packed = (SR ? pack_bytes2(c) : pack_bytes0(c)) ^ 0x80808080u;       // stored = unsigned code - 128
                reinterpret_cast<uint32_t *>(o.q8)[j] = packed;
                if (o.rowsum8) rs[u] = __dp4a((int)packed, 0x01010101, 0);
                if (TOTALS && o.chansum8) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) cs8[e] = __dp4a((int)packed, 1 << (8 * e), cs8[e]);
                }
            }
            if (want16) {
                const uint32_t r[4] = {b16.x, b16.y, b16.z, b16.w};
                uint32_t c[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (PERCH) {
                        if (table) { const float2 t = s_qp[cols + c0 + e]; p16.inv = t.x; p16.zp_u = t.y; }
                        else p16 = load_qp(qp16 + c0 + e, 16);
                        if (SR) { p16.inv *= 65536.0f; p16.zp_u *= 65536.0f; }
                    }
                    // (stochastic: the code sits in the upper half of the word, i.e. bytes 3 and 2)
                    c[e] = SR ? quantize_sr16_top_half(xs[e], p16.inv, p16.zp_u, r[e])
                              : (uint32_t)quantize_code<SR>(xs[e], p16.inv, p16.zp_u, 65535.0f, r[e]);
                }
                if (TOTALS && o.chansum16) {
                    // unsigned codes here (the offset of 32768 per element is taken off when the block adds its totals up)
#pragma unroll
                    for (int e = 0; e < 4; ++e) cs16[e] += SR ? c[e] >> 16 : c[e];
                }
                // stored = unsigned code - 32768: flip the top bit of every code (of every high byte)
                if (o.q16)
                    reinterpret_cast<uint2 *>(o.q16)[j] = make_uint2(__byte_perm(c[0], c[1], SR ? 0x7632 : 0x5410) ^ 0x80008000u,
                                                                     __byte_perm(c[2], c[3], SR ? 0x7632 : 0x5410) ^ 0x80008000u);
                if (SR && o.hi && o.lo) {
                    // (low, low, high, high) bytes of two codes each, then the two words: four permutes for both limbs
                    const uint32_t t01 = __byte_perm(c[0], c[1], 0x7362), t23 = __byte_perm(c[2], c[3], 0x7362);
                    reinterpret_cast<uint32_t *>(o.hi)[j] = __byte_perm(t01, t23, 0x7632) ^ 0x80808080u;
                    reinterpret_cast<uint32_t *>(o.lo)[j] = __byte_perm(t01, t23, 0x5410) ^ o.lo_flip;
                } else {
                    if (o.hi) reinterpret_cast<uint32_t *>(o.hi)[j] = (SR ? pack_bytes3(c) : pack_bytes1(c)) ^ 0x80808080u;
                    if (o.lo) reinterpret_cast<uint32_t *>(o.lo)[j] = (SR ? pack_bytes2(c) : pack_bytes0(c)) ^ o.lo_flip;
                }
            }
        }
        if (o.rowsum8) {
            // a row is rs_group consecutive lanes (groups are aligned: the lane index is j mod 32)
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                int sum = rs[u];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1)
                    if (off < o.rs_group) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                const int64_t j = base + u * kThreads + threadIdx.x;
                if (ok[u] && (threadIdx.x & (o.rs_group - 1)) == 0) o.rowsum8[j >> o.rs_shift] = sum;
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (int64_t i = nv << 2; i < n; ++i)
            quantize_scalar<SR>(x, i, cols, PERCH, qp8, id8, qp16, id16, keys, o, index_base);
    if (TOTALS && !PERCH && (o.chansum8 || o.chansum16)) {
        // (cols / 4 divides the block size and the grid stride: the thread's channels are 4 * (threadIdx.x mod cols / 4) ...)
        // (a block sees fewer than 65536 rows -- the launcher's rule -- so its totals fit int32)
        int *s_cs = reinterpret_cast<int *>(s_qp);           // [cols] 8-bit totals, then [cols] 16-bit ones
        for (int c = threadIdx.x; c < 2 * cols; c += kThreads) s_cs[c] = 0;
        __syncthreads();
        const int c0 = 4 * (threadIdx.x & ((cols >> 2) - 1));
        // how many elements this thread quantised per channel: the 16-bit totals were taken over unsigned codes
        int64_t mine = 0;
        for (int64_t base = (int64_t)blockIdx.x * kThreads * kUnroll; base < nv; base += stride)
            for (int u = 0; u < kUnroll; ++u) mine += (base + u * kThreads + threadIdx.x < nv) ? 1 : 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (o.chansum8 && cs8[e]) atomicAdd(&s_cs[c0 + e], cs8[e]);
            if (o.chansum16) atomicAdd(&s_cs[cols + c0 + e], (int)((long long)cs16[e] - mine * 32768));
        }
        __syncthreads();
        for (int c = threadIdx.x; c < cols; c += kThreads) {
            if (o.chansum8 && s_cs[c]) atomicAdd(o.chansum8 + c, (unsigned long long)(long long)s_cs[c]);
            if (o.chansum16 && s_cs[cols + c]) atomicAdd(o.chansum16 + c, (unsigned long long)(long long)s_cs[cols + c]);
        }
    }
}

// Row sums of stored 8-bit codes: a group of G lanes per row (G = smallest power
// of two covering cols/16, at most 32), 16-byte loads.
template <bool IS_SIGNED>
__global__ void __launch_bounds__(kThreads) rowsum_kernel(const uint8_t *__restrict__ q, int64_t rows, int cols,
                                                          int G, int32_t *__restrict__ sums)
{
    const int lane = threadIdx.x & 31;
    const int gl = lane % G;
    const int64_t groups_per_block = kThreads / G;
    const int cv = cols >> 4;
    for (int64_t r = (int64_t)blockIdx.x * groups_per_block + threadIdx.x / G; r < rows;
         r += (int64_t)gridDim.x * groups_per_block) {
        int acc = 0;
        const uint4 *row = reinterpret_cast<const uint4 *>(q + r * cols);
        for (int c = gl; c < cv; c += G) {
            uint4 v = __ldg(row + c);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k)
                acc = IS_SIGNED ? __dp4a((int)w[k], 0x01010101, acc) : (int)__dp4a(w[k], 0x01010101u, (uint32_t)acc);
        }
        for (int o = G >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (gl == 0) sums[r] = acc;
    }
}

// Column sums (over rows) of stored 8-bit codes (signed or unsigned) into int64.  blockIdx.y
// selects a slab of up to 256 column groups (16 codes each); inside a slab a
// thread owns one group and every (256 / groups)-th row.  Block partials meet in
// shared memory, then one atomic per column and block.  The destination must be
// zeroed beforehand.
template <bool IS_SIGNED>
__global__ void __launch_bounds__(kThreads) colsum_kernel(const uint8_t *__restrict__ q, int64_t rows, int cols,
                                                          unsigned long long *__restrict__ sums)
{
    const int cv = cols >> 4;
    const int slab0 = blockIdx.y * kThreads;                 // first column group of this slab
    const int tw = (cv - slab0) < kThreads ? (cv - slab0) : kThreads;
    const int rpb = kThreads / tw;
    const int tx = threadIdx.x % tw, ty = threadIdx.x / tw;
    __shared__ int s_acc[kThreads * 16];
    for (int c = threadIdx.x; c < tw * 16; c += kThreads) s_acc[c] = 0;
    __syncthreads();
    if (ty < rpb) {
        int acc[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = 0;
        for (int64_t r = (int64_t)blockIdx.x * rpb + ty; r < rows; r += (int64_t)gridDim.x * rpb) {
            uint4 v = __ldg(reinterpret_cast<const uint4 *>(q + r * cols) + slab0 + tx);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    acc[k * 4 + b] += IS_SIGNED ? (int)(int8_t)(w[k] >> (8 * b)) : (int)((w[k] >> (8 * b)) & 0xFFu);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) atomicAdd(&s_acc[tx * 16 + e], acc[e]);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < tw * 16; c += kThreads)
        atomicAdd(&sums[slab0 * 16 + c], (unsigned long long)(long long)s_acc[c]);
}

// ----------------------------------------------------------------- launchers
// One wave: `bps` resident blocks per SM (the kernel's occupancy), never more blocks than work groups.
static int grid_for(int bps, int64_t n_groups)
{
    int64_t want = (int64_t)sm_count() * bps;
    int64_t g = n_groups < want ? n_groups : want;
    return (int)(g < 1 ? 1 : g);
}

// after_range (nullable): recorded on the stream once the parameters are enqueued -- a caller that has work for
// another stream which needs only them (and not the codes) starts it from there.
static int launch_range(const float *x, int64_t n, float2 *partials, qbp_qparams *qp8, qbp_qparams *qp16,
                        cudaStream_t st, cudaEvent_t after_range = nullptr, int keep_rev = 0)
{
    int nparts = 0;
    if (n > 0) {
        const bool vec = aligned16(x);
        const int64_t per_block = (int64_t)kThreads * kRangeUnroll * (vec ? 4 : 1);
        nparts = grid_for(vec ? blocks_per_sm(range_partial_kernel<4>, kThreads) : blocks_per_sm(range_partial_kernel<1>, kThreads),
                          (n + per_block - 1) / per_block);
        if (nparts > kMaxParts) nparts = kMaxParts;
        QBP_TRACE_BEGIN(st);
        if (vec) range_partial_kernel<4><<<nparts, kThreads, 0, st>>>(x, n, partials, keep_rev);
        else     range_partial_kernel<1><<<nparts, kThreads, 0, st>>>(x, n, partials, keep_rev);
        QBP_LAUNCH_OK("range_partial_kernel");
    }
    QBP_TRACE_BEGIN(st);
    range_finalize_kernel<<<1, kThreads, 0, st>>>(partials, nparts, qp8, qp16);
    QBP_LAUNCH_OK("range_finalize_kernel");
    if (after_range) QBP_CUDA_OK(cudaEventRecord(after_range, st));
    return QBP_OK;
}

// The per-tensor scan for callers in other files: *qp receives the 8-bit parameters of the tensor's range widened to
// hold 0 (vmin = min(lowest, 0), vmax = max(highest, 0)).
size_t range_scan_ws_bytes() { return align_up(sizeof(float2) * kMaxParts, 256); }
int range_scan(const float *x, int64_t n, void *ws, size_t ws_bytes, qbp_qparams *qp, cudaStream_t st)
{
    if (!ws || ws_bytes < range_scan_ws_bytes()) return fail(QBP_ERR_WORKSPACE, "range scan: workspace too small");
    return launch_range(x, n, static_cast<float2 *>(ws), qp, nullptr, st);
}

static int launch_chan_range(const float *x, int64_t rows, int64_t cols, int bits, float *part_lo, float *part_hi,
                             qbp_qparams *qp, cudaStream_t st)
{
    const bool v4 = aligned16(x) && cols % 4 == 0;
    ScanGeom g = scan_geom(rows, cols, aligned16(x), v4 ? blocks_per_sm(chan_range_partial_kernel<4>, kScanThreads)
                                                        : blocks_per_sm(chan_range_partial_kernel<1>, kScanThreads));
    int nparts = 0;
    if (rows > 0) {
        nparts = g.nbx;
        dim3 grid(g.nbx, g.slabs);
        QBP_TRACE_BEGIN(st);
        if (g.vec == 4) chan_range_partial_kernel<4><<<grid, kScanThreads, 0, st>>>(x, rows, (int)cols, g.tw, part_lo, part_hi);
        else            chan_range_partial_kernel<1><<<grid, kScanThreads, 0, st>>>(x, rows, (int)cols, g.tw, part_lo, part_hi);
        QBP_LAUNCH_OK("chan_range_partial_kernel");
    }
    QBP_TRACE_BEGIN(st);
    chan_range_finalize_kernel<<<(int)((cols + 7) / 8), kThreads, 0, st>>>(part_lo, part_hi, nparts, (int)cols, bits, qp);
    QBP_LAUNCH_OK("chan_range_finalize_kernel");
    return QBP_OK;
}

static int launch_quantize(const float *x, int64_t n, int64_t cols, int perch, int rounding,
                           const qbp_qparams *qp8, uint32_t id8, const qbp_qparams *qp16, uint32_t id16,
                           uint64_t seed, const QuantOut &o, cudaStream_t st, uint64_t index_base = 0)
{
    if (n == 0) return QBP_OK;
    const bool vec = aligned16(x) && (!perch || cols % 4 == 0) &&
                     (!o.q8 || ((uintptr_t)o.q8 & 3) == 0) && (!o.q16 || ((uintptr_t)o.q16 & 7) == 0) &&
                     (!o.hi || ((uintptr_t)o.hi & 3) == 0) && (!o.lo || ((uintptr_t)o.lo & 3) == 0);
    if (o.rowsum8 && !vec) return fail(QBP_ERR_INVALID_ARG, "quantize: fused row sums need the vector path");
    const int64_t per_block = (int64_t)kThreads * (vec ? 4 * kUnroll : 1);
    const bool sr = rounding == QBP_ROUND_STOCHASTIC;
    const PhiloxKeys key = philox_keys_host(seed);
    const int c = (int)cols;
    // per-channel parameter table: 2 x cols x 8 bytes of dynamic shared memory when that stays within 32 KB
    const int smem_cols = (perch && vec && cols <= 2048) ? c : 0;
    const bool totals = o.chansum8 || o.chansum16;
    // (fewer than 2^22 rows: with a grid of at least one block per SM, or one block per 1024 vectors, a block sees
    // fewer than 65536 of them, and its int32 totals of 16-bit codes cannot overflow)
    if (totals && !(vec && !perch && cols % 4 == 0 && cols / 4 <= kThreads && ((cols / 4) & (cols / 4 - 1)) == 0 && n / cols < (1ll << 22)))
        return fail(QBP_ERR_INVALID_ARG, "quantize: per-channel totals need the vector path and cols / 4 a power of two <= %d", kThreads);
    const size_t smem = totals ? (size_t)cols * 2 * sizeof(int) : (size_t)smem_cols * 2 * sizeof(float2);
    const int64_t groups = (n + per_block - 1) / per_block;
#define QBP_QUANT2(SR_, VEC_, PC_, TOT_)                                                                                \
    do {                                                                                                                \
        const int grid = grid_for(blocks_per_sm(quantize_kernel<SR_, VEC_, PC_, TOT_>, kThreads), groups);              \
        QBP_TRACE_BEGIN(st);                                                                                            \
        quantize_kernel<SR_, VEC_, PC_, TOT_><<<grid, kThreads, (VEC_) == 4 ? smem : 0, st>>>(x, n, c, qp8, id8, qp16, id16,  \
                                                                                         key, o, (VEC_) == 4 ? smem_cols : 0, index_base); \
    } while (0)
#define QBP_QUANT(SR_, VEC_, PC_) QBP_QUANT2(SR_, VEC_, PC_, false)
    if (totals) {           // (vector path, per tensor: checked above)
        if (sr) QBP_QUANT2(true, 4, false, true); else QBP_QUANT2(false, 4, false, true);
    } else if (sr) {
        if (vec) { if (perch) QBP_QUANT(true, 4, true); else QBP_QUANT(true, 4, false); }
        else     { if (perch) QBP_QUANT(true, 1, true); else QBP_QUANT(true, 1, false); }
    } else {
        if (vec) { if (perch) QBP_QUANT(false, 4, true); else QBP_QUANT(false, 4, false); }
        else     { if (perch) QBP_QUANT(false, 1, true); else QBP_QUANT(false, 1, false); }
    }
#undef QBP_QUANT
#undef QBP_QUANT2
    QBP_LAUNCH_OK("quantize_kernel");
    return QBP_OK;
}

// Whether the quantising kernel itself can emit the row sums of its 8-bit codes: per-tensor, 16-byte aligned
// tensors whose rows are 4, 8, ..., 128 elements (a row is then a power-of-two group of lanes of one warp).
static bool can_fuse_rowsums(const float *x, const void *q8, int64_t cols, const QuantOut &o)
{
    const int64_t g = cols / 4;
    return cols % 4 == 0 && g >= 1 && g <= 32 && (g & (g - 1)) == 0 && aligned16(x) && ((uintptr_t)q8 & 3) == 0 &&
           (!o.q16 || ((uintptr_t)o.q16 & 7) == 0) && (!o.hi || ((uintptr_t)o.hi & 3) == 0) && (!o.lo || ((uintptr_t)o.lo & 3) == 0);
}

// Row / column sums of stored codes; used by the quantiser's optional outputs
// and by the integer products' zero-point corrections.
int launch_rowsum(const void *q, bool is_signed, int64_t rows, int64_t cols, int32_t *sums, cudaStream_t st)
{
    if (rows == 0) return QBP_OK;
    if (cols % 16 || !aligned16(q)) return fail(QBP_ERR_INVALID_ARG, "row sums need 16-byte aligned rows (cols %% 16 == 0)");
    int G = 1; while (G < 32 && G < cols / 16) G <<= 1;
    const int64_t groups = kThreads / G;
    const int grid = grid_for(is_signed ? blocks_per_sm(rowsum_kernel<true>, kThreads) : blocks_per_sm(rowsum_kernel<false>, kThreads),
                              (rows + groups - 1) / groups);
    QBP_TRACE_BEGIN(st);
    if (is_signed) rowsum_kernel<true><<<grid, kThreads, 0, st>>>((const uint8_t *)q, rows, (int)cols, G, sums);
    else           rowsum_kernel<false><<<grid, kThreads, 0, st>>>((const uint8_t *)q, rows, (int)cols, G, sums);
    QBP_LAUNCH_OK("rowsum_kernel");
    return QBP_OK;
}

int launch_colsum(const void *q, bool is_signed, int64_t rows, int64_t cols, int64_t *sums, cudaStream_t st)
{
    if (cols % 16 || !aligned16(q)) return fail(QBP_ERR_INVALID_ARG, "column sums need cols %% 16 == 0");
    QBP_CUDA_OK(cudaMemsetAsync(sums, 0, sizeof(int64_t) * cols, st));
    if (rows == 0) return QBP_OK;
    const int cv = (int)(cols / 16);
    const int slabs = (cv + kThreads - 1) / kThreads;
    const int rpb = kThreads / (cv < kThreads ? cv : kThreads);
    // each thread keeps int32 partials over at most 2^22 rows: 255 * 2^22 < 2^31
    int64_t min_blocks = (rows >> 22) + 1;
    int64_t grid = grid_for(blocks_per_sm(colsum_kernel<true>, kThreads), (rows + rpb - 1) / rpb) / slabs;
    if (grid < min_blocks) grid = min_blocks;
    QBP_TRACE_BEGIN(st);
    if (is_signed) colsum_kernel<true><<<dim3((unsigned)grid, (unsigned)slabs), kThreads, 0, st>>>((const uint8_t *)q, rows, (int)cols, (unsigned long long *)sums);
    else           colsum_kernel<false><<<dim3((unsigned)grid, (unsigned)slabs), kThreads, 0, st>>>((const uint8_t *)q, rows, (int)cols, (unsigned long long *)sums);
    QBP_LAUNCH_OK("colsum_kernel");
    return QBP_OK;
}

static int check_common(const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                        const qbp_qparams *qp_out)
{
    if (rows < 0 || cols <= 0) return fail(QBP_ERR_INVALID_ARG, "quantize: rows must be >= 0 and cols > 0");
    if (granularity != QBP_PER_TENSOR && granularity != QBP_PER_CHANNEL)
        return fail(QBP_ERR_INVALID_ARG, "quantize: granularity must be QBP_PER_TENSOR or QBP_PER_CHANNEL");
    if (rounding != QBP_ROUND_NEAREST && rounding != QBP_ROUND_STOCHASTIC)
        return fail(QBP_ERR_INVALID_ARG, "quantize: rounding must be QBP_ROUND_NEAREST or QBP_ROUND_STOCHASTIC");
    if (!qp_out) return fail(QBP_ERR_INVALID_ARG, "quantize: qp_out is NULL");
    if (!x && rows * cols > 0) return fail(QBP_ERR_INVALID_ARG, "quantize: x is NULL");
    if (((uintptr_t)x & 3) != 0) return fail(QBP_ERR_INVALID_ARG, "quantize: x is not 4-byte aligned");
    return QBP_OK;
}

static size_t quant_ws_bytes(int64_t cols, int granularity)
{
    if (granularity == QBP_PER_CHANNEL) return 2 * align_up(sizeof(float) * kScanMaxStrips * (size_t)cols, 256) + 256;
    return align_up(sizeof(float2) * kMaxParts, 256) + 256;
}

// Shared body of the 8- and 16-bit entry points.
static int quantize_any(int bits, const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                        uint64_t seed, uint32_t tensor_id, const qbp_qparams *range_in, const QuantOut &o,
                        qbp_qparams *qp_out, void *ws, size_t ws_bytes, cudaStream_t st, cudaEvent_t after_range = nullptr,
                        int keep_rev = 0)
{
    int rc = check_common(x, rows, cols, granularity, rounding, qp_out);
    if (rc) return rc;
    const int perch = granularity == QBP_PER_CHANNEL;
    if (range_in) {
        const int count = perch ? (int)cols : 1;
        QBP_TRACE_BEGIN(st);
        qparams_from_range_kernel<<<(count + 255) / 256, 256, 0, st>>>(range_in, count, bits, qp_out);
        QBP_LAUNCH_OK("qparams_from_range_kernel");
    } else {
        if (!ws || ws_bytes < quant_ws_bytes(cols, granularity))
            return fail(QBP_ERR_WORKSPACE, "quantize: workspace of %zu bytes needed, %zu given",
                        quant_ws_bytes(cols, granularity), ws_bytes);
        WsCarver w(ws, ws_bytes);
        if (perch) {
            float *plo = w.take<float>((size_t)kScanMaxStrips * cols);
            float *phi = w.take<float>((size_t)kScanMaxStrips * cols);
            rc = launch_chan_range(x, rows, cols, bits, plo, phi, qp_out, st);
        } else {
            float2 *parts = w.take<float2>(kMaxParts);
            rc = launch_range(x, rows * cols, parts, bits == 8 ? qp_out : nullptr, bits == 16 ? qp_out : nullptr, st, after_range, keep_rev);
        }
        if (rc) return rc;
    }
    return launch_quantize(x, rows * cols, cols, perch, rounding, qp_out, tensor_id, qp_out, tensor_id, seed, o, st);
}

// ------------------------------------------------- built-in scratch (no allocation)
// Scratch of qbp_quantize_s8_static: lives in the library's device image, so every GPU that loads the
// library holds these bytes until the process exits.  Sized for the per-channel range scan of
// QBP_STATIC_MAX_CHANNELS channels (two float partial tables of kScanMaxStrips rows), which also covers the
// per-tensor scan.  Host code must not pass this name to a kernel: it is resolved per device below.
constexpr size_t kStaticScratchBytes = 2 * sizeof(float) * (size_t)kScanMaxStrips * QBP_STATIC_MAX_CHANNELS + 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static std::mutex g_static_mu;
static void *g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device, looked up once per device.
static int static_scratch_address(void **out)
{
    int dev = -1;
    QBP_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(QBP_ERR_CUDA, "quantize_s8_static: device ordinal %d not supported", dev);
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        QBP_CUDA_OK(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return fail(QBP_ERR_CUDA, "quantize_s8_static: the built-in scratch has no device address");
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return QBP_OK;
}

// The quantising half of the bifurcation, once qp8 / qp16 are known.
static int bifurcate_tail(const float *g, int64_t rows, int64_t cols, uint64_t seed, uint32_t tensor_id8,
                          uint32_t tensor_id16, int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi, uint8_t *lo,
                          qbp_qparams *qp16, cudaStream_t st, uint64_t index_base = 0, int64_t *tot16 = nullptr,
                          bool lo_signed = false)
{
    QuantOut o = {q8, nullptr, hi, lo, nullptr, 0, 0, nullptr, nullptr, lo_signed ? 0x80808080u : 0u};
    if (tot16 && rows * cols > 0) {                       // (the caller asked quantizer_totals_supported(cols) first)
        QBP_CUDA_OK(cudaMemsetAsync(tot16, 0, sizeof(int64_t) * (size_t)cols, st));
        o.chansum16 = reinterpret_cast<unsigned long long *>(tot16);
    }
    const bool fused = row_sums8 && rows * cols > 0 && can_fuse_rowsums(g, q8, cols, o);
    if (fused) { o.rowsum8 = row_sums8; o.rs_group = (int)(cols / 4); o.rs_shift = 31 - __builtin_clz((unsigned)o.rs_group); }
    int rc = launch_quantize(g, rows * cols, cols, 0, QBP_ROUND_STOCHASTIC, qp8, tensor_id8, qp16, tensor_id16, seed, o, st, index_base);
    if (rc) return rc;
    if (row_sums8 && !fused) return launch_rowsum(q8, true, rows, cols, row_sums8, st);
    return QBP_OK;
}

// Bifurcation of a gradient whose range partials (min, max per block) were left by the kernel that wrote it.
int bifurcate_with_range_partials(const float *g, int64_t rows, int64_t cols, uint64_t seed, uint32_t tensor_id8,
                                  uint32_t tensor_id16, int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi,
                                  uint8_t *lo, qbp_qparams *qp16, const float2 *partials, int nparts, cudaStream_t st,
                                  int64_t *tot16, bool lo_signed, cudaEvent_t after_range)
{
    QBP_TRACE_BEGIN(st);
    range_finalize_kernel<<<1, kThreads, 0, st>>>(partials, nparts, qp8, qp16);
    QBP_LAUNCH_OK("range_finalize_kernel");
    if (after_range) QBP_CUDA_OK(cudaEventRecord(after_range, st));
    return bifurcate_tail(g, rows, cols, seed, tensor_id8, tensor_id16, q8, qp8, row_sums8, hi, lo, qp16, st, 0, tot16, lo_signed);
}

// The parameters of both copies from per-block (or per-channel) (min, max) pairs.
int launch_range_finalize(const float2 *partials, int nparts, qbp_qparams *qp8, qbp_qparams *qp16, cudaStream_t st,
                          cudaEvent_t after_range)
{
    QBP_TRACE_BEGIN(st);
    range_finalize_kernel<<<1, kThreads, 0, st>>>(partials, nparts, qp8, qp16);
    QBP_LAUNCH_OK("range_finalize_kernel");
    if (after_range) QBP_CUDA_OK(cudaEventRecord(after_range, st));
    return QBP_OK;
}

bool quantizer_totals_supported(int64_t cols)
{
    return cols % 4 == 0 && cols / 4 <= kThreads && ((cols / 4) & (cols / 4 - 1)) == 0;
}

// The layer's activation quantiser: qbp_quantize_s8 (per tensor, nearest) that also leaves the per-channel totals
// of the codes (tot8 [cols], zeroed here) when the tensor's shape allows it; *left says whether it did.
int quantize_s8_with_totals(const float *x, int64_t rows, int64_t cols, int8_t *q, qbp_qparams *qp_out, int32_t *row_sums,
                            int64_t *tot8, bool *left, void *ws, size_t ws_bytes, cudaStream_t st, cudaEvent_t after_range)
{
    *left = false;
    QuantOut o = {q, nullptr, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    const bool fused = row_sums && rows * cols > 0 && can_fuse_rowsums(x, q, cols, o);
    if (fused) { o.rowsum8 = row_sums; o.rs_group = (int)(cols / 4); o.rs_shift = 31 - __builtin_clz((unsigned)o.rs_group); }
    if (tot8 && rows * cols > 0 && quantizer_totals_supported(cols) && aligned16(x) && ((uintptr_t)q & 3) == 0) {
        QBP_CUDA_OK(cudaMemsetAsync(tot8, 0, sizeof(int64_t) * (size_t)cols, st));
        o.chansum8 = reinterpret_cast<unsigned long long *>(tot8);
        *left = true;
    }
    int rc = quantize_any(8, x, rows, cols, QBP_PER_TENSOR, QBP_ROUND_NEAREST, 0, 0, nullptr, o, qp_out, ws, ws_bytes, st, after_range, 1);
    if (rc) return rc;
    if (row_sums && !fused) return launch_rowsum(q, true, rows, cols, row_sums, st);
    return QBP_OK;
}

}  // namespace qbp

using namespace qbp;

extern "C" __attribute__((visibility("default"))) const char *qbp_last_error(void) { return g_err; }

extern "C" __attribute__((visibility("default"))) int qbp_trace_enable(int on)
{
    for (TraceRec &r : g_trace) { g_event_pool.push_back(r.a); g_event_pool.push_back(r.b); }
    g_trace.clear();
    g_trace_on = on != 0;
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) int qbp_trace_count(void) { return (int)g_trace.size(); }

extern "C" __attribute__((visibility("default"))) int qbp_trace_read(int index, char *name, int name_cap, float *ms)
{
    if (index < 0 || index >= (int)g_trace.size() || !name || name_cap <= 0 || !ms)
        return fail(QBP_ERR_INVALID_ARG, "trace_read: bad index or NULL output");
    const TraceRec &r = g_trace[index];
    if (!r.name) return fail(QBP_ERR_INVALID_ARG, "trace_read: record %d was never closed", index);
    snprintf(name, (size_t)name_cap, "%s", r.name);
    QBP_CUDA_OK(cudaEventElapsedTime(ms, r.a, r.b));
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) size_t qbp_range_chunked_workspace_bytes(void)
{
    return 2 * align_up(sizeof(float2) * kMaxParts, 256) + 256;
}

extern "C" __attribute__((visibility("default"))) int qbp_range_chunked(const float *x, int64_t rows, int64_t cols, int64_t chunks,
                                                                       qbp_qparams *range_out, void *ws, size_t ws_bytes,
                                                                       void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (!x || !range_out) return fail(QBP_ERR_INVALID_ARG, "range_chunked: NULL argument");
    if (rows <= 0 || cols <= 0) return fail(QBP_ERR_INVALID_ARG, "range_chunked: empty tensor");
    if (chunks < 1 || chunks > kMaxParts || rows % chunks)
        return fail(QBP_ERR_INVALID_ARG, "range_chunked: rows (%lld) must be a multiple of chunks (%lld), at most %d chunks",
                    (long long)rows, (long long)chunks, kMaxParts);
    if (!ws || ws_bytes < qbp_range_chunked_workspace_bytes())
        return fail(QBP_ERR_WORKSPACE, "range_chunked: workspace of %zu bytes needed, %zu given",
                    qbp_range_chunked_workspace_bytes(), ws_bytes);
    WsCarver w(ws, ws_bytes);
    float2 *parts = w.take<float2>(kMaxParts);
    float2 *per_chunk = w.take<float2>(kMaxParts);
    const int64_t n_chunk = rows / chunks * cols;
    const bool vec = aligned16(x) && n_chunk % 4 == 0;
    // about one wave of blocks in all, at least one per chunk
    const int64_t per_block = (int64_t)kThreads * kRangeUnroll * (vec ? 4 : 1);
    const int wave = grid_for(vec ? blocks_per_sm(chunk_range_partial_kernel<4>, kThreads) : blocks_per_sm(chunk_range_partial_kernel<1>, kThreads),
                              (rows * cols + per_block - 1) / per_block);
    int bpc = (int)std::max<int64_t>(1, std::min<int64_t>((n_chunk + per_block - 1) / per_block, wave / chunks));
    bpc = (int)std::min<int64_t>(bpc, kMaxParts / chunks);
    QBP_TRACE_BEGIN(st);
    if (vec) chunk_range_partial_kernel<4><<<dim3(bpc, (unsigned)chunks), kThreads, 0, st>>>(x, n_chunk, parts);
    else     chunk_range_partial_kernel<1><<<dim3(bpc, (unsigned)chunks), kThreads, 0, st>>>(x, n_chunk, parts);
    QBP_LAUNCH_OK("chunk_range_partial_kernel");
    QBP_TRACE_BEGIN(st);
    chunk_range_finalize_kernel<<<1, kThreads, 0, st>>>(parts, (int)chunks, bpc, per_chunk, range_out);
    QBP_LAUNCH_OK("chunk_range_finalize_kernel");
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) size_t qbp_quantize_workspace_bytes(int64_t rows, int64_t cols, int granularity)
{
    (void)rows;
    return quant_ws_bytes(cols > 0 ? cols : 1, granularity);
}

extern "C" __attribute__((visibility("default"))) int qbp_quantize_s8(const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                               uint64_t seed, uint32_t tensor_id, const qbp_qparams *range_in, int8_t *q,
                               qbp_qparams *qp_out, int32_t *row_sums, int64_t *col_sums, void *ws, size_t ws_bytes,
                               void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (!q && rows * cols > 0) return fail(QBP_ERR_INVALID_ARG, "quantize_s8: q is NULL");
    if ((row_sums || col_sums) && granularity != QBP_PER_TENSOR)
        return fail(QBP_ERR_INVALID_ARG, "quantize_s8: row/column sums are per-tensor only");
    QuantOut o = {q, nullptr, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    const bool fused = row_sums && rows * cols > 0 && can_fuse_rowsums(x, q, cols, o);
    if (fused) { o.rowsum8 = row_sums; o.rs_group = (int)(cols / 4); o.rs_shift = 31 - __builtin_clz((unsigned)o.rs_group); }
    int rc = quantize_any(8, x, rows, cols, granularity, rounding, seed, tensor_id, range_in, o, qp_out, ws, ws_bytes, st);
    if (rc) return rc;
    if (row_sums && !fused) { rc = launch_rowsum(q, true, rows, cols, row_sums, st); if (rc) return rc; }
    if (col_sums) { rc = launch_colsum(q, true, rows, cols, col_sums, st); if (rc) return rc; }
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) int qbp_quantize_s16(const float *x, int64_t rows, int64_t cols, int granularity, int rounding,
                                uint64_t seed, uint32_t tensor_id, const qbp_qparams *range_in, int16_t *q,
                                int8_t *hi, uint8_t *lo, qbp_qparams *qp_out, void *ws, size_t ws_bytes, void *stream)
{
    if (!q && !hi && !lo) return fail(QBP_ERR_INVALID_ARG, "quantize_s16: q, hi and lo are all NULL");
    QuantOut o = {nullptr, q, hi, lo, nullptr, 0, 0, nullptr, nullptr};
    return quantize_any(16, x, rows, cols, granularity, rounding, seed, tensor_id, range_in, o, qp_out, ws, ws_bytes,
                        (cudaStream_t)stream);
}

extern "C" __attribute__((visibility("default"))) int qbp_bifurcate(const float *g, int64_t rows, int64_t cols, uint64_t seed, uint32_t tensor_id8,
                             uint32_t tensor_id16, int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi,
                             uint8_t *lo, qbp_qparams *qp16, void *ws, size_t ws_bytes, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (rows < 0 || cols <= 0) return fail(QBP_ERR_INVALID_ARG, "bifurcate: rows must be >= 0 and cols > 0");
    if (!qp8 || !qp16) return fail(QBP_ERR_INVALID_ARG, "bifurcate: qp8 / qp16 is NULL");
    if (rows * cols > 0 && (!g || !q8 || !hi || !lo)) return fail(QBP_ERR_INVALID_ARG, "bifurcate: NULL tensor");
    if (((uintptr_t)g & 3) != 0) return fail(QBP_ERR_INVALID_ARG, "bifurcate: g is not 4-byte aligned");
    if (!ws || ws_bytes < quant_ws_bytes(cols, QBP_PER_TENSOR))
        return fail(QBP_ERR_WORKSPACE, "bifurcate: workspace of %zu bytes needed, %zu given",
                    quant_ws_bytes(cols, QBP_PER_TENSOR), ws_bytes);
    WsCarver w(ws, ws_bytes);
    float2 *parts = w.take<float2>(kMaxParts);
    int rc = launch_range(g, rows * cols, parts, qp8, qp16, st);
    if (rc) return rc;
    return bifurcate_tail(g, rows, cols, seed, tensor_id8, tensor_id16, q8, qp8, row_sums8, hi, lo, qp16, st);
}

// Both parameter records from clamping values the caller supplies.
__global__ void qparams_pair_from_range_kernel(const qbp_qparams *__restrict__ in, qbp_qparams *__restrict__ qp8,
                                               qbp_qparams *__restrict__ qp16)
{
    *qp8 = make_qparams(in->vmin, in->vmax, 8);
    *qp16 = make_qparams(in->vmin, in->vmax, 16);
}

extern "C" __attribute__((visibility("default"))) int qbp_bifurcate_shard(const float *g, int64_t rows, int64_t cols, uint64_t seed,
                                   uint32_t tensor_id8, uint32_t tensor_id16, uint64_t index_base, const qbp_qparams *range_in,
                                   int8_t *q8, qbp_qparams *qp8, int32_t *row_sums8, int8_t *hi, uint8_t *lo,
                                   qbp_qparams *qp16, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (rows < 0 || cols <= 0) return fail(QBP_ERR_INVALID_ARG, "bifurcate_shard: rows must be >= 0 and cols > 0");
    if (!qp8 || !qp16 || !range_in) return fail(QBP_ERR_INVALID_ARG, "bifurcate_shard: qp8 / qp16 / range_in is NULL");
    if (rows * cols > 0 && (!g || !q8 || !hi || !lo)) return fail(QBP_ERR_INVALID_ARG, "bifurcate_shard: NULL tensor");
    if (((uintptr_t)g & 3) != 0) return fail(QBP_ERR_INVALID_ARG, "bifurcate_shard: g is not 4-byte aligned");
    if (index_base % 4) return fail(QBP_ERR_INVALID_ARG, "bifurcate_shard: index_base must be a multiple of 4");
    QBP_TRACE_BEGIN(st);
    qparams_pair_from_range_kernel<<<1, 1, 0, st>>>(range_in, qp8, qp16);
    QBP_LAUNCH_OK("qparams_pair_from_range_kernel");
    return bifurcate_tail(g, rows, cols, seed, tensor_id8, tensor_id16, q8, qp8, row_sums8, hi, lo, qp16, st, index_base);
}

// out = (float)acc * (sa * sb): the dequantisation of a weight gradient whose int64 accumulators were added up
// over several GPUs first (integer addition is exact, so the sum does not depend on the order of the GPUs).
__global__ void dequant_s64_kernel(const long long *__restrict__ acc, int64_t n, const qbp_qparams *qa,
                                   const qbp_qparams *qb, float *__restrict__ out)
{
    const float s = __fmul_rn(qa->scale, qb->scale);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = __fmul_rn((float)acc[i], s);
}

extern "C" __attribute__((visibility("default"))) int qbp_dequant_s64(const int64_t *acc, int64_t count, const qbp_qparams *qa,
                               const qbp_qparams *qb, float *out, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (count < 0 || (count > 0 && (!acc || !out)) || !qa || !qb) return fail(QBP_ERR_INVALID_ARG, "dequant_s64: NULL argument");
    if (count == 0) return QBP_OK;
    const int grid = (int)std::min<int64_t>((count + 255) / 256, (int64_t)sm_count() * 8);
    QBP_TRACE_BEGIN(st);
    dequant_s64_kernel<<<grid, 256, 0, st>>>((const long long *)acc, count, qa, qb, out);
    QBP_LAUNCH_OK("dequant_s64_kernel");
    return QBP_OK;
}

// fp32 master-weight update (Section 6 "Putting it all together": the updates stay in float32 and run once per
// minibatch): g = dw + wd * w;  v = mu * v + g (with a momentum buffer);  w = w - lr * v.  Every operation is
// rounded on its own, in this order.
__global__ void __launch_bounds__(256) sgd_update_kernel(float *__restrict__ w, const float *__restrict__ dw,
                                                         float *__restrict__ vbuf, int64_t n, float lr, float mu, float wd)
{
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256) {
        const float wi = w[i];
        float g = __fadd_rn(dw[i], __fmul_rn(wd, wi));
        if (vbuf) { g = __fadd_rn(__fmul_rn(mu, vbuf[i]), g); vbuf[i] = g; }
        w[i] = __fsub_rn(wi, __fmul_rn(lr, g));
    }
}

extern "C" __attribute__((visibility("default"))) int qbp_sgd_update(float *w, const float *dw, float *momentum_buf, int64_t count,
                              float lr, float momentum, float weight_decay, void *stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    if (count < 0 || (count > 0 && (!w || !dw))) return fail(QBP_ERR_INVALID_ARG, "sgd_update: NULL tensor");
    if (count == 0) return QBP_OK;
    const int grid = (int)std::min<int64_t>((count + 255) / 256, (int64_t)sm_count() * 8);
    QBP_TRACE_BEGIN(st);
    sgd_update_kernel<<<grid, 256, 0, st>>>(w, dw, momentum_buf, count, lr, momentum, weight_decay);
    QBP_LAUNCH_OK("sgd_update_kernel");
    return QBP_OK;
}

extern "C" __attribute__((visibility("default"))) int qbp_quantize_s8_static(const float *x, int64_t rows, int64_t cols, int granularity,
                                      int rounding, uint64_t seed, uint32_t tensor_id, int8_t *q,
                                      qbp_qparams *qp_out, void *stream)
{
    if (!q && rows * cols > 0) return fail(QBP_ERR_INVALID_ARG, "quantize_s8_static: q is NULL");
    int rc = check_common(x, rows, cols, granularity, rounding, qp_out);
    if (rc) return rc;
    if (granularity == QBP_PER_CHANNEL && cols > QBP_STATIC_MAX_CHANNELS)
        return fail(QBP_ERR_UNSUPPORTED_SHAPE,
                    "quantize_s8_static: %lld channels exceed the built-in scratch (at most %d per-channel ranges); "
                    "use qbp_quantize_s8 with a caller workspace",
                    (long long)cols, QBP_STATIC_MAX_CHANNELS);
    if (quant_ws_bytes(cols, granularity) > kStaticScratchBytes)
        return fail(QBP_ERR_UNSUPPORTED_SHAPE, "quantize_s8_static: the scan needs %zu scratch bytes, %zu are built in",
                    quant_ws_bytes(cols, granularity), kStaticScratchBytes);
    void *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc) return rc;
    // every partial the finalising kernel reads was written by this call's scan: nothing has to start at zero
    QuantOut o = {q, nullptr, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    return quantize_any(8, x, rows, cols, granularity, rounding, seed, tensor_id, nullptr, o, qp_out, scratch,
                        kStaticScratchBytes, (cudaStream_t)stream);
}
