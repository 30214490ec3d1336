// Shared host/device helpers of libqbp: error reporting, launch checks, small
// numeric helpers with a pinned IEEE operation order, Philox4x32-10, and thin
// wrappers over the sm_100a PTX used by the tensor-core kernels (mbarrier,
// TMA, tcgen05).  No kernel lives here.
#pragma once

#include <cuda_runtime.h>
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "../../include/qbp.h"

namespace qbp {

// ---------------------------------------------------------------- host side
void set_error(const char *fmt, ...);          // defined in qbp_quant.cu
int fail(int status, const char *fmt, ...);    // sets the message, returns status

#define QBP_CUDA_OK(expr)                                                         \
    do {                                                                          \
        cudaError_t e_ = (expr);                                                  \
        if (e_ != cudaSuccess)                                                    \
            return ::qbp::fail(QBP_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

// Optional per-kernel timing (qbp_trace_enable): an event pair around every launch.
void trace_begin(cudaStream_t st);
void trace_end(const char *name, cudaStream_t st);
#define QBP_TRACE_BEGIN(st) ::qbp::trace_begin(st)

// Placed after every kernel launch; expects the stream in a variable named `st`.
#define QBP_LAUNCH_OK(name)                                                       \
    do {                                                                          \
        ::qbp::trace_end(name, st);                                               \
        cudaError_t e_ = cudaGetLastError();                                      \
        if (e_ != cudaSuccess)                                                    \
            return ::qbp::fail(QBP_ERR_CUDA, "launch of %s: %s", name, cudaGetErrorString(e_)); \
    } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
int sm_count();                                // cached multiprocessor count of the current device

// Function attributes (the opt-in to more than 48 KB of dynamic shared memory) belong to a device: set them once
// per device ordinal, whichever host thread gets there first.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    bool done[kMaxDevices] = {};
    // true when the caller still has to do the set-up for the current device (and then calls mark())
    bool pending(int *dev_out)
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); *dev_out = -1; return true; }
        *dev_out = dev;
        return !__atomic_load_n(&done[dev], __ATOMIC_ACQUIRE);
    }
    void mark(int dev) { if (dev >= 0) __atomic_store_n(&done[dev], true, __ATOMIC_RELEASE); }
};
#define QBP_SMEM_OPT_IN(once, kernel, bytes)                                                                       \
    do {                                                                                                           \
        int dev_ = -1;                                                                                             \
        if ((once).pending(&dev_)) {                                                                               \
            QBP_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes)));  \
            (once).mark(dev_);                                                                                     \
        }                                                                                                          \
    } while (0)

// Carves 256-byte aligned pieces out of the caller's workspace.
struct WsCarver {
    char *base; size_t off; size_t cap;
    WsCarver(void *ws, size_t bytes) : base(static_cast<char *>(ws)), off(0), cap(bytes) {}
    template <typename T> T *take(size_t count) {
        size_t bytes = align_up(count * sizeof(T), 256);
        T *p = reinterpret_cast<T *>(base + off);
        off += bytes;
        return p;
    }
    bool ok() const { return base != nullptr && off <= cap; }
};

// -------------------------------------------------------------- device side
#ifdef __CUDACC__

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies
// (one wide multiply each); the round keys are key + r * (0x9E3779B9, 0xBB67AE85).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * c.x;
        const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c.z;
        const uint32_t k0 = k.x + (uint32_t)r * 0x9E3779B9u, k1 = k.y + (uint32_t)r * 0xBB67AE85u;
        c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ k0, (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ k1, (uint32_t)p0);
    }
    return c;
}

// Scale and zero-point from clamping values (Appendix B), fp32, fixed order.
__device__ __forceinline__ qbp_qparams make_qparams(float vmin, float vmax, int bits)
{
    const int L = (1 << bits) - 1;
    vmin = fminf(vmin, 0.0f);
    vmax = fmaxf(vmax, 0.0f);
    float range = __fsub_rn(vmax, vmin);
    float s = (range == 0.0f) ? 1.0f : __fdiv_rn(range, (float)L);
    float z = rintf(__fdiv_rn(-vmin, s));
    z = fminf(fmaxf(z, 0.0f), (float)L);
    qbp_qparams q;
    q.scale = s;
    q.zero_point = (int)z - (1 << (bits - 1));
    q.vmin = vmin;
    q.vmax = vmax;
    return q;
}

// One element to its unsigned code in [0, L].  rnd is the element's Philox word; stochastic rounding takes a
// 16-bit draw from it: the high half-word for an 8-bit code, the low half-word for a 16-bit code (the two copies
// of one gradient then round independently from one word).
template <bool STOCHASTIC>
__device__ __forceinline__ int quantize_code(float x, float inv_scale, float zp_u, float Lf, uint32_t rnd)
{
    float t = __fmaf_rn(x, inv_scale, zp_u);
    float c;
    if (!STOCHASTIC) {
        c = rintf(t);
    } else {
        float f = floorf(t);
        float frac = __fsub_rn(t, f);
        const uint32_t draw = (Lf == 255.0f) ? (rnd >> 16) : (rnd & 0xFFFFu);
        float u = __fmul_rn((float)draw, 0x1p-16f);
        c = (u < frac) ? __fadd_rn(f, 1.0f) : f;
    }
    // c is integral: the saturating conversion is the clamp to [0, 2^bits - 1] (Lf selects the width)
    uint32_t code;
    if (Lf == 255.0f) asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(code) : "f"(c));
    else              asm("cvt.rni.sat.u16.f32 %0, %1;" : "=r"(code) : "f"(c));
    return (int)code;
}

// The stochastic codes of one element in fixed point: the same results as quantize_code<true> with fewer
// instructions.  With t = fma(x, inv, zp), f = floor(t), frac = t - f and a 16-bit draw d, the code is
// f + [d * 2^-16 < frac] = f + [d < ceil(frac * 2^16)] (d is an integer).  t * 2^16 is exact in fp32 and
// ceil(t * 2^16) = f * 2^16 + ceil(frac * 2^16), so adding 0xFFFF - d carries into bit 16 exactly when the code
// rounds up.  The conversion saturates negative t to 0 (code 0, as the clamp gives) and the minimum with
// L * 2^16 is the clamp at the top (then nothing can carry).
// The caller passes inv_scale and zp_u already multiplied by 2^16: scaling by a power of two commutes with the
// rounding of the fused multiply-add, so fma(x, inv * 2^16, zp * 2^16) is exactly 2^16 * fma(x, inv, zp).
// 8 bits: the code is byte 2 of the result; the draw is the high half of rnd.
__device__ __forceinline__ uint32_t quantize_sr8_byte2(float x, float inv_scale_2p16, float zp_u_2p16, uint32_t rnd)
{
    uint32_t tc;
    asm("cvt.rpi.sat.u32.f32 %0, %1;" : "=r"(tc) : "f"(__fmaf_rn(x, inv_scale_2p16, zp_u_2p16)));
    return min(tc, 0x00FF0000u) + ((~rnd) >> 16);
}
// 16 bits: the code is the upper half of the result (high byte = byte 3, low byte = byte 2); the draw is the low half of rnd.
__device__ __forceinline__ uint32_t quantize_sr16_top_half(float x, float inv_scale_2p16, float zp_u_2p16, uint32_t rnd)
{
    uint32_t tc;
    asm("cvt.rpi.sat.u32.f32 %0, %1;" : "=r"(tc) : "f"(__fmaf_rn(x, inv_scale_2p16, zp_u_2p16)));
    return min(tc, 0xFFFF0000u) + ((~rnd) & 0xFFFFu);
}

// Philox4x32-10 with the ten round keys precomputed (they depend on the key only); passed to a kernel by value,
// they sit in its constant parameter space and cost no registers.
struct PhiloxKeys { uint32_t k0[10], k1[10]; };
inline PhiloxKeys philox_keys_host(uint64_t seed)
{
    PhiloxKeys r;
    for (int i = 0; i < 10; ++i) {
        r.k0[i] = (uint32_t)seed + (uint32_t)i * 0x9E3779B9u;
        r.k1[i] = (uint32_t)(seed >> 32) + (uint32_t)i * 0xBB67AE85u;
    }
    return r;
}
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const PhiloxKeys &k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * c.x;
        const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c.z;
        c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ k.k0[r], (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ k.k1[r], (uint32_t)p0);
    }
    return c;
}

// Range BN (Section 3, Eq. (range)): xhat and y of one element and the per-channel scale 1 / (C(n) (max - min)).
// The order of operations is part of the contract: every kernel that normalises (the apply passes, the fused
// epilogue of a product) must produce the same bits, so that forward, backward and requantisation agree.
__device__ __forceinline__ float bn_xhat(float x, float mu, float s) { return __fmul_rn(__fsub_rn(x, mu), s); }
__device__ __forceinline__ float bn_y(float xh, float g, float b) { return __fadd_rn(__fmul_rn(g, xh), b); }
// One element of the Range BN backward (the derivative stated with Eq. (rangebn) in Section 3, ties as in the forward):
// dx = s * (gamma * dy - m1 - k2 * ind), ind = [x == max] - [x == min].  Every operation is rounded on its own and
// none is contracted, so the value is a monotone function of dy for fixed (s >= 0, gamma, m1, k2, ind): the extremes of
// dx over a set of positions are this function of the extremes of dy (which is how the gradient's range is known
// before the gradient is written).
__device__ __forceinline__ float bn_dx(float d, float ind, float s, float g, float m1, float k2)
{
    return __fmul_rn(s, __fsub_rn(__fsub_rn(__fmul_rn(g, d), m1), __fmul_rn(k2, ind)));
}
// Floats as integers that compare the same way (and back): for atomic minima and maxima of floats.
__device__ __forceinline__ int float_order(float f) { const int b = __float_as_int(f); return b ^ ((b >> 31) & 0x7fffffff); }
__device__ __forceinline__ float order_float(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }
__device__ __forceinline__ float bn_scale(float lo, float hi, float Cn);
// The rectifier's mask of a Range BN output as a threshold on the input.  y(x) = bn_y(bn_xhat(x, mu, s), g, b) is a
// monotone function of x (every operation is rounded on its own and monotone, s >= 0): rising for g >= 0, falling for
// g < 0, so {x : y(x) > 0} is a ray, and its end is found by bisection over the floats in their order (33 evaluations
// of y).  Returns (t, sgn) with  y(x) > 0  <=>  sgn * x >= t  for finite x (sgn = +-1; t = +-inf: none / all).
__device__ inline float2 relu_threshold(float mu, float s, float g, float b)
{
    const bool rising = !(g < 0.0f);
    long long lo = float_order(-3.402823466e38f), hi = float_order(3.402823466e38f);
    auto on = [&](long long k) { return bn_y(bn_xhat(order_float((int)k), mu, s), g, b) > 0.0f; };
    const float sgn = rising ? 1.0f : -1.0f;
    // (towards `far` the output rises: the ray is [threshold, far])
    const bool at_far = on(rising ? hi : lo), at_near = on(rising ? lo : hi);
    if (!at_far) return make_float2(INFINITY, sgn);
    if (at_near) return make_float2(-INFINITY, sgn);
    if (rising) {                       // smallest key that is on
        while (hi - lo > 1) { const long long mid = lo + (hi - lo) / 2; if (on(mid)) hi = mid; else lo = mid; }
        return make_float2(order_float((int)hi), 1.0f);
    }
    while (hi - lo > 1) { const long long mid = lo + (hi - lo) / 2; if (on(mid)) lo = mid; else hi = mid; }   // largest key that is on
    return make_float2(-order_float((int)lo), -1.0f);
}
__device__ __forceinline__ float bn_scale(float lo, float hi, float Cn)
{
    float r = __fsub_rn(hi, lo);
    return r > 0.0f ? __fdiv_rn(1.0f, __fmul_rn(Cn, r)) : 0.0f;
}

__device__ __forceinline__ float warp_min(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// ---- sm_100a PTX wrappers ---------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` SM clock cycles (by default about a second) and reports false; the
// caller then raises the kernel's status word and leaves through its normal exit.
constexpr long long kWaitLimitCycles = 2000000000ll;
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, long long limit = kWaitLimitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit) return false;
    return true;
}

// The same wait by every lane of a converged warp; the answer is the same in all of them.
__device__ __forceinline__ bool mbar_wait_uniform(uint64_t *bar, uint32_t parity, long long limit = kWaitLimitCycles)
{
    const bool ok = mbar_wait(bar, parity, limit);
    return __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
}

// The same wait for a whole warp: one lane polls (with a short sleep between polls, so that waiting warps
// leave the shared-memory pipe to the warps that feed the tensor core), the result is shared by shuffle.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t *bar, uint32_t parity, long long limit = kWaitLimitCycles)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0 && !mbar_try_wait(bar, parity)) {
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity)) {
            if (clock64() - t0 > limit) { ok = 0; break; }
            __nanosleep(40);
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}

// A kernel whose bounded wait ran out records it here; the word only ever goes from 0 to QBP_ERR_TIMEOUT.
__device__ __forceinline__ void raise_timeout(int *status) { atomicExch(status, (int)QBP_ERR_TIMEOUT); }

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// TMA tiled loads, completion reported on an mbarrier as transferred bytes.
__device__ __forceinline__ void tma_load_2d(void *dst, const void *map, uint64_t *bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *dst, const void *map, uint64_t *bar, int x, int y, int z, int w)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
// TMA tiled stores (shared -> global) as bulk groups of the issuing thread; elements of the box that fall
// outside the tensor are not written.  The x coordinate times the element size must be a multiple of 16.
__device__ __forceinline__ void tma_store_2d(const void *map, const void *src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_4d(const void *map, const void *src, int x, int y, int z, int w)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z), "r"(w)
                 : "memory");
}
// Per-thread asynchronous 16-byte copies global -> shared (L2 only), in groups a thread commits and waits for itself:
// what a thread copies and reads back itself needs no barrier.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// ... until at most N of this thread's groups are still in flight
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until every store group of this thread has finished reading its shared-memory source.
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// Until all but the latest store group of this thread have finished reading their sources.
__device__ __forceinline__ void tma_store_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// Until every store group of this thread is complete.
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Named barrier over `count` threads (a multiple of 32) of the CTA.
__device__ __forceinline__ void named_barrier(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const void *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Tensor memory (TMEM) management; executed by one full warp.
__device__ __forceinline__ void tmem_alloc(uint32_t *slot_in_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// Three-input minimum / maximum (one instruction on sm_100).
__device__ __forceinline__ float fmin3(float a, float b, float c)
{
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// True in exactly one lane of a converged warp.  The MMA warps run whole and put this around each tcgen05.mma and
// commit, rather than branching on the lane index once around the loop: the instruction takes its operands from
// warp-uniform registers, and only in code the compiler knows to be convergent are descriptors that change from
// one MMA to the next kept there (measured: 63 against 110 cycles per 128 x 64 x 32 MMA).
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}

// D[tmem] (+)= A[smem] * B[smem], 8-bit integer operands, int32 accumulator.  Volatile keeps it in order with
// the barrier waits and commits around it; there is no memory clobber, so that the issuing thread's loads of
// the next descriptors can be scheduled across it (that thread is bound by its own instruction latency).
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate));
}
// Arrive on an mbarrier once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns of the accumulator into registers.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

#endif  // __CUDACC__
}  // namespace qbp
