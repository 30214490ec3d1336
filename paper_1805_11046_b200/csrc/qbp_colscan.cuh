// Per-channel scans of a [rows x C] fp32 matrix with the channel innermost
// (NHWC): the thread/row mapping shared by the per-channel range scan of the
// quantiser and by both passes of Range BN.
//
// Mapping: the matrix is read as vectors of VEC floats (4 when C % 4 == 0 and
// the base is 16-byte aligned, else 1).  A 256-thread block is TW vector
// columns wide (at most kScanMaxTw) and 256/TW rows high; blockIdx.y selects
// the slab of TW vector columns, blockIdx.x the strip of rows, strips advance
// by gridDim.x.  A thread therefore stays on the same VEC channels for its
// whole life and a warp always reads 32*VEC consecutive floats.  Every block
// leaves one partial per channel of its slab, so narrow slabs (many rows per
// block, few channels) keep the partial arrays small: with 2048 channels, slabs
// of 256 vectors cost 20 % extra traffic for the partials, slabs of 64 a
// quarter of that.
#pragma once

#include "qbp_common.cuh"

namespace qbp {

constexpr int kScanThreads = 256;
constexpr int kScanUnroll = 4;
constexpr int kScanMaxStrips = 1024;     // bound on gridDim.x, sizes the partial buffers
constexpr int kScanMaxTw = 64;           // widest block in vector columns (64 float4 = 1 KB of a row)

struct ScanGeom {
    int vec;        // 4 or 1
    int cv;         // vector columns = C / vec
    int tw;         // threads across = min(pow2ceil(cv), kScanMaxTw)
    int rpb;        // rows per block step = 256 / tw
    int slabs;      // ceil(cv / tw)
    int nbx;        // row strips (gridDim.x)
};

inline int pow2ceil(int v) { int p = 1; while (p < v) p <<= 1; return p; }

// Resident blocks per SM of a kernel at `threads` threads and no dynamic shared memory.
template <typename Kernel>
inline int blocks_per_sm(Kernel kernel, int threads)
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, 0) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = 1;
    }
    return n;
}

// nbx is chosen so that all strips are resident at once (a single wave: `bps`
// blocks per SM, the occupancy of the kernel that will run) and no strip is empty.
inline ScanGeom scan_geom(int64_t rows, int64_t C, bool aligned, int bps)
{
    ScanGeom g;
    g.vec = (aligned && C % 4 == 0) ? 4 : 1;
    g.cv = (int)(C / g.vec);
    g.tw = pow2ceil(g.cv) < kScanMaxTw ? pow2ceil(g.cv) : kScanMaxTw;
    g.rpb = kScanThreads / g.tw;
    g.slabs = (g.cv + g.tw - 1) / g.tw;
    int64_t steps = (rows + g.rpb - 1) / g.rpb;
    int64_t want = (int64_t)sm_count() * bps / g.slabs;
    if (want < 1) want = 1;
    if (want > kScanMaxStrips) want = kScanMaxStrips;
    g.nbx = (int)(steps < want ? (steps > 0 ? steps : 1) : want);
    return g;
}

#ifdef __CUDACC__

template <int VEC> struct VecF;
template <> struct VecF<4> {
    float v[4];
    __device__ __forceinline__ void load(const float *p) {
        float4 t = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    // read-once data of a reduction pass: evict-first, so that it does not push out what a later pass re-reads
    __device__ __forceinline__ void load_stream(const float *p) {
        float4 t = __ldcs(reinterpret_cast<const float4 *>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    __device__ __forceinline__ void store(float *p) const {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
    // written once, not read again soon: evict-first (measured 6.1 against 5.5 TB/s in the Range BN apply pass)
    __device__ __forceinline__ void store_stream(float *p) const {
        __stcs(reinterpret_cast<float4 *>(p), make_float4(v[0], v[1], v[2], v[3]));
    }
};
template <> struct VecF<1> {
    float v[1];
    __device__ __forceinline__ void load(const float *p) { v[0] = __ldg(p); }
    __device__ __forceinline__ void load_stream(const float *p) { v[0] = __ldcs(p); }
    __device__ __forceinline__ void store(float *p) const { *p = v[0]; }
    __device__ __forceinline__ void store_stream(float *p) const { __stcs(p, v[0]); }
};

// Calls f(row, first_channel, vec_index_in_unroll) for every vector this thread
// owns; loads are expected to be grouped by the caller via the unroll index.
struct ScanPos {
    int tx, ty, col;      // col = first channel of this thread's vector
    bool active;
};

template <int VEC>
__device__ __forceinline__ ScanPos scan_pos(int C, int tw)
{
    ScanPos p;
    p.tx = threadIdx.x % tw;
    p.ty = threadIdx.x / tw;
    int cv = blockIdx.y * tw + p.tx;
    p.col = cv * VEC;
    p.active = p.col < C;
    return p;
}

#endif  // __CUDACC__
}  // namespace qbp
