"""ctypes loader and numpy front end for the CPU oracle (oracle/qbp_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
cpu-baseline / reference legs of the benchmark.  It never touches the CUDA
library, and the CUDA library never touches it.

The layer-level functions at the bottom compose the C steps in the order the
paper gives them (Section 4): quantise -> integer product -> Range BN, and in
the backward direction Range BN backward -> two quantised copies of the
gradient (8-bit and 16-bit, both stochastically rounded) -> layer gradient and
weight gradient.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "qbp_oracle.c"
_LIB = _HERE / "_build" / "libqbp_oracle.so"
_CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-shared", "-fPIC"]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no-op when the library is newer than the source)."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    _LIB.parent.mkdir(exist_ok=True)
    tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
    subprocess.run(["gcc", *_CFLAGS, "-o", str(tmp), str(_SRC), "-lm"], check=True)
    os.replace(tmp, _LIB)
    return _LIB


class ConvDesc(C.Structure):
    _fields_ = [(k, C.c_int64) for k in
                ("N", "H", "W", "C", "K", "R", "S", "stride", "pad", "P", "Q")]


def conv_desc(N, H, W, Cin, K, R, S, stride=1, pad=0) -> ConvDesc:
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    return ConvDesc(N, H, W, Cin, K, R, S, stride, pad, P, Q)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build()))
        _lib.qbo_random_word.restype = C.c_uint32
        _lib.qbo_random_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        _lib.qbo_rangebn_C.restype = C.c_double
        _lib.qbo_rangebn_C.argtypes = [C.c_int64]
        _lib.qbo_gemm_s8.restype = C.c_int64
        _lib.qbo_conv_s8.restype = C.c_int64
        _lib.qbo_random_word_sample.restype = C.c_uint32
        _lib.qbo_random_word_sample.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32]
        _lib.qbo_stc_tern.restype = C.c_float
        _lib.qbo_stc_tern.argtypes = [C.c_void_p, C.c_int64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p]
        _lib.qbo_tbp_update.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_uint64,
                                        C.c_uint32, C.c_void_p]
    return _lib


def _p(a, t=C.c_void_p):
    return None if a is None else a.ctypes.data_as(t)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle use."""
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else (os.cpu_count() or 1)


# ----------------------------------------------------------------- Philox
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32); k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().qbo_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def random_word(seed: int, tensor_id: int, i: int) -> int:
    return int(lib().qbo_random_word(seed, tensor_id, i))


# -------------------------------------------------------------- quantiser
@dataclass
class Quantized:
    q: np.ndarray            # signed stored codes, int8 or int16, same shape as x
    scale: np.ndarray        # float32 [1] or [cols]
    zero_point: np.ndarray   # int32   [1] or [cols]  (stored, i.e. signed)
    vmin: np.ndarray
    vmax: np.ndarray
    bits: int


def tensor_range(x, per_channel=False):
    x = _f32(x); cols = x.shape[-1]; rows = x.size // cols
    nq = cols if per_channel else 1
    lo = np.zeros(nq, np.float32); hi = np.zeros(nq, np.float32)
    lib().qbo_range(_p(x), C.c_int64(rows), C.c_int64(cols), int(per_channel), _p(lo), _p(hi))
    return lo, hi


def qparams(vmin: float, vmax: float, bits: int):
    s = C.c_float(); z = C.c_int32(); lo = C.c_float(); hi = C.c_float()
    lib().qbo_qparams(C.c_float(vmin), C.c_float(vmax), bits,
                      C.byref(s), C.byref(z), C.byref(lo), C.byref(hi))
    return np.float32(s.value), int(z.value), np.float32(lo.value), np.float32(hi.value)


def quantize(x, bits=8, per_channel=False, rounding=0, seed=0, tensor_id=0,
             range_in=None, index_base=0) -> Quantized:
    """rounding 0 = nearest (ties to even), 1 = stochastic.  range_in = (vmin, vmax).
    index_base: flat index of x[0] in the larger tensor x is a block of rows of."""
    x = _f32(x); cols = x.shape[-1]; rows = x.size // cols
    nq = cols if per_channel else 1
    q = np.zeros(x.shape, np.int8 if bits == 8 else np.int16)
    scale = np.zeros(nq, np.float32); zp = np.zeros(nq, np.int32)
    lo = np.zeros(nq, np.float32); hi = np.zeros(nq, np.float32)
    rng = None
    if range_in is not None:
        rng = np.concatenate([np.asarray(range_in[0], np.float32).reshape(nq),
                              np.asarray(range_in[1], np.float32).reshape(nq)])
    lib().qbo_quantize_at(_p(x), C.c_int64(rows), C.c_int64(cols), bits, int(per_channel),
                          int(rounding), C.c_uint64(seed), C.c_uint32(tensor_id), C.c_uint64(index_base), _p(rng),
                          _p(q) if bits == 8 else None, _p(q) if bits == 16 else None,
                          _p(scale), _p(zp), _p(lo), _p(hi))
    return Quantized(q, scale, zp, lo, hi, bits)


def range_chunked(x, chunks):
    """Appendix B's clamping values for activations: (mean of the chunk minima, mean of the chunk maxima) over
    `chunks` equal contiguous groups of rows.  Feed them to quantize(range_in=...)."""
    x = _f32(x); cols = x.shape[-1]; rows = x.size // cols
    if chunks < 1 or rows % chunks:
        raise ValueError("rows must be a multiple of chunks")
    lo = np.zeros(1, np.float32); hi = np.zeros(1, np.float32)
    lib().qbo_range_chunked(_p(x), C.c_int64(rows), C.c_int64(cols), C.c_int64(chunks), _p(lo), _p(hi))
    return float(lo[0]), float(hi[0])


def dequantize(qt: Quantized) -> np.ndarray:
    """Per-tensor only."""
    out = np.zeros(qt.q.shape, np.float32)
    fn = lib().qbo_dequantize_s8 if qt.bits == 8 else lib().qbo_dequantize_s16
    fn(_p(qt.q), C.c_int64(qt.q.size), C.c_float(qt.scale[0]), int(qt.zero_point[0]), _p(out))
    return out


def limb_split(q16):
    q16 = np.ascontiguousarray(q16, np.int16)
    hi = np.zeros(q16.shape, np.int8); lo = np.zeros(q16.shape, np.uint8)
    lib().qbo_limb_split(_p(q16), C.c_int64(q16.size), _p(hi), _p(lo))
    return hi, lo


# -------------------------------------------------------- integer products
def gemm_s8(A, za, B, zb, sa=1.0, sb=1.0, transA=False, transB=False):
    """acc = (op(A)-za) @ (op(B)-zb) with op = transpose when asked.  Returns (acc int32, out fp32, n_overflow)."""
    A = np.ascontiguousarray(A, np.int8); B = np.ascontiguousarray(B, np.int8)
    if transA: K, M = A.shape; a_rs, a_cs = 1, A.shape[1]
    else:      M, K = A.shape; a_rs, a_cs = A.shape[1], 1
    if transB: N, K2 = B.shape; b_rs, b_cs = 1, B.shape[1]
    else:      K2, N = B.shape; b_rs, b_cs = B.shape[1], 1
    assert K == K2
    acc = np.zeros((M, N), np.int32); out = np.zeros((M, N), np.float32)
    i64 = C.c_int64
    bad = lib().qbo_gemm_s8(i64(M), i64(N), i64(K), _p(A), i64(a_rs), i64(a_cs), int(za),
                            _p(B), i64(b_rs), i64(b_cs), int(zb), _p(acc),
                            C.c_float(sa), C.c_float(sb), _p(out))
    return acc, out, int(bad)


def gemm_s16s8(X, zx, G16, zg, sx=1.0, sg=1.0):
    """Linear-layer weight gradient: acc[k,n] = sum_m (X[m,k]-zx)(G16[m,n]-zg), int64."""
    X = np.ascontiguousarray(X, np.int8); G16 = np.ascontiguousarray(G16, np.int16)
    M, K = X.shape; M2, N = G16.shape; assert M == M2
    acc = np.zeros((K, N), np.int64); out = np.zeros((K, N), np.float32)
    i64 = C.c_int64
    lib().qbo_gemm_s16s8(i64(M), i64(N), i64(K), _p(X), int(zx), _p(G16), int(zg), _p(acc),
                         C.c_float(sx), C.c_float(sg), _p(out))
    return acc, out


def gemm_limbs(X, zx, Ghi, Glo, zg):
    X = np.ascontiguousarray(X, np.int8)
    Ghi = np.ascontiguousarray(Ghi, np.int8); Glo = np.ascontiguousarray(Glo, np.uint8)
    M, K = X.shape; _, N = Ghi.shape
    acc = np.zeros((K, N), np.int64)
    i64 = C.c_int64
    lib().qbo_gemm_limbs(i64(M), i64(N), i64(K), _p(X), int(zx), _p(Ghi), _p(Glo), int(zg), _p(acc))
    return acc


def conv_s8(mode, d: ConvDesc, inp, z_in, w, zw, s_in=1.0, s_w=1.0, idx=None):
    """mode 0: forward, input x [N,H,W,C] -> [N,P,Q,K]; mode 1: layer gradient,
    input g [N,P,Q,K] -> [N,H,W,C].  idx: flat output indices (sampled evaluation).
    Returns (acc int32, out fp32, n_overflow), shaped like the output (or like idx)."""
    inp = np.ascontiguousarray(inp, np.int8); w = np.ascontiguousarray(w, np.int8)
    shape = (d.N, d.P, d.Q, d.K) if mode == 0 else (d.N, d.H, d.W, d.C)
    if idx is not None:
        idx = np.ascontiguousarray(idx, np.int64); count = idx.size; oshape = idx.shape
    else:
        count = int(np.prod(shape)); oshape = shape
    acc = np.zeros(oshape, np.int32); out = np.zeros(oshape, np.float32)
    bad = lib().qbo_conv_s8(int(mode), C.byref(d), _p(inp), int(z_in), _p(w), int(zw), _p(idx),
                            C.c_int64(count), _p(acc), C.c_float(s_in), C.c_float(s_w), _p(out))
    return acc, out, int(bad)


def conv_wgrad_s16(d: ConvDesc, x, zx, g16, zg, sx=1.0, sg=1.0, idx=None):
    """acc[k,r,s,c] int64 (or the sampled flat indices idx)."""
    x = np.ascontiguousarray(x, np.int8); g16 = np.ascontiguousarray(g16, np.int16)
    shape = (d.K, d.R, d.S, d.C)
    if idx is not None:
        idx = np.ascontiguousarray(idx, np.int64); count = idx.size; oshape = idx.shape
    else:
        count = int(np.prod(shape)); oshape = shape
    acc = np.zeros(oshape, np.int64); out = np.zeros(oshape, np.float32)
    lib().qbo_conv_wgrad_s16(C.byref(d), _p(x), int(zx), _p(g16), int(zg), _p(idx),
                             C.c_int64(count), _p(acc), C.c_float(sx), C.c_float(sg), _p(out))
    return acc, out


# ---------------------------------------------------------------- Range BN
def rangebn_C(n: int) -> float:
    return float(lib().qbo_rangebn_C(n))


def rangebn_fwd(x, gamma=None, beta=None, relu=False):
    """x [..., C] -> (y fp64, mean fp64 [C], min fp32 [C], max fp32 [C]); n = x.size / C."""
    x = _f32(x); Cc = x.shape[-1]; n = x.size // Cc
    g = None if gamma is None else _f32(gamma); b = None if beta is None else _f32(beta)
    y = np.zeros(x.shape, np.float64); mean = np.zeros(Cc, np.float64)
    lo = np.zeros(Cc, np.float32); hi = np.zeros(Cc, np.float32)
    lib().qbo_rangebn_fwd(_p(x), C.c_int64(n), C.c_int64(Cc), _p(g), _p(b), int(relu),
                          _p(y), _p(mean), _p(lo), _p(hi))
    return y, mean, lo, hi


def rangebn_bwd(dy, x, save_mean, save_min, save_max, gamma=None, beta=None, relu=False):
    """Returns (dx fp64, dgamma fp64 [C], dbeta fp64 [C])."""
    dy = _f32(dy); x = _f32(x); Cc = x.shape[-1]; n = x.size // Cc
    g = None if gamma is None else _f32(gamma); b = None if beta is None else _f32(beta)
    mu = _f32(save_mean); lo = _f32(save_min); hi = _f32(save_max)
    dx = np.zeros(x.shape, np.float64); dg = np.zeros(Cc, np.float64); db = np.zeros(Cc, np.float64)
    lib().qbo_rangebn_bwd(_p(dy), _p(x), C.c_int64(n), C.c_int64(Cc), _p(g), _p(b), int(relu),
                          _p(mu), _p(lo), _p(hi), _p(dx), _p(dg), _p(db))
    return dx, dg, db


# ----------------------------------------------------------- weight update
def sgd_update(w, dw, vbuf=None, lr=0.1, momentum=0.0, weight_decay=0.0):
    """fp32 step of the master weights (Section 6): returns (new w, new momentum buffer or None); inputs untouched."""
    w = _f32(w).copy(); dw = _f32(dw)
    v = None if vbuf is None else _f32(vbuf).copy()
    lib().qbo_sgd_update(_p(w), _p(dw), _p(v), C.c_int64(w.size), C.c_float(lr), C.c_float(momentum), C.c_float(weight_decay))
    return w, v


# ------------------------------------------------------------------- layer
@dataclass
class LayerSaved:
    qx: Quantized
    qw: Quantized
    z: np.ndarray            # fp32 pre-BN output of the integer product
    mean: np.ndarray
    vmin: np.ndarray
    vmax: np.ndarray


def layer_fwd(x, w, gamma=None, beta=None, relu=False, conv: ConvDesc | None = None):
    """Quantised layer forward.  Linear: x [B,K], w [K,N] (y = x w).  Conv: x NHWC, w KRSC.
    Returns (y fp64, saved, acc int32)."""
    qx = quantize(x, 8, rounding=0); qw = quantize(w, 8, rounding=0)
    if conv is None:
        acc, z, bad = gemm_s8(qx.q, qx.zero_point[0], qw.q, qw.zero_point[0], qx.scale[0], qw.scale[0])
    else:
        acc, z, bad = conv_s8(0, conv, qx.q, qx.zero_point[0], qw.q, qw.zero_point[0],
                              qx.scale[0], qw.scale[0])
    assert bad == 0
    y, mean, lo, hi = rangebn_fwd(z, gamma, beta, relu)
    return y, LayerSaved(qx, qw, z, mean, lo, hi), acc


def bifurcate(g, seed, id8, id16):
    """The two copies of the layer gradient: 8-bit and 16-bit, both stochastically rounded,
    drawn from independent Philox streams (different tensor ids)."""
    return (quantize(g, 8, rounding=1, seed=seed, tensor_id=id8),
            quantize(g, 16, rounding=1, seed=seed, tensor_id=id16))


def layer_bwd_products(g, saved: LayerSaved, seed, id8, id16, conv: ConvDesc | None = None):
    """From the fp32 gradient g at the product's output: (dx fp32, dw fp32, acc_dx int32, acc_dw int64, g8, g16)."""
    g8, g16 = bifurcate(g, seed, id8, id16)
    qx, qw = saved.qx, saved.qw
    if conv is None:
        acc_dx, dx, bad = gemm_s8(g8.q, g8.zero_point[0], qw.q, qw.zero_point[0],
                                  g8.scale[0], qw.scale[0], transB=True)
        acc_dw, dw = gemm_s16s8(qx.q, qx.zero_point[0], g16.q, g16.zero_point[0],
                                qx.scale[0], g16.scale[0])
    else:
        acc_dx, dx, bad = conv_s8(1, conv, g8.q, g8.zero_point[0], qw.q, qw.zero_point[0],
                                  g8.scale[0], qw.scale[0])
        acc_dw, dw = conv_wgrad_s16(conv, qx.q, qx.zero_point[0], g16.q, g16.zero_point[0],
                                    qx.scale[0], g16.scale[0])
    assert bad == 0
    return dx, dw, acc_dx, acc_dw, g8, g16


# ------------------------------------------------- Appendix C: low-bit variants
def random_word_sample(seed: int, tensor_id: int, i: int, sample: int) -> int:
    return int(lib().qbo_random_word_sample(seed, tensor_id, i, sample))


def binarize(x) -> np.ndarray:
    """+1 for x >= 0, else -1 (int8, the shape of x)."""
    x = _f32(x); b = np.empty(x.shape, dtype=np.int8)
    lib().qbo_binarize(_p(x), C.c_int64(x.size), _p(b))
    return b


def pack_bits(codes, mask=False) -> np.ndarray:
    """[rows x cols] int8 -> [rows x ceil(cols / 32)] uint32 bit rows (bit = code > 0, or code != 0 with mask)."""
    b = np.ascontiguousarray(codes, dtype=np.int8); rows, cols = b.shape
    w = np.zeros((rows, (cols + 31) // 32), dtype=np.uint32)
    lib().qbo_pack_bits(_p(b), C.c_int64(rows), C.c_int64(cols), C.c_int(1 if mask else 0), _p(w))
    return w


def xnor_gemm(A_bits, B_bits, K) -> np.ndarray:
    """C [M x N] int32 = K - 2 popcount(a xor b) for bit rows A [M x words], B [N x words]."""
    A = np.ascontiguousarray(A_bits, dtype=np.uint32); Bm = np.ascontiguousarray(B_bits, dtype=np.uint32)
    out = np.zeros((A.shape[0], Bm.shape[0]), dtype=np.int32)
    lib().qbo_xnor_gemm(C.c_int64(A.shape[0]), C.c_int64(Bm.shape[0]), C.c_int64(K), _p(A), _p(Bm), _p(out))
    return out


def stc_tern(g, seed=0, tensor_id=0, sample=0):
    """(t int8 in {-1, 0, 1} of g's shape, s = max |g|): one stochastic ternarisation of g."""
    g = _f32(g); t = np.empty(g.shape, dtype=np.int8)
    s = lib().qbo_stc_tern(_p(g), g.size, seed, tensor_id, sample, _p(t))
    return t, np.float32(s)


def gated_xnor_gemm(nz_bits, sign_bits, B_bits, K) -> np.ndarray:
    """C [M x N] int32 = sum_k t b for ternary rows (non-zero and sign bit planes) against binary rows."""
    nz = np.ascontiguousarray(nz_bits, dtype=np.uint32); sg = np.ascontiguousarray(sign_bits, dtype=np.uint32)
    Bm = np.ascontiguousarray(B_bits, dtype=np.uint32)
    out = np.zeros((nz.shape[0], Bm.shape[0]), dtype=np.int32)
    lib().qbo_gated_xnor_gemm(C.c_int64(nz.shape[0]), C.c_int64(Bm.shape[0]), C.c_int64(K), _p(nz), _p(sg), _p(Bm), _p(out))
    return out


def tbp_update(g, a_bin, samples, seed=0, tensor_id=0) -> np.ndarray:
    """Algorithm 1: gW [K x N] float64 from g [rows x N] and the binarised activations a [rows x K]."""
    g = _f32(g); a = np.ascontiguousarray(a_bin, dtype=np.int8)
    rows, N = g.shape; K = a.shape[1]
    out = np.zeros((K, N), dtype=np.float64)
    lib().qbo_tbp_update(_p(g), _p(a), rows, N, K, samples, seed, tensor_id, _p(out))
    return out
