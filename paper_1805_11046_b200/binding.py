"""Thin Python binding over the C ABI of libqbp (include/qbp.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are torch CUDA tensors used as device memory (their
data_ptr() is what crosses the boundary); work is enqueued on torch's current
stream.  There is no CPU fallback: importing this module without the built
library raises, and every non-zero status raises QbpError with the library's
message.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libqbp.so"

QBP_PER_TENSOR, QBP_PER_CHANNEL = 0, 1
QBP_ROUND_NEAREST, QBP_ROUND_STOCHASTIC = 0, 1
QBP_CONV_FPROP, QBP_CONV_DGRAD = 0, 1
QBP_ERR_TIMEOUT = -6

EXPORTS = (
    "qbp_last_error", "qbp_trace_enable", "qbp_trace_count", "qbp_trace_read",
    "qbp_device_status", "qbp_selftest_bounded_wait",
    "qbp_quantize_workspace_bytes", "qbp_quantize_s8", "qbp_quantize_s8_static", "qbp_quantize_s16", "qbp_bifurcate",
    "qbp_bifurcate_shard", "qbp_dequant_s64", "qbp_sgd_update",
    "qbp_range_chunked_workspace_bytes", "qbp_range_chunked",
    "qbp_gemm_s8_workspace_bytes", "qbp_gemm_s8", "qbp_gemm_s8_sums",
    "qbp_conv_s8_workspace_bytes", "qbp_conv_s8_implicit",
    "qbp_wgrad_s16_workspace_bytes", "qbp_wgrad_s16",
    "qbp_rangebn_workspace_bytes", "qbp_rangebn_fwd", "qbp_rangebn_bwd", "qbp_rangebn_fwd_q8",
    "qbp_rangebn_fwd_stats", "qbp_rangebn_fwd_apply", "qbp_rangebn_bwd_stats", "qbp_rangebn_bwd_apply",
    "qbp_layer_workspace_bytes", "qbp_layer_fwd", "qbp_layer_fwd_chained", "qbp_layer_bwd",
    "qbp_binarize_s8", "qbp_stc_ternarize_workspace_bytes", "qbp_stc_ternarize_s8",
    "qbp_tbp_weight_gradient_workspace_bytes", "qbp_tbp_weight_gradient",
    "qbp_pack_bits", "qbp_xnor_gemm_bits", "qbp_gated_xnor_gemm_bits",
)


class QbpError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"libqbp status {status}: {message}")
        self.status = status


class ConvDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("N", "H", "W", "C", "K", "R", "S", "stride", "pad")]


class LayerDesc(C.Structure):
    _fields_ = [("conv", ConvDesc), ("batch", C.c_int64), ("in_features", C.c_int64),
                ("out_features", C.c_int64), ("relu", C.c_int32), ("seed", C.c_uint64),
                ("tensor_id8", C.c_uint32), ("tensor_id16", C.c_uint32)]


class LayerCtx(C.Structure):
    _fields_ = [("x_codes", C.c_void_p), ("qx", C.c_void_p), ("w_codes", C.c_void_p), ("qw", C.c_void_p),
                ("z", C.c_void_p), ("save_mean", C.c_void_p), ("save_min", C.c_void_p), ("save_max", C.c_void_p),
                ("g", C.c_void_p), ("g8", C.c_void_p), ("qg8", C.c_void_p), ("g_hi", C.c_void_p), ("g_lo", C.c_void_p),
                ("qg16", C.c_void_p), ("x_chan_sums", C.c_void_p)]


class Requant(C.Structure):
    """qbp_requant: where a pass writes the 8-bit codes of the activation it produces (q, qp) and, optionally,
    each row's code sum."""
    _fields_ = [("q", C.c_void_p), ("qp", C.c_void_p), ("row_sums", C.c_void_p), ("chan_sums", C.c_void_p)]


def requant(q, qp, row_sums=None, chan_sums=None) -> Requant:
    return Requant(q.data_ptr(), qp.data_ptr(), row_sums.data_ptr() if row_sums is not None else None,
                   chan_sums.data_ptr() if chan_sums is not None else None)


def _load() -> C.CDLL:
    if not _LIB_PATH.exists():
        raise ImportError(f"{_LIB_PATH} is missing: build it with "
                          f"`python -m paper_1805_11046_b200.build` (needs nvcc); there is no fallback path")
    lib = C.CDLL(str(_LIB_PATH))
    lib.qbp_last_error.restype = C.c_char_p
    missing = [name for name in EXPORTS if not hasattr(lib, name)]
    if missing:
        raise ImportError(f"{_LIB_PATH} lacks {missing}: rebuild it with `python -m paper_1805_11046_b200.build`")
    for name in EXPORTS:
        if name.endswith("_workspace_bytes"):
            getattr(lib, name).restype = C.c_size_t
    lib.qbp_quantize_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int]
    lib.qbp_gemm_s8_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int64]
    lib.qbp_conv_s8_workspace_bytes.argtypes = [C.c_int, C.c_void_p]
    lib.qbp_wgrad_s16_workspace_bytes.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
    lib.qbp_rangebn_workspace_bytes.argtypes = [C.c_int64, C.c_int64]
    lib.qbp_layer_workspace_bytes.argtypes = [C.c_void_p]
    lib.qbp_range_chunked_workspace_bytes.argtypes = []
    lib.qbp_stc_ternarize_workspace_bytes.argtypes = []
    lib.qbp_tbp_weight_gradient_workspace_bytes.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
    return lib


lib = _load()


def _check(status: int) -> None:
    if status != 0:
        raise QbpError(status, lib.qbp_last_error().decode())


def _ptr(t) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, int):
        return C.c_void_p(t)
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


_ws_cache: dict = {}


def workspace(nbytes: int, device=None) -> torch.Tensor:
    """A cached device scratch buffer of at least nbytes (grown on demand, 256-byte aligned by torch); one per
    device and host thread, since calls of different threads may interleave on a stream."""
    import threading
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    key = (dev, threading.get_ident())
    t = _ws_cache.get(key)
    if t is None or t.numel() < nbytes:
        t = torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device=dev)
        _ws_cache[key] = t
    return t


def new_qparams(count: int = 1, device="cuda") -> torch.Tensor:
    """Device storage for `count` qbp_qparams records: int32 [count, 4] = (scale bits, zero_point, vmin bits, vmax bits)."""
    return torch.zeros((count, 4), dtype=torch.int32, device=device)


def read_qparams(qp: torch.Tensor):
    """Host copy of qbp_qparams records -> (scale, zero_point, vmin, vmax) numpy arrays."""
    h = qp.detach().cpu()
    f = h.view(torch.float32)
    return f[:, 0].numpy().copy(), h[:, 1].numpy().copy(), f[:, 2].numpy().copy(), f[:, 3].numpy().copy()


def range_qparams(vmin, vmax, device="cuda") -> torch.Tensor:
    """qbp_qparams records carrying only clamping values (for range_in)."""
    lo = torch.as_tensor(vmin, dtype=torch.float32).reshape(-1)
    hi = torch.as_tensor(vmax, dtype=torch.float32).reshape(-1)
    qp = torch.zeros((lo.numel(), 4), dtype=torch.float32)
    qp[:, 2] = lo
    qp[:, 3] = hi
    return qp.view(torch.int32).to(device)


def status_word(ws: torch.Tensor) -> int:
    """qbp_device_status of a workspace: synchronises the current stream; 0, or QBP_ERR_TIMEOUT if a bounded
    device-side wait of a call that used `ws` gave up."""
    return int(lib.qbp_device_status(_ptr(ws), _stream()))


def qbp_selftest_bounded_wait(limit_cycles: int = 4096, ws=None):
    """Launches the library's wait self-test (a wait that nothing ends, with a short limit) and returns the
    workspace whose status word it raises."""
    if ws is None: ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    _check(lib.qbp_selftest_bounded_wait(_ptr(ws), C.c_size_t(ws.numel()), C.c_uint32(limit_cycles), _stream()))
    return ws


# ------------------------------------------------------------------ quantiser
def qbp_quantize_s8(x, granularity=QBP_PER_TENSOR, rounding=QBP_ROUND_NEAREST, seed=0, tensor_id=0,
                    range_in=None, q=None, qp_out=None, row_sums=None, col_sums=None, ws=None):
    cols = x.shape[-1]; rows = x.numel() // cols if cols else 0
    if q is None: q = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    if qp_out is None: qp_out = new_qparams(cols if granularity else 1, x.device)
    if ws is None: ws = workspace(lib.qbp_quantize_workspace_bytes(rows, cols, granularity), x.device)
    _check(lib.qbp_quantize_s8(_ptr(x), C.c_int64(rows), C.c_int64(cols), granularity, rounding,
                               C.c_uint64(seed), C.c_uint32(tensor_id), _ptr(range_in), _ptr(q), _ptr(qp_out),
                               _ptr(row_sums), _ptr(col_sums), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return q, qp_out


def qbp_range_chunked(x, chunks, range_out=None, ws=None):
    """Appendix B's clamping values for activations (averages of the chunks' minima / maxima over `chunks` equal
    groups of rows) as a qparams record to pass to qbp_quantize_s8(range_in=...)."""
    cols = x.shape[-1]; rows = x.numel() // cols if cols else 0
    if range_out is None: range_out = new_qparams(1, x.device)
    if ws is None: ws = workspace(lib.qbp_range_chunked_workspace_bytes(), x.device)
    _check(lib.qbp_range_chunked(_ptr(x), C.c_int64(rows), C.c_int64(cols), C.c_int64(chunks), _ptr(range_out), _ptr(ws),
                                 C.c_size_t(ws.numel()), _stream()))
    return range_out


QBP_STATIC_MAX_CHANNELS = 256


def qbp_quantize_s8_static(x, q, qp_out, granularity=QBP_PER_TENSOR, rounding=QBP_ROUND_NEAREST, seed=0, tensor_id=0):
    """qbp_quantize_s8 on the library's built-in scratch: no workspace argument and no allocation inside the
    call, for callers that may not allocate device memory (see include/qbp.h).  The outputs q (int8, shape of
    x) and qp_out (new_qparams(cols or 1)) are the caller's.  Per-channel granularity is limited to
    QBP_STATIC_MAX_CHANNELS columns; calls that overlap on the GPU share, and race on, the one scratch array."""
    cols = x.shape[-1]; rows = x.numel() // cols if cols else 0
    _check(lib.qbp_quantize_s8_static(_ptr(x), C.c_int64(rows), C.c_int64(cols), granularity, rounding,
                                      C.c_uint64(seed), C.c_uint32(tensor_id), _ptr(q), _ptr(qp_out), _stream()))
    return q, qp_out


def qbp_quantize_s16(x, granularity=QBP_PER_TENSOR, rounding=QBP_ROUND_NEAREST, seed=0, tensor_id=0,
                     range_in=None, q=None, hi=None, lo=None, qp_out=None, want=("q", "hi", "lo"), ws=None):
    cols = x.shape[-1]; rows = x.numel() // cols if cols else 0
    if q is None and "q" in want: q = torch.empty(x.shape, dtype=torch.int16, device=x.device)
    if hi is None and "hi" in want: hi = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    if lo is None and "lo" in want: lo = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    if qp_out is None: qp_out = new_qparams(cols if granularity else 1, x.device)
    if ws is None: ws = workspace(lib.qbp_quantize_workspace_bytes(rows, cols, granularity), x.device)
    _check(lib.qbp_quantize_s16(_ptr(x), C.c_int64(rows), C.c_int64(cols), granularity, rounding,
                                C.c_uint64(seed), C.c_uint32(tensor_id), _ptr(range_in), _ptr(q), _ptr(hi), _ptr(lo),
                                _ptr(qp_out), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return q, hi, lo, qp_out


def qbp_bifurcate(g, seed, tensor_id8, tensor_id16, q8=None, hi=None, lo=None, qp8=None, qp16=None,
                  row_sums8=None, ws=None):
    cols = g.shape[-1]; rows = g.numel() // cols if cols else 0
    if q8 is None: q8 = torch.empty(g.shape, dtype=torch.int8, device=g.device)
    if hi is None: hi = torch.empty(g.shape, dtype=torch.int8, device=g.device)
    if lo is None: lo = torch.empty(g.shape, dtype=torch.uint8, device=g.device)
    if qp8 is None: qp8 = new_qparams(1, g.device)
    if qp16 is None: qp16 = new_qparams(1, g.device)
    if ws is None: ws = workspace(lib.qbp_quantize_workspace_bytes(rows, cols, 0), g.device)
    _check(lib.qbp_bifurcate(_ptr(g), C.c_int64(rows), C.c_int64(cols), C.c_uint64(seed), C.c_uint32(tensor_id8),
                             C.c_uint32(tensor_id16), _ptr(q8), _ptr(qp8), _ptr(row_sums8), _ptr(hi), _ptr(lo),
                             _ptr(qp16), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return q8, qp8, hi, lo, qp16


def qbp_bifurcate_shard(g, seed, tensor_id8, tensor_id16, index_base, range_in, q8=None, hi=None, lo=None, qp8=None,
                        qp16=None, row_sums8=None):
    """qbp_bifurcate for a block of rows of a larger gradient tensor: index_base = flat index of g[0] in it,
    range_in = the whole tensor's clamping values."""
    cols = g.shape[-1]; rows = g.numel() // cols if cols else 0
    if q8 is None: q8 = torch.empty(g.shape, dtype=torch.int8, device=g.device)
    if hi is None: hi = torch.empty(g.shape, dtype=torch.int8, device=g.device)
    if lo is None: lo = torch.empty(g.shape, dtype=torch.uint8, device=g.device)
    if qp8 is None: qp8 = new_qparams(1, g.device)
    if qp16 is None: qp16 = new_qparams(1, g.device)
    _check(lib.qbp_bifurcate_shard(_ptr(g), C.c_int64(rows), C.c_int64(cols), C.c_uint64(seed), C.c_uint32(tensor_id8),
                                   C.c_uint32(tensor_id16), C.c_uint64(index_base), _ptr(range_in), _ptr(q8), _ptr(qp8),
                                   _ptr(row_sums8), _ptr(hi), _ptr(lo), _ptr(qp16), _stream()))
    return q8, qp8, hi, lo, qp16


def qbp_dequant_s64(acc, qa, qb, out=None):
    """out = float(acc) * (qa.scale * qb.scale) for int64 accumulators combined outside the product."""
    if out is None: out = torch.empty(acc.shape, dtype=torch.float32, device=acc.device)
    _check(lib.qbp_dequant_s64(_ptr(acc), C.c_int64(acc.numel()), _ptr(qa), _ptr(qb), _ptr(out), _stream()))
    return out


# ------------------------------------------------------------------- products
class Epilogue(C.Structure):
    """qbp_epilogue: device pointers [N] that receive the per-column sum / min / max of the fp32 output, and / or
    the ReLU + requantisation of the output (clamping values requant_range -> codes q_out, parameters qp_out, each
    row's code sum row_sums_out)."""
    _fields_ = [("col_sum", C.c_void_p), ("col_min", C.c_void_p), ("col_max", C.c_void_p), ("relu", C.c_int32),
                ("requant_range", C.c_void_p), ("q_out", C.c_void_p), ("qp_out", C.c_void_p), ("row_sums_out", C.c_void_p)]


def _epilogue(col_stats, n, device, relu=False, requant=None):
    """col_stats: None, True (allocate), or a (sum f64, min f32, max f32) triple of device tensors.
    requant: None or (range qparams, q int8 [M x N], qp_out, row_sums int32 [M] or None)."""
    if not col_stats and not relu and requant is None:
        return None, None
    ep = Epilogue()
    if col_stats:
        if col_stats is True:
            col_stats = (torch.empty(n, dtype=torch.float64, device=device), torch.empty(n, dtype=torch.float32, device=device),
                         torch.empty(n, dtype=torch.float32, device=device))
        ep.col_sum, ep.col_min, ep.col_max = (t.data_ptr() for t in col_stats)
    ep.relu = int(bool(relu))
    if requant is not None:
        rng, q, qp, rs = requant
        ep.requant_range, ep.q_out, ep.qp_out = rng.data_ptr(), q.data_ptr(), qp.data_ptr()
        ep.row_sums_out = rs.data_ptr() if rs is not None else None
    return ep, col_stats


def qbp_gemm_s8(A, qa, B, qb, transA=False, transB=False, want_acc=False, want_out=True, acc_out=None, out=None, ws=None,
                col_stats=None, relu=False, requant=None, a_sums=None, b_sums=None):
    if transA: K, M = A.shape
    else:      M, K = A.shape
    N = B.shape[0] if transB else B.shape[1]
    if want_acc and acc_out is None: acc_out = torch.empty((M, N), dtype=torch.int32, device=A.device)
    if want_out and out is None: out = torch.empty((M, N), dtype=torch.float32, device=A.device)
    if ws is None: ws = workspace(lib.qbp_gemm_s8_workspace_bytes(M, N, K), A.device)
    ep, stats = _epilogue(col_stats, N, A.device, relu, requant)
    if a_sums is not None or b_sums is not None:
        _check(lib.qbp_gemm_s8_sums(int(transA), int(transB), C.c_int64(M), C.c_int64(N), C.c_int64(K), _ptr(A), _ptr(qa),
                                    _ptr(a_sums), _ptr(B), _ptr(qb), _ptr(b_sums), _ptr(acc_out), _ptr(out),
                                    C.byref(ep) if ep else None, _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    else:
        _check(lib.qbp_gemm_s8(int(transA), int(transB), C.c_int64(M), C.c_int64(N), C.c_int64(K), _ptr(A), _ptr(qa),
                               _ptr(B), _ptr(qb), _ptr(acc_out), _ptr(out), C.byref(ep) if ep else None, _ptr(ws),
                               C.c_size_t(ws.numel()), _stream()))
    return (acc_out, out, ws, stats) if col_stats else (acc_out, out, ws)


def conv_desc(N, H, W, C_in, K, R, S, stride=1, pad=0) -> ConvDesc:
    return ConvDesc(N, H, W, C_in, K, R, S, stride, pad)


def qbp_conv_s8_implicit(mode, d: ConvDesc, inp, q_in, w, q_w, want_acc=False, want_out=True, acc_out=None, out=None, ws=None,
                         col_stats=None, relu=False, requant=None):
    shape = (d.N, d.H, d.W, d.K) if mode == QBP_CONV_FPROP else (d.N, d.H, d.W, d.C)
    if want_acc and acc_out is None: acc_out = torch.empty(shape, dtype=torch.int32, device=inp.device)
    if want_out and out is None: out = torch.empty(shape, dtype=torch.float32, device=inp.device)
    if ws is None: ws = workspace(lib.qbp_conv_s8_workspace_bytes(mode, C.byref(d)), inp.device)
    ep, stats = _epilogue(col_stats, shape[3], inp.device, relu, requant)
    _check(lib.qbp_conv_s8_implicit(mode, C.byref(d), _ptr(inp), _ptr(q_in), _ptr(w), _ptr(q_w), _ptr(acc_out),
                                    _ptr(out), C.byref(ep) if ep else None, _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return (acc_out, out, ws, stats) if col_stats else (acc_out, out, ws)


def qbp_wgrad_s16(x, qx, g_hi, g_lo, qg16, d: ConvDesc | None = None, want_acc=False, want_out=True,
                  acc_out=None, dW=None, ws=None):
    if d is None:
        M, K = x.shape; N = g_hi.shape[1]; shape = (K, N)
        dref = None
    else:
        M = d.N * d.H * d.W; K = d.C; N = d.K; shape = (d.K, d.R, d.S, d.C)
        dref = C.byref(d)
    if want_acc and acc_out is None: acc_out = torch.empty(shape, dtype=torch.int64, device=x.device)
    if want_out and dW is None: dW = torch.empty(shape, dtype=torch.float32, device=x.device)
    if ws is None: ws = workspace(lib.qbp_wgrad_s16_workspace_bytes(dref, M, N, K), x.device)
    _check(lib.qbp_wgrad_s16(dref, C.c_int64(M), C.c_int64(N), C.c_int64(K), _ptr(x), _ptr(qx), _ptr(g_hi),
                             _ptr(g_lo), _ptr(qg16), _ptr(acc_out), _ptr(dW), _ptr(ws), C.c_size_t(ws.numel()),
                             _stream()))
    return acc_out, dW, ws


# ------------------------------------------------- Appendix C: 1-bit operands, ternary gradients
def qbp_binarize_s8(x, q=None, qp_out=None):
    if q is None: q = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    if qp_out is None: qp_out = new_qparams(1, x.device)
    _check(lib.qbp_binarize_s8(_ptr(x), C.c_int64(x.numel()), _ptr(q), _ptr(qp_out), _stream()))
    return q, qp_out


def qbp_stc_ternarize_s8(g, samples=1, seed=0, tensor_id=0, q=None, qp_out=None, ws=None):
    if q is None: q = torch.empty(g.shape, dtype=torch.int8, device=g.device)
    if qp_out is None: qp_out = new_qparams(1, g.device)
    if ws is None: ws = workspace(lib.qbp_stc_ternarize_workspace_bytes(), g.device)
    _check(lib.qbp_stc_ternarize_s8(_ptr(g), C.c_int64(g.numel()), int(samples), C.c_uint64(seed), C.c_uint32(tensor_id),
                                    _ptr(q), _ptr(qp_out), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return q, qp_out


def qbp_tbp_weight_gradient(a_codes, qa, g, samples, seed=0, tensor_id=0, d: ConvDesc | None = None, want_acc=False, ws=None):
    """Algorithm 1: (acc int64 or None, gW fp32, t_hi, t_lo, qp_t)."""
    if d is None:
        rows, K = a_codes.shape; N = g.shape[1]; shape = (K, N); dref = None
    else:
        rows = d.N * d.H * d.W; K = d.C; N = d.K; shape = (d.K, d.R, d.S, d.C); dref = C.byref(d)
    dev = g.device
    t_hi = torch.empty(g.shape, dtype=torch.int8, device=dev); t_lo = torch.empty(g.shape, dtype=torch.uint8, device=dev)
    qp_t = new_qparams(1, dev)
    acc = torch.empty(shape, dtype=torch.int64, device=dev) if want_acc else None
    gW = torch.empty(shape, dtype=torch.float32, device=dev)
    if ws is None: ws = workspace(lib.qbp_tbp_weight_gradient_workspace_bytes(dref, rows, N, K), dev)
    _check(lib.qbp_tbp_weight_gradient(dref, C.c_int64(rows), C.c_int64(N), C.c_int64(K), _ptr(a_codes), _ptr(qa), _ptr(g),
                                       int(samples), C.c_uint64(seed), C.c_uint32(tensor_id), _ptr(t_hi), _ptr(t_lo), _ptr(qp_t),
                                       _ptr(acc), _ptr(gW), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return acc, gW, t_hi, t_lo, qp_t


def qbp_pack_bits(codes, mask=False, words=None):
    rows, cols = codes.shape
    if words is None: words = torch.empty((rows, (cols + 31) // 32), dtype=torch.int32, device=codes.device)
    _check(lib.qbp_pack_bits(_ptr(codes), C.c_int64(rows), C.c_int64(cols), int(mask), _ptr(words), _stream()))
    return words


def qbp_xnor_gemm_bits(A_bits, B_bits, K, out=None):
    M, N = A_bits.shape[0], B_bits.shape[0]
    if out is None: out = torch.empty((M, N), dtype=torch.int32, device=A_bits.device)
    _check(lib.qbp_xnor_gemm_bits(C.c_int64(M), C.c_int64(N), C.c_int64(K), _ptr(A_bits), _ptr(B_bits), _ptr(out), _stream()))
    return out


def qbp_gated_xnor_gemm_bits(nz_bits, sign_bits, B_bits, K, out=None):
    M, N = nz_bits.shape[0], B_bits.shape[0]
    if out is None: out = torch.empty((M, N), dtype=torch.int32, device=nz_bits.device)
    _check(lib.qbp_gated_xnor_gemm_bits(C.c_int64(M), C.c_int64(N), C.c_int64(K), _ptr(nz_bits), _ptr(sign_bits), _ptr(B_bits),
                                        _ptr(out), _stream()))
    return out


# ------------------------------------------------------------------- Range BN
def qbp_rangebn_fwd(x, gamma=None, beta=None, relu=False, y=None, want_range=False, ws=None):
    Cc = x.shape[-1]; n = x.numel() // Cc
    if y is None: y = torch.empty_like(x)
    mean = torch.empty(Cc, dtype=torch.float32, device=x.device)
    vmin = torch.empty_like(mean); vmax = torch.empty_like(mean)
    out_range = new_qparams(1, x.device) if want_range else None
    if ws is None: ws = workspace(lib.qbp_rangebn_workspace_bytes(n, Cc), x.device)
    _check(lib.qbp_rangebn_fwd(_ptr(x), C.c_int64(n), C.c_int64(Cc), _ptr(gamma), _ptr(beta), int(relu), _ptr(y),
                               _ptr(mean), _ptr(vmin), _ptr(vmax), _ptr(out_range), _ptr(ws), C.c_size_t(ws.numel()),
                               _stream()))
    return y, mean, vmin, vmax, out_range


def qbp_rangebn_fwd_q8(x, gamma=None, beta=None, relu=False, y=None, want_y=True, q=None, qp=None, row_sums=None,
                       want_row_sums=False, ws=None, chan_sums=None):
    """Range BN forward that also (or only: want_y=False) writes the 8-bit codes of its output for the next layer.
    Returns (y or None, mean, vmin, vmax, q, qp, row_sums or None)."""
    Cc = x.shape[-1]; n = x.numel() // Cc
    if y is None and want_y: y = torch.empty_like(x)
    if q is None: q = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    if qp is None: qp = new_qparams(1, x.device)
    if row_sums is None and want_row_sums: row_sums = torch.empty(n, dtype=torch.int32, device=x.device)
    mean = torch.empty(Cc, dtype=torch.float32, device=x.device)
    vmin = torch.empty_like(mean); vmax = torch.empty_like(mean)
    if ws is None: ws = workspace(lib.qbp_rangebn_workspace_bytes(n, Cc), x.device)
    rq = requant(q, qp, row_sums, chan_sums)
    _check(lib.qbp_rangebn_fwd_q8(_ptr(x), C.c_int64(n), C.c_int64(Cc), _ptr(gamma), _ptr(beta), int(relu), _ptr(y),
                                  _ptr(mean), _ptr(vmin), _ptr(vmax), None, C.byref(rq), _ptr(ws), C.c_size_t(ws.numel()),
                                  _stream()))
    return y, mean, vmin, vmax, q, qp, row_sums


def qbp_rangebn_fwd_stats(x, col_sum=None, col_min=None, col_max=None, ws=None):
    """This GPU's per-channel (sum fp64, min, max) of x, to be combined over the GPUs that share the minibatch."""
    Cc = x.shape[-1]; n = x.numel() // Cc
    if col_sum is None: col_sum = torch.empty(Cc, dtype=torch.float64, device=x.device)
    if col_min is None: col_min = torch.empty(Cc, dtype=torch.float32, device=x.device)
    if col_max is None: col_max = torch.empty(Cc, dtype=torch.float32, device=x.device)
    if ws is None: ws = workspace(lib.qbp_rangebn_workspace_bytes(n, Cc), x.device)
    _check(lib.qbp_rangebn_fwd_stats(_ptr(x), C.c_int64(n), C.c_int64(Cc), _ptr(col_sum), _ptr(col_min), _ptr(col_max),
                                     _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return col_sum, col_min, col_max


def qbp_rangebn_fwd_apply(x, n_stat, col_sum, col_min, col_max, gamma=None, beta=None, relu=False, y=None, want_y=True,
                          rq: Requant | None = None, want_range=False):
    """Normalise this GPU's rows with the combined statistics of n_stat rows.  Returns (y, mean, vmin, vmax, out_range)."""
    Cc = x.shape[-1]; n = x.numel() // Cc
    if y is None and want_y: y = torch.empty_like(x)
    mean = torch.empty(Cc, dtype=torch.float32, device=x.device)
    vmin = torch.empty_like(mean); vmax = torch.empty_like(mean)
    out_range = new_qparams(1, x.device) if want_range else None
    _check(lib.qbp_rangebn_fwd_apply(_ptr(x), C.c_int64(n), C.c_int64(n_stat), C.c_int64(Cc), _ptr(col_sum), _ptr(col_min),
                                     _ptr(col_max), _ptr(gamma), _ptr(beta), int(relu), _ptr(y), _ptr(mean), _ptr(vmin),
                                     _ptr(vmax), _ptr(out_range), C.byref(rq) if rq is not None else None, _stream()))
    return y, mean, vmin, vmax, out_range


def qbp_rangebn_bwd_stats(dy, x, n_stat, mean, vmin, vmax, gamma=None, beta=None, relu=False, ws=None):
    """This GPU's per-channel (sum dy, sum dy*xhat), fp64, to be added up over the GPUs."""
    Cc = x.shape[-1]; n = x.numel() // Cc
    sdy = torch.empty(Cc, dtype=torch.float64, device=x.device); sdyx = torch.empty_like(sdy)
    if ws is None: ws = workspace(lib.qbp_rangebn_workspace_bytes(n, Cc), x.device)
    _check(lib.qbp_rangebn_bwd_stats(_ptr(dy), _ptr(x), C.c_int64(n), C.c_int64(n_stat), C.c_int64(Cc), _ptr(gamma),
                                     _ptr(beta), int(relu), _ptr(mean), _ptr(vmin), _ptr(vmax), _ptr(sdy), _ptr(sdyx),
                                     _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return sdy, sdyx


def qbp_rangebn_bwd_apply(dy, x, n_stat, mean, vmin, vmax, sum_dy, sum_dyxhat, gamma=None, beta=None, relu=False,
                          dx=None, ws=None):
    Cc = x.shape[-1]; n = x.numel() // Cc
    if dx is None: dx = torch.empty_like(x)
    dgamma = torch.empty(Cc, dtype=torch.float32, device=x.device); dbeta = torch.empty_like(dgamma)
    if ws is None: ws = workspace(lib.qbp_rangebn_workspace_bytes(n, Cc), x.device)
    _check(lib.qbp_rangebn_bwd_apply(_ptr(dy), _ptr(x), C.c_int64(n), C.c_int64(n_stat), C.c_int64(Cc), _ptr(gamma),
                                     _ptr(beta), int(relu), _ptr(mean), _ptr(vmin), _ptr(vmax), _ptr(sum_dy),
                                     _ptr(sum_dyxhat), _ptr(dx), _ptr(dgamma), _ptr(dbeta), _ptr(ws),
                                     C.c_size_t(ws.numel()), _stream()))
    return dx, dgamma, dbeta


def qbp_rangebn_bwd(dy, x, mean, vmin, vmax, gamma=None, beta=None, relu=False, dx=None, ws=None):
    Cc = x.shape[-1]; n = x.numel() // Cc
    if dx is None: dx = torch.empty_like(x)
    dgamma = torch.empty(Cc, dtype=torch.float32, device=x.device); dbeta = torch.empty_like(dgamma)
    if ws is None: ws = workspace(lib.qbp_rangebn_workspace_bytes(n, Cc), x.device)
    _check(lib.qbp_rangebn_bwd(_ptr(dy), _ptr(x), C.c_int64(n), C.c_int64(Cc), _ptr(gamma), _ptr(beta), int(relu),
                               _ptr(mean), _ptr(vmin), _ptr(vmax), _ptr(dx), _ptr(dgamma), _ptr(dbeta), _ptr(ws),
                               C.c_size_t(ws.numel()), _stream()))
    return dx, dgamma, dbeta


def qbp_sgd_update(w, dw, momentum_buf=None, lr=0.1, momentum=0.0, weight_decay=0.0):
    """In-place fp32 update of master weights (Section 6): v = momentum*v + (dw + wd*w); w -= lr*v."""
    _check(lib.qbp_sgd_update(_ptr(w), _ptr(dw), _ptr(momentum_buf), C.c_int64(w.numel()), C.c_float(lr),
                              C.c_float(momentum), C.c_float(weight_decay), _stream()))
    return w


# ---------------------------------------------------------------------- layer
def qbp_layer_workspace_bytes(L: LayerDesc) -> int:
    return int(lib.qbp_layer_workspace_bytes(C.byref(L)))


def qbp_layer_fwd(L: LayerDesc, x, w, gamma, beta, y, ctx: LayerCtx, ws):
    _check(lib.qbp_layer_fwd(C.byref(L), _ptr(x), _ptr(w), _ptr(gamma), _ptr(beta), _ptr(y), C.byref(ctx), _ptr(ws),
                             C.c_size_t(ws.numel()), _stream()))
    return y


def qbp_layer_fwd_chained(L: LayerDesc, x, rq_in, w, gamma, beta, y, rq_out, ctx: LayerCtx, ws):
    """qbp_layer_fwd with the input already quantised by the previous layer (rq_in, x None) and / or the output's
    8-bit codes written for the next one (rq_out; y may then be None)."""
    _check(lib.qbp_layer_fwd_chained(C.byref(L), _ptr(x), C.byref(rq_in) if rq_in is not None else None, _ptr(w),
                                     _ptr(gamma), _ptr(beta), _ptr(y), C.byref(rq_out) if rq_out is not None else None,
                                     C.byref(ctx), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return y


def qbp_layer_bwd(L: LayerDesc, ctx: LayerCtx, dy, gamma, beta, dx, dw, dgamma, dbeta, ws):
    _check(lib.qbp_layer_bwd(C.byref(L), C.byref(ctx), _ptr(dy), _ptr(gamma), _ptr(beta), _ptr(dx), _ptr(dw),
                             _ptr(dgamma), _ptr(dbeta), _ptr(ws), C.c_size_t(ws.numel()), _stream()))
    return dx, dw, dgamma, dbeta


# ---------------------------------------------------------------- diagnostics
def trace_enable(on: bool) -> None:
    _check(lib.qbp_trace_enable(int(on)))


def trace_records():
    """[(kernel name, device milliseconds)] of every launch since trace_enable(True); synchronises first."""
    torch.cuda.synchronize()
    out = []
    name = C.create_string_buffer(64); ms = C.c_float()
    for i in range(lib.qbp_trace_count()):
        _check(lib.qbp_trace_read(i, name, 64, C.byref(ms)))
        out.append((name.value.decode(), float(ms.value)))
    return out
