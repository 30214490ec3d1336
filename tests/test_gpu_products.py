"""GPU integer products (tcgen05 int8 GEMM, implicit-GEMM convolution, limb-split weight gradient)
vs the CPU oracle: int32 / int64 accumulators bit for bit, fp32 outputs identical (same single multiply)."""
import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth
from tests.util import random_codes, set_qparams, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


def _qp(B, scale, zp):
    return set_qparams(B.new_qparams(1), scale, zp)


# ------------------------------------------------------------------ GEMM
GEMMS = [(128, 128, 128), (64, 128, 256), (64, 256, 128), (16, 16, 16), (208, 80, 144), (256, 384, 512),
         (384, 640, 1040), (128, 272, 33024)]


@pytest.mark.parametrize("M,N,K", GEMMS)
@pytest.mark.parametrize("tA,tB", [(False, False), (False, True), (True, False), (True, True)])
def test_gemm_s8(B, M, N, K, tA, tB):
    A = random_codes((K, M) if tA else (M, K), 1); Bm = random_codes((N, K) if tB else (K, N), 2)
    za, zb, sa, sb = 3, -128, 0.5, 0.25
    if K > 30000:                       # keep the exact sum inside int32: small codes at the longest legal K
        A = (A // 4).astype(np.int8); Bm = (Bm // 4).astype(np.int8); zb = -5
    acc, out, ws = B.qbp_gemm_s8(to_dev(A), _qp(B, sa, za), to_dev(Bm), _qp(B, sb, zb), transA=tA, transB=tB, want_acc=True)
    oacc, oout, bad = O.gemm_s8(A, za, Bm, zb, sa, sb, transA=tA, transB=tB)
    assert bad == 0 and B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc)
    assert np.array_equal(to_host(out), oout)


def test_gemm_extreme_codes_and_zero_points(B):
    M, N, K = 128, 128, 33024 // 2
    A = np.full((M, K), -128, np.int8); Bm = np.full((K, N), 127, np.int8)
    acc, _, ws = B.qbp_gemm_s8(to_dev(A), _qp(B, 1, 127), to_dev(Bm), _qp(B, 1, -128), want_acc=True, want_out=False)
    assert B.status_word(ws) == 0
    assert np.all(to_host(acc) == (-255) * 255 * K)


def test_gemm_dense_sweep_shape_sampled_rows(B):
    """4096^3 from the dense sweep, operands quantised from N(0,1); oracle on 192 sampled rows."""
    case = synth.dense_gemm(4096, 4096, 4096)
    qa, qpa = B.qbp_quantize_s8(to_dev(case["a"])); qb, qpb = B.qbp_quantize_s8(to_dev(case["b"]))
    oa = O.quantize(case["a"], 8); ob = O.quantize(case["b"], 8)
    assert np.array_equal(to_host(qa), oa.q) and np.array_equal(to_host(qb), ob.q)
    acc, out, ws = B.qbp_gemm_s8(qa, qpa, qb, qpb, want_acc=True)
    assert B.status_word(ws) == 0
    rows = np.unique(np.concatenate([[0, 127, 128, 4095, 3968], np.random.Generator(np.random.PCG64(5)).integers(0, 4096, 187)]))
    oacc, oout, bad = O.gemm_s8(oa.q[rows], oa.zero_point[0], ob.q, ob.zero_point[0], oa.scale[0], ob.scale[0])
    assert bad == 0
    assert np.array_equal(to_host(acc)[rows], oacc) and np.array_equal(to_host(out)[rows], oout)


def test_gemm_dense_sweep_8192_sampled_rows_and_corner_tiles(B):
    """8192^3 from the dense sweep in the benchmark's launch configuration (256 x 256 tiles, several tiles per CTA);
    oracle on 64 random rows plus the rows of the four corner tiles' edges."""
    n = 8192
    case = synth.dense_gemm(n, n, n)
    qa, qpa = B.qbp_quantize_s8(to_dev(case["a"])); qb, qpb = B.qbp_quantize_s8(to_dev(case["b"]))
    oa = O.quantize(case["a"], 8); ob = O.quantize(case["b"], 8)
    assert np.array_equal(to_host(qa), oa.q) and np.array_equal(to_host(qb), ob.q)
    acc, out, ws = B.qbp_gemm_s8(qa, qpa, qb, qpb, want_acc=True)
    assert B.status_word(ws) == 0
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, n - 256, n - 129, n - 128, n - 1],
                                     np.random.Generator(np.random.PCG64(6)).integers(0, n, 64)]))
    oacc, oout, bad = O.gemm_s8(oa.q[rows], oa.zero_point[0], ob.q, ob.zero_point[0], oa.scale[0], ob.scale[0])
    assert bad == 0
    assert np.array_equal(to_host(acc[rows]), oacc) and np.array_equal(to_host(out[rows]), oout)


def _dense_gemm_sampled(B, M, N, K, seed, n_random=64):
    """One product of the dense sweep in the benchmark's launch configuration: operands quantised from N(0,1) on both
    sides (codes compared in full), accumulators and fp32 outputs compared on the rows at the tile edges plus
    n_random random rows, every column."""
    case = synth.dense_gemm(M, N, K, parts=("a", "b"))
    qa, qpa = B.qbp_quantize_s8(to_dev(case["a"])); qb, qpb = B.qbp_quantize_s8(to_dev(case["b"]))
    oa = O.quantize(case["a"], 8); ob = O.quantize(case["b"], 8)
    del case
    assert np.array_equal(to_host(qa), oa.q) and np.array_equal(to_host(qb), ob.q)
    acc, out, ws = B.qbp_gemm_s8(qa, qpa, qb, qpb, want_acc=True)
    assert B.status_word(ws) == 0
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, 511, 512, M - 512, M - 257, M - 256, M - 129, M - 128, M - 1],
                                     np.random.Generator(np.random.PCG64(seed)).integers(0, M, n_random)]))
    oacc, oout, bad = O.gemm_s8(oa.q[rows], oa.zero_point[0], ob.q, ob.zero_point[0], oa.scale[0], ob.scale[0])
    assert bad == 0
    assert np.array_equal(to_host(acc[rows]), oacc) and np.array_equal(to_host(out[rows]), oout)


def test_gemm_dense_sweep_16384_sampled_rows(B):
    """The largest cube of the dense sweep (16384^3, 512 x 256 pair tiles, 32 x 64 of them over 74 CTA pairs)."""
    _dense_gemm_sampled(B, 16384, 16384, 16384, 8, n_random=32)


# (M, N, K) combinations of the sweep that are not cubes: tall, wide, deep and shallow ones
NONCUBE = [(4096, 16384, 8192), (16384, 4096, 4096), (8192, 4096, 16384), (4096, 8192, 16384)]


@pytest.mark.parametrize("M,N,K", NONCUBE)
def test_gemm_dense_sweep_noncube_sampled_rows(B, M, N, K):
    _dense_gemm_sampled(B, M, N, K, 9 + M // 4096 + N // 2048, n_random=48)


def _dense_wgrad_sampled(B, M, N, K, seed, n_cols):
    """The limb-split 16 x 8-bit product dW [K x N] = X [M x K]^T G [M x N] of the dense sweep: operands quantised from
    N(0,1) (nearest for the 8-bit side, stochastic for the 16-bit side, codes compared in full); int64
    accumulators and fp32 outputs compared on the output columns at the tile edges plus random ones, every row."""
    case = synth.dense_gemm(M, N, K, parts=("x", "g"))
    qx, qpx = B.qbp_quantize_s8(to_dev(case["x"]))
    q16, hi, lo, qpg = B.qbp_quantize_s16(to_dev(case["g"]), rounding=B.QBP_ROUND_STOCHASTIC, seed=3, tensor_id=7)
    ox = O.quantize(case["x"], 8); og = O.quantize(case["g"], 16, rounding=1, seed=3, tensor_id=7)
    del case
    assert np.array_equal(to_host(qx), ox.q) and np.array_equal(to_host(q16), og.q)
    del q16
    acc, dW, ws = B.qbp_wgrad_s16(qx, qpx, hi, lo, qpg, want_acc=True)
    assert B.status_word(ws) == 0
    cols = np.unique(np.concatenate([[0, 127, 128, N - 129, N - 128, N - 1],
                                     np.random.Generator(np.random.PCG64(seed)).integers(0, N, n_cols)]))
    oacc, oout = O.gemm_s16s8(ox.q, ox.zero_point[0], np.ascontiguousarray(og.q[:, cols]), og.zero_point[0], ox.scale[0], og.scale[0])
    assert np.array_equal(to_host(acc[:, cols]), oacc) and np.array_equal(to_host(dW[:, cols]), oout)


@pytest.mark.parametrize("n,n_cols", [(8192, 48), (16384, 16)])
def test_wgrad_dense_sweep_large_cubes_sampled_columns(B, n, n_cols):
    """8192^3 and 16384^3: the reduction over M is split over CTAs in chunks of at most 65536 rows and summed in int64."""
    _dense_wgrad_sampled(B, n, n, n, 10 + n // 8192, n_cols)


@pytest.mark.parametrize("M,N,K", NONCUBE)
def test_wgrad_dense_sweep_noncube_sampled_columns(B, M, N, K):
    _dense_wgrad_sampled(B, M, N, K, 20 + M // 4096 + K // 2048, 24)


# Shapes the CTA-pair kernel takes (at least eight rounds of 256 x 256 tiles over the SM pairs) with ragged edges in
# every dimension: 512 x 256 pair tiles (M >= 2048) and 256 x 256 pair tiles (short M, wide N).
PAIR_GEMMS = [(8208, 8464, 208), (1104, 38000, 144), (2048, 19216, 400)]


@pytest.mark.parametrize("M,N,K", PAIR_GEMMS)
@pytest.mark.parametrize("tA,tB", [(False, False), (False, True), (True, False), (True, True)])
def test_gemm_s8_pair_kernel_ragged_sampled_rows(B, M, N, K, tA, tB):
    """Oracle on the rows at the tile and pair-half edges, the ragged last rows and 48 random ones; every column."""
    A = random_codes((K, M) if tA else (M, K), 11); Bm = random_codes((N, K) if tB else (K, N), 12)
    za, zb, sa, sb = -7, 19, 0.125, 0.5
    acc, out, ws = B.qbp_gemm_s8(to_dev(A), _qp(B, sa, za), to_dev(Bm), _qp(B, sb, zb), transA=tA, transB=tB, want_acc=True)
    assert B.status_word(ws) == 0
    edge = [0, 127, 128, 255, 256, 383, 384, 511, 512, M - 1, M - 2, (M // 512) * 512 - 1, (M // 256) * 256 - 1,
            min((M // 256) * 256, M - 1), min((M // 128) * 128, M - 1)]
    rows = np.unique(np.concatenate([edge, np.random.Generator(np.random.PCG64(M)).integers(0, M, 48)]))
    Arows = np.ascontiguousarray(A[:, rows]) if tA else A[rows]
    oacc, oout, bad = O.gemm_s8(Arows, za, Bm, zb, sa, sb, transA=tA, transB=tB)
    assert bad == 0
    assert np.array_equal(to_host(acc[rows]), oacc) and np.array_equal(to_host(out[rows]), oout)


# ------------------------------------------- column statistics from the epilogue
def _check_col_stats(out, stats):
    o = to_host(out).reshape(-1, out.shape[-1]).astype(np.float64)
    csum, cmin, cmax = (to_host(t) for t in stats)
    assert np.array_equal(cmin, o.min(axis=0).astype(np.float32)) and np.array_equal(cmax, o.max(axis=0).astype(np.float32))
    # partial sums of at most 32 fp32 values in fp32, the rest in fp64
    assert np.allclose(csum, o.sum(axis=0), rtol=0, atol=1e-6 * np.abs(o).sum(axis=0).max())


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (208, 80, 144), (1024, 256, 512), (2000, 64, 64)])
def test_gemm_epilogue_column_statistics(B, M, N, K):
    """Section 3: the sum, minimum and maximum of every output column, as the following Range BN needs them, taken
    from the fp32 outputs in the product's epilogue; the product itself is unchanged."""
    A = random_codes((M, K), 21); Bm = random_codes((K, N), 22)
    za, zb, sa, sb = 5, -9, 0.5, 0.125
    acc, out, ws, stats = B.qbp_gemm_s8(to_dev(A), _qp(B, sa, za), to_dev(Bm), _qp(B, sb, zb), want_acc=True, col_stats=True)
    oacc, oout, bad = O.gemm_s8(A, za, Bm, zb, sa, sb)
    assert bad == 0 and B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc) and np.array_equal(to_host(out), oout)
    _check_col_stats(out, stats)


@pytest.mark.parametrize("N,H,W,C,K,R", [(2, 56, 56, 64, 64, 3), (3, 10, 12, 32, 48, 3), (4, 7, 7, 256, 128, 1), (2, 20, 17, 128, 32, 3)])
@pytest.mark.parametrize("mode", [0, 1])
def test_conv_epilogue_channel_statistics(B, N, H, W, C, K, R, mode):
    """The same for a convolution (ragged pixel boxes: positions outside the image must not count)."""
    pad = (R - 1) // 2
    d = B.conv_desc(N, H, W, C, K, R, R, 1, pad); od = O.conv_desc(N, H, W, C, K, R, R, 1, pad)
    inp = random_codes((N, H, W, C if mode == 0 else K), 23); w = random_codes((K, R, R, C), 24)
    zi, zw = -3, 11
    acc, out, ws, stats = B.qbp_conv_s8_implicit(mode, d, to_dev(inp), _qp(B, 0.5, zi), to_dev(w), _qp(B, 0.25, zw),
                                                 want_acc=True, col_stats=True)
    oacc, oout, bad = O.conv_s8(mode, od, inp, zi, w, zw, 0.5, 0.25)
    assert bad == 0 and B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc) and np.array_equal(to_host(out), oout)
    _check_col_stats(out, stats)


@pytest.mark.parametrize("N,H,W,C,K,R,mode", [(8, 14, 14, 128, 512, 1, 0), (2, 9, 9, 64, 768, 1, 0), (2, 10, 10, 640, 64, 3, 1),
                                              (64, 28, 28, 128, 512, 1, 0), (64, 14, 14, 64, 768, 1, 0)])
def test_conv_epilogue_channel_statistics_of_wide_outputs(B, N, H, W, C, K, R, mode):
    """More than 256 output channels: several column tiles, each CTA keeping the statistics of the one it meets (two
    and three column tiles, a ragged last one, grids smaller than and as large as the device)."""
    pad = (R - 1) // 2
    d = B.conv_desc(N, H, W, C, K, R, R, 1, pad); od = O.conv_desc(N, H, W, C, K, R, R, 1, pad)
    inp = random_codes((N, H, W, C if mode == 0 else K), 25); w = random_codes((K, R, R, C), 26)
    zi, zw = 7, -2
    acc, out, ws, stats = B.qbp_conv_s8_implicit(mode, d, to_dev(inp), _qp(B, 0.5, zi), to_dev(w), _qp(B, 0.25, zw),
                                                 want_acc=True, col_stats=True)
    oacc, oout, bad = O.conv_s8(mode, od, inp, zi, w, zw, 0.5, 0.25)
    assert bad == 0 and B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc) and np.array_equal(to_host(out), oout)
    _check_col_stats(out, stats)


def test_wgrad_dense_sweep_shape_sampled_columns(B):
    """The limb-split 16 x 8-bit product at 4096^3 (dense sweep): operands quantised from N(0,1) (nearest for the
    8-bit side, stochastic for the 16-bit side); oracle on 96 sampled output columns (all 4096 rows of each)."""
    n = 4096
    case = synth.dense_gemm(n, n, n)
    qx, qpx = B.qbp_quantize_s8(to_dev(case["x"]))
    q16, hi, lo, qpg = B.qbp_quantize_s16(to_dev(case["g"]), rounding=B.QBP_ROUND_STOCHASTIC, seed=3, tensor_id=7)
    ox = O.quantize(case["x"], 8); og = O.quantize(case["g"], 16, rounding=1, seed=3, tensor_id=7)
    assert np.array_equal(to_host(qx), ox.q) and np.array_equal(to_host(q16), og.q)
    acc, dW, ws = B.qbp_wgrad_s16(qx, qpx, hi, lo, qpg, want_acc=True)
    assert B.status_word(ws) == 0
    cols = np.unique(np.concatenate([[0, 127, 128, n - 1], np.random.Generator(np.random.PCG64(7)).integers(0, n, 92)]))
    oacc, oout = O.gemm_s16s8(ox.q, ox.zero_point[0], np.ascontiguousarray(og.q[:, cols]), og.zero_point[0], ox.scale[0], og.scale[0])
    assert np.array_equal(to_host(acc)[:, cols], oacc) and np.array_equal(to_host(dW)[:, cols], oout)


# ----------------------------------------------------------- convolution
CONVS = [(2, 8, 8, 64, 64, 1), (2, 8, 8, 64, 64, 3), (3, 10, 12, 32, 48, 3), (2, 14, 14, 128, 256, 3),
         (4, 7, 7, 256, 128, 1), (1, 1, 1, 16, 16, 3), (5, 9, 3, 80, 16, 3), (3, 28, 28, 128, 128, 3),
         (2, 56, 56, 64, 64, 3), (1, 5, 130, 16, 272, 3),
         # boxes loaded once with their border (taps as shifted windows): 128-, 64- and 32-byte channel chunks,
         # several chunks per tile, ragged boxes in both directions
         (2, 20, 17, 128, 32, 3), (2, 20, 17, 32, 128, 3), (1, 33, 9, 192, 32, 3), (2, 16, 8, 256, 16, 3),
         (1, 40, 24, 16, 64, 3)]


@pytest.mark.parametrize("N,H,W,C,K,R", CONVS)
@pytest.mark.parametrize("mode", [0, 1])
def test_conv_s8(B, N, H, W, C, K, R, mode):
    pad = (R - 1) // 2
    d = B.conv_desc(N, H, W, C, K, R, R, 1, pad); od = O.conv_desc(N, H, W, C, K, R, R, 1, pad)
    inp = random_codes((N, H, W, C if mode == 0 else K), 3); w = random_codes((K, R, R, C), 4)
    zi, zw = 7, -128
    acc, out, ws = B.qbp_conv_s8_implicit(mode, d, to_dev(inp), _qp(B, 0.5, zi), to_dev(w), _qp(B, 0.25, zw), want_acc=True)
    oacc, oout, bad = O.conv_s8(mode, od, inp, zi, w, zw, 0.5, 0.25)
    assert bad == 0 and B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc)
    assert np.array_equal(to_host(out), oout)


# --------------------------------------------------------- weight gradient
def _g16(shape, seed):
    return random_codes(shape, seed, -32768, 32767, np.int16)


# (the last four run on CTA pairs: ragged in every dimension, a short and a long reduction)
WGRADS = [(128, 128, 128), (64, 128, 256), (1000, 64, 64), (70000, 32, 48), (4096, 256, 384), (130, 16, 16),
          (1000, 272, 400), (520, 528, 256), (2064, 1040, 784), (4096, 2304, 512)]


@pytest.mark.parametrize("M,N,K", WGRADS)
def test_wgrad_plain(B, M, N, K):
    X = random_codes((M, K), 5); G = _g16((M, N), 6)
    hi, lo = O.limb_split(G)
    zx, zg = -128, 32767
    acc, dW, ws = B.qbp_wgrad_s16(to_dev(X), _qp(B, 0.5, zx), to_dev(hi), to_dev(lo), _qp(B, 0.25, zg), want_acc=True)
    oacc, oout = O.gemm_s16s8(X, zx, G, zg, 0.5, 0.25)
    assert B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc) and np.array_equal(to_host(dW), oout)


def test_wgrad_long_reduction_extreme_codes(B):
    """131072 rows of extreme codes: each CTA's int32 chunk stays in range, the int64 total is exact."""
    M, N, K = 131072, 32, 32
    X = np.full((M, K), -128, np.int8); G = np.full((M, N), 32767, np.int16)
    G[::2] = -32768
    hi, lo = O.limb_split(G)
    acc, _, ws = B.qbp_wgrad_s16(to_dev(X), _qp(B, 1, 127), to_dev(hi), to_dev(lo), _qp(B, 1, 0), want_acc=True, want_out=False)
    assert B.status_word(ws) == 0
    assert np.all(to_host(acc) == (-255) * (32767 - 32768) * (M // 2))


def test_wgrad_pair_kernel_longest_reduction_extreme_codes(B):
    """65536 rows, the most one CTA pair accumulates in int32: every low-limb product at 128 * 255, every high-limb
    product at 128 * 128; the int64 combination must still be exact."""
    M, N, K = 65536, 256, 256
    X = np.full((M, K), -128, np.int8); G = np.full((M, N), -32513, np.int16)        # hi = -128, lo = 255
    hi, lo = O.limb_split(G)
    assert hi.min() == hi.max() == -128 and lo.min() == lo.max() == 255
    acc, _, ws = B.qbp_wgrad_s16(to_dev(X), _qp(B, 1, 0), to_dev(hi), to_dev(lo), _qp(B, 1, 0), want_acc=True, want_out=False)
    assert B.status_word(ws) == 0
    assert np.all(to_host(acc) == (-128) * (-32513) * M)


WCONVS = [(2, 8, 8, 64, 64, 1), (2, 8, 8, 64, 64, 3), (3, 10, 12, 32, 96, 3), (2, 14, 14, 128, 256, 3),
          (4, 7, 7, 256, 128, 1), (1, 1, 1, 32, 32, 3), (2, 28, 28, 128, 128, 3), (3, 9, 5, 96, 160, 3)]


@pytest.mark.parametrize("N,H,W,C,K,R", WCONVS)
def test_wgrad_conv(B, N, H, W, C, K, R):
    pad = (R - 1) // 2
    d = B.conv_desc(N, H, W, C, K, R, R, 1, pad); od = O.conv_desc(N, H, W, C, K, R, R, 1, pad)
    X = random_codes((N, H, W, C), 7); G = _g16((N, H, W, K), 8)
    hi, lo = O.limb_split(G)
    zx, zg = 5, -300
    acc, dW, ws = B.qbp_wgrad_s16(to_dev(X), _qp(B, 0.5, zx), to_dev(hi), to_dev(lo), _qp(B, 0.25, zg), d=d, want_acc=True)
    oacc, oout = O.conv_wgrad_s16(od, X, zx, G, zg, 0.5, 0.25)
    assert B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc) and np.array_equal(to_host(dW), oout)


# ------------------------------------------- ReLU and requantisation in the epilogue (no Range BN after the product)
def _check_requant(B, out_dev, q_dev, qp_dev, rs_dev, oout, relu, rng):
    want = np.maximum(oout, 0) if relu else oout
    if out_dev is not None:
        assert np.array_equal(to_host(out_dev), want)
    o = O.quantize(want, 8, range_in=rng)                # values beyond the clamp saturate
    s_, z_, lo_, hi_ = B.read_qparams(qp_dev)
    assert s_[0] == o.scale[0] and z_[0] == o.zero_point[0] and lo_[0] == o.vmin[0] and hi_[0] == o.vmax[0]
    assert np.array_equal(to_host(q_dev), o.q)
    if rs_dev is not None:
        assert np.array_equal(to_host(rs_dev), o.q.reshape(-1, o.q.shape[-1]).astype(np.int32).sum(1))


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (208, 80, 144), (1024, 256, 512), (2000, 64, 64), (384, 640, 256)])
@pytest.mark.parametrize("relu,keep_out", [(True, True), (False, False), (True, False)])
def test_gemm_epilogue_relu_and_requantisation(B, M, N, K, relu, keep_out):
    import torch
    A = random_codes((M, K), 31); Bm = random_codes((K, N), 32)
    za, zb, sa, sb = 5, -9, 0.5, 0.125
    _, oout, bad = O.gemm_s8(A, za, Bm, zb, sa, sb)
    assert bad == 0
    hi = np.float32(0.6 * oout.max()); lo = np.float32(0.0 if relu else 0.5 * oout.min())      # a clamp that cuts the tails
    q = torch.empty((M, N), dtype=torch.int8, device="cuda"); qp = B.new_qparams(1); rs = torch.empty(M, dtype=torch.int32, device="cuda")
    res = B.qbp_gemm_s8(to_dev(A), _qp(B, sa, za), to_dev(Bm), _qp(B, sb, zb), want_out=keep_out, relu=relu,
                        requant=(B.range_qparams(lo, hi), q, qp, rs))
    assert B.status_word(res[2]) == 0
    _check_requant(B, res[1] if keep_out else None, q, qp, rs, oout, relu, (lo, hi))


@pytest.mark.parametrize("N_,H,W,C_,K_,R", [(2, 56, 56, 64, 64, 3), (3, 10, 12, 32, 48, 3), (4, 7, 7, 256, 128, 1), (1, 5, 130, 16, 272, 3)])
@pytest.mark.parametrize("mode", [0, 1])
def test_conv_epilogue_relu_and_requantisation(B, N_, H, W, C_, K_, R, mode):
    import torch
    pad = (R - 1) // 2
    d = B.conv_desc(N_, H, W, C_, K_, R, R, 1, pad); od = O.conv_desc(N_, H, W, C_, K_, R, R, 1, pad)
    inp = random_codes((N_, H, W, C_ if mode == 0 else K_), 33); w = random_codes((K_, R, R, C_), 34)
    zi, zw = -3, 11
    _, oout, bad = O.conv_s8(mode, od, inp, zi, w, zw, 0.5, 0.25)
    assert bad == 0
    hi = np.float32(0.7 * oout.max()); lo = np.float32(0.0)
    q = torch.empty(oout.shape, dtype=torch.int8, device="cuda"); qp = B.new_qparams(1)
    rs = torch.empty(oout.size // oout.shape[-1], dtype=torch.int32, device="cuda")
    res = B.qbp_conv_s8_implicit(mode, d, to_dev(inp), _qp(B, 0.5, zi), to_dev(w), _qp(B, 0.25, zw), relu=True,
                                 requant=(B.range_qparams(lo, hi), q, qp, rs))
    assert B.status_word(res[2]) == 0
    _check_requant(B, res[1], q, qp, rs, oout, True, (lo, hi))


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (208, 80, 144), (1024, 512, 256)])
@pytest.mark.parametrize("tA,tB", [(False, False), (False, True), (True, False), (True, True)])
def test_gemm_with_caller_code_sums(B, M, N, K, tA, tB):
    """The code sums along the reduction handed in (as a chain of calls has them from the quantiser): same product,
    and no sum kernel in the launch list."""
    A = random_codes((K, M) if tA else (M, K), 41); Bm = random_codes((N, K) if tB else (K, N), 42)
    za, zb, sa, sb = 3, -11, 0.5, 0.25
    a_sums = (A.astype(np.int32).sum(0 if tA else 1)).astype(np.int32); b_sums = (Bm.astype(np.int32).sum(1 if tB else 0)).astype(np.int32)
    B.trace_enable(True)
    acc, out, ws = B.qbp_gemm_s8(to_dev(A), _qp(B, sa, za), to_dev(Bm), _qp(B, sb, zb), transA=tA, transB=tB, want_acc=True,
                                 a_sums=to_dev(a_sums), b_sums=to_dev(b_sums))
    names = [n for n, _ in B.trace_records()]
    B.trace_enable(False)
    assert "rowsum_kernel" not in names and "colsum_kernel" not in names
    oacc, oout, bad = O.gemm_s8(A, za, Bm, zb, sa, sb, transA=tA, transB=tB)
    assert bad == 0 and B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), oacc) and np.array_equal(to_host(out), oout)


@pytest.mark.parametrize("mode", ["fprop", "dgrad"])
def test_conv_at_full_size_is_reproducible(B, mode):
    """The 64-channel 3x3 convolution of the benchmark, twenty times on the same codes: every run must write the same
    bits.  (Integer accumulators and one fp32 scale leave no room for run-to-run differences; a difference means a
    race -- one was found this way: an output slab refilled while the store of the tile before was still reading it,
    in tiles whose rows lie partly outside the image.)  Each run starts from an output filled with NaN."""
    import torch
    cfg = synth.conv3x3_layer()
    c = cfg["conv"]
    d = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    src = to_dev(cfg["x"] if mode == "fprop" else cfg["dy"])
    q_in, p_in = B.qbp_quantize_s8(src)
    w = to_dev(cfg["w"])
    q_w, p_w = B.qbp_quantize_s8(w.reshape(c["K"], -1))
    out = torch.empty((c["N"], c["H"], c["W"], 64), dtype=torch.float32, device="cuda")
    ref = None
    for rep in range(20):
        out.fill_(float("nan"))
        B.qbp_conv_s8_implicit(B.QBP_CONV_FPROP if mode == "fprop" else B.QBP_CONV_DGRAD, d, q_in, p_in, q_w.reshape(w.shape), p_w, out=out)
        torch.cuda.synchronize()
        bits = out.view(torch.int32)
        if ref is None:
            ref = bits.clone()
            assert not bool(torch.isnan(out).any())
        else:
            assert int((bits != ref).sum()) == 0, f"run {rep} differs from run 0"
