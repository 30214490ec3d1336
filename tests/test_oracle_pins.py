"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible slip in the oracle (a dropped term, a wrong sign or index, a
transposed operand, 2^M instead of 2^M - 1 levels, a wrong Philox constant)
fails it.
"""
import itertools
import math
from pathlib import Path

import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth

GOLDEN = Path(__file__).parent / "golden"


def _paper_constants():
    out = {}
    for line in (GOLDEN / "paper_constants.txt").read_text().splitlines():
        line = line.split("#")[0].split()
        if len(line) == 3:
            out[line[0]] = (float(line[1]), float(line[2]))
    return out


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    n = 0
    for line in (GOLDEN / "philox4x32_10_kat.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        v = [int(t, 16) for t in line.split()]
        assert list(O.philox4x32_10(v[:4], v[4:6])) == v[6:]
        n += 1
    assert n == 3


def test_random_word_indexing():
    # element i -> block i//4 keyed by (seed lo, seed hi), counter (j lo, j hi, tensor id, 0), word i%4
    seed = 0x1234_5678_9ABC_DEF0
    for i in (0, 1, 2, 3, 4, 7, 2**34 + 5):
        j = i >> 2
        blk = O.philox4x32_10([j & 0xFFFFFFFF, j >> 32, 9, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert O.random_word(seed, 9, i) == int(blk[i & 3])
    assert O.random_word(seed, 9, 5) != O.random_word(seed, 10, 5)


# --------------------------------------------------------------- quantiser
CASES = {
    "gauss": lambda: synth.normal((257, 33), 100),
    "relu": lambda: synth.relu_normal((64, 130), 101),
    "positive": lambda: synth.uniform((50, 40), 102, 1.0) + np.float32(2.0),
    "negative": lambda: -(synth.uniform((50, 40), 103, 1.0) + np.float32(2.0)),
    "tiny": lambda: synth.normal((31, 7), 104, std=1e-6),
}


@pytest.mark.parametrize("bits,slack", [(8, 1e-4), (16, 1e-2)])
@pytest.mark.parametrize("name", list(CASES))
def test_nearest_error_bound_and_end_codes(name, bits, slack):
    x = CASES[name]()
    qt = O.quantize(x, bits)
    L = 2**bits - 1; half = 2**(bits - 1)
    s = float(qt.scale[0]); zp = int(qt.zero_point[0])
    err = np.abs(O.dequantize(qt).astype(np.float64) - x.astype(np.float64))
    assert err.max() <= s * (0.5 + slack)
    codes = qt.q.astype(np.int64) + half
    assert codes.min() >= 0 and codes.max() <= L
    # the interval always contains 0, and its ends land on the end codes
    lo, hi = min(float(x.min()), 0.0), max(float(x.max()), 0.0)
    assert qt.vmin[0] == np.float32(lo) and qt.vmax[0] == np.float32(hi)
    assert math.isclose(s, (hi - lo) / L, rel_tol=1e-6)
    if x.min() <= 0:
        assert codes.flat[np.argmin(x)] == 0
    if x.max() >= 0:
        assert codes.flat[np.argmax(x)] == L
    # real zero is exactly a code
    z = O.quantize(np.zeros((1, 4), np.float32), bits, range_in=(qt.vmin, qt.vmax))
    assert np.all(z.q == zp) and np.all(O.dequantize(z) == 0.0)


def test_integer_grid_is_reproduced_exactly():
    x = np.arange(-128, 128, dtype=np.float32).reshape(16, 16)
    qt = O.quantize(x, 8)
    assert qt.scale[0] == 1.0 and qt.zero_point[0] == 0
    assert np.array_equal(qt.q.astype(np.float32), x)
    x16 = np.linspace(-32768, 32767, 65536, dtype=np.float32).reshape(256, 256)
    q16 = O.quantize(x16, 16)
    assert q16.scale[0] == 1.0 and np.array_equal(q16.q.astype(np.float32), x16)


def test_nearest_is_monotone_and_ties_go_to_even():
    x = np.sort(synth.normal((1, 5000), 105).ravel()).reshape(1, -1)
    q = O.quantize(x, 8).q.ravel().astype(np.int32)
    assert np.all(np.diff(q) >= 0)
    # scale exactly 1 over [-128,127]; halves round to the even code
    t = np.array([[-128.0, 127.0, 0.5, 1.5, 2.5, -0.5, -1.5]], np.float32)
    assert list(O.quantize(t, 8).q.ravel()[2:]) == [0, 2, 2, 0, -2]


def test_degenerate_ranges():
    qt = O.quantize(np.zeros((3, 5), np.float32), 8)
    assert qt.scale[0] == 1.0 and np.all(qt.q == qt.zero_point[0]) and qt.zero_point[0] == -128
    c = O.quantize(np.full((3, 5), 2.5, np.float32), 8)      # all equal, positive: range [0, 2.5]
    assert c.zero_point[0] == -128 and np.all(c.q == 127)
    e = O.quantize(np.zeros((0, 5), np.float32), 8, range_in=(np.float32(-1), np.float32(1)))
    assert e.q.size == 0


def test_supplied_range_and_per_channel():
    x = synth.channel_gaussian((4, 6, 6, 8), 106, 107)
    lo, hi = O.tensor_range(x)
    assert lo[0] == x.min() and hi[0] == x.max()
    a = O.quantize(x, 8); b = O.quantize(x, 8, range_in=(lo, hi))
    assert np.array_equal(a.q, b.q) and a.scale == b.scale
    pc = O.quantize(x, 8, per_channel=True)
    for c in range(8):
        one = O.quantize(np.ascontiguousarray(x[..., c:c + 1]), 8)
        assert np.array_equal(pc.q[..., c], one.q[..., 0])
        assert pc.scale[c] == one.scale[0] and pc.zero_point[c] == one.zero_point[0]


def test_chunk_averaged_clamp_values():
    """Appendix B (activations): clamping values = the average over K chunks of the chunks' maxima and minima."""
    # worked by hand: chunk 0 = rows 0-1 (min -3, max 5), chunk 1 = rows 2-3 (min -7, max 9)
    x = np.array([[1, 5], [-3, 2], [0, 9], [-7, 4]], np.float32)
    assert O.range_chunked(x, 2) == (-5.0, 7.0)
    assert O.range_chunked(x, 4) == ((1 - 3 + 0 - 7) / 4, (5 + 2 + 9 + 4) / 4)
    # one chunk: the tensor's own minimum and maximum
    r = np.random.Generator(np.random.PCG64(7)).standard_normal((96, 40)).astype(np.float32)
    assert O.range_chunked(r, 1) == (float(r.min()), float(r.max()))
    # averages of chunk extremes lie inside the global range, shrink (weakly) as the chunks get finer when the chunks
    # nest, and do not depend on the order of the elements inside a chunk
    lo1, hi1 = O.range_chunked(r, 1)
    prev = (lo1, hi1)
    for k in (2, 4, 8, 16, 32, 96):
        lo, hi = O.range_chunked(r, k)
        assert lo1 <= prev[0] <= lo <= hi <= prev[1] <= hi1
        prev = (lo, hi)
    shuffled = r.reshape(4, -1).copy()
    for row in shuffled:
        np.random.Generator(np.random.PCG64(1)).shuffle(row)
    assert O.range_chunked(shuffled.reshape(r.shape), 4) == O.range_chunked(r, 4)
    # values beyond the clamp saturate at the end codes; inside it the error bound of the quantiser holds
    lo, hi = O.range_chunked(r, 8)
    qt = O.quantize(r, 8, range_in=(lo, hi))
    assert np.all(qt.q[r >= hi] == 127) and np.all(qt.q[r <= lo] == -128)
    inside = (r > lo) & (r < hi)
    assert np.max(np.abs(O.dequantize(qt)[inside] - r[inside])) <= float(qt.scale[0]) * (0.5 + 1e-4)
    with pytest.raises(ValueError):
        O.range_chunked(r, 7)


@pytest.mark.parametrize("bits", [8, 16])
def test_stochastic_rounding_brackets_and_is_unbiased(bits):
    # many copies of a few values inside a fixed range: the mean code tends to t
    n = 1 << 17
    vals = np.array([0.3137, -0.7771, 0.05, 0.9], np.float32)
    rng = (np.float32(-1.0), np.float32(1.0))
    L = 2**bits - 1; half = 2**(bits - 1)
    for k, v in enumerate(vals):
        x = np.full((n // 64, 64), v, np.float32)
        qt = O.quantize(x, bits, rounding=1, seed=7, tensor_id=k, range_in=rng)
        s = np.float64(qt.scale[0]); zp_u = int(qt.zero_point[0]) + half
        t = np.float64(v) / s + zp_u
        codes = qt.q.astype(np.float64).ravel() + half
        assert set(np.unique(codes)) <= {math.floor(t), math.floor(t) + 1}
        frac = t - math.floor(t)
        sigma = math.sqrt(max(frac * (1 - frac), 1e-12) / n)
        assert abs(codes.mean() - t) <= 4.5 * sigma + 2e-3   # 2e-3: fp32 rounding of t at 16 bits
    # values exactly on the grid (scale 1, integer inputs) never move
    g = O.quantize(np.array([[-half, half - 1, 0.0, 5.0, -17.0]], np.float32), bits, rounding=1, seed=3, tensor_id=1)
    assert g.scale[0] == 1.0 and list(g.q.ravel().astype(int)) == [-half, half - 1, 0, 5, -17]


def test_stochastic_codes_depend_only_on_position_seed_and_id():
    x = synth.normal((40, 50), 108, std=0.1)
    rng = O.tensor_range(x)
    full = O.quantize(x, 8, rounding=1, seed=11, tensor_id=5, range_in=rng)
    again = O.quantize(x, 8, rounding=1, seed=11, tensor_id=5, range_in=rng)
    other = O.quantize(x, 8, rounding=1, seed=11, tensor_id=6, range_in=rng)
    assert np.array_equal(full.q, again.q) and not np.array_equal(full.q, other.q)
    # the first 12 rows quantised alone (same flat positions) give the same codes
    head = O.quantize(x[:12], 8, rounding=1, seed=11, tensor_id=5, range_in=rng)
    assert np.array_equal(head.q, full.q[:12])
    # ... and so do the last 28 when told where they start in the whole tensor
    tail = O.quantize(x[12:], 8, rounding=1, seed=11, tensor_id=5, range_in=rng, index_base=12 * 50)
    assert np.array_equal(tail.q, full.q[12:])
    # rebuild every code from the published random word: floor(t) + [u < frac]
    s = full.scale[0]; zp_u = np.float32(int(full.zero_point[0]) + 128)
    inv = np.float32(1.0) / s
    t = (x.astype(np.float64) * np.float64(inv) + np.float64(zp_u)).astype(np.float32)  # fma: one rounding
    f = np.floor(t); frac = t - f
    # (8-bit codes draw from the word's high half, 16-bit codes from its low half)
    words = np.array([O.random_word(11, 5, i) for i in range(x.size)], np.uint64)
    u = (words >> 16).astype(np.float64) / 2.0**16
    want = np.clip(f.ravel() + (u < frac.ravel()), 0, 255) - 128
    assert np.array_equal(full.q.ravel().astype(np.int64), want.astype(np.int64))
    full16 = O.quantize(x, 16, rounding=1, seed=11, tensor_id=5, range_in=rng)
    s16 = full16.scale[0]; zp16 = np.float32(int(full16.zero_point[0]) + 32768)
    t16 = (x.astype(np.float64) * np.float64(np.float32(1.0) / s16) + np.float64(zp16)).astype(np.float32)
    f16 = np.floor(t16); frac16 = t16 - f16
    u16 = (words & 0xFFFF).astype(np.float64) / 2.0**16
    want16 = np.clip(f16.ravel() + (u16 < frac16.ravel()), 0, 65535) - 32768
    assert np.array_equal(full16.q.ravel().astype(np.int64), want16.astype(np.int64))


def test_the_two_copies_of_a_gradient_round_independently():
    """Gradients Bifurcation quantises one tensor twice (8 and 16 bits) under one (seed, tensor id): the two
    round-up decisions of an element come from disjoint halves of its word, so over many elements they are
    uncorrelated, and each is unbiased on its own."""
    n = 1 << 18
    x = np.full((n // 64, 64), 0.3137, np.float32)
    rng = (np.float32(-1.0), np.float32(1.0))
    q8 = O.quantize(x, 8, rounding=1, seed=21, tensor_id=4, range_in=rng)
    q16 = O.quantize(x, 16, rounding=1, seed=21, tensor_id=4, range_in=rng)
    up8 = (q8.q.ravel() - q8.q.min()).astype(np.float64); up16 = (q16.q.ravel() - q16.q.min()).astype(np.float64)
    assert set(np.unique(up8)) == {0.0, 1.0} and set(np.unique(up16)) == {0.0, 1.0}
    corr = np.corrcoef(up8, up16)[0, 1]
    assert abs(corr) < 5.0 / math.sqrt(n)


def test_limb_split_exhaustive():
    q = np.arange(-32768, 32768, dtype=np.int16)
    hi, lo = O.limb_split(q)
    assert hi.dtype == np.int8 and lo.dtype == np.uint8
    assert np.array_equal(256 * hi.astype(np.int32) + lo.astype(np.int32), q.astype(np.int32))


def test_cosine_similarity_of_gaussian_weights_meets_the_bound():
    # Section 5, last bound: cos >= 2^M / (2^M + sqrt(ln N)/sqrt 6); the min/max grid spans
    # about twice max|W|, hence M - 1 effective bits on each side.
    N = 1 << 16
    w = synth.normal((256, 256), 109)
    for bits in (8, 16):
        d = O.dequantize(O.quantize(w, bits)).astype(np.float64).ravel()
        wv = w.astype(np.float64).ravel()
        cos = d @ wv / np.linalg.norm(d) / np.linalg.norm(wv)
        m = bits - 1
        assert cos >= 2**m / (2**m + math.sqrt(math.log(N)) / math.sqrt(6))


# -------------------------------------------------------- integer products
def _codes(shape, seed, lo=-128, hi=127, dtype=np.int8):
    g = np.random.Generator(np.random.PCG64(seed))
    return g.integers(lo, hi + 1, size=shape).astype(dtype)


def test_gemm_s8_brute_force_tiny():
    A = _codes((3, 5), 1); B = _codes((5, 4), 2); za, zb = -7, 19
    acc, out, bad = O.gemm_s8(A, za, B, zb, 0.5, 0.25)
    for m, n in itertools.product(range(3), range(4)):
        ref = sum((int(A[m, k]) - za) * (int(B[k, n]) - zb) for k in range(5))
        assert acc[m, n] == ref and out[m, n] == np.float32(ref) * np.float32(0.125)
    assert bad == 0


@pytest.mark.parametrize("tA,tB", [(False, False), (True, False), (False, True), (True, True)])
def test_gemm_s8_matches_fp64_matmul_with_transposes(tA, tB):
    M, N, K = 37, 29, 211
    A = _codes((K, M) if tA else (M, K), 3); B = _codes((N, K) if tB else (K, N), 4)
    za, zb = 5, -128
    acc, _, bad = O.gemm_s8(A, za, B, zb, transA=tA, transB=tB)
    a = (A.T if tA else A).astype(np.float64) - za; b = (B.T if tB else B).astype(np.float64) - zb
    assert bad == 0 and np.array_equal(acc.astype(np.float64), a @ b)


def test_gemm_s8_special_case_plain_integer_matmul_and_overflow_flag():
    A = _codes((8, 16), 5); B = _codes((16, 8), 6)
    acc, out, _ = O.gemm_s8(A, 0, B, 0)
    assert np.array_equal(acc, A.astype(np.int32) @ B.astype(np.int32))
    assert np.array_equal(out, acc.astype(np.float32))
    K = 33100                                    # 255*255*K > 2^31 - 1: flagged, not silently wrapped
    _, _, bad = O.gemm_s8(np.full((1, K), 127, np.int8), -128, np.full((K, 1), 127, np.int8), -128)
    assert bad == 1


def test_weight_gradient_product_and_limb_form():
    M, N, K = 301, 9, 13
    X = _codes((M, K), 7); G = _codes((M, N), 8, -32768, 32767, np.int16); zx, zg = -128, 1234
    acc, out = O.gemm_s16s8(X, zx, G, zg, 0.5, 2.0)
    ref = (X.astype(np.int64) - zx).T @ (G.astype(np.int64) - zg)
    assert np.array_equal(acc, ref) and np.array_equal(out, ref.astype(np.float32))
    for k, n in ((0, 0), (12, 8)):
        assert acc[k, n] == sum((int(X[m, k]) - zx) * (int(G[m, n]) - zg) for m in range(M))
    hi, lo = O.limb_split(G)
    assert np.array_equal(O.gemm_limbs(X, zx, hi, lo, zg), ref)


def _im2col(xc, d):
    """Centred integer input [N,H,W,C] -> [N*P*Q, R*S*C] with real-zero padding (written out here
    independently of the oracle's loops)."""
    xp = np.pad(xc, ((0, 0), (d.pad, d.pad), (d.pad, d.pad), (0, 0)))
    cols = np.zeros((d.N, d.P, d.Q, d.R, d.S, d.C), np.int64)
    for r in range(d.R):
        for s in range(d.S):
            cols[:, :, :, r, s, :] = xp[:, r:r + d.stride * d.P:d.stride, s:s + d.stride * d.Q:d.stride, :]
    return cols.reshape(d.N * d.P * d.Q, d.R * d.S * d.C)


CONVS = [dict(N=2, H=7, W=6, Cin=5, K=4, R=3, S=3, stride=1, pad=1),
         dict(N=1, H=9, W=8, Cin=3, K=6, R=3, S=3, stride=2, pad=1),
         dict(N=2, H=5, W=5, Cin=7, K=3, R=1, S=1, stride=1, pad=0),
         dict(N=1, H=6, W=7, Cin=2, K=2, R=3, S=3, stride=1, pad=0)]


@pytest.mark.parametrize("cfg", CONVS)
def test_conv_products_against_im2col_and_adjoints(cfg):
    d = O.conv_desc(**cfg)
    x = _codes((d.N, d.H, d.W, d.C), 9); w = _codes((d.K, d.R, d.S, d.C), 10)
    g8 = _codes((d.N, d.P, d.Q, d.K), 11); g16 = _codes((d.N, d.P, d.Q, d.K), 12, -32768, 32767, np.int16)
    zx, zw, zg8, zg16 = -100, 3, 17, -2000
    xc = x.astype(np.int64) - zx; wc = w.astype(np.int64) - zw
    cols = _im2col(xc, d); wm = wc.reshape(d.K, -1)
    # forward == im2col x filter matrix
    acc, out, bad = O.conv_s8(0, d, x, zx, w, zw, 0.5, 0.5)
    assert bad == 0 and np.array_equal(acc.reshape(-1, d.K), cols @ wm.T)
    assert np.array_equal(out, acc.astype(np.float32) * np.float32(0.25))
    # sampled evaluation agrees with the full one
    idx = np.array([0, acc.size - 1, acc.size // 2, 5], np.int64)
    assert np.array_equal(O.conv_s8(0, d, x, zx, w, zw, idx=idx)[0], acc.ravel()[idx])
    # weight gradient == cols^T g
    gc16 = g16.astype(np.int64) - zg16
    aw, _ = O.conv_wgrad_s16(d, x, zx, g16, zg16)
    assert np.array_equal(aw.reshape(d.K, -1), gc16.reshape(-1, d.K).T @ cols)
    # layer gradient: adjoint of the forward map, <fprop(x,W), g> == <x, dgrad(g,W)> exactly
    gc8 = g8.astype(np.int64) - zg8
    ad, _, bad = O.conv_s8(1, d, g8, zg8, w, zw)
    assert bad == 0
    fwd = (cols @ wm.T).reshape(d.N, d.P, d.Q, d.K)
    assert int((fwd * gc8).sum()) == int((xc * ad.astype(np.int64)).sum())
    assert int((fwd * gc16).sum()) == int((wc * aw).sum())
    # and dgrad is that adjoint for every basis input, not just in the sum: check a few coordinates
    for o in (0, x.size - 1, x.size // 3):
        e = np.zeros(x.size, np.int64); e[o] = 1
        col_e = _im2col(e.reshape(xc.shape), d)
        assert int(((col_e @ wm.T).reshape(fwd.shape) * gc8).sum()) == int(ad.ravel()[o])


def test_conv_1x1_is_a_gemm():
    d = O.conv_desc(N=2, H=4, W=4, Cin=8, K=5, R=1, S=1)
    x = _codes((2, 4, 4, 8), 13); w = _codes((5, 1, 1, 8), 14)
    a, _, _ = O.conv_s8(0, d, x, 4, w, -9)
    b, _, _ = O.gemm_s8(x.reshape(32, 8), 4, w.reshape(5, 8), -9, transB=True)
    assert np.array_equal(a.reshape(32, 5), b)


# ---------------------------------------------------------------- Range BN
def test_C_of_n_closed_form_and_paper_number():
    assert math.isclose(O.rangebn_C(64), 1 / math.sqrt(2 * math.log(64)), rel_tol=1e-15)
    assert abs(O.rangebn_C(64) - 0.346734) < 1e-6 and abs(O.rangebn_C(802816) - 0.191770) < 1e-6
    val, tol = _paper_constants()["sqrt_2ln_last_resnet50_layer_batch1024"]
    assert abs(1.0 / O.rangebn_C(3 * 3 * 2048 * 1024) - val) <= tol


@pytest.mark.parametrize("n", [2, 64, 1000])
def test_rangebn_output_range_is_exactly_one_over_C(n):
    x = synth.channel_gaussian((n, 1, 1, 6), 30, 31)
    y, mean, lo, hi = O.rangebn_fwd(x)
    y = y.reshape(n, 6)
    assert np.allclose(y.max(0) - y.min(0), math.sqrt(2 * math.log(n)), rtol=1e-12)
    assert np.allclose(y.mean(0), 0, atol=1e-12)
    assert np.array_equal(lo, x.reshape(n, 6).min(0)) and np.array_equal(hi, x.reshape(n, 6).max(0))
    assert np.allclose(mean, x.reshape(n, 6).astype(np.float64).mean(0), rtol=1e-13, atol=1e-15)


def test_rangebn_affine_invariance_gamma_beta_relu_and_zero_range():
    x = synth.normal((128, 5), 32)
    y0, *_ = O.rangebn_fwd(x)
    y1, *_ = O.rangebn_fwd(x * np.float32(4.0) + np.float32(0.5))     # exact in fp32: power-of-two scale
    assert np.allclose(y0, y1, rtol=0, atol=1e-6)
    g = np.array([2, -1, 0.5, 1, 3], np.float32); b = np.array([0, 1, -1, 0.25, -3], np.float32)
    y2, *_ = O.rangebn_fwd(x, g, b)
    assert np.allclose(y2, y0 * g + b, rtol=1e-14, atol=1e-14)
    y3, *_ = O.rangebn_fwd(x, g, b, relu=True)
    assert np.array_equal(y3, np.maximum(y2, 0))
    xc = x.copy(); xc[:, 2] = 7.0
    y4, *_ = O.rangebn_fwd(xc, g, b)
    assert np.all(y4[:, 2] == b[2])


def test_rangebn_scale_tracks_sigma_within_the_papers_bounds():
    consts = _paper_constants()
    lo_b = consts["rangebn_lower_bound_in_sigma"][0]; hi_b = consts["rangebn_upper_bound_in_sigma"][0]
    ratios = []
    for n in (64, 1024, 16384):
        x = synth.normal((n, 64), 33 + n)
        _, _, lo, hi = O.rangebn_fwd(x)
        ratio = float(np.mean(O.rangebn_C(n) * (hi - lo)))          # sigma = 1
        assert lo_b <= ratio <= hi_b
        ratios.append(ratio)
        _, _, lo3, hi3 = O.rangebn_fwd(x * np.float32(3.0))
        assert np.allclose(hi3 - lo3, 3.0 * (hi - lo), rtol=1e-6)   # proportional to sigma
    assert ratios[0] < ratios[1] < ratios[2]                        # creeps up with n, stays below 2


def _bn_loss(x, wgt, gamma, beta, relu):
    y, *_ = O.rangebn_fwd(x, gamma, beta, relu)
    return float((y * wgt).sum())


@pytest.mark.parametrize("relu", [False, True])
def test_rangebn_backward_against_central_differences(relu):
    n, Cc = 16, 3
    g = np.random.Generator(np.random.PCG64(40))
    # inputs on a 2^-10 grid so that x +- h is exact in fp32; distinct values, no ties
    x = (g.permutation(4096)[: n * Cc].reshape(n, Cc).astype(np.float32) - 2048) / 1024
    gamma = np.array([1.5, -0.75, 1.0], np.float32); beta = np.array([0.25, 0.5, -0.125], np.float32)
    wgt = g.standard_normal((n, Cc)).astype(np.float32)
    _, mean, lo, hi = O.rangebn_fwd(x, gamma, beta, relu)
    dx, dg, db = O.rangebn_bwd(wgt, x, mean, lo, hi, gamma, beta, relu)
    h = np.float32(2.0**-13)
    for i in range(n):
        for c in range(Cc):
            xp = x.copy(); xm = x.copy(); xp[i, c] += h; xm[i, c] -= h
            num = (_bn_loss(xp, wgt, gamma, beta, relu) - _bn_loss(xm, wgt, gamma, beta, relu)) / (2 * float(h))
            assert abs(num - dx[i, c]) <= 2e-6 * max(1.0, abs(num)), (i, c, num, dx[i, c])
    y, *_ = O.rangebn_fwd(x, gamma, beta, relu)
    mask = (y > 0) if relu else np.ones_like(y, bool)
    xhat, *_ = O.rangebn_fwd(x)
    assert np.allclose(db, (wgt.astype(np.float64) * mask).sum(0), rtol=1e-12)
    assert np.allclose(dg, (wgt.astype(np.float64) * mask * xhat).sum(0), rtol=1e-6, atol=1e-9)


def test_rangebn_backward_sum_identities_and_ties():
    n, Cc = 200, 4
    x = synth.channel_gaussian((n, 1, 1, Cc), 41, 42).reshape(n, Cc)
    dy = synth.normal((n, Cc), 43)
    gamma = np.array([1, 2, -1, 0.5], np.float32)
    _, mean, lo, hi = O.rangebn_fwd(x, gamma)
    dx, _, _ = O.rangebn_bwd(dy, x, mean, lo, hi, gamma)
    scale = np.abs(dx).sum(0)
    # invariance of the output to x -> x + b and x -> a x  ==>  sum dx = 0 and sum x dx = 0
    assert np.all(np.abs(dx.sum(0)) <= 1e-9 * scale)
    assert np.all(np.abs((dx * (x.astype(np.float64) - mean)).sum(0)) <= 1e-6 * scale)
    # ties: every coordinate attaining the maximum carries the same extra term
    xt = x.copy(); j1, j2 = 3, 77; xt[j1, 0] = xt[j2, 0] = x[:, 0].max() + np.float32(1.0)
    _, mt, lt, ht = O.rangebn_fwd(xt, gamma)
    dxt, _, _ = O.rangebn_bwd(dy, xt, mt, lt, ht, gamma)
    s = 1.0 / (O.rangebn_C(n) * (float(ht[0]) - float(lt[0])))
    extra = lambda j: dxt[j, 0] - s * float(gamma[0]) * float(dy[j, 0])
    plain = extra(10)                                               # neither max nor min
    assert abs((extra(j1) - plain) - (extra(j2) - plain)) < 1e-12 and abs(extra(j1) - plain) > 1e-6


# ------------------------------------------------------------------- layer
def test_layer_composition_on_the_linear_config():
    cfg = synth.linear_layer()
    y, saved, acc = O.layer_fwd(cfg["x"], cfg["w"])
    # a quantised product stays close to the fp32 one (8 bits on each operand)
    ref = cfg["x"].astype(np.float64) @ cfg["w"].astype(np.float64)
    assert np.abs(saved.z - ref).max() <= 0.02 * np.abs(ref).max()
    assert np.allclose(y.max(0) - y.min(0), math.sqrt(2 * math.log(64)), rtol=1e-12)
    dz, _, _ = O.rangebn_bwd(cfg["dy"], saved.z, saved.mean, saved.vmin, saved.vmax)
    dx, dw, acc_dx, acc_dw, g8, g16 = O.layer_bwd_products(dz.astype(np.float32), saved, 0, 1, 2)
    refdx = dz @ cfg["w"].astype(np.float64).T; refdw = cfg["x"].astype(np.float64).T @ dz
    assert np.abs(dx - refdx).max() <= 0.05 * np.abs(refdx).max()
    assert np.abs(dw - refdw).max() <= 0.02 * np.abs(refdw).max()
    # the 16-bit copy is the finer one
    e8 = np.abs(O.dequantize(g8) - dz).max(); e16 = np.abs(O.dequantize(g16) - dz).max()
    assert e16 < e8 / 100


# ------------------------------------------------------------------ fp32 weight update
def test_sgd_update_closed_forms():
    """Values chosen dyadic so that every fp32 operation is exact and the closed forms hold to the bit."""
    w0 = np.array([1.0, -2.0, 0.5, 8.0], np.float32); g = np.array([0.25, -0.5, 1.0, 0.0], np.float32)
    # plain SGD, constant gradient: w_k = w_0 - k lr g
    w = w0
    for k in range(1, 6):
        w, _ = O.sgd_update(w, g, lr=0.5)
        assert np.array_equal(w, w0 - k * 0.5 * g)
    # momentum 1/2, constant gradient: v_k = g (2 - 2^(1-k)), w_k = w_0 - lr sum_j v_j
    w, v = w0, np.zeros(4, np.float32)
    total = np.zeros(4, np.float64)
    for k in range(1, 8):
        w, v = O.sgd_update(w, g, v, lr=0.25, momentum=0.5)
        assert np.array_equal(v, (g * (2.0 - 2.0 ** (1 - k))).astype(np.float32))
        total += v
        assert np.array_equal(w, (w0 - 0.25 * total).astype(np.float32))
    # weight decay alone: w_k = w_0 (1 - lr wd)^k
    w = w0
    for k in range(1, 6):
        w, _ = O.sgd_update(w, np.zeros(4, np.float32), lr=0.5, weight_decay=0.25)
        assert np.array_equal(w, (w0 * 0.875 ** k).astype(np.float32))
    # a dropped or mis-signed term shows: decay and gradient together, one step, by hand
    w, v = O.sgd_update(np.array([2.0], np.float32), np.array([1.0], np.float32), np.array([4.0], np.float32), lr=0.5, momentum=0.5,
                        weight_decay=0.25)
    assert v[0] == 0.5 * 4.0 + (1.0 + 0.25 * 2.0) and w[0] == 2.0 - 0.5 * v[0]
