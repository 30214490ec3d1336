"""Appendix C on the GPU against the CPU oracle: binarisation, stochastic ternarisation (one sample and the sum of
several), the XNOR-popcount forward product and the gated-XNOR backward product as int8 tensor-core products on +-1
and ternary bytes, and Algorithm 1.  Codes and integer accumulators bit for bit."""
import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth
from tests.util import set_qparams, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


def _tern_sum(g, samples, seed, tid):
    tot = np.zeros(g.shape, dtype=np.int32)
    s = np.float32(0)
    for k in range(samples):
        t, s = O.stc_tern(g, seed, tid, k)
        tot += t
    return tot, s


@pytest.mark.parametrize("n", [1, 3, 4, 1027, 64 * 256, 1 << 20])
def test_binarize(B, n):
    x = synth.normal((n,), 31)
    x[:: 7] = 0.0
    if n > 2: x[2] = -0.0
    q, qp = B.qbp_binarize_s8(to_dev(x))
    assert np.array_equal(to_host(q), O.binarize(x))
    s, z, lo, hi = B.read_qparams(qp)
    assert s[0] == 1.0 and z[0] == 0 and lo[0] == -1.0 and hi[0] == 1.0
    # a tensor that starts 4 bytes into a 16-byte line takes the element-wise path
    if n > 8:
        import torch
        buf = to_dev(np.concatenate([[np.float32(0)], x]))
        q2, _ = B.qbp_binarize_s8(buf[1:], q=torch.empty(n, dtype=torch.int8, device="cuda"))
        assert np.array_equal(to_host(q2), O.binarize(x))


@pytest.mark.parametrize("n,samples", [(1, 1), (5, 3), (1027, 1), (4096, 6), (64 * 300 + 2, 2), (1 << 18, 20)])
def test_stochastic_ternarisation_codes(B, n, samples):
    g = synth.normal((n,), 32, std=0.3)
    g[:: 5] = 0.0
    q, qp = B.qbp_stc_ternarize_s8(to_dev(g), samples=samples, seed=77, tensor_id=9)
    want, s = _tern_sum(g, samples, 77, 9)
    assert np.array_equal(to_host(q).astype(np.int32), want)
    sc, z, lo, hi = B.read_qparams(qp)
    assert z[0] == 0 and hi[0] == s and lo[0] == -s
    assert sc[0] == (np.float32(s) / np.float32(samples) if s > 0 else np.float32(1))
    if n > 8:
        import torch
        buf = to_dev(np.concatenate([[np.float32(0)], g]))
        q2, _ = B.qbp_stc_ternarize_s8(buf[1:], samples=samples, seed=77, tensor_id=9)
        assert np.array_equal(to_host(q2).astype(np.int32), want)


def test_ternarisation_of_zeros_and_of_the_full_size_gradient(B):
    q, qp = B.qbp_stc_ternarize_s8(to_dev(np.zeros(100, dtype=np.float32)), samples=4)
    assert not to_host(q).any() and B.read_qparams(qp)[0][0] == 1.0
    g = synth.normal((256 * 56 * 56 * 64,), 33, std=0.05)           # the benchmark layer's gradient tensor
    q, qp = B.qbp_stc_ternarize_s8(to_dev(g), samples=1, seed=5, tensor_id=6)
    want, s = O.stc_tern(g, 5, 6, 0)
    assert np.array_equal(to_host(q), want) and B.read_qparams(qp)[3][0] == s


@pytest.mark.parametrize("M,N,K", [(64, 48, 128), (256, 128, 1024), (16, 16, 16), (512, 272, 2064)])
def test_forward_product_equals_xnor_popcount(B, M, N, K):
    """Appendix C: the forward MACs of a binarised layer as XNOR + popcount; here the int8 tensor-core product on the
    +-1 bytes, whose accumulators must be the popcount results."""
    a = synth.normal((M, K), 34); w = synth.normal((N, K), 35)
    qa, pa = B.qbp_binarize_s8(to_dev(a)); qw, pw = B.qbp_binarize_s8(to_dev(w))
    acc, out, ws = B.qbp_gemm_s8(qa, pa, qw, pw, transB=True, want_acc=True)
    want = O.xnor_gemm(O.pack_bits(O.binarize(a)), O.pack_bits(O.binarize(w)), K)
    assert B.status_word(ws) == 0
    assert np.array_equal(to_host(acc), want) and np.array_equal(to_host(out), want.astype(np.float32))


@pytest.mark.parametrize("M,N,K", [(64, 128, 48), (256, 512, 128), (16, 32, 16)])
def test_backward_product_equals_gated_xnor(B, M, N, K):
    """The layer gradient of a binarised layer from a ternary gradient: dx [M x K] = t [M x N] . W [N x K]."""
    g = synth.normal((M, N), 36, std=0.2); w = synth.normal((N, K), 37)
    t, pt = B.qbp_stc_ternarize_s8(to_dev(g), samples=1, seed=3, tensor_id=4)
    qw, pw = B.qbp_binarize_s8(to_dev(w))
    acc, out, ws = B.qbp_gemm_s8(t, pt, qw, pw, want_acc=True)
    ot, s = O.stc_tern(g, 3, 4, 0)
    wb = O.binarize(w)
    want = O.gated_xnor_gemm(O.pack_bits(ot, mask=True), O.pack_bits(ot), O.pack_bits(np.ascontiguousarray(wb.T)), N)
    assert B.status_word(ws) == 0 and np.array_equal(to_host(acc), want)
    assert np.array_equal(to_host(out), (want.astype(np.float32) * np.float32(s)))      # in units of g: s * t


@pytest.mark.parametrize("rows,K,N,samples", [(256, 64, 48, 1), (256, 64, 48, 6), (1024, 128, 256, 12), (70000, 32, 32, 3)])
def test_algorithm_1_linear(B, rows, K, N, samples):
    g = synth.normal((rows, N), 38, std=0.1); a = synth.normal((rows, K), 39)
    qa, pa = B.qbp_binarize_s8(to_dev(a))
    acc, gW, t_hi, t_lo, pt = B.qbp_tbp_weight_gradient(qa, pa, to_dev(g), samples, seed=11, tensor_id=12, want_acc=True)
    tsum, s = _tern_sum(g, samples, 11, 12)
    ab = O.binarize(a).astype(np.int64)
    want = ab.T @ tsum.astype(np.int64)                                  # the sum of the samples' products (exact integers)
    assert np.array_equal(to_host(acc), want)
    # the limbs hold the summed samples as a 16-bit code
    assert np.array_equal(to_host(t_hi).astype(np.int32) * 256 + to_host(t_lo).astype(np.int32), tsum)
    scale = np.float32(s) / np.float32(samples)
    assert np.array_equal(to_host(gW), want.astype(np.float32) * scale)
    if rows <= 1024:
        ref = O.tbp_update(g, O.binarize(a), samples, seed=11, tensor_id=12)
        assert np.max(np.abs(to_host(gW) - ref)) <= 1e-6 * max(1.0, np.max(np.abs(ref)))


@pytest.mark.parametrize("N,H,W,C,K,R,samples", [(2, 8, 8, 32, 32, 3, 3), (4, 14, 14, 64, 64, 3, 2), (2, 7, 7, 64, 128, 1, 4)])
def test_algorithm_1_convolution(B, N, H, W, C, K, R, samples):
    """Algorithm 1 for a convolution layer, in the algorithm's order on the oracle's side: one weight-gradient product
    per sample, added up."""
    pad = (R - 1) // 2
    d = B.conv_desc(N, H, W, C, K, R, R, 1, pad); od = O.conv_desc(N, H, W, C, K, R, R, 1, pad)
    a = synth.normal((N, H, W, C), 40); g = synth.normal((N, H, W, K), 41, std=0.1)
    qa, pa = B.qbp_binarize_s8(to_dev(a))
    acc, gW, _, _, pt = B.qbp_tbp_weight_gradient(qa, pa, to_dev(g), samples, seed=21, tensor_id=22, d=d, want_acc=True)
    ab = O.binarize(a)
    want = np.zeros((K, R, R, C), dtype=np.int64)
    s = np.float32(0)
    for k in range(samples):
        t, s = O.stc_tern(g, 21, 22, k)
        oacc, _ = O.conv_wgrad_s16(od, ab, 0, t.astype(np.int16), 0, 1.0, 1.0)
        want += oacc.reshape(want.shape)
    assert np.array_equal(to_host(acc), want)
    assert np.array_equal(to_host(gW), want.astype(np.float32) * (np.float32(s) / np.float32(samples)))


@pytest.mark.parametrize("rows,cols", [(1, 1), (3, 35), (64, 64), (130, 257), (7, 4096)])
def test_bit_rows(B, rows, cols):
    t = np.random.Generator(np.random.PCG64(50 + cols)).integers(-1, 2, (rows, cols)).astype(np.int8)
    assert np.array_equal(to_host(B.qbp_pack_bits(to_dev(t))).view(np.uint32), O.pack_bits(t))
    assert np.array_equal(to_host(B.qbp_pack_bits(to_dev(t), mask=True)).view(np.uint32), O.pack_bits(t, mask=True))


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (5, 7, 70), (64, 64, 1024), (130, 67, 1057), (256, 300, 4096)])
def test_popcount_products_on_bit_rows(B, M, N, K):
    """The literal XNOR + popcount and gated-XNOR products on bit rows (ragged sizes) against the oracle's, and against
    the tensor-core route on the byte codes where its shape rules allow."""
    rng = np.random.Generator(np.random.PCG64(60 + K))
    a = (rng.integers(0, 2, (M, K)) * 2 - 1).astype(np.int8); b = (rng.integers(0, 2, (N, K)) * 2 - 1).astype(np.int8)
    t = rng.integers(-1, 2, (M, K)).astype(np.int8)
    ab, bb = B.qbp_pack_bits(to_dev(a)), B.qbp_pack_bits(to_dev(b))
    got = to_host(B.qbp_xnor_gemm_bits(ab, bb, K))
    assert np.array_equal(got, O.xnor_gemm(O.pack_bits(a), O.pack_bits(b), K))
    nz, sg = B.qbp_pack_bits(to_dev(t), mask=True), B.qbp_pack_bits(to_dev(t))
    gated = to_host(B.qbp_gated_xnor_gemm_bits(nz, sg, bb, K))
    assert np.array_equal(gated, O.gated_xnor_gemm(O.pack_bits(t, mask=True), O.pack_bits(t), O.pack_bits(b), K))
    if M % 16 == 0 and N % 16 == 0 and K % 16 == 0:
        one = set_qparams(B.new_qparams(1), 1.0, 0)
        acc, _, _ = B.qbp_gemm_s8(to_dev(a), one, to_dev(b), one, transB=True, want_acc=True)
        assert np.array_equal(to_host(acc), got)


@pytest.mark.parametrize("kind,samples", [("conv", 1), ("conv", 4), ("linear", 3)])
def test_ternarized_layer_stagewise(B, kind, samples):
    """The low-bit layer (1-bit x and w, Range BN, ternary gradient, Algorithm 1) stage by stage against the oracle."""
    from paper_1805_11046_b200 import layer
    from tests.util import FP32_TOL, rel_err
    relu = True
    if kind == "conv":
        N, H, W, C, K, R = 2, 8, 8, 32, 64, 3
        d = B.conv_desc(N, H, W, C, K, R, R, 1, 1); od = O.conv_desc(N, H, W, C, K, R, R, 1, 1)
        x = synth.normal((N, H, W, C), 80); w = synth.normal((K, R, R, C), 81); dy = synth.normal((N, H, W, K), 82, std=0.1)
    else:
        d = od = None
        x = synth.normal((64, 128), 80); w = synth.normal((128, 64), 81); dy = synth.normal((64, 64), 82, std=0.1)
        K = 64
    gamma = synth.normal((K,), 83) * np.float32(0.5) + np.float32(1); beta = synth.normal((K,), 84) * np.float32(0.1)
    L = layer.TernarizedLayer(conv=d, relu=relu, seed=9, tensor_id=5, samples=samples)
    y = L.forward(to_dev(x), to_dev(w), to_dev(gamma), to_dev(beta))
    dx, dw, dgamma, dbeta = L.backward(to_dev(dy))
    ab, wb = O.binarize(x), O.binarize(w)
    assert np.array_equal(to_host(L.saved["a"]), ab) and np.array_equal(to_host(L.saved["wb"]), wb)
    if od is not None:
        _, oz, bad = O.conv_s8(0, od, ab, 0, wb, 0, 1.0, 1.0)
    else:
        _, oz, bad = O.gemm_s8(ab, 0, wb, 0, 1.0, 1.0)
    z = to_host(L.saved["z"])
    assert bad == 0 and np.array_equal(z.ravel(), np.asarray(oz).ravel())
    z2 = z.reshape(-1, K); dy2 = dy.reshape(-1, K)
    oy, om, olo, ohi = O.rangebn_fwd(z2, gamma, beta, relu=relu)
    assert rel_err(to_host(y).reshape(-1, K), oy)[0] <= FP32_TOL
    mean, vmin, vmax = (to_host(L.saved[k]) for k in ("mean", "vmin", "vmax"))
    og, odg, odb = O.rangebn_bwd(dy2, z2, mean, vmin, vmax, gamma, beta, relu=relu)
    g = to_host(L.g)
    assert rel_err(g.reshape(-1, K), og)[0] <= FP32_TOL
    assert rel_err(to_host(dgamma), odg)[0] <= FP32_TOL and rel_err(to_host(dbeta), odb)[0] <= FP32_TOL
    ot, s = O.stc_tern(g, 9, 5, 0)
    assert np.array_equal(to_host(L.t), ot)
    if od is not None:
        _, odx, bad = O.conv_s8(1, od, ot, 0, wb, 0, float(s), 1.0)
        assert bad == 0 and np.array_equal(to_host(dx).ravel(), np.asarray(odx).ravel())
        want = np.zeros(w.shape, dtype=np.int64)
        for k in range(samples):
            tk, s2 = O.stc_tern(g, 9, 6, k)
            oacc, _ = O.conv_wgrad_s16(od, ab, 0, tk.astype(np.int16), 0, 1.0, 1.0)
            want += np.asarray(oacc).reshape(want.shape)
    else:
        _, odx, bad = O.gemm_s8(ot, 0, wb, 0, float(s), 1.0, transB=True)
        assert bad == 0 and np.array_equal(to_host(dx), odx)
        tot = np.zeros(g.shape, dtype=np.int64)
        for k in range(samples):
            tk, s2 = O.stc_tern(g, 9, 6, k)
            tot += tk
        want = ab.astype(np.int64).T @ tot
    assert np.array_equal(to_host(dw), want.astype(np.float32) * (np.float32(s2) / np.float32(samples)))
