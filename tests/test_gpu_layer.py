"""Whole-layer parity, stage by stage: each stage of the oracle is fed the fp32 tensor the GPU actually
produced for that stage, so that codes and integer accumulators must agree bit for bit even where an
upstream fp32 sum differs in its last bit."""
import ctypes as C

import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth
from tests.util import FP32_TOL, rel_err, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


def _run_layer(B, cfg, relu, conv=None):
    import torch
    from paper_1805_11046_b200 import layer
    x, w, dy = cfg["x"], cfg["w"], cfg["dy"]
    L = layer.QuantizedLayer(conv=conv, batch=x.shape[0], in_features=x.shape[-1], out_features=w.shape[-1] if conv is None else None,
                             relu=relu, seed=cfg["seed"], tensor_id8=cfg["id8"], tensor_id16=cfg["id16"])
    y = L.forward(to_dev(x), to_dev(w))
    dx, dw, dgamma, dbeta = L.backward(to_dev(dy))
    torch.cuda.synchronize()
    return L, y, dx, dw, dgamma, dbeta


def _check_layer(B, cfg, relu, conv_kw=None, sample=None, want_y=False):
    conv = None if conv_kw is None else B.conv_desc(conv_kw["N"], conv_kw["H"], conv_kw["W"], conv_kw["C"], conv_kw["K"],
                                                    conv_kw["R"], conv_kw["S"], conv_kw["stride"], conv_kw["pad"])
    oconv = None if conv_kw is None else O.conv_desc(conv_kw["N"], conv_kw["H"], conv_kw["W"], conv_kw["C"], conv_kw["K"],
                                                     conv_kw["R"], conv_kw["S"], conv_kw["stride"], conv_kw["pad"])
    L, y, dx, dw, dgamma, dbeta = _run_layer(B, cfg, relu, conv)
    x, w, dy = cfg["x"], cfg["w"], cfg["dy"]
    # stage 1: quantisers (inputs are the shared synthetic tensors)
    ox = O.quantize(x, 8); ow = O.quantize(w, 8)
    assert np.array_equal(to_host(L.x_codes), ox.q) and np.array_equal(to_host(L.w_codes), ow.q)
    sx, zx, _, _ = B.read_qparams(L.qx); sw, zw, _, _ = B.read_qparams(L.qw)
    assert sx[0] == ox.scale[0] and zx[0] == ox.zero_point[0] and sw[0] == ow.scale[0] and zw[0] == ow.zero_point[0]
    # stage 2: the forward product (bit-exact fp32: integer accumulator times one fp32 scale)
    z = to_host(L.z)
    if oconv is None:
        _, oz, bad = O.gemm_s8(ox.q, ox.zero_point[0], ow.q, ow.zero_point[0], ox.scale[0], ow.scale[0])
        assert bad == 0 and np.array_equal(z, oz)
    else:
        idx = sample(z.size)
        _, oz, bad = O.conv_s8(0, oconv, ox.q, ox.zero_point[0], ow.q, ow.zero_point[0], ox.scale[0], ow.scale[0], idx=idx)
        assert bad == 0 and np.array_equal(z.ravel()[idx], oz)
    # stage 3: Range BN forward on the GPU's z
    Cc = z.shape[-1]
    chans = list(range(Cc)) if z.size < 1 << 22 else sorted({0, Cc // 2, Cc - 1})
    z2 = z.reshape(-1, Cc)
    oy, om, olo, ohi = O.rangebn_fwd(np.ascontiguousarray(z2[:, chans]), relu=relu)
    assert rel_err(to_host(y).reshape(-1, Cc)[:, chans], oy)[0] <= FP32_TOL
    # stage 4: Range BN backward from the GPU's saved statistics
    mean, vmin, vmax = to_host(L.save_mean), to_host(L.save_min), to_host(L.save_max)
    dy2 = dy.reshape(-1, Cc)
    og, odg, odb = O.rangebn_bwd(np.ascontiguousarray(dy2[:, chans]), np.ascontiguousarray(z2[:, chans]), mean[chans], vmin[chans],
                                 vmax[chans], relu=relu)
    g = to_host(L.g)
    assert rel_err(g.reshape(-1, Cc)[:, chans], og)[0] <= FP32_TOL
    assert rel_err(to_host(dgamma)[chans], odg)[0] <= FP32_TOL and rel_err(to_host(dbeta)[chans], odb)[0] <= FP32_TOL
    # stage 5: bifurcation of the GPU's fp32 gradient
    g8, g16 = O.bifurcate(g, cfg["seed"], cfg["id8"], cfg["id16"])
    ohi_, olo_ = O.limb_split(g16.q)
    assert np.array_equal(to_host(L.g8), g8.q) and np.array_equal(to_host(L.ghi), ohi_) and np.array_equal(to_host(L.glo) ^ np.uint8(0x80), olo_)     # (the layer stores lo - 128)
    # stage 6: the two backward products from those codes
    if oconv is None:
        _, odx, bad = O.gemm_s8(g8.q, g8.zero_point[0], ow.q, ow.zero_point[0], g8.scale[0], ow.scale[0], transB=True)
        _, odw = O.gemm_s16s8(ox.q, ox.zero_point[0], g16.q, g16.zero_point[0], ox.scale[0], g16.scale[0])
        assert bad == 0 and np.array_equal(to_host(dx), odx) and np.array_equal(to_host(dw), odw)
    else:
        idx = sample(x.size)
        _, odx, bad = O.conv_s8(1, oconv, g8.q, g8.zero_point[0], ow.q, ow.zero_point[0], g8.scale[0], ow.scale[0], idx=idx)
        assert bad == 0 and np.array_equal(to_host(dx).ravel()[idx], odx)
        widx = sample(w.size, 96)
        _, odw = O.conv_wgrad_s16(oconv, ox.q, ox.zero_point[0], g16.q, g16.zero_point[0], ox.scale[0], g16.scale[0], idx=widx)
        assert np.array_equal(to_host(dw).ravel()[widx], odw)
    if want_y:
        return to_host(y)


def _sampler(seed):
    rng = np.random.Generator(np.random.PCG64(seed))

    def sample(size, count=4096):
        if size <= count:
            return np.arange(size, dtype=np.int64)
        return np.unique(np.concatenate([[0, size - 1], rng.integers(0, size, count)])).astype(np.int64)
    return sample


@pytest.mark.parametrize("relu", [False, True])
def test_linear_layer_config(B, relu):
    _check_layer(B, synth.linear_layer(), relu)


@pytest.mark.parametrize("relu", [False, True])
def test_small_conv_layer(B, relu):
    cfg = synth.conv3x3_layer(batch=4, hw=14)
    _check_layer(B, cfg, relu, cfg["conv"], _sampler(1))


def test_conv2_x_layer_full_size(B):
    """ResNet-18 conv2_x 3x3 at batch 256 in the benchmark's launch configuration; products on sampled outputs."""
    cfg = synth.conv3x3_layer()
    _check_layer(B, cfg, True, cfg["conv"], _sampler(2))


@pytest.mark.parametrize("kind", ["linear", "conv_small", "conv_wide", "conv2_x"])
def test_backward_without_the_fp32_gradient_buffer(B, kind):
    """keep_g=False: the gradient arriving at the product is quantised as the Range BN backward computes it and never
    written as fp32.  Everything the backward leaves must equal, bit for bit, what the layer that keeps the buffer
    leaves (that layer is the one the stage-wise tests check against the oracle)."""
    import torch
    from paper_1805_11046_b200 import layer
    if kind == "linear":
        cfg, conv = synth.linear_layer(), None
    else:
        cfg = {"conv_small": lambda: synth.conv3x3_layer(batch=4, hw=14), "conv_wide": lambda: synth.conv3x3_layer(batch=2, hw=9, c_in=32, k_out=160),
               "conv2_x": lambda: synth.conv3x3_layer()}[kind]()
        c = cfg["conv"]
        conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    x, w, dy = to_dev(cfg["x"]), to_dev(cfg["w"]), to_dev(cfg["dy"])
    outs = []
    for keep_g in (True, False):
        L = layer.QuantizedLayer(conv=conv, batch=cfg["x"].shape[0], in_features=cfg["x"].shape[-1],
                                 out_features=cfg["w"].shape[-1] if conv is None else None, relu=True, seed=cfg["seed"],
                                 tensor_id8=cfg["id8"], tensor_id16=cfg["id16"], keep_g=keep_g)
        L.forward(x, w)
        dx, dw, dgamma, dbeta = L.backward(dy)
        torch.cuda.synchronize()
        assert L.status() == 0 and (L.g is None) == (not keep_g)
        outs.append([to_host(t) for t in (L.g8, L.ghi, L.glo, dx, dw, dgamma, dbeta)] + [B.read_qparams(L.qg8), B.read_qparams(L.qg16)])
    for a_, b_ in zip(outs[0][:7], outs[1][:7]):
        assert np.array_equal(a_, b_)
    for qa, qb in zip(outs[0][7:], outs[1][7:]):
        assert all(np.array_equal(u, v) for u, v in zip(qa, qb))


def test_layer_step_at_full_size_is_reproducible(B):
    """Eight forward + backward steps of the benchmark's layer on the same tensors: every output and every kept
    intermediate must come out with the same bits each time (integers, fixed summation orders, counter-based random
    numbers: nothing in the path depends on timing)."""
    import torch
    from paper_1805_11046_b200 import layer
    cfg = synth.conv3x3_layer()
    c = cfg["conv"]
    conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    x, w, dy = to_dev(cfg["x"]), to_dev(cfg["w"]), to_dev(cfg["dy"])
    L = layer.QuantizedLayer(conv=conv, relu=True, seed=cfg["seed"], tensor_id8=cfg["id8"], tensor_id16=cfg["id16"], keep_g=False)
    ref = None
    for rep in range(8):
        L.forward(x, w)
        dx, dw, dgamma, dbeta = L.backward(dy)
        torch.cuda.synchronize()
        outs = [t.contiguous().view(torch.uint8).clone() for t in (L.x_codes, L.z, L.y, L.g8, L.ghi, L.glo, dx, dw, dgamma, dbeta, L.save_mean)]
        if ref is None:
            ref = outs
        else:
            assert all(int((a_ != b_).sum()) == 0 for a_, b_ in zip(outs, ref)), f"step {rep} differs from step 0"
    assert L.status() == 0


def test_bottleneck_stack_stagewise(B):
    """conv3_x bottleneck (1x1, 3x3, 1x1, each + Range BN + ReLU) at a reduced batch; every layer checked
    stage-wise on the activations the GPU handed to it."""
    import torch
    from paper_1805_11046_b200 import layer
    st = synth.bottleneck_stack(batch=8, hw=28)
    a = st["x"]
    layers = []
    for i, (w, c) in enumerate(zip(st["w"], st["convs"])):
        cfg = dict(x=a, w=w, dy=synth.normal((c["N"], c["H"], c["W"], c["K"]), 50 + i, std=0.1), seed=0, id8=2 * i + 1, id16=2 * i + 2)
        _check_layer(B, cfg, True, c, _sampler(3 + i))
        conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
        L = layer.QuantizedLayer(conv=conv, relu=True, seed=0, tensor_id8=2 * i + 1, tensor_id16=2 * i + 2)
        a = to_host(L.forward(to_dev(a), to_dev(w)))
        layers.append(L)
    torch.cuda.synchronize()
    assert a.shape == (8, 28, 28, 512) and a.min() == 0.0


def test_bottleneck_stack_full_batch_stagewise(B):
    """conv3_x bottleneck at the full batch of 256 (input [256,28,28,256]), every layer in the launch configuration
    a benchmark of it would use; products checked on sampled outputs, Range BN on three channels."""
    st = synth.bottleneck_stack(batch=256, hw=28)
    a = st["x"]
    for i, (w, c) in enumerate(zip(st["w"], st["convs"])):
        cfg = dict(x=a, w=w, dy=synth.normal((c["N"], c["H"], c["W"], c["K"]), 60 + i, std=0.1), seed=0, id8=2 * i + 1, id16=2 * i + 2)
        a = _check_layer(B, cfg, True, c, _sampler(13 + i), want_y=True)
    assert a.shape == (256, 28, 28, 512) and a.min() == 0.0


# ------------------------------------------------ chained layers: the quantiser's range from the Range BN before it
def test_rangebn_fused_requantisation_equals_quantising_the_output(B):
    """Section 4: the range of a Range BN output is known from the statistics, so its 8-bit codes are written by the
    apply pass itself.  They must be, bit for bit, what the quantiser makes of the materialised fp32 output (range
    scan included), the row sums must be the sums of those codes, and leaving y unwritten must not change them."""
    for shape, relu in (((4, 14, 14, 64), True), ((3, 5, 7, 48), False), ((64, 128), True), ((2, 9, 9, 256), True),
                        ((5, 3, 3, 6), False), ((1000, 512), True)):
        x = synth.channel_gaussian(shape, 20, 21)
        C_ = shape[-1]
        gamma = synth.uniform((C_,), 23, 1.0) + np.float32(1.5); beta = synth.uniform((C_,), 24, 0.5)
        gamma[::3] *= -1
        import torch
        cs = torch.empty(C_, dtype=torch.int64, device="cuda")
        y, mean, vmin, vmax, q, qp, rs = B.qbp_rangebn_fwd_q8(to_dev(x), to_dev(gamma), to_dev(beta), relu, want_row_sums=True,
                                                              chan_sums=cs)
        yh = to_host(y)
        o = O.quantize(yh, 8)                        # scans yh for its range
        s_, z_, lo_, hi_ = B.read_qparams(qp)
        assert s_[0] == o.scale[0] and z_[0] == o.zero_point[0] and lo_[0] == o.vmin[0] and hi_[0] == o.vmax[0]
        assert np.array_equal(to_host(q), o.q)
        assert np.array_equal(to_host(rs), o.q.reshape(-1, C_).astype(np.int32).sum(1))
        assert np.array_equal(to_host(cs), o.q.reshape(-1, C_).astype(np.int64).sum(0))
        _, _, _, _, q2, qp2, _ = B.qbp_rangebn_fwd_q8(to_dev(x), to_dev(gamma), to_dev(beta), relu, want_y=False)
        assert np.array_equal(to_host(q2), o.q) and np.array_equal(to_host(qp2), to_host(qp))


def _chained_stack(B, batch, keep_y):
    import torch
    from paper_1805_11046_b200 import layer
    st = synth.bottleneck_stack(batch=batch, hw=28)
    layers = []
    for i, c in enumerate(st["convs"]):
        conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
        last = i == len(st["convs"]) - 1
        layers.append(layer.QuantizedLayer(conv=conv, relu=True, seed=0, tensor_id8=2 * i + 1, tensor_id16=2 * i + 2,
                                           input_from=layers[-1] if layers else None, emit_codes=not last,
                                           keep_y=keep_y or last))
    ws = [to_dev(w) for w in st["w"]]
    layers[0].forward(to_dev(st["x"]), ws[0])
    for L, w in zip(layers[1:], ws[1:]):
        L.forward(None, w)
    torch.cuda.synchronize()
    return st, layers


@pytest.mark.parametrize("batch", [8, 256])
def test_chained_bottleneck_stack_needs_no_scan_between_layers(B, batch):
    """The conv3_x bottleneck with every inner activation handed on as 8-bit codes written by the Range BN that made
    it: stage-wise parity (each stage of the oracle is fed what the GPU produced for it), no range scan and no
    quantisation pass between the layers, and the same results whether or not the fp32 activations are kept."""
    st, layers = _chained_stack(B, batch, keep_y=True)
    rng = np.random.Generator(np.random.PCG64(40 + batch))
    codes_in = None
    for i, (L, c) in enumerate(zip(layers, st["convs"])):
        od = O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
        ow = O.quantize(st["w"][i], 8)
        if i == 0:
            ox = O.quantize(st["x"], 8)
            assert np.array_equal(to_host(L.x_codes), ox.q)
            xq, xz, xs = ox.q, ox.zero_point[0], ox.scale[0]
        else:
            xq, xz, xs = codes_in
            assert np.array_equal(to_host(L.x_codes), xq)        # the very buffer the previous layer wrote
        z = to_host(L.z)
        idx = np.unique(np.concatenate([[0, z.size - 1], rng.integers(0, z.size, 4096)])).astype(np.int64)
        _, oz, bad = O.conv_s8(0, od, xq, xz, ow.q, ow.zero_point[0], xs, ow.scale[0], idx=idx)
        assert bad == 0 and np.array_equal(z.ravel()[idx], oz)
        Cc = z.shape[-1]
        chans = sorted({0, Cc // 2, Cc - 1})
        oy, _, _, _ = O.rangebn_fwd(np.ascontiguousarray(z.reshape(-1, Cc)[:, chans]), relu=True)
        yh = to_host(L.y)
        assert rel_err(yh.reshape(-1, Cc)[:, chans], oy)[0] <= FP32_TOL
        if L.rq_out is not None:
            o = O.quantize(yh, 8)
            s_, z_, lo_, hi_ = B.read_qparams(L.q_out)
            assert s_[0] == o.scale[0] and z_[0] == o.zero_point[0] and lo_[0] == o.vmin[0] and hi_[0] == o.vmax[0]
            assert np.array_equal(to_host(L.out_codes), o.q)
            assert np.array_equal(to_host(L.out_row_sums), o.q.reshape(-1, Cc).astype(np.int32).sum(1))
            codes_in = (o.q, o.zero_point[0], o.scale[0])
        assert L.status() == 0
    # the same stack without the inner fp32 activations
    _, lean = _chained_stack(B, batch, keep_y=False)
    for L, M in zip(layers, lean):
        assert np.array_equal(to_host(L.z), to_host(M.z))
        if L.rq_out is not None:
            assert np.array_equal(to_host(L.out_codes), to_host(M.out_codes))
    assert np.array_equal(to_host(layers[-1].y), to_host(lean[-1].y))
    # and the launch list of a chained inner layer holds no scan and no stand-alone quantiser for its input
    import torch
    B.trace_enable(True)
    lean[1].forward(None, to_dev(st["w"][1]))
    names = [n for n, _ in B.trace_records()]
    B.trace_enable(False)
    # (one scan and one quantisation: the filter's -- in one launch of its own when it is small; none for the activation)
    assert names.count("range_partial_kernel") + names.count("filter_prep_kernel") == 1
    assert names.count("quantize_kernel") + names.count("filter_prep_kernel") == 1


def test_chained_stack_backward_runs_on_the_handed_on_codes(B):
    """Backward through a chained pair: the weight gradient of the second layer uses the codes the first layer's
    Range BN wrote; stage-wise parity of its products."""
    import torch
    st, layers = _chained_stack(B, 8, keep_y=True)
    L = layers[1]; c = st["convs"][1]
    dy = synth.normal(L.z_shape, 70, std=0.1)
    dx, dw, _, _ = L.backward(to_dev(dy))
    torch.cuda.synchronize()
    assert L.status() == 0
    od = O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    g = to_host(L.g)
    g8, g16 = O.bifurcate(g, 0, 3, 4)
    assert np.array_equal(to_host(L.g8), g8.q)
    ow = O.quantize(st["w"][1], 8)
    xq = to_host(L.x_codes); s_, z_, _, _ = B.read_qparams(L.qx)
    _, odx, bad = O.conv_s8(1, od, g8.q, g8.zero_point[0], ow.q, ow.zero_point[0], g8.scale[0], ow.scale[0])
    _, odw = O.conv_wgrad_s16(od, xq, z_[0], g16.q, g16.zero_point[0], np.float32(s_[0]), g16.scale[0])
    assert bad == 0 and np.array_equal(to_host(dx), odx) and np.array_equal(to_host(dw), odw)


# ------------------------------------------------ fp32 master-weight update and a whole training step of a stack
@pytest.mark.parametrize("momentum,wd", [(0.0, 0.0), (0.9, 1e-4)])
def test_sgd_update_matches_the_fp32_statement_bit_for_bit(B, momentum, wd):
    w = synth.normal((4099,), 81); dw = synth.normal((4099,), 82, std=0.01); v = synth.normal((4099,), 83, std=0.01)
    wd_ = to_dev(w); vd = to_dev(v) if momentum else None
    ow, ov = w, (v if momentum else None)
    for _ in range(3):
        B.qbp_sgd_update(wd_, to_dev(dw), vd, lr=0.05, momentum=momentum, weight_decay=wd)
        ow, ov = O.sgd_update(ow, dw, ov, lr=0.05, momentum=momentum, weight_decay=wd)
    assert np.array_equal(to_host(wd_), ow)
    if momentum:
        assert np.array_equal(to_host(vd), ov)


def test_training_steps_of_the_chained_bottleneck_stack(B):
    """Two whole training steps (forward chain on handed-on codes, backward chain, fp32 updates of w, gamma, beta) of
    the conv3_x bottleneck at a reduced batch.  After each step the updated tensors equal the fp32 statement of the
    update applied to the gradients the GPU produced, and the next forward quantises exactly those weights."""
    import torch
    from paper_1805_11046_b200 import layer
    st = synth.bottleneck_stack(batch=8, hw=28)
    convs = [B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"]) for c in st["convs"]]
    S = layer.QuantizedStack(convs, [to_dev(w) for w in st["w"]], lr=0.05, momentum=0.9, weight_decay=1e-4)
    x, dy = to_dev(st["x"]), to_dev(st["dy"])
    ow = [w.copy() for w in st["w"]]; ovw = [np.zeros_like(w) for w in ow]
    og = [np.ones(L.cout, np.float32) for L in S.layers]; ovg = [np.zeros_like(g) for g in og]
    ob = [np.zeros(L.cout, np.float32) for L in S.layers]; ovb = [np.zeros_like(b) for b in ob]
    for step in range(2):
        S.train_step(x, dy)
        torch.cuda.synchronize()
        assert S.status() == 0
        for i, L in enumerate(S.layers):
            # the forward of this step quantised the weights as they stood before the update
            assert np.array_equal(to_host(L.w_codes), O.quantize(ow[i], 8).q)
            ow[i], ovw[i] = O.sgd_update(ow[i], to_host(L.dw), ovw[i], 0.05, 0.9, 1e-4)
            og[i], ovg[i] = O.sgd_update(og[i], to_host(L.dgamma), ovg[i], 0.05, 0.9, 0.0)
            ob[i], ovb[i] = O.sgd_update(ob[i], to_host(L.dbeta), ovb[i], 0.05, 0.9, 0.0)
            assert np.array_equal(to_host(S.w[i]), ow[i]) and np.array_equal(to_host(S.gamma[i]), og[i])
            assert np.array_equal(to_host(S.beta[i]), ob[i])
        if step == 0:
            # the gradient chain: a layer's dy is the next layer's dx (straight-through estimator through the
            # quantiser); gamma = 1, beta = 0 in the first step
            for a, b_ in zip(S.layers[:-1], S.layers[1:]):
                og_, _, _ = O.rangebn_bwd(to_host(b_.dx), to_host(a.z), to_host(a.save_mean), to_host(a.save_min),
                                          to_host(a.save_max), relu=True)
                assert rel_err(to_host(a.g), og_)[0] <= FP32_TOL
    assert not np.array_equal(ow[0], st["w"][0])


def test_chained_and_unchained_stacks_agree(B):
    """The chained stack (codes handed on by the Range BN) and the unfused composition (every layer scans and
    quantises the fp32 activation of the one before) compute the same thing: same codes, same outputs, same gradients."""
    import torch
    from paper_1805_11046_b200 import layer
    st = synth.bottleneck_stack(batch=8, hw=28)
    convs = [B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"]) for c in st["convs"]]
    x, dy = to_dev(st["x"]), to_dev(st["dy"])
    A = layer.QuantizedStack(convs, [to_dev(w) for w in st["w"]], chained=True)
    U = layer.QuantizedStack(convs, [to_dev(w) for w in st["w"]], chained=False)
    da = A.train_step(x, dy); du = U.train_step(x, dy)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(da), to_host(du))
    for La, Lu in zip(A.layers, U.layers):
        assert np.array_equal(to_host(La.x_codes), to_host(Lu.x_codes)) and np.array_equal(to_host(La.z), to_host(Lu.z))
        assert np.array_equal(to_host(La.dw), to_host(Lu.dw))
    for wa, wu in zip(A.w, U.w):
        assert np.array_equal(to_host(wa), to_host(wu))


# ------------------------------------------------ recompute instead of store: conv -> Range BN -> ReLU -> 8-bit codes
@pytest.mark.parametrize("batch,hw,cin,cout", [(4, 14, 64, 64), (3, 9, 32, 96), (2, 20, 128, 32), (256, 56, 64, 64)])
def test_recompute_fusion_writes_the_same_codes_without_storing_the_product(B, batch, hw, cin, cout):
    """The convolution run twice (statistics only, then normalise + ReLU + requantise in the epilogue) must leave,
    bit for bit, the codes, parameters, row sums and saved statistics of the path that stores the fp32 product and
    normalises it in a pass of its own -- and those are checked against the oracle (quantising the fp32 output)."""
    import torch
    from paper_1805_11046_b200 import layer
    cfg = synth.conv3x3_layer(batch=batch, hw=hw, c_in=cin, k_out=cout)
    c = cfg["conv"]
    conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    gamma = to_dev(synth.uniform((cout,), 23, 1.0) + np.float32(1.5)); beta = to_dev(synth.uniform((cout,), 24, 0.5))
    x, w = to_dev(cfg["x"]), to_dev(cfg["w"])
    kept = layer.QuantizedLayer(conv=conv, relu=True, emit_codes=True, keep_y=True)
    kept.forward(x, w, gamma, beta)
    lean = layer.QuantizedLayer(conv=conv, relu=True, emit_codes=True, keep_y=False, keep_z=False)
    lean.forward(x, w, gamma, beta)
    torch.cuda.synchronize()
    assert kept.status() == 0 and lean.status() == 0
    assert np.array_equal(to_host(lean.out_codes), to_host(kept.out_codes))
    assert np.array_equal(to_host(lean.q_out), to_host(kept.q_out))
    assert np.array_equal(to_host(lean.out_row_sums), to_host(kept.out_row_sums))
    for a, b_ in ((lean.save_mean, kept.save_mean), (lean.save_min, kept.save_min), (lean.save_max, kept.save_max)):
        assert np.array_equal(to_host(a), to_host(b_))
    # and against the oracle: the codes are those of the fp32 output the storing path wrote
    o = O.quantize(to_host(kept.y), 8)
    s_, z_, lo_, hi_ = B.read_qparams(lean.q_out)
    assert s_[0] == o.scale[0] and z_[0] == o.zero_point[0] and lo_[0] == o.vmin[0] and hi_[0] == o.vmax[0]
    assert np.array_equal(to_host(lean.out_codes), o.q)
    # the backward pass needs the stored product and says so
    with pytest.raises(B.QbpError):
        lean.backward(to_dev(cfg["dy"]))


@pytest.mark.parametrize("batch,hw,cin,cout,R", [(3, 9, 32, 96, 3), (2, 12, 64, 32, 3), (2, 7, 96, 64, 3), (4, 6, 128, 128, 3),
                                                   (3, 10, 64, 128, 1), (2, 5, 32, 32, 3), (2, 6, 32, 320, 1)])
def test_conv_layers_of_other_shapes_stagewise(B, batch, hw, cin, cout, R):
    """Forward and backward of convolution layers whose shapes take the other routes to the weight gradient's
    zero-point sums (with and without a spare chunk for the row of ones, channel counts the epilogue warps do or
    do not take, 1x1 filters, output rows wider than one block of the backward pass with a partly filled last slab),
    each stage against the oracle."""
    pad = (R - 1) // 2
    cfg = dict(x=synth.relu_normal((batch, hw, hw, cin), 90), w=synth.kaiming_normal((cout, R, R, cin), 91),
               dy=synth.normal((batch, hw, hw, cout), 92, std=0.1), seed=5, id8=7, id16=7,
               conv=dict(N=batch, H=hw, W=hw, C=cin, K=cout, R=R, S=R, stride=1, pad=pad))
    _check_layer(B, cfg, True, cfg["conv"], _sampler(50 + cin + cout))


@pytest.mark.parametrize("kind", ["conv", "linear"])
def test_backward_with_mixed_gamma_and_beta(B, kind):
    """The layer's backward with a rectifier and per-channel gamma of both signs, zero and tiny, beta of both signs: the
    second pass takes the rectifier's mask as a per-channel threshold on the product's output, which must agree with
    the forward formula for rising, falling and constant channels.  Gradient against the oracle, codes of the GPU's
    gradient bit for bit."""
    import torch
    from paper_1805_11046_b200 import layer
    if kind == "conv":
        cfg = dict(x=synth.relu_normal((3, 10, 10, 32), 60), w=synth.kaiming_normal((64, 3, 3, 32), 61),
                   dy=synth.normal((3, 10, 10, 64), 62, std=0.1))
        conv = B.conv_desc(3, 10, 10, 32, 64, 3, 3, 1, 1)
        L = layer.QuantizedLayer(conv=conv, relu=True, seed=4, tensor_id8=3, tensor_id16=3)
    else:
        cfg = dict(x=synth.relu_normal((96, 128), 60), w=synth.kaiming_normal((128, 64), 61), dy=synth.normal((96, 64), 62, std=0.1))
        L = layer.QuantizedLayer(batch=96, in_features=128, out_features=64, relu=True, seed=4, tensor_id8=3, tensor_id16=3)
    K = 64
    gamma = synth.normal((K,), 63)
    gamma[0] = 0.0; gamma[1] = -0.0; gamma[2] = 1e-30; gamma[3] = -1e-30; gamma[4] = -2.5; gamma[5] = 3.0
    beta = synth.normal((K,), 64) * np.float32(0.5)
    beta[0] = 0.25; beta[1] = -0.25; beta[6] = 0.0; beta[7] = 100.0; beta[8] = -100.0
    gd, bd = to_dev(gamma), to_dev(beta)
    y = L.forward(to_dev(cfg["x"]), to_dev(cfg["w"]), gd, bd)
    dx, dw, dgamma, dbeta = L.backward(to_dev(cfg["dy"]))
    torch.cuda.synchronize()
    assert L.status() == 0
    z2 = to_host(L.z).reshape(-1, K); dy2 = cfg["dy"].reshape(-1, K)
    oy, _, _, _ = O.rangebn_fwd(z2, gamma, beta, relu=True)
    assert rel_err(to_host(y).reshape(-1, K), oy)[0] <= FP32_TOL
    mean, vmin, vmax = to_host(L.save_mean), to_host(L.save_min), to_host(L.save_max)
    og, odg, odb = O.rangebn_bwd(dy2, z2, mean, vmin, vmax, gamma, beta, relu=True)
    g = to_host(L.g)
    # per channel: a wrong mask in one channel must not hide behind the others
    got = g.reshape(-1, K)
    for c in range(K):
        den = max(float(np.abs(og[:, c]).max()), 1e-30)
        assert float(np.abs(got[:, c] - og[:, c]).max()) / den <= FP32_TOL or float(np.abs(og[:, c]).max()) < 1e-20, c
    assert rel_err(to_host(dgamma), odg)[0] <= FP32_TOL and rel_err(to_host(dbeta), odb)[0] <= FP32_TOL
    g8, g16 = O.bifurcate(g, 4, 3, 3)
    ohi, olo = O.limb_split(g16.q)
    assert np.array_equal(to_host(L.g8), g8.q) and np.array_equal(to_host(L.ghi), ohi)
    assert np.array_equal(to_host(L.glo) ^ np.uint8(0x80), olo)
