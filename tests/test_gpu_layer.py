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
    assert np.array_equal(to_host(L.g8), g8.q) and np.array_equal(to_host(L.ghi), ohi_) and np.array_equal(to_host(L.glo), olo_)
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
