"""GPU Range BN forward / backward vs the CPU oracle (fp64): max|a - b| / max|b| <= 1e-5 per channel."""
import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth
from tests.util import FP32_TOL, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


CANCEL = 1.0 / 32.0


def _per_channel_rel(got, want, terms=None):
    """Worst channel of max|got - want| / max|want| (the tolerance definition used for every fp32 output).

    `terms` (per channel) is the magnitude of the terms the output is a sum of.  A fp32 sum carries an absolute
    error of a few 2^-24 of its largest term, so a channel whose whole reference lies below 1/32 of that magnitude
    (a ReLU that cut everything but values next to zero; n = 2, where dx cancels to zero identically) cannot
    meet a bound relative to the result in any fp32 evaluation: such a channel, and only such a channel, is measured
    against terms / 32 instead.  A channel whose reference is identically zero must agree to within 1e-5 of terms."""
    C = want.shape[-1]
    g = np.asarray(got, np.float64).reshape(-1, C); w = np.asarray(want, np.float64).reshape(-1, C)
    den = np.abs(w).max(0)
    if terms is not None:
        den = np.maximum(den, CANCEL * np.asarray(terms, np.float64))
    den[den == 0] = 1.0
    return float((np.abs(g - w).max(0) / den).max())


def _scales(x, dy, vmin, vmax, gamma, beta):
    """Magnitude of the terms per channel: |gamma| * max|xhat| + |beta| for y, s * |gamma| * max|dy| for dx."""
    C = x.shape[-1]; n = x.size // C
    g = np.ones(C) if gamma is None else np.abs(gamma.astype(np.float64))
    b = np.zeros(C) if beta is None else np.abs(beta.astype(np.float64))
    r = vmax.astype(np.float64) - vmin
    s = np.where(r > 0, 1.0 / (O.rangebn_C(n) * np.where(r > 0, r, 1.0)), 0.0)
    return g / O.rangebn_C(n) + b, s * g * np.abs(dy.reshape(-1, C)).max(0)


def _run(B, x, dy, gamma, beta, relu):
    gd = None if gamma is None else to_dev(gamma); bd = None if beta is None else to_dev(beta)
    xd = to_dev(x)
    y, mean, vmin, vmax, rng = B.qbp_rangebn_fwd(xd, gd, bd, relu, want_range=True)
    oy, om, olo, ohi = O.rangebn_fwd(x, gamma, beta, relu)
    assert np.array_equal(to_host(vmin), olo) and np.array_equal(to_host(vmax), ohi)
    assert np.abs(to_host(mean) - om).max() <= 1e-6 * max(1.0, np.abs(om).max())
    y_scale, dx_scale = _scales(x, dy, olo, ohi, gamma, beta)
    assert _per_channel_rel(to_host(y), oy, y_scale) <= FP32_TOL
    # the advertised output range is the exact range of the output just written
    _, _, lo, hi = B.read_qparams(rng)
    yh = to_host(y)
    assert lo[0] == yh.min() and hi[0] == yh.max()
    # backward, fed with the forward's own saved statistics
    dx, dg, db = B.qbp_rangebn_bwd(to_dev(dy), xd, mean, vmin, vmax, gd, bd, relu)
    odx, odg, odb = O.rangebn_bwd(dy, x, to_host(mean), to_host(vmin), to_host(vmax), gamma, beta, relu)
    assert _per_channel_rel(to_host(dx), odx, dx_scale) <= FP32_TOL
    # the two channel-sum vectors: per tensor, max|a - b| / max|b|
    assert np.abs(to_host(dg) - odg).max() <= FP32_TOL * np.abs(odg).max()
    assert np.abs(to_host(db) - odb).max() <= FP32_TOL * np.abs(odb).max()


CASES = [(2, 1, 1, 4), (64, 1, 1, 128), (4, 7, 7, 64), (3, 5, 5, 6), (2, 3, 3, 2048), (5, 4, 4, 96), (1001, 1, 1, 1)]


@pytest.mark.parametrize("shape", CASES)
@pytest.mark.parametrize("relu", [False, True])
def test_forward_backward(B, shape, relu):
    case_x = synth.channel_gaussian(shape, 20, 21); dy = synth.normal(shape, 22)
    C = shape[-1]
    gamma = synth.uniform((C,), 23, 1.0) + np.float32(1.5); beta = synth.uniform((C,), 24, 0.5)
    gamma[::3] *= -1                                       # negative gains flip the extremes
    _run(B, case_x, dy, gamma, beta, relu)
    _run(B, case_x, dy, None, None, relu)


def test_ties_and_constant_channel(B):
    x = synth.normal((256, 8), 25)
    x = np.round(x * 4) / 4                                # coarse grid: many ties at the extremes
    x[:, 3] = 2.0                                          # zero range
    dy = synth.normal((256, 8), 26)
    _run(B, x.astype(np.float32), dy, None, None, False)
    _run(B, x.astype(np.float32), dy, None, None, True)


@pytest.mark.parametrize("hw,C", synth.RANGEBN_SWEEP)
def test_sweep_shapes_full_size(B, hw, C):
    """Batch 256 at every shape of the sweep; compared on sampled channels plus the statistics of all."""
    case = synth.rangebn_case(256, hw, C)
    x, dy = case["x"], case["dy"]
    xd = to_dev(x)
    y, mean, vmin, vmax, _ = B.qbp_rangebn_fwd(xd, relu=True)
    dx, dg, db = B.qbp_rangebn_bwd(to_dev(dy), xd, mean, vmin, vmax, relu=True)
    n = x.size // C
    x2 = x.reshape(n, C); dy2 = dy.reshape(n, C)
    assert np.array_equal(to_host(vmin), x2.min(0)) and np.array_equal(to_host(vmax), x2.max(0))
    chans = sorted({0, C // 2, C - 1, 17 % C})
    xs = np.ascontiguousarray(x2[:, chans]); dys = np.ascontiguousarray(dy2[:, chans])
    # the oracle's C(n) depends on n only, so a channel subset is a valid instance
    oy, om, _, _ = O.rangebn_fwd(xs, relu=True)
    assert _per_channel_rel(to_host(y).reshape(n, C)[:, chans], oy) <= FP32_TOL
    mh, lo, hi = to_host(mean)[chans], to_host(vmin)[chans], to_host(vmax)[chans]
    odx, odg, odb = O.rangebn_bwd(dys, xs, mh, lo, hi, relu=True)
    assert _per_channel_rel(to_host(dx).reshape(n, C)[:, chans], odx) <= FP32_TOL
    assert np.abs(to_host(dg)[chans] - odg).max() <= FP32_TOL * np.abs(odg).max()
    assert np.abs(to_host(db)[chans] - odb).max() <= FP32_TOL * np.abs(odb).max()
    # properties that hold at any size: output range per channel is 1/C(n) (before the ReLU cut: check max side)
    yh = to_host(y).reshape(n, C)
    s = 1.0 / (O.rangebn_C(n) * (to_host(vmax).astype(np.float64) - to_host(vmin)))
    want_max = (to_host(vmax).astype(np.float64) - to_host(mean)) * s
    assert np.allclose(yh.max(0), np.maximum(want_max, 0), rtol=1e-5)
