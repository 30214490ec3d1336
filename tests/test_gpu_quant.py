"""GPU quantiser vs the CPU oracle: codes, scale, zero-point and limbs bit for bit."""
import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth
from tests.util import to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


def _same_params(B, qp, o):
    s, z, lo, hi = B.read_qparams(qp)
    assert np.array_equal(s, o.scale) and np.array_equal(z, o.zero_point)
    assert np.array_equal(lo, o.vmin) and np.array_equal(hi, o.vmax)


SHAPES = [(64, 256), (256, 128), (1, 1), (3, 5), (1, 4099), (257, 33), (1000, 64), (4, 7, 7, 96)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("kind", ["gauss", "relu", "positive"])
def test_nearest_s8_and_s16(B, shape, kind):
    x = {"gauss": synth.normal, "relu": synth.relu_normal}.get(kind, lambda s, seed: synth.uniform(s, seed, 1.0) + np.float32(3))(shape, 7)
    q, qp = B.qbp_quantize_s8(to_dev(x))
    o = O.quantize(x, 8)
    _same_params(B, qp, o)
    assert np.array_equal(to_host(q), o.q)
    q16, hi, lo, qp16 = B.qbp_quantize_s16(to_dev(x))
    o16 = O.quantize(x, 16)
    _same_params(B, qp16, o16)
    assert np.array_equal(to_host(q16), o16.q)
    ohi, olo = O.limb_split(o16.q)
    assert np.array_equal(to_host(hi), ohi) and np.array_equal(to_host(lo), olo)


@pytest.mark.parametrize("shape", [(64, 128), (3, 5), (1, 4099), (513, 96)])
def test_stochastic_rounding_is_bit_exact(B, shape):
    g = synth.normal(shape, 3, std=0.1)
    for seed, tid in ((0, 1), (0x1234_5678_9ABC_DEF0, 77)):
        q, qp = B.qbp_quantize_s8(to_dev(g), rounding=B.QBP_ROUND_STOCHASTIC, seed=seed, tensor_id=tid)
        o = O.quantize(g, 8, rounding=1, seed=seed, tensor_id=tid)
        _same_params(B, qp, o)
        assert np.array_equal(to_host(q), o.q)
        q16, _, _, qp16 = B.qbp_quantize_s16(to_dev(g), rounding=B.QBP_ROUND_STOCHASTIC, seed=seed, tensor_id=tid)
        o16 = O.quantize(g, 16, rounding=1, seed=seed, tensor_id=tid)
        assert np.array_equal(to_host(q16), o16.q)


def test_unaligned_input_takes_the_scalar_path(B):
    import torch
    g = synth.normal((1, 1001), 5)
    buf = torch.empty(1002, dtype=torch.float32, device="cuda")
    view = buf[1:]                                   # 4-byte aligned only
    view.copy_(to_dev(g).ravel())
    q, qp = B.qbp_quantize_s8(view.reshape(1, 1001), rounding=B.QBP_ROUND_STOCHASTIC, seed=9, tensor_id=2)
    o = O.quantize(g, 8, rounding=1, seed=9, tensor_id=2)
    assert np.array_equal(to_host(q), o.q)


@pytest.mark.parametrize("shape", [(4, 7, 7, 64), (100, 5), (33, 2048), (64, 96)])
def test_per_channel(B, shape):
    x = synth.channel_gaussian(shape if len(shape) == 4 else (shape[0], 1, 1, shape[1]), 20, 21).reshape(shape)
    for rounding in (0, 1):
        q, qp = B.qbp_quantize_s8(to_dev(x), granularity=B.QBP_PER_CHANNEL, rounding=rounding, seed=4, tensor_id=3)
        o = O.quantize(x, 8, per_channel=True, rounding=rounding, seed=4, tensor_id=3)
        _same_params(B, qp, o)
        assert np.array_equal(to_host(q), o.q)


def test_supplied_range_and_empty_tensor(B):
    x = synth.normal((17, 40), 8)
    rng = B.range_qparams(-5.0, 6.0)
    q, qp = B.qbp_quantize_s8(to_dev(x), range_in=rng)
    o = O.quantize(x, 8, range_in=(np.float32(-5), np.float32(6)))
    _same_params(B, qp, o)
    assert np.array_equal(to_host(q), o.q)
    import torch
    e = torch.empty((0, 8), dtype=torch.float32, device="cuda")
    q, qp = B.qbp_quantize_s8(e)
    s, z, lo, hi = B.read_qparams(qp)
    assert q.numel() == 0 and s[0] == 1.0 and z[0] == -128 and lo[0] == 0 and hi[0] == 0


@pytest.mark.parametrize("shape,chunks", [((64, 256), 1), ((64, 256), 8), ((96, 40), 96), ((256, 33), 16), ((12, 5, 7, 24), 4),
                                          ((4096, 3), 4096), ((1000, 64), 125)])
def test_chunk_averaged_clamp(B, shape, chunks):
    """Appendix B's clamping values for activations (averages over K chunks of the chunks' extremes): the two values
    bit for bit, then the codes of the quantiser that clamps to them."""
    x = synth.channel_gaussian(shape, 31, 32) if len(shape) == 4 else synth.normal(shape, 33)
    rng = B.qbp_range_chunked(to_dev(x), chunks)
    lo, hi = O.range_chunked(x, chunks)
    _, _, glo, ghi = B.read_qparams(rng)
    assert glo[0] == np.float32(lo) and ghi[0] == np.float32(hi)
    q, qp = B.qbp_quantize_s8(to_dev(x), range_in=rng)
    o = O.quantize(x, 8, range_in=(np.float32(lo), np.float32(hi)))
    _same_params(B, qp, o)
    assert np.array_equal(to_host(q), o.q)


def test_chunk_averaged_clamp_refuses_rows_that_do_not_divide(B):
    with pytest.raises(B.QbpError):
        B.qbp_range_chunked(to_dev(synth.normal((10, 8), 1)), 3)


def test_bifurcate_and_code_sums(B):
    import torch
    g = synth.normal((130, 64), 12, std=0.1)
    rows = torch.empty(130, dtype=torch.int32, device="cuda")
    q8, qp8, hi, lo, qp16 = B.qbp_bifurcate(to_dev(g), 0, 1, 2, row_sums8=rows)
    o8 = O.quantize(g, 8, rounding=1, seed=0, tensor_id=1); o16 = O.quantize(g, 16, rounding=1, seed=0, tensor_id=2)
    _same_params(B, qp8, o8); _same_params(B, qp16, o16)
    ohi, olo = O.limb_split(o16.q)
    assert np.array_equal(to_host(q8), o8.q) and np.array_equal(to_host(hi), ohi) and np.array_equal(to_host(lo), olo)
    assert np.array_equal(to_host(rows), o8.q.astype(np.int32).sum(1))
    cols = torch.empty(64, dtype=torch.int64, device="cuda")
    q, _ = B.qbp_quantize_s8(to_dev(g), row_sums=rows, col_sums=cols)
    on = O.quantize(g, 8)
    assert np.array_equal(to_host(rows), on.q.astype(np.int32).sum(1))
    assert np.array_equal(to_host(cols), on.q.astype(np.int64).sum(0))


@pytest.mark.parametrize("rows,cols", [(130, 128), (77, 256), (300, 512), (33, 2048), (9, 96), (5, 4096)])
def test_row_sums_of_rows_of_any_width(B, rows, cols):
    """Row sums taken inside the quantising kernel (power-of-two rows up to 128 elements) or by the pass over the codes
    (other widths): the same sums, nearest and stochastic."""
    import torch
    g = synth.normal((rows, cols), 14, std=0.5)
    rs = torch.full((rows,), 12345, dtype=torch.int32, device="cuda")
    q, _ = B.qbp_quantize_s8(to_dev(g), row_sums=rs)
    on = O.quantize(g, 8)
    assert np.array_equal(to_host(q), on.q) and np.array_equal(to_host(rs), on.q.astype(np.int32).sum(1))
    rs.fill_(-7)
    q8, qp8, hi, lo, qp16 = B.qbp_bifurcate(to_dev(g), 3, 1, 2, row_sums8=rs)
    o8 = O.quantize(g, 8, rounding=1, seed=3, tensor_id=1)
    assert np.array_equal(to_host(q8), o8.q) and np.array_equal(to_host(rs), o8.q.astype(np.int32).sum(1))


def test_full_size_activation_tensor(B):
    """The 51.4M-element conv2_x activation, nearest and stochastic, every code."""
    x = synth.relu_normal((256, 56, 56, 64), 10)
    xd = to_dev(x)
    q, qp = B.qbp_quantize_s8(xd)
    o = O.quantize(x, 8)
    _same_params(B, qp, o)
    assert np.array_equal(to_host(q), o.q)
    q8, qp8, hi, lo, qp16 = B.qbp_bifurcate(xd, 0, 1, 2)
    o16 = O.quantize(x, 16, rounding=1, seed=0, tensor_id=2)
    ohi, olo = O.limb_split(o16.q)
    assert np.array_equal(to_host(hi), ohi) and np.array_equal(to_host(lo), olo)
    o8 = O.quantize(x, 8, rounding=1, seed=0, tensor_id=1)
    assert np.array_equal(to_host(q8), o8.q)
