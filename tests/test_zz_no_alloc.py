"""qbp_quantize_s8_static -- the quantiser for callers that cannot hand over a workspace.

Some users of the library run where device memory may not be allocated (a fixed memory plan, a plugin that is
given its tensors and nothing else), so this entry point keeps the range scan's scratch in an array built into
the library instead of taking a workspace.  It must produce exactly what qbp_quantize_s8 produces.  The array is
shared by all calls and keeps the previous call's contents, hence the check on two calls in a row with
different inputs.  This file sorts last on purpose: a run that stops at the first failure has then already run
every other test."""
import ctypes as C

import numpy as np
import pytest

from oracle import qbp_oracle as O
from paper_1805_11046_b200 import synth
from tests.util import to_dev, to_host


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


def test_static_variant_rejects_what_its_scratch_cannot_hold(B):
    """Host-side refusals come before anything touches a device: too many per-channel columns, NULL outputs."""
    one = C.c_void_p(256)       # never dereferenced: the call must fail first
    too_wide = B.QBP_STATIC_MAX_CHANNELS + 4
    st = B.lib.qbp_quantize_s8_static(one, C.c_int64(8), C.c_int64(too_wide), B.QBP_PER_CHANNEL, B.QBP_ROUND_NEAREST,
                                      C.c_uint64(0), C.c_uint32(0), one, one, C.c_void_p(0))
    assert st == -2 and b"exceed the built-in scratch" in B.lib.qbp_last_error()
    st = B.lib.qbp_quantize_s8_static(one, C.c_int64(8), C.c_int64(16), B.QBP_PER_TENSOR, B.QBP_ROUND_NEAREST,
                                      C.c_uint64(0), C.c_uint32(0), C.c_void_p(0), one, C.c_void_p(0))
    assert st == -1
    st = B.lib.qbp_quantize_s8_static(one, C.c_int64(8), C.c_int64(16), B.QBP_PER_TENSOR, 7,
                                      C.c_uint64(0), C.c_uint32(0), one, one, C.c_void_p(0))
    assert st == -1


@pytest.mark.gpu
@pytest.mark.parametrize("granularity,rounding", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_static_variant_matches_the_workspace_variant_twice_in_a_row(B, granularity, rounding):
    import torch
    cases = [synth.channel_gaussian((3, 37, 29, 256), 20, 21),          # ragged rows, the widest per-channel case
             synth.normal((1031, 64), 77, std=0.1) - np.float32(0.05)]  # a different shape and range right after it
    for k, x in enumerate(cases):
        xd = to_dev(x)
        cols = x.shape[-1]
        want_q, want_qp = B.qbp_quantize_s8(xd, granularity=granularity, rounding=rounding, seed=5, tensor_id=9 + k)
        q = torch.empty(x.shape, dtype=torch.int8, device="cuda")
        qp = B.new_qparams(cols if granularity else 1)
        B.qbp_quantize_s8_static(xd, q, qp, granularity=granularity, rounding=rounding, seed=5, tensor_id=9 + k)
        torch.cuda.synchronize()
        assert np.array_equal(to_host(q), to_host(want_q))              # codes bit for bit
        assert np.array_equal(to_host(qp), to_host(want_qp))            # scale, zero-point, range bit for bit
        # and directly against the CPU statement of the quantiser
        o = O.quantize(x, 8, per_channel=bool(granularity), rounding=rounding, seed=5, tensor_id=9 + k)
        scale, zp, lo, hi = B.read_qparams(qp)
        assert np.array_equal(to_host(q), o.q) and np.array_equal(scale, o.scale) and np.array_equal(zp, o.zero_point)
        assert np.array_equal(lo, o.vmin) and np.array_equal(hi, o.vmax)


@pytest.mark.gpu
def test_static_variant_allocates_no_device_memory(B):
    """The point of the entry point: after a first call (which resolves the built-in array's address and loads the
    kernels) further calls leave the device's free memory and torch's allocator untouched."""
    import torch
    x = to_dev(synth.normal((515, 128), 79))
    q = torch.empty(x.shape, dtype=torch.int8, device="cuda")
    for granularity in (0, 1):
        qp = B.new_qparams(128 if granularity else 1)
        B.qbp_quantize_s8_static(x, q, qp, granularity=granularity, rounding=1, seed=1, tensor_id=2)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info(); alloc0 = torch.cuda.memory_allocated(); reserved0 = torch.cuda.memory_reserved()
        for _ in range(3):
            B.qbp_quantize_s8_static(x, q, qp, granularity=granularity, rounding=1, seed=1, tensor_id=2)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0 and torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


@pytest.mark.gpu
def test_static_variant_large_per_tensor_input(B):
    """Per-tensor granularity has no size limit: 8.4 M elements, several waves of the scan."""
    import torch
    x = synth.normal((4099, 2051), 78)
    xd = to_dev(x)
    want_q, want_qp = B.qbp_quantize_s8(xd)
    q = torch.empty(x.shape, dtype=torch.int8, device="cuda"); qp = B.new_qparams(1)
    for _ in range(2):
        q.zero_()
        B.qbp_quantize_s8_static(xd, q, qp)
        torch.cuda.synchronize()
        assert np.array_equal(to_host(q), to_host(want_q)) and np.array_equal(to_host(qp), to_host(want_qp))
