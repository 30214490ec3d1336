"""The device status word: a bounded wait that runs out raises it, the kernel ends normally, the host reads
QBP_ERR_TIMEOUT through the C ABI, and the device stays usable.  The wait that runs out is the library's own
self-test (a barrier that nothing signals, a limit of a few thousand cycles): no product kernel is disturbed."""
import numpy as np
import pytest

from oracle import qbp_oracle as O
from tests.util import random_codes, set_qparams, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_1805_11046_b200.binding as binding
    return binding


@pytest.mark.parametrize("limit", [2000, 200000])
def test_a_wait_that_runs_out_raises_the_status_word(B, limit):
    import torch
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    B.qbp_selftest_bounded_wait(limit, ws)
    assert B.status_word(ws) == B.QBP_ERR_TIMEOUT
    assert b"bounded device-side wait" in B.lib.qbp_last_error()
    # the context is intact and the next product on the same workspace clears the word again
    A = random_codes((128, 128), 1); Bm = random_codes((128, 128), 2)
    big = B.workspace(B.lib.qbp_gemm_s8_workspace_bytes(128, 128, 128))
    B.qbp_selftest_bounded_wait(limit, big)
    acc, _, ws2 = B.qbp_gemm_s8(to_dev(A), set_qparams(B.new_qparams(1), 1.0, 3), to_dev(Bm), set_qparams(B.new_qparams(1), 1.0, -4),
                                want_acc=True, want_out=False, ws=big)
    assert B.status_word(ws2) == 0
    assert np.array_equal(to_host(acc), O.gemm_s8(A, 3, Bm, -4)[0])


def test_selftest_refuses_bad_arguments(B):
    import ctypes as C
    import torch
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert B.lib.qbp_selftest_bounded_wait(C.c_void_p(ws.data_ptr()), C.c_size_t(256), C.c_uint32(0), C.c_void_p(0)) == -1
    assert B.lib.qbp_selftest_bounded_wait(C.c_void_p(0), C.c_size_t(256), C.c_uint32(1000), C.c_void_p(0)) == -4
    assert B.lib.qbp_device_status(C.c_void_p(0), C.c_void_p(0)) == -1


def test_layer_status_word_is_sticky_across_the_step(B):
    """The layer keeps one word at the head of its workspace: the forward clears it, nothing in the backward
    does, so a flag raised in between (here by hand) is still there after the backward call."""
    import torch
    from paper_1805_11046_b200 import layer, synth
    cfg = synth.conv3x3_layer(batch=2, hw=8)
    c = cfg["conv"]
    conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    L = layer.QuantizedLayer(conv=conv, relu=True)
    L.forward(to_dev(cfg["x"]), to_dev(cfg["w"]))
    assert L.status() == 0
    L.ws[:4].view(torch.int32).fill_(B.QBP_ERR_TIMEOUT)       # as a product of the forward would have left it
    L.backward(to_dev(cfg["dy"]))
    assert L.status() == B.QBP_ERR_TIMEOUT
    L.forward(to_dev(cfg["x"]), to_dev(cfg["w"]))
    L.backward(to_dev(cfg["dy"]))
    assert L.status() == 0
