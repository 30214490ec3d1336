"""One minibatch spread over two shards (data parallelism, Section 3: Range BN's statistics are the whole
minibatch's): the library's split entry points with the four exchange steps between them must give each shard the
rows of what the undivided layer gives -- codes and integer accumulators bit for bit, fp32 within 1e-5 -- and that
is checked against the CPU oracle run on the whole batch.  One GPU: the two shards run as two host threads whose
"all-reduce" is a host-side rendezvous (no kernel waits for another)."""
import threading

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


class HostRendezvous:
    """All-reduce among `world` host threads sharing one GPU: deposit, wait, combine, wait, copy back."""

    def __init__(self, world):
        self.world, self.slots = world, [None] * world
        self.barrier = threading.Barrier(world)
        self.local = threading.local()

    def reduce_for(self, rank):
        import torch

        def reduce(t, op):
            torch.cuda.synchronize()
            self.slots[rank] = t.clone()
            self.barrier.wait()
            stack = torch.stack(self.slots)
            res = {"sum": lambda s: s.sum(0), "min": lambda s: s.min(0).values, "max": lambda s: s.max(0).values}[op](stack)
            self.barrier.wait()
            t.copy_(res.to(t.dtype))
            torch.cuda.synchronize()
            return t
        return reduce


def _run_sharded(B, make_layer, x, w, dy, splits, relu):
    """splits: row boundaries of the shards along the batch axis.  Returns per-shard results."""
    from paper_1805_11046_b200 import dist
    world = len(splits) - 1
    rv = HostRendezvous(world)
    out, errs = [None] * world, []

    def work(r):
        try:
            import torch
            torch.cuda.set_device(0)
            L = make_layer(r, rv.reduce_for(r))
            y = L.forward(to_dev(x[splits[r]:splits[r + 1]]), to_dev(w))
            dx, dw, dgamma, dbeta = L.backward(to_dev(dy[splits[r]:splits[r + 1]]))
            torch.cuda.synchronize()
            out[r] = dict(L=L, y=to_host(y), dx=to_host(dx), dw=to_host(dw), dgamma=to_host(dgamma), dbeta=to_host(dbeta),
                          x_codes=to_host(L.x_codes), z=to_host(L.z), g=to_host(L.g), g8=to_host(L.g8), ghi=to_host(L.ghi),
                          glo=to_host(L.glo), acc=to_host(L.acc_dw))
        except Exception as exc:            # let the other thread's barrier time out rather than hang
            errs.append(exc)
            rv.barrier.abort()

    ts = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in ts: t.start()
    for t in ts: t.join()
    if errs:
        raise errs[0]
    return out


@pytest.mark.parametrize("splits", [(0, 3, 6), (0, 4, 6)])
def test_conv_layer_over_two_shards_equals_the_whole_batch(B, splits):
    from paper_1805_11046_b200 import dist
    cfg = synth.conv3x3_layer(batch=6, hw=14)
    c = cfg["conv"]; relu = True
    HW = c["H"] * c["W"]

    def make_layer(r, reduce):
        n = splits[r + 1] - splits[r]
        conv = B.conv_desc(n, c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
        return dist.DataParallelLayer(B, conv=conv, relu=relu, seed=cfg["seed"], tensor_id8=cfg["id8"], tensor_id16=cfg["id16"],
                                      rows_total=6 * HW, row_offset=splits[r] * HW, reduce=reduce)

    parts = _run_sharded(B, make_layer, cfg["x"], cfg["w"], cfg["dy"], splits, relu)
    cat = lambda k: np.concatenate([p[k] for p in parts])
    # the oracle on the undivided batch, stage by stage on what the GPU produced
    od = O.conv_desc(6, c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    ox = O.quantize(cfg["x"], 8); ow = O.quantize(cfg["w"], 8)
    assert np.array_equal(cat("x_codes"), ox.q)
    _, oz, bad = O.conv_s8(0, od, ox.q, ox.zero_point[0], ow.q, ow.zero_point[0], ox.scale[0], ow.scale[0])
    z = cat("z")
    assert bad == 0 and np.array_equal(z, oz)
    oy, om, olo, ohi = O.rangebn_fwd(z, relu=relu)
    assert rel_err(cat("y"), oy)[0] <= FP32_TOL
    L0 = parts[0]["L"]
    for p in parts:                                    # every shard holds the whole minibatch's statistics
        assert np.array_equal(to_host(p["L"].vmin), olo) and np.array_equal(to_host(p["L"].vmax), ohi)
        assert np.array_equal(to_host(p["L"].mean), to_host(L0.mean))
    assert np.abs(to_host(L0.mean) - om).max() <= 1e-6 * max(1.0, np.abs(om).max())
    og, odg, odb = O.rangebn_bwd(cfg["dy"], z, to_host(L0.mean), olo, ohi, relu=relu)
    g = cat("g")
    assert rel_err(g, og)[0] <= FP32_TOL
    for p in parts:
        assert rel_err(p["dgamma"], odg)[0] <= FP32_TOL and rel_err(p["dbeta"], odb)[0] <= FP32_TOL
    g8, g16 = O.bifurcate(g, cfg["seed"], cfg["id8"], cfg["id16"])
    ohi_, olo_ = O.limb_split(g16.q)
    assert np.array_equal(cat("g8"), g8.q) and np.array_equal(cat("ghi"), ohi_) and np.array_equal(cat("glo"), olo_)
    _, odx, bad = O.conv_s8(1, od, g8.q, g8.zero_point[0], ow.q, ow.zero_point[0], g8.scale[0], ow.scale[0])
    assert bad == 0 and np.array_equal(cat("dx"), odx)
    oacc, odw = O.conv_wgrad_s16(od, ox.q, ox.zero_point[0], g16.q, g16.zero_point[0], ox.scale[0], g16.scale[0])
    for p in parts:                                    # the exact integer sum, and its one dequantisation, on every shard
        assert np.array_equal(p["acc"], oacc) and np.array_equal(p["dw"], odw)


def test_linear_layer_over_two_shards_equals_the_whole_batch(B):
    from paper_1805_11046_b200 import dist
    cfg = synth.linear_layer()
    splits = (0, 32, 64)

    def make_layer(r, reduce):
        return dist.DataParallelLayer(B, batch=splits[r + 1] - splits[r], in_features=256, out_features=128, relu=False,
                                      seed=cfg["seed"], tensor_id8=cfg["id8"], tensor_id16=cfg["id16"], rows_total=64,
                                      row_offset=splits[r], reduce=reduce)

    parts = _run_sharded(B, make_layer, cfg["x"], cfg["w"], cfg["dy"], splits, False)
    cat = lambda k: np.concatenate([p[k] for p in parts])
    ox = O.quantize(cfg["x"], 8); ow = O.quantize(cfg["w"], 8)
    assert np.array_equal(cat("x_codes"), ox.q)
    _, oz, _ = O.gemm_s8(ox.q, ox.zero_point[0], ow.q, ow.zero_point[0], ox.scale[0], ow.scale[0])
    z = cat("z")
    assert np.array_equal(z, oz)
    oy, om, olo, ohi = O.rangebn_fwd(z)
    assert rel_err(cat("y"), oy)[0] <= FP32_TOL
    L0 = parts[0]["L"]
    og, odg, odb = O.rangebn_bwd(cfg["dy"], z, to_host(L0.mean), olo, ohi)
    g = cat("g")
    assert rel_err(g, og)[0] <= FP32_TOL
    g8, g16 = O.bifurcate(g, cfg["seed"], cfg["id8"], cfg["id16"])
    assert np.array_equal(cat("g8"), g8.q)
    _, odx, _ = O.gemm_s8(g8.q, g8.zero_point[0], ow.q, ow.zero_point[0], g8.scale[0], ow.scale[0], transB=True)
    assert np.array_equal(cat("dx"), odx)
    oacc, odw = O.gemm_s16s8(ox.q, ox.zero_point[0], g16.q, g16.zero_point[0], ox.scale[0], g16.scale[0])
    for p in parts:
        assert np.array_equal(p["acc"], oacc) and np.array_equal(p["dw"], odw)
