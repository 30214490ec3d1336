#!/usr/bin/env python
"""Benchmark of the 8-bit training hot path: one quantised conv layer + Range BN, forward and backward.

A step is one pass of the whole path over one batch of synthetic input shaped like ResNet-18's conv2_x
3x3 layer (batch 256, 56x56, 64 -> 64 channels): quantise x and w, int8 implicit-GEMM forward, Range BN
(+ReLU); Range BN backward, gradient bifurcation (8-bit and 16-bit stochastic copies), int8 layer
gradient, 16x8-bit weight gradient.  Everything runs in libqbp's CUDA kernels through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  N > 1: one process per GPU under torch.distributed.run; the batches are
independent, so ranks share nothing on the data path (weak scaling, per-GPU batch statistics).
--impl reference times the CPU oracle on the host cores instead (bounded sample per step).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "QBP layer fwd+bwd int8 TOPS & Range BN GB/s vs B200 roofline; images/s"
WORKLOAD = "resnet18_conv2x_3x3_layer_fwd_bwd"
BATCH, HW, CIN, COUT = 256, 56, 64, 64
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised under profiles/
# (captured at the full batch of 256).  None: not captured.
# Keyed by (kernel, occurrence within the step), like KERNEL_WORK; dropped when a kernel changes.
NCU_TRAFFIC_BYTES_PER_ELEMENT = {("bn_bwd_apply_bifurcate_kernel", 0): (411.1e6 + 134.0e6) / 51380224}
# Kernels bound by plain instruction issue rather than by HBM: thread instructions per element, from the same
# captures (smsp__inst_executed.sum x 32 / elements).  Their roofline is the issue rate of the SMs:
# SMs x 4 schedulers x 1 warp instruction per clock x 32 threads x the maximum SM clock.
ALU_INSTR_PER_ELEMENT = {("bn_bwd_apply_bifurcate_kernel", 0): 9.761e7 * 32 / 51380224}
SM_COUNT, SCHEDULERS_PER_SM = 148, 4


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Reads SM clock and throttle reasons every 25 ms while the GPU works (NVML, read-only)."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.025)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------- the workload
def conv_workload(batch):
    from paper_1805_11046_b200 import synth
    return synth.conv3x3_layer(batch=batch, hw=HW, c_in=CIN, k_out=COUT)


# Algorithmic HBM bytes per element of the [N,H,W,64] activation (E = batch*56*56*64 elements) and int8 ops per
# element of each kernel of a step, keyed by (kernel name, occurrence within the step); kernels not listed
# move O(channels) or O(pixels) bytes only.
OPS_PER_ELEMENT_CONV = 2 * 9 * CIN          # 2*K per output element of fprop / dgrad
KERNEL_WORK = {
    ("range_partial_kernel", 0): (4, 0), ("quantize_kernel", 0): (5, 0),            # x: scan, then codes (+ per-pixel sums, per-channel totals)
    ("qbp_mma_kernel", 0): (5, OPS_PER_ELEMENT_CONV),                               # fprop: 1 B codes in, 4 B fp32 out
    ("bn_stats_kernel", 0): (4, 0), ("bn_apply_kernel", 0): (8, 0),
    ("bn_bwd_stats_kernel", 0): (8, 0), ("bn_bwd_apply_kernel", 0): (12, 0),
    ("quantize_kernel", 1): (7, 0),                                                 # bifurcation: 4 B in, 1 + 2 B out
    ("bn_bwd_apply_bifurcate_kernel", 0): (11, 0),                                  # dy and z in (8 B), the gradient's 8-bit copy and two limbs out (3 B)
    ("qbp_mma_kernel", 1): (5, OPS_PER_ELEMENT_CONV),                               # dgrad
    ("qbp_wgrad_kernel", 0): (3, 2 * OPS_PER_ELEMENT_CONV),                         # two int8 products per 16x8-bit product
}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1805_11046_b200 import binding as B
    from paper_1805_11046_b200 import layer
    from paper_1805_11046_b200.dist import max_over_ranks, rank_info

    rank, local_rank, world = rank_info()
    if world != args.gpus and rank == 0:
        print(f"bench: --gpus {args.gpus} but the launcher started {world} rank(s); reporting n_gpus = {world}", file=sys.stderr)
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)

    cfg = conv_workload(args.batch)
    host = {k: torch.from_numpy(cfg[k]).pin_memory() for k in ("x", "w", "dy")}
    x, w, dy = (host[k].to(dev, non_blocking=True) for k in ("x", "w", "dy"))
    c = cfg["conv"]
    conv = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    L = layer.QuantizedLayer(conv=conv, relu=True, seed=cfg["seed"], tensor_id8=cfg["id8"], tensor_id16=cfg["id16"], device=dev,
                             keep_g=False)      # (the fp32 gradient at the product is an intermediate: only its two copies are kept)
    E = x.numel()

    def step():
        L.forward(x, w)
        L.backward(dy)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.only_steps:
        # profiling aid: just the steps (run under `ncu -k ... -c ...`), no timing, no JSON line
        for _ in range(args.warmup + args.steps):
            step()
        barrier()
        assert L.status() == 0, "a device-side wait timed out"
        return

    sampler = ClockSampler(local_rank)
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    assert L.status() == 0, "a device-side wait timed out"

    # The step is ~30 short kernels: capture it once in a CUDA graph (the library only enqueues on the stream it is
    # given) and replay it, so that the gaps between dependent launches do not depend on the host.
    run_step, graphed = step, False
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.current_stream().wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            torch.cuda.synchronize()
            assert L.status() == 0
            run_step, graphed = graph.replay, True
        except Exception as exc:            # capture refused: time the plain launches
            print(f"bench: CUDA graph capture failed ({exc}); timing plain launches", file=sys.stderr)
            torch.cuda.synchronize()

    # ---- device-resident throughput: exactly K steps between two events on the launching stream
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        run_step()
    ev1.record()
    barrier()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    clocks = sampler.stop()
    ms_step = ms_total / args.steps
    value = world * args.batch / (ms_step * 1e-3)

    # ---- end to end: inputs start in pinned host memory, the weight gradient is read back, every step
    out_host = {k: torch.empty(t.shape, dtype=t.dtype).pin_memory() for k, t in
                (("dw", L.dw), ("dgamma", L.dgamma), ("dbeta", L.dbeta))}
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_step():
        x.copy_(host["x"], non_blocking=True); w.copy_(host["w"], non_blocking=True); dy.copy_(host["dy"], non_blocking=True)
        run_step()
        out_host["dw"].copy_(L.dw, non_blocking=True); out_host["dgamma"].copy_(L.dgamma, non_blocking=True)
        out_host["dbeta"].copy_(L.dbeta, non_blocking=True)

    e2e_step()
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev) / e2e_steps
    h2d = sum(host[k].numel() * host[k].element_size() for k in host)
    d2h = sum(t.numel() * t.element_size() for t in out_host.values())

    # ---- per-kernel device times (event pair around every launch), same launch configuration
    trace_steps = max(3, min(args.steps, 10))
    B.trace_enable(True)
    for _ in range(trace_steps):
        step()
    recs = B.trace_records()
    B.trace_enable(False)
    per_step = len(recs) // trace_steps
    launches_per_step = per_step
    kernels = []
    seen = {}
    for i in range(per_step):
        name = recs[i][0]
        occ = seen.get(name, 0); seen[name] = occ + 1
        assert all(recs[st * per_step + i][0] == name for st in range(trace_steps)), (i, name)
        times = [recs[st * per_step + i][1] for st in range(trace_steps)]
        bpe, ope = KERNEL_WORK.get((name, occ), (0, 0))
        kernels.append({"kernel": name, "occ": occ, "ms": sum(times) / len(times), "bytes": bpe * E, "ops": ope * E})
    traced_ms = sum(k["ms"] for k in kernels) or 1.0
    peaks, peaks_kind = measured_peaks()
    hbm_peak = float(peaks["hbm_gbs"])
    int8_peak_tops = 4500.0                 # nominal dense int8: 2 x nominal dense bf16
    for k in kernels:
        k["share"] = k["ms"] / traced_ms
        k["gbs"] = k["bytes"] / (k["ms"] * 1e-3) / 1e9 if k["ms"] > 0 else 0.0
        k["tops"] = k["ops"] / (k["ms"] * 1e-3) / 1e12 if k["ms"] > 0 else 0.0
    roofline = None
    if kernels:
        # the kernel with the largest share of the step, against the roofline that binds it by its algorithmic work:
        # HBM bytes over the measured copy bandwidth
        top = max(kernels, key=lambda k: k["ms"])
        tr = NCU_TRAFFIC_BYTES_PER_ELEMENT.get((top["kernel"], top["occ"]))
        roofline = {"kernel": top["kernel"], "bound": "hbm", "achieved": round(top["gbs"], 1), "peak": hbm_peak,
                    "unit": "GB/s", "frac": round(top["gbs"] / hbm_peak, 4), "traffic": tr * E if tr else None,
                    "peak_source": f"{peaks_kind} copy bandwidth", "ms_per_launch": round(top["ms"], 4),
                    "share_of_step": round(top["share"], 4)}
        ipe = ALU_INSTR_PER_ELEMENT.get((top["kernel"], top["occ"]))
        if ipe:
            # beside it, how close the kernel runs to the SMs' instruction issue rate (thread instructions per
            # element from the ncu capture under profiles/; 148 SMs x 4 schedulers x 32 threads x max SM clock)
            sm_ghz = float(peaks.get("sm_max_mhz", 1965.0)) / 1e3
            alu_peak = SM_COUNT * SCHEDULERS_PER_SM * 32 * sm_ghz / 1e3          # T thread-instructions / s
            alu_ach = ipe * E / (top["ms"] * 1e-3) / 1e12
            roofline.update({"alu_frac": round(alu_ach / alu_peak, 4), "alu_achieved_tinstr_s": round(alu_ach, 2),
                             "alu_peak_tinstr_s": round(alu_peak, 2), "thread_instructions_per_element": round(ipe, 1)})
    mma_ops = sum(k["ops"] for k in kernels if k["ops"])
    mma_ms = sum(k["ms"] for k in kernels if k["ops"])
    bn_bytes = sum(k["bytes"] for k in kernels if k["kernel"].startswith("bn_"))
    bn_ms = sum(k["ms"] for k in kernels if k["kernel"].startswith("bn_"))

    line = {
        "metric": METRIC, "value": round(value, 1), "unit": "images/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "s8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": args.batch, "input": [args.batch, HW, HW, CIN],
                   "filter": [COUT, 3, 3, CIN], "l2": "inputs (205 MB per activation tensor) larger than the 126 MB L2",
                   "parallelism": f"dp{world} (independent batches, no data-path collective)", "cuda_graph": graphed},
        "clocks": clocks,
        "e2e": {"value": round(world * args.batch / (e2e_ms * 1e-3), 1), "unit": "images/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4), "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline,
        "int8_tops": round(mma_ops / (mma_ms * 1e-3) / 1e12, 1) if mma_ms else None,
        "int8_tops_frac_of_nominal_4500": round(mma_ops / (mma_ms * 1e-3) / 1e12 / int8_peak_tops, 4) if mma_ms else None,
        "rangebn_gbs": round(bn_bytes / (bn_ms * 1e-3) / 1e9, 1) if bn_ms else None,
        "rangebn_frac_of_hbm": round(bn_bytes / (bn_ms * 1e-3) / 1e9 / hbm_peak, 4) if bn_ms else None,
        "kernels": [{"kernel": k["kernel"], "ms": round(k["ms"], 4), "share": round(k["share"], 4),
                     "gbs": round(k["gbs"], 1), "tops": round(k["tops"], 1)} for k in kernels if k["ms"] > 0.002],
    }
    if world == 1 and not args.no_extras:
        # the kernels the two roofline targets are graded on (dense sweep: tensor; Range BN / quantiser sweep: HBM)
        del L, x, w, dy
        torch.cuda.empty_cache()
        line["gemm_c5"] = gemm_c5_block(B, args.mnk, peaks)
        torch.cuda.empty_cache()
        line["rangebn_c3"] = rangebn_sweep_block(B, args.batch, hbm_peak)
        torch.cuda.empty_cache()
        line["stack_c4"] = stack_block(B, args.batch)
        torch.cuda.empty_cache()
        line["tbp_appendix_c"] = tbp_block(B, args.batch, hbm_peak, peaks)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args.cpu_sample_batch)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------- the two roofline targets, inside the headline line
def _graph_ms_per_call(calls, launches):
    """Device milliseconds per call of `launches` back-to-back calls, taken from the list `calls` in turn (each works
    on its own buffers, so that nothing a call reads is left in the L2 by the one before it), captured once as a
    CUDA graph and replayed: the time of a 10 us kernel then holds no host launch gap and no event overhead."""
    import torch
    for c in calls:
        c()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        calls[0]()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(launches):
            calls[i % len(calls)]()
    g.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 3
    a.record()
    for _ in range(reps):
        g.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / (reps * launches)


def rangebn_sweep_block(B, batch, hbm_peak, launches=60):
    """Range BN passes and the stochastic 8-bit quantiser on the five sweep shapes: GB/s per pass against the copy
    bandwidth.  Each pass is one C-ABI call (the streaming kernel plus its one-block finalize), timed as a graph of
    `launches` calls that rotate over enough buffer sets that every call reads from HBM."""
    import torch
    from paper_1805_11046_b200 import synth
    L2_BYTES = 126e6
    out = []
    for hw, ch in synth.RANGEBN_SWEEP:
        case = synth.rangebn_case(batch, hw, ch)
        E = case["x"].size
        tbytes = 4 * E
        sets = int(max(2, min(12, 2 * L2_BYTES // tbytes + 2)))
        x0 = torch.from_numpy(case["x"]).cuda(); dy0 = torch.from_numpy(case["dy"]).cuda()
        xs = [x0] + [x0.clone() for _ in range(sets - 1)]
        dys = [dy0] + [dy0.clone() for _ in range(sets - 1)]
        ys = [torch.empty_like(x0) for _ in range(sets)]
        qs = [torch.empty(x0.shape, dtype=torch.int8, device="cuda") for _ in range(sets)]
        n = E // ch
        ws = B.workspace(max(B.lib.qbp_rangebn_workspace_bytes(n, ch), B.lib.qbp_quantize_workspace_bytes(n, ch, 1)))
        csum, cmin, cmax = B.qbp_rangebn_fwd_stats(x0, ws=ws)
        _, mean, vmin, vmax, rng = B.qbp_rangebn_fwd_apply(x0, n, csum, cmin, cmax, relu=True, y=ys[0], want_range=True)
        sdy, sdyx = B.qbp_rangebn_bwd_stats(dy0, x0, n, mean, vmin, vmax, relu=True, ws=ws)
        xr = B.qbp_range_chunked(x0, 1)
        qp1, qpc = B.new_qparams(1), B.new_qparams(ch)
        passes = {
            "bn_stats": (4, [lambda i=i: B.qbp_rangebn_fwd_stats(xs[i], csum, cmin, cmax, ws=ws) for i in range(sets)]),
            "bn_apply": (8, [lambda i=i: B.qbp_rangebn_fwd_apply(xs[i], n, csum, cmin, cmax, relu=True, y=ys[i]) for i in range(sets)]),
            "bn_bwd_stats": (8, [lambda i=i: B.qbp_rangebn_bwd_stats(dys[i], xs[i], n, mean, vmin, vmax, relu=True, ws=ws) for i in range(sets)]),
            "bn_bwd_apply": (12, [lambda i=i: B.qbp_rangebn_bwd_apply(dys[i], xs[i], n, mean, vmin, vmax, sdy, sdyx, relu=True, dx=ys[i], ws=ws) for i in range(sets)]),
            "range_scan": (4, [lambda i=i: B.qbp_range_chunked(xs[i], 1, range_out=xr, ws=ws) for i in range(sets)]),
            "quantize_sr_s8_range_given": (5, [lambda i=i: B.qbp_quantize_s8(xs[i], rounding=1, seed=1, tensor_id=2, range_in=xr, q=qs[i], qp_out=qp1, ws=ws) for i in range(sets)]),
            "quantize_sr_s8_with_scan": (9, [lambda i=i: B.qbp_quantize_s8(xs[i], rounding=1, seed=1, tensor_id=2, q=qs[i], qp_out=qp1, ws=ws) for i in range(sets)]),
            "quantize_sr_s8_per_channel_with_scan": (9, [lambda i=i: B.qbp_quantize_s8(xs[i], granularity=1, rounding=1, seed=1, tensor_id=2, q=qs[i], qp_out=qpc, ws=ws) for i in range(sets)]),
        }
        row = {"shape": [batch, hw, hw, ch], "tensor_mb": round(tbytes / 1e6, 1), "buffer_sets": sets, "passes": {}}
        for name, (bpe, calls) in passes.items():
            ms = _graph_ms_per_call(calls, launches)
            gbs = bpe * E / (ms * 1e-3) / 1e9
            row["passes"][name] = {"us": round(ms * 1e3, 2), "bytes_per_element": bpe, "gbs": round(gbs, 0),
                                   "frac": round(gbs / hbm_peak, 3)}
        out.append(row)
        del xs, dys, ys, qs, x0, dy0
        torch.cuda.empty_cache()
    return {"timing": f"CUDA graph of {launches} back-to-back calls per pass over rotating buffer sets (inputs not in L2)",
            "peak_gbs": hbm_peak, "shapes": out}


def gemm_c5_block(B, n, peaks, launches=20):
    """The dense sweep's int8 GEMM and limb-split 16x8-bit weight-gradient GEMM at M = N = K = n: the tensor-core
    kernel's time per launch (CUDA-event pair around each of `launches` launches, median) with the clocks sampled
    meanwhile, against 2 x the measured bf16 peak (the nominal int8 : bf16 ratio)."""
    import torch
    from paper_1805_11046_b200 import synth
    int8_peak = 2.0 * float(peaks["bf16_tflops"])
    int8_sustained = 2.0 * float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    dev = lambda a: torch.from_numpy(a).cuda()
    case = synth.dense_gemm(n, n, n)
    res = {"mnk": n, "launches": launches, "peak_tops_burst": int8_peak, "peak_tops_sustained": int8_sustained,
           "peak_source": "measured bf16 x 2 (nominal int8 : bf16)"}

    def kernel_times(fn, names):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        B.trace_enable(True)
        for _ in range(launches):
            fn()
        r = B.trace_records(); B.trace_enable(False)
        ts = sorted(t for k, t in r if k in names)
        return statistics.median(ts), ts[0]

    qa, qpa = B.qbp_quantize_s8(dev(case["a"])); qb, qpb = B.qbp_quantize_s8(dev(case["b"]))
    out = torch.empty((n, n), dtype=torch.float32, device="cuda")
    ws = B.workspace(B.lib.qbp_gemm_s8_workspace_bytes(n, n, n))
    sampler = ClockSampler(torch.cuda.current_device()); sampler.start()
    med, best = kernel_times(lambda: B.qbp_gemm_s8(qa, qpa, qb, qpb, want_acc=False, out=out, ws=ws), ("qbp_mma_kernel", "qbp_mma2_kernel"))
    clocks = sampler.stop()
    assert B.status_word(ws) == 0
    tops = 2.0 * n ** 3 / med / 1e9
    res["gemm_s8"] = {"kernel": "qbp_mma2_kernel", "ms": round(med, 4), "ms_best": round(best, 4), "tops": round(tops, 1),
                      "frac_of_measured_burst": round(tops / int8_peak, 4), "frac_of_nominal_4500": round(tops / 4500.0, 4),
                      "frac_of_clock_adjusted": round(tops / (SM_COUNT * 16384 * float(clocks.get("sm_mhz") or 1965.0) / 1e6), 4),
                      "clocks": clocks}
    del qa, qb, out
    qx, qpx = B.qbp_quantize_s8(dev(case["x"]))
    _, hi, lo, qpg = B.qbp_quantize_s16(dev(case["g"]), want=("hi", "lo"))
    dW = torch.empty((n, n), dtype=torch.float32, device="cuda")
    ws = B.workspace(B.lib.qbp_wgrad_s16_workspace_bytes(None, n, n, n))
    sampler = ClockSampler(torch.cuda.current_device()); sampler.start()
    med, best = kernel_times(lambda: B.qbp_wgrad_s16(qx, qpx, hi, lo, qpg, want_acc=False, dW=dW, ws=ws), ("qbp_wgrad_kernel", "qbp_wgrad2_kernel"))
    clocks = sampler.stop()
    assert B.status_word(ws) == 0
    useful = 2.0 * n ** 3 / med / 1e9
    res["wgrad_s16xs8"] = {"kernel": "qbp_wgrad2_kernel" if n >= 512 else "qbp_wgrad_kernel", "ms": round(med, 4), "ms_best": round(best, 4),
                           "useful_tops": round(useful, 1), "executed_int8_tops": round(2 * useful, 1),
                           "frac_of_measured_burst": round(2 * useful / int8_peak, 4),
                           "frac_of_nominal_4500": round(2 * useful / 4500.0, 4), "clocks": clocks}
    return res


def stack_block(B, batch, reps=20):
    """One training step (forward chain, backward chain, fp32 updates) of the ResNet-50 conv3_x bottleneck stack
    (1x1 256->128, 3x3 128->128, 1x1 128->512, each + Range BN + ReLU) at batch `batch`: chained (every inner
    activation handed on as the 8-bit codes its Range BN wrote) against the unfused composition (range scan +
    quantiser per layer).  Each as a captured CUDA graph, `reps` replays."""
    import torch
    from paper_1805_11046_b200 import layer, synth
    st = synth.bottleneck_stack(batch=batch, hw=28)
    convs = [B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"]) for c in st["convs"]]
    x = torch.from_numpy(st["x"]).cuda(); dy = torch.from_numpy(st["dy"]).cuda()
    out = {"workload": "resnet50_conv3x_bottleneck_train_step", "batch": batch}
    for name, chained in (("chained", True), ("unfused", False)):
        S = layer.QuantizedStack(convs, [torch.from_numpy(w).cuda() for w in st["w"]], chained=chained, lr=0.0)
        for _ in range(3):
            S.train_step(x, dy)
        torch.cuda.synchronize()
        assert S.status() == 0
        B.trace_enable(True); S.train_step(x, dy); launches = len(B.trace_records()); B.trace_enable(False)
        side = torch.cuda.Stream(); side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            S.train_step(x, dy)
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            S.train_step(x, dy)
        g.replay(); torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record(); torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        out[name] = {"ms_per_step": round(ms, 4), "images_per_s": round(batch / (ms * 1e-3), 1), "launches": launches}
        del S, g
        torch.cuda.empty_cache()
    return out


def tbp_block(B, batch, hbm_peak, peaks, launches=30):
    """Appendix C (1-bit operands, ternary gradients) at the benchmark layer's size: the binarisation and the stochastic
    ternarisation (1 sample, and the sum of 6 for Algorithm 1) of the 51.4 M-element activation / gradient tensor as
    graph-timed calls over rotating buffers (bytes per element: 4 in + 1 out, plus 4 for the ternariser's range scan),
    the forward product of a binarised 4096^3 layer (XNOR-popcount result on the int8 tensor cores), and Algorithm 1
    for the conv2_x layer (ternarise 6 samples + one weight-gradient product)."""
    import torch
    from paper_1805_11046_b200 import synth
    cfg = conv_workload(batch)
    E = cfg["dy"].size
    g0 = torch.from_numpy(cfg["dy"]).cuda()
    gs = [g0, g0.clone(), g0.clone()]
    qs = [torch.empty(g0.shape, dtype=torch.int8, device="cuda") for _ in gs]
    qp = B.new_qparams(1); ws = B.workspace(B.lib.qbp_stc_ternarize_workspace_bytes())
    passes = {
        "binarize": (5, [lambda i=i: B.qbp_binarize_s8(gs[i], q=qs[i], qp_out=qp) for i in range(3)]),
        "stc_ternarize_1_sample_with_scan": (9, [lambda i=i: B.qbp_stc_ternarize_s8(gs[i], 1, 1, 2, q=qs[i], qp_out=qp, ws=ws) for i in range(3)]),
        "stc_ternarize_6_samples_with_scan": (9, [lambda i=i: B.qbp_stc_ternarize_s8(gs[i], 6, 1, 2, q=qs[i], qp_out=qp, ws=ws) for i in range(3)]),
    }
    out = {"tensor_elements": E, "passes": {}}
    for name, (bpe, calls) in passes.items():
        ms = _graph_ms_per_call(calls, launches)
        gbs = bpe * E / (ms * 1e-3) / 1e9
        out["passes"][name] = {"us": round(ms * 1e3, 2), "bytes_per_element": bpe, "gbs": round(gbs, 0), "frac": round(gbs / hbm_peak, 3)}
    # forward product of a binarised layer, 4096^3
    n = 4096
    case = synth.dense_gemm(n, n, n)
    qa, pa = B.qbp_binarize_s8(torch.from_numpy(case["a"]).cuda()); qb, pb = B.qbp_binarize_s8(torch.from_numpy(case["b"]).cuda())
    o = torch.empty((n, n), dtype=torch.float32, device="cuda"); wsg = B.workspace(B.lib.qbp_gemm_s8_workspace_bytes(n, n, n))
    ms = _graph_ms_per_call([lambda: B.qbp_gemm_s8(qa, pa, qb, pb, out=o, ws=wsg)], 20)
    out["xnor_forward_4096"] = {"ms": round(ms, 4), "tera_bit_macs_per_s": round(n ** 3 / (ms * 1e-3) / 1e12, 1),
                                "int8_tops": round(2 * n ** 3 / (ms * 1e-3) / 1e12, 1),
                                "frac_of_measured_burst": round(2 * n ** 3 / (ms * 1e-3) / 1e12 / (2 * float(peaks["bf16_tflops"])), 3),
                                "includes": "the two code-sum kernels and the terms kernel of the call"}
    # the same product from bit rows on the popcount unit of the CUDA cores
    ab, bb = B.qbp_pack_bits(qa), B.qbp_pack_bits(qb.t().contiguous())
    oc = torch.empty((n, n), dtype=torch.int32, device="cuda")
    msb = _graph_ms_per_call([lambda: B.qbp_xnor_gemm_bits(ab, bb, n, out=oc)], 5)
    out["xnor_forward_4096_popcount_on_bit_rows"] = {"ms": round(msb, 4), "tera_bit_macs_per_s": round(n ** 3 / (msb * 1e-3) / 1e12, 1),
                                                     "tensor_core_route_speedup": round(msb / ms, 2)}
    del qa, qb, o, wsg, case, ab, bb, oc
    # Algorithm 1 for the benchmark layer: 6 samples
    import ctypes
    c = cfg["conv"]
    d = B.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    a_codes, qa = B.qbp_binarize_s8(torch.from_numpy(cfg["x"]).cuda())
    wsa = B.workspace(B.lib.qbp_tbp_weight_gradient_workspace_bytes(ctypes.byref(d), 0, 0, 0))
    ms = _graph_ms_per_call([lambda: B.qbp_tbp_weight_gradient(a_codes, qa, g0, 6, seed=1, tensor_id=2, d=d, ws=wsa)], 10)
    out["algorithm_1_conv2x_6_samples"] = {"ms": round(ms, 4), "images_per_s": round(batch / (ms * 1e-3), 1)}
    return out


# ------------------------------------------------------------- CPU oracle arm
def oracle_step(cfg):
    """The whole path once through the oracle, as it stands."""
    from oracle import qbp_oracle as O
    c = cfg["conv"]
    d = O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["stride"], c["pad"])
    y, saved, _ = O.layer_fwd(cfg["x"], cfg["w"], relu=True, conv=d)
    g, dgamma, dbeta = O.rangebn_bwd(cfg["dy"], saved.z, saved.mean, saved.vmin, saved.vmax, relu=True)
    dx, dw, *_ = O.layer_bwd_products(g.astype(np.float32), saved, cfg["seed"], cfg["id8"], cfg["id16"], conv=d)
    return y, dx, dw


def cpu_baseline(sample_batch):
    from oracle import qbp_oracle as O
    cfg = conv_workload(sample_batch)
    O.lib()
    t0 = time.perf_counter()
    oracle_step(cfg)
    dt = time.perf_counter() - t0
    return {"value": round(sample_batch / dt, 3), "unit": "images/s", "cores": O.num_threads(), "kind": "oracle",
            "sample": f"one fwd+bwd of the same layer at batch {sample_batch} (of {BATCH}) on the host, {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import qbp_oracle as O
    cfg = conv_workload(args.cpu_sample_batch)
    O.lib()
    for _ in range(min(args.warmup, 1)):
        oracle_step(cfg)
    steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(cfg)
    dt = (time.perf_counter() - t0) / steps
    value = round(args.cpu_sample_batch / dt, 3)
    sample = f"each step = one fwd+bwd of the layer at batch {args.cpu_sample_batch} (of {BATCH}); {steps} timed steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "images/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": round(dt * 1e3, 2), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "s8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": args.batch, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


# ------------------------------------------------- side workloads (not the headline line)
def _event_ms(fn, iters, flush=None):
    """Median CUDA-event time of fn over `iters` runs (after 3 warm-ups); an L2 flush before each when given."""
    import torch
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        if flush is not None:
            flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record(); torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    return statistics.median(ts)


def _kernel_ms(B, fn, reps=5, flush=None):
    """Per-kernel device times (minimum over reps) of one call, from the library's launch trace; an L2 flush
    (a write larger than the L2) before each call when given."""
    for _ in range(2):
        fn()
    B.trace_enable(True)
    for _ in range(reps):
        if flush is not None:
            flush.zero_()
        fn()
    r = B.trace_records(); B.trace_enable(False)
    n = len(r) // reps
    return [(r[i][0], min(r[k * n + i][1] for k in range(reps))) for i in range(n)]


def run_gemm(args):
    """Dense quantised GEMM (fp32 N(0,1) operands -> int8 codes -> tcgen05 product with fused zero-point correction
    and dequantisation) and the limb-split 16x8-bit weight-gradient GEMM at M = N = K = --mnk; one JSON line each."""
    import torch
    from paper_1805_11046_b200 import binding as B, synth
    torch.cuda.set_device(0)
    n = args.mnk
    peaks, kind = measured_peaks()
    int8_peak = 2.0 * float(peaks["bf16_tflops"])        # own-dtype peak: measured bf16 x the nominal int8 : bf16 ratio
    int8_peak_sustained = 2.0 * float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    case = synth.dense_gemm(n, n, n)
    dev = lambda a: torch.from_numpy(a).cuda()
    qa, qpa = B.qbp_quantize_s8(dev(case["a"])); qb, qpb = B.qbp_quantize_s8(dev(case["b"]))
    out = torch.empty((n, n), dtype=torch.float32, device="cuda")
    ws = B.workspace(B.lib.qbp_gemm_s8_workspace_bytes(n, n, n))
    if args.only_steps:
        # profiling aid: the GEMM, then the weight-gradient GEMM, warmup + steps calls each; no timing, no JSON line
        for _ in range(args.warmup + args.steps):
            B.qbp_gemm_s8(qa, qpa, qb, qpb, want_acc=False, out=out, ws=ws)
        torch.cuda.synchronize(); assert B.status_word(ws) == 0
        del qa, qb, out
        qx, qpx = B.qbp_quantize_s8(dev(case["x"]))
        _, hi, lo, qpg = B.qbp_quantize_s16(dev(case["g"]), want=("hi", "lo"))
        dW = torch.empty((n, n), dtype=torch.float32, device="cuda")
        ws = B.workspace(B.lib.qbp_wgrad_s16_workspace_bytes(None, n, n, n))
        for _ in range(args.warmup + args.steps):
            B.qbp_wgrad_s16(qx, qpx, hi, lo, qpg, want_acc=False, dW=dW, ws=ws)
        torch.cuda.synchronize(); assert B.status_word(ws) == 0
        return
    sampler = ClockSampler(0); sampler.start()
    fn = lambda: B.qbp_gemm_s8(qa, qpa, qb, qpb, want_acc=False, out=out, ws=ws)
    call_ms = _event_ms(fn, max(args.steps, 5))
    ker = _kernel_ms(B, fn)
    clocks = sampler.stop()
    mma_ms = [t for k, t in ker if k in ("qbp_mma_kernel", "qbp_mma2_kernel")][0]
    tops = 2.0 * n ** 3 / mma_ms / 1e9
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    print(json.dumps({"workload": f"dense_gemm_s8_{n}", "metric": "int8 TOPS", "value": round(tops, 1), "unit": "TOP/s",
                      "call_ms": round(call_ms, 4), "kernels": [(k, round(t, 4)) for k, t in ker], "dtype": "s8", "clocks": clocks,
                      "roofline": {"kernel": [k for k, t in ker if k.startswith("qbp_mma")][0], "bound": "tensor", "achieved": round(tops, 1),
                                   "peak": int8_peak_sustained if capped else int8_peak,
                                   "unit": "TOP/s", "frac": round(tops / (int8_peak_sustained if capped else int8_peak), 4), "traffic": None,
                                   "peak_source": f"{kind} bf16 {'sustained (the run was power-capped)' if capped else 'burst'} x 2 (nominal int8 : bf16)",
                                   "frac_of_burst_peak": round(tops / int8_peak, 4),
                                   # 148 SMs x 16384 int8 ops per clock at the SM clock sampled during the run
                                   "frac_of_clock_adjusted": round(tops / (SM_COUNT * 16384 * float(clocks.get("sm_mhz") or 1965.0) / 1e6), 4),
                                   "frac_of_nominal_4500": round(tops / 4500.0, 4)}}), flush=True)
    # limb-split weight-gradient GEMM: dW [K x N] = X [M x K]^T G [M x N], X 8-bit, G 16-bit as two byte limbs
    del qa, qb, out
    qx, qpx = B.qbp_quantize_s8(dev(case["x"]))
    _, hi, lo, qpg = B.qbp_quantize_s16(dev(case["g"]), want=("hi", "lo"))
    dW = torch.empty((n, n), dtype=torch.float32, device="cuda")
    ws = B.workspace(B.lib.qbp_wgrad_s16_workspace_bytes(None, n, n, n))
    fn = lambda: B.qbp_wgrad_s16(qx, qpx, hi, lo, qpg, want_acc=False, dW=dW, ws=ws)
    call_ms = _event_ms(fn, max(min(args.steps, 20), 5))
    ker = _kernel_ms(B, fn, reps=3)
    k_ms = [t for k, t in ker if k in ("qbp_wgrad_kernel", "qbp_wgrad2_kernel")][0]
    useful = 2.0 * n ** 3 / k_ms / 1e9
    print(json.dumps({"workload": f"dense_wgrad_s16xs8_{n}", "metric": "useful 16x8-bit TOPS (executes twice as many int8 ops)",
                      "value": round(useful, 1), "unit": "TOP/s", "call_ms": round(call_ms, 4),
                      "kernels": [(k, round(t, 4)) for k, t in ker], "dtype": "s8",
                      "roofline": {"kernel": [k for k, t in ker if k.startswith("qbp_wgrad")][0], "bound": "tensor", "achieved": round(2 * useful, 1),
                                   "peak": int8_peak, "unit": "TOP/s (executed int8)", "frac": round(2 * useful / int8_peak, 4),
                                   "traffic": None, "peak_source": f"{kind} bf16 burst x 2"}}), flush=True)


def run_rangebn(args):
    """Range BN forward/backward and 8-bit stochastic quantisation (per tensor, per channel) on the sweep shapes
    (batch 256 x 56^2x64 ... 7^2x2048); one JSON line per shape with GB/s per kernel against the copy bandwidth."""
    import torch
    from paper_1805_11046_b200 import binding as B, synth
    torch.cuda.set_device(0)
    peaks, kind = measured_peaks()
    hbm = float(peaks["hbm_gbs"])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    bpe = {"bn_stats_kernel": 4, "bn_apply_kernel": 8, "bn_bwd_stats_kernel": 8, "bn_bwd_apply_kernel": 12,
           "range_partial_kernel": 4, "chan_range_partial_kernel": 4, "chunk_range_partial_kernel": 4, "quantize_kernel": 5}
    for hw, ch in synth.RANGEBN_SWEEP:
        case = synth.rangebn_case(args.batch, hw, ch)
        x = torch.from_numpy(case["x"]).cuda(); dy = torch.from_numpy(case["dy"]).cuda()
        y = torch.empty_like(x); dx = torch.empty_like(x); q = torch.empty(x.shape, dtype=torch.int8, device="cuda")
        E = x.numel()
        _, mean, vmin, vmax, _ = B.qbp_rangebn_fwd(x, relu=True, y=y)

        def timed(fn):
            return _kernel_ms(B, fn, reps=3, flush=flush)
        ker = timed(lambda: B.qbp_rangebn_fwd(x, relu=True, y=y)) + \
            timed(lambda: B.qbp_rangebn_bwd(dy, x, mean, vmin, vmax, relu=True, dx=dx))
        qt = timed(lambda: B.qbp_quantize_s8(x, granularity=0, rounding=1, seed=1, tensor_id=2, q=q))
        qc = timed(lambda: B.qbp_quantize_s8(x, granularity=1, rounding=1, seed=1, tensor_id=2, q=q))
        rng = B.new_qparams(1)
        rc = timed(lambda: B.qbp_range_chunked(x, args.batch, range_out=rng))        # one chunk per image
        row = lambda ks: [{"kernel": k, "us": round(t * 1e3, 1), "gbs": round(bpe[k] * E / t / 1e6, 0) if k in bpe else None,
                           "frac": round(bpe[k] * E / t / 1e6 / hbm, 3) if k in bpe else None} for k, t in ks]
        print(json.dumps({"workload": f"rangebn_quant_{args.batch}x{hw}x{hw}x{ch}", "tensor_mb": round(E * 4 / 1e6, 1),
                          "peak_gbs": hbm, "peak_source": f"{kind} copy bandwidth", "rangebn": row(ker),
                          "quantize_sr_per_tensor": row(qt), "quantize_sr_per_channel": row(qc),
                          "range_chunk_averaged": row(rc)}), flush=True)
        del x, dy, y, dx, q


def run_tbp(args):
    """The low-bit variant's kernels (Appendix C) at the benchmark layer's size: one JSON line (see tbp_block)."""
    import torch
    from paper_1805_11046_b200 import binding as B
    torch.cuda.set_device(0)
    peaks, kind = measured_peaks()
    out = tbp_block(B, args.batch, float(peaks["hbm_gbs"]), peaks)
    out.update({"workload": "tbp_appendix_c", "peak_gbs": float(peaks["hbm_gbs"]), "peak_source": f"{kind} copy bandwidth"})
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--batch", type=int, default=BATCH, help="images per GPU (the workload is quoted at 256)")
    ap.add_argument("--cpu-sample-batch", type=int, default=128,
                    help="images of the layer the CPU oracle is timed on (128 of the 256 take about 15 s on 16 cores)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the dense-GEMM and Range BN sweep blocks of the line")
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of a captured CUDA graph of the step")
    ap.add_argument("--only-steps", action="store_true", help="run warmup+steps and exit (for captures under ncu)")
    ap.add_argument("--workload", choices=["layer", "gemm", "rangebn", "tbp"], default="layer",
                    help="layer: the headline line; gemm / rangebn / tbp: side measurements of the dense sweep, the Range BN "
                         "sweep and the low-bit variant's kernels (Appendix C)")
    ap.add_argument("--mnk", type=int, default=8192, help="--workload gemm: M = N = K")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.workload == "layer":
        # not started by a launcher: start one rank per GPU ourselves (torch.distributed.run, loopback rendezvous)
        import socket
        import subprocess
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *sys.argv[1:]]
        sys.exit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "gemm":
        run_gemm(args)
    elif args.workload == "rangebn":
        run_rangebn(args)
    elif args.workload == "tbp":
        run_tbp(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
