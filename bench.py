#!/usr/bin/env python
"""Benchmark of the HBMM hot path on B200.

One step = one pass of the whole path over one synthetic batch: for each of the four ResNet-18
3x3 convolution shapes at batch 64, the convolution as HBMM (im2col gather + Hadamard
binarization + packed contraction, beta_a = beta_w = 32, fp32 scales) and the same convolution
in HBWN mode (bf16 activations x Hadamard-binary weights, beta_w = 32).  Weights are binarized
once outside the timed region.  The eight calls of a step share no buffer; the timed schedule
runs the four HBMM calls on one stream and the four HBWN calls on a second one, joined every
step (the one-stream time is reported beside it).  The metric is effective binary TOPS =
2*M*N*K summed over the eight products / step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (torchrun, one rank per GPU) every rank runs its own batch of 64 images (weak
scaling, no data-path collective); the time is the max over ranks.  `--impl reference` times
the CPU checker under oracle/ on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

BETA = 32
# Planning figures used only when the arithmetic-rate loops could not be timed (they always are on a GPU):
# 16 population counts and 128 fp32 additions per clock and multiprocessor.
PLAN_POPC_PER_CLK_SM = 16
PLAN_FADD_PER_CLK_SM = 128
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126e6
PAPER_CONTEXT = ("paper, Section 4.2 / Fig. 5: xHBNN is approximately 10x faster than a full-precision (32-bit) matrix "
                 "multiply on square matrices at beta = 16, on an Intel Xeon Gold 6128 CPU (3.40 GHz, 19.25 MB cache); "
                 "no absolute times are given")


# ----------------------------------------------------------------------------- distributed plumbing
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Max of a per-rank scalar (all-reduce MAX); identity for one rank."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed_offset(rank: int) -> int:
    """Each rank draws its own batch: global image index = 64 * rank + local index."""
    return 1000 * rank


def aggregate(work_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job throughput in TOPS from per-rank work (ops per step) and the max-over-ranks step time."""
    return work_per_rank * world / (ms_per_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def wait_ready(self, rows: int = 2, timeout: float = 5.0):
        """nvidia-smi needs a moment to start: block until it has delivered a few samples."""
        t = time.time()
        while self.proc is not None and len(self.rows) < rows and time.time() - t < timeout:
            time.sleep(0.02)

    def stop(self, t0: float, t1: float, t_end: float = None):
        """Samples inside [t0, t1] (the timed region); when that short region caught fewer than three, the
        samples of the legs that follow it under the same load (up to t_end) are used and `window` says so."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        window = "timed region"
        inside = sum(1 for ts, _ in self.rows if t0 <= ts <= t1 + 0.1)
        if inside < 3 and t_end is not None:
            t1 = t_end
            window = "timed region and the legs after it (weight-expansion step, end-to-end leg)"
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.rows:
            if ts < t0 or ts > t1 + 0.1:
                continue
            f = [s.strip() for s in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "window": window}


FALLBACK_BF16_TFLOPS = 1590.0


def measured_peaks():
    """(HBM GB/s, dense bf16 TFLOP/s burst, 'measured' | 'fallback')."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


# ----------------------------------------------------------------------------- workload
def layer_ops(shapes):
    return [2.0 * s.M * s.N * s.K for s in shapes]


def build_workload(torch, hbmm, inputs, rank: int, device, only=None):
    """Device-resident inputs, weights (binarized once), outputs and workspaces for every layer
    (or for the one layer named by ``only``)."""
    shapes = [s for s in inputs.resnet18_convs(64) if only is None or s.name == only]
    if not shapes:
        raise SystemExit("unknown layer %r" % only)
    off = rank_seed_offset(rank)
    layers = []
    for li, s in enumerate(shapes):
        x = inputs.conv_activation(s, inputs.SEEDS["resnet_hbmm"][0] + li + off)            # post-ReLU, fp32
        xs = inputs.conv_activation(s, inputs.SEEDS["resnet_hbwn"][0] + li + off, signed=False)
        xb_bits, _ = inputs.as_bf16(xs)
        w = inputs.he_normal(s.N, s.K, inputs.SEEDS["resnet_hbmm"][1] + li)
        wd = torch.from_numpy(w).to(device)
        Wop = hbmm.quantize(wd, hbmm.alloc_operand(s.N, s.K, BETA, hbmm.F32, device=device))
        geom = hbmm.make_geom(s.B, s.C, s.H, s.W, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
        x_host = torch.from_numpy(x).pin_memory()
        xb_host = torch.from_numpy(xb_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
        ws_bytes = hbmm.conv_workspace_bytes(geom, BETA, hbmm.F32, Wop)
        wsb_bytes = hbmm.conv_workspace_bytes(geom, 1, hbmm.F32, Wop)
        layers.append(dict(
            shape=s, geom=geom, W=Wop,
            x_host=x_host, xb_host=xb_host,
            x=x_host.to(device), xb=xb_host.to(device),
            C=torch.empty((s.M, s.N), device=device), Cb=torch.empty((s.M, s.N), device=device),
            C_host=torch.empty((s.M, s.N), dtype=torch.float32).pin_memory(),
            Cb_host=torch.empty((s.M, s.N), dtype=torch.float32).pin_memory(),
            # one workspace per product, so that the expanded weights each call leaves there survive the other
            ws=torch.empty(ws_bytes, dtype=torch.uint8, device=device),
            wsb=torch.empty(wsb_bytes, dtype=torch.uint8, device=device),
        ))
    return shapes, layers


def run_step(hbmm, layers, flags=0):
    """flags = CONV_WEIGHTS_PREPARED: the weights are fixed at inference time, so their expansion into the
    contraction's tile layout (left in each workspace by an earlier step) is not repeated per batch."""
    for L in layers:
        hbmm.conv_im2col(L["x"], L["geom"], BETA, hbmm.F32, L["W"], L["C"], L["ws"], flags=flags)      # rows I, Q, G
        hbmm.conv_im2col(L["xb"], L["geom"], 1, hbmm.F32, L["W"], L["Cb"], L["wsb"], flags=flags)      # rows I, H


class TwoStreamStep:
    """The same step with the two products on two streams: the HBMM calls of all layers on one, the HBWN calls
    on the other, forked from and joined to the current stream every step.  The two chains share no buffer
    (each has its own workspaces and outputs).  Each contraction is a persistent kernel of one block per SM
    whose last wave leaves SMs idle on the smaller layers; blocks of the other chain take them."""

    def __init__(self, torch):
        self.torch = torch
        self.sa, self.sb = torch.cuda.Stream(), torch.cuda.Stream()
        self.fork, self.ja, self.jb = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()

    def __call__(self, hbmm, layers, flags=0):
        torch = self.torch
        cur = torch.cuda.current_stream()
        self.fork.record(cur)
        self.sa.wait_event(self.fork)
        self.sb.wait_event(self.fork)
        with torch.cuda.stream(self.sa):
            for L in layers:
                hbmm.conv_im2col(L["x"], L["geom"], BETA, hbmm.F32, L["W"], L["C"], L["ws"], flags=flags)   # rows I, Q, G
        with torch.cuda.stream(self.sb):
            for L in layers:
                hbmm.conv_im2col(L["xb"], L["geom"], 1, hbmm.F32, L["W"], L["Cb"], L["wsb"], flags=flags)   # rows I, H
        self.ja.record(self.sa)
        self.jb.record(self.sb)
        cur.wait_event(self.ja)
        cur.wait_event(self.jb)


# per layer: gather+binarize+pack (+ weight expansion in the same launch), contraction; NHWC bf16 copy + weight pieces (one launch), HBWN contraction
LAUNCHES_PER_STEP = 4 * (2 + 2)


class E2EPipeline:
    """End-to-end step with host buffers: every step copies every layer's inputs from pinned host memory,
    runs the path through the C ABI and copies both outputs back.  Three streams (upload, compute,
    download) with per-layer events, so that the copies of one layer overlap the kernels of another; a
    layer's device buffers are reused every step, hence the waits on the previous step's events."""

    def __init__(self, torch, layers):
        self.torch = torch
        self.up, self.comp, self.down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        n = len(layers)
        self.in_ready = [torch.cuda.Event() for _ in range(n)]
        self.comp_done = [torch.cuda.Event() for _ in range(n)]
        self.out_done = [torch.cuda.Event() for _ in range(n)]
        self.started = False

    def step(self, hbmm, layers, flags=0):
        torch = self.torch
        for i, L in enumerate(layers):
            with torch.cuda.stream(self.up):
                if self.started:
                    self.up.wait_event(self.comp_done[i])          # the previous step has read these inputs
                L["x"].copy_(L["x_host"], non_blocking=True)
                L["xb"].copy_(L["xb_host"], non_blocking=True)
                self.in_ready[i].record(self.up)
            with torch.cuda.stream(self.comp):
                self.comp.wait_event(self.in_ready[i])
                if self.started:
                    self.comp.wait_event(self.out_done[i])         # the previous step's outputs have left
                hbmm.conv_im2col(L["x"], L["geom"], BETA, hbmm.F32, L["W"], L["C"], L["ws"], flags=flags)
                hbmm.conv_im2col(L["xb"], L["geom"], 1, hbmm.F32, L["W"], L["Cb"], L["wsb"], flags=flags)
                self.comp_done[i].record(self.comp)
            with torch.cuda.stream(self.down):
                self.down.wait_event(self.comp_done[i])
                L["C_host"].copy_(L["C"], non_blocking=True)
                L["Cb_host"].copy_(L["Cb"], non_blocking=True)
                self.out_done[i].record(self.down)
        self.started = True

    def join(self, stream):
        """Makes `stream` wait for everything the three streams have been given."""
        for s in (self.up, self.comp, self.down):
            ev = self.torch.cuda.Event()
            ev.record(s)
            stream.wait_event(ev)


def time_loop(torch, fn, iters: int) -> float:
    """Average milliseconds per call, CUDA events on the current stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def time_rotating(torch, fns, rounds: int) -> float:
    """Average milliseconds per call of a list of equivalent calls on different buffer sets, walked in turn, so
    that a call finds none of its operands in L2 (the sets together exceed it)."""
    for fn in fns:
        fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(rounds):
        for fn in fns:
            fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (rounds * len(fns))


def time_graph(torch, fns, rounds: int, replays: int = 5) -> float:
    """Average milliseconds per call with the calls captured in a CUDA graph (`rounds` passes over `fns`) and
    the graph replayed: for kernels of a few microseconds, whose back-to-back issue from Python (about 10 us
    per call) would otherwise be what is timed.  The library enqueues on the capturing stream and neither
    allocates nor synchronises, so its calls can be captured."""
    for fn in fns:
        fn()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(rounds):
            for fn in fns:
                fn()
    graph.replay()
    return time_loop(torch, graph.replay, replays) / (rounds * len(fns))


def measure_alu_rates(torch, hbmm, clock_reader):
    """Issue rates of the units the two ALU rooflines are built on, from the library's register-only loops:
    32-bit population counts per second and fp32 additions per second over the whole GPU, with the SM clock
    seen while they ran.  `at_max_clock` scales the measured rate by max clock / observed clock."""
    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    sms = props.multi_processor_count
    blocks = sms * 2                       # two blocks of 1024 threads fill a multiprocessor
    sink = torch.empty(blocks * 1024, dtype=torch.int32, device="cuda")
    out = {"sm_count": sms}
    for name, kind, iters in (("popc", hbmm.ALU_POPC, 1 << 15), ("fadd", hbmm.ALU_FADD, 1 << 17), ("ffma", hbmm.ALU_FFMA, 1 << 17)):
        ops = hbmm.bench_alu_rate(kind, blocks, iters, sink)          # warm-up
        for _ in range(2):
            hbmm.bench_alu_rate(kind, blocks, iters, sink)
        best = None
        mhz = []
        for _ in range(5):
            ms = time_loop(torch, lambda: hbmm.bench_alu_rate(kind, blocks, iters, sink), 2)
            best = ms if best is None else min(best, ms)
            c = clock_reader()
            if c:
                mhz.append(c)
        rate = ops / (best * 1e-3)
        sm_mhz = statistics.median(mhz) if mhz else None
        out[name] = {"ops_per_s": rate, "ms_per_launch": best, "ops_per_launch": ops,
                     "per_clk_per_sm": rate / (sms * sm_mhz * 1e6) if sm_mhz else None, "sm_mhz": sm_mhz}
    return out


def read_sm_clock(index: int):
    """(current, max) SM clock in MHz from nvidia-smi, or None."""
    try:
        o = subprocess.run(["nvidia-smi", "-i", str(index), "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits"],
                           capture_output=True, text=True, timeout=10).stdout.strip().split(",")
        return float(o[0]), float(o[1])
    except Exception:
        return None


def kernel_breakdown(torch, hbmm, layers, rounds: int):
    """Per-kernel average launch durations in the launch configuration of the step, L2-cold: every call of a
    family walks a ring of buffer sets (input, workspace, output) that together exceed L2, as in the step,
    where ~0.7 GB pass between two uses of a buffer.  Three timings per layer: the packed front end alone
    (hbmm_conv_im2col_ex with HBMM_CONV_PACK_ONLY: gather + binarize + pack), the HBMM contraction alone
    (hbmm_gemm_ex on the packed operand a front end left in the set's workspace, expanded weights reused),
    and the whole HBWN convolution call (layout copy + contraction: one call, two launches)."""
    out = {"hbmm_contraction": [], "hbwn_conv": [], "front_end_pack": [], "hbmm_conv_call": [], "sets": []}
    PREP = hbmm.CONV_WEIGHTS_PREPARED
    for L in layers:
        s = L["shape"]
        bb, sb, lw, ls = hbmm.operand_bytes(s.M, s.K, BETA, hbmm.F32)
        x_bytes = L["x"].numel() * 4
        c_bytes = s.M * s.N * 4
        per_set = min(x_bytes + bb + sb, bb + sb + c_bytes, L["xb"].numel() * 2 + c_bytes)
        n_sets = max(2, min(32, int(2 * L2_BYTES / per_set) + 1))
        xs = [L["x"]] + [L["x"].clone() for _ in range(n_sets - 1)]
        xbs = [L["xb"]] + [L["xb"].clone() for _ in range(n_sets - 1)]
        wss = [L["ws"]] + [torch.empty_like(L["ws"]) for _ in range(n_sets - 1)]
        wsbs = [L["wsb"]] + [torch.empty_like(L["wsb"]) for _ in range(n_sets - 1)]
        Cs = [L["C"]] + [torch.empty_like(L["C"]) for _ in range(n_sets - 1)]
        for i in range(n_sets):          # every set's workspace gets its own expanded weights and packed operand
            hbmm.conv_im2col(xs[i], L["geom"], BETA, hbmm.F32, L["W"], Cs[i], wss[i])
            hbmm.conv_im2col(xbs[i], L["geom"], 1, hbmm.F32, L["W"], Cs[i], wsbs[i])
        bits_off = (bb + 255) // 256 * 256
        ops_pk = []
        for i in range(n_sets):
            bits = wss[i][:bb].view(torch.int32).reshape(s.M, lw)
            scales = wss[i][bits_off: bits_off + sb].view(torch.float32).reshape(s.M, ls)
            ops_pk.append(hbmm.wrap_packed(bits, scales, s.K, BETA))
        gws_off = (bits_off + sb + 255) // 256 * 256
        gws = [wss[i][gws_off:] for i in range(n_sets)]
        t_front = time_rotating(torch, [
            (lambda i=i: hbmm.conv_im2col(xs[i], L["geom"], BETA, hbmm.F32, L["W"], None, wss[i], flags=PREP | hbmm.CONV_PACK_ONLY))
            for i in range(n_sets)], rounds)
        t_gemm = time_rotating(torch, [
            (lambda i=i: hbmm.gemm_ex(ops_pk[i], L["W"], Cs[i], hbmm.PATH_FOLDED_PREPARED, gws[i])) for i in range(n_sets)], rounds)
        t_call = time_rotating(torch, [
            (lambda i=i: hbmm.conv_im2col(xs[i], L["geom"], BETA, hbmm.F32, L["W"], Cs[i], wss[i], flags=PREP)) for i in range(n_sets)], rounds)
        t_hbwn = time_rotating(torch, [
            (lambda i=i: hbmm.conv_im2col(xbs[i], L["geom"], 1, hbmm.F32, L["W"], Cs[i], wsbs[i], flags=PREP)) for i in range(n_sets)], rounds)
        out["front_end_pack"].append(t_front)
        out["hbmm_contraction"].append(t_gemm)
        out["hbmm_conv_call"].append(t_call)
        out["hbwn_conv"].append(t_hbwn)
        out["sets"].append(n_sets)
        del xs, xbs, wss, wsbs, Cs, ops_pk, gws
    return out


def side_measurements(torch, hbmm, inputs, peaks, iters: int):
    """Rows of the hot path that the convolution step only runs in fused form, timed on their own on the
    conv3_x matrix view (M = 50176, K = 1152, N = 128; 231 MB of fp32 input, larger than L2):
    hbmm_quantize alone (HBM bound), the gradient through the binarization (Eq. 6, HBM bound: 8 bytes read
    and 4 written per element), and the folded-scale contraction at the sub-word group sizes of the
    paper's experiments.  Reported beside the step, not part of it."""
    hbm_gbs, bf16_tflops, _ = peaks
    M, N, K = 50176, 128, 1152
    g = torch.Generator(device="cuda")
    g.manual_seed(19160)
    a = torch.randn((M, K), device="cuda", generator=g)
    w = torch.randn((N, K), device="cuda", generator=g) * (2.0 / K) ** 0.5
    out = []
    for beta in (32, 4):
        A = hbmm.alloc_operand(M, K, beta, hbmm.F32)
        ms = time_loop(torch, lambda: hbmm.quantize(a, A), iters)
        by = 4.0 * M * K + A.bits.numel() * 4.0 + A.scales.numel() * 4.0
        out.append({"kernel": "hbmm_quantize/beta%d" % beta, "shape": [M, K], "ms": round(ms, 5), "bound": "hbm",
                    "achieved": by / (ms * 1e-3) / 1e9, "peak": hbm_gbs, "unit": "GB/s", "frac": by / (ms * 1e-3) / 1e9 / hbm_gbs})
    gy = torch.randn((M, K), device="cuda", generator=g)
    gx = torch.empty_like(a)
    for beta in (4, 32):
        ms = time_loop(torch, lambda: hbmm.binarize_backward(a, gy, beta, gx), iters)
        by = 12.0 * M * K
        out.append({"kernel": "hbmm_binarize_backward/beta%d" % beta, "shape": [M, K], "ms": round(ms, 5), "bound": "hbm",
                    "achieved": by / (ms * 1e-3) / 1e9, "peak": hbm_gbs, "unit": "GB/s", "frac": by / (ms * 1e-3) / 1e9 / hbm_gbs})
    # Eq. 3 on a conv2_x-shaped activation map (256 x 64 x 56 x 56 fp32, beyond L2): lines of 56, groups of 8
    amap = torch.randn((256 * 64 * 56, 56), device="cuda", generator=g)
    for odt, name, ob in ((hbmm.BF16, "bf16", 2.0), (hbmm.F32, "f32", 4.0)):
        om = torch.empty(amap.shape, device="cuda", dtype=torch.bfloat16 if odt == hbmm.BF16 else torch.float32)
        ms = time_loop(torch, lambda: hbmm.binarize_dense(amap, 8, odt, om), iters)
        by = (4.0 + ob) * amap.numel()
        out.append({"kernel": "hbmm_binarize_dense/beta8_%s" % name, "shape": list(amap.shape), "ms": round(ms, 5), "bound": "hbm",
                    "achieved": by / (ms * 1e-3) / 1e9, "peak": hbm_gbs, "unit": "GB/s", "frac": by / (ms * 1e-3) / 1e9 / hbm_gbs})
    for ba, bw in ((16, 16), (8, 8), (4, 4), (2, 16)):
        A = hbmm.quantize(a, hbmm.alloc_operand(M, K, ba, hbmm.F32))
        W = hbmm.quantize(w, hbmm.alloc_operand(N, K, bw, hbmm.F32))
        ws = torch.empty(max(hbmm.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
        C = torch.empty((M, N), device="cuda")
        hbmm.gemm_ex(A, W, C, hbmm.PATH_FOLDED, ws)
        ms = time_loop(torch, lambda: hbmm.gemm_ex(A, W, C, hbmm.PATH_FOLDED_PREPARED, ws), iters)
        ach = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        out.append({"kernel": "hbmm_fold_kernel/beta_a%d_beta_w%d" % (ba, bw), "shape": [M, N, K], "ms": round(ms, 5), "bound": "tensor",
                    "achieved": ach, "peak": bf16_tflops, "unit": "TFLOP/s", "frac": ach / bf16_tflops})
        if ba != 8:
            # the same product with no workspace: masked popcounts on the integer pipe, one multiply-add per output and group
            msp = time_loop(torch, lambda: hbmm.gemm_ex(A, W, C, hbmm.PATH_POPC), max(3, iters // 4))
            out.append({"kernel": "gemm_popc_sub_kernel (no workspace)/beta_a%d_beta_w%d" % (ba, bw), "shape": [M, N, K], "ms": round(msp, 5),
                        "tops": 2.0 * M * N * K / (msp * 1e-3) / 1e12, "multiply_adds_per_output": K // min(ba, bw)})
    # the whole convolution call (packing front end + contraction) on conv3_x at the group sizes of the paper's experiments
    # (Section 5: beta_a / beta_w = 16/16, 4/4, 2/16) and at 64/64, beside 32/32
    sh3 = inputs.resnet18_convs(64)[1]
    x3 = torch.randn((sh3.B, sh3.C, sh3.H, sh3.W), device="cuda", generator=g)
    geomc = hbmm.make_geom(sh3.B, sh3.C, sh3.H, sh3.W, 3, 3, (1, 1), (1, 1))
    c3 = torch.empty((sh3.M, sh3.N), device="cuda")
    for ba, bw in ((32, 32), (64, 64), (16, 16), (4, 4), (2, 16)):
        W3 = hbmm.quantize(w, hbmm.alloc_operand(N, K, bw, hbmm.F32))
        ws3 = torch.empty(hbmm.conv_workspace_bytes(geomc, ba, hbmm.F32, W3), dtype=torch.uint8, device="cuda")
        hbmm.conv_im2col(x3, geomc, ba, hbmm.F32, W3, c3, ws3)
        ms = time_loop(torch, lambda: hbmm.conv_im2col(x3, geomc, ba, hbmm.F32, W3, c3, ws3, flags=hbmm.CONV_WEIGHTS_PREPARED), iters)
        msp = time_loop(torch, lambda: hbmm.conv_im2col(x3, geomc, ba, hbmm.F32, W3, None, ws3,
                                                        flags=hbmm.CONV_WEIGHTS_PREPARED | hbmm.CONV_PACK_ONLY), iters)
        out.append({"kernel": "hbmm_conv_im2col/conv3_x/beta_a%d_beta_w%d" % (ba, bw), "shape": [M, N, K], "ms": round(ms, 5),
                    "ms_front_end_alone": round(msp, 5), "tops": 2.0 * M * N * K / (ms * 1e-3) / 1e12})
    del x3, c3
    # AlexNet-style fully connected layer at batch 256 (4096 -> 4096, beta 64): product + binarization of its
    # rows for the next layer, as two calls (fp32 product stored, then hbmm_quantize) and fused in the epilogue
    Mf, Kf, Nf, bf = 256, 4096, 4096, 64
    af = torch.randn((Mf, Kf), device="cuda", generator=g)
    wf = torch.randn((Nf, Kf), device="cuda", generator=g) * (2.0 / Kf) ** 0.5
    Af = hbmm.quantize(af, hbmm.alloc_operand(Mf, Kf, bf, hbmm.F32))
    Wf = hbmm.quantize(wf, hbmm.alloc_operand(Nf, Kf, bf, hbmm.F32))
    wsf = torch.empty(max(hbmm.gemm_workspace_bytes(Af, Wf), 16), dtype=torch.uint8, device="cuda")
    Cf = torch.empty((Mf, Nf), device="cuda")
    nxt = hbmm.alloc_operand(Mf, Nf, bf, hbmm.F32)

    def two_calls():
        hbmm.gemm(Af, Wf, Cf, wsf)
        hbmm.quantize(Cf, nxt)

    ms2 = time_loop(torch, two_calls, iters)
    ms1 = time_loop(torch, lambda: hbmm.gemm_binarize_next(Af, Wf, nxt, wsf), iters)
    out.append({"kernel": "fc_4096x4096_b256_beta64: hbmm_gemm + hbmm_quantize", "shape": [Mf, Nf, Kf], "ms": round(ms2, 5)})
    out.append({"kernel": "fc_4096x4096_b256_beta64: hbmm_gemm_binarize_next", "shape": [Mf, Nf, Kf], "ms": round(ms1, 5)})
    # conv2_x with the activations grouped along map rows (Eq. 3 as printed): binarize the map, then the HBWN convolution
    Bc, Cc, Hc, Nc = 64, 64, 56, 64
    xm = torch.randn((Bc, Cc, Hc, Hc), device="cuda", generator=g)
    wc = torch.randn((Nc, Cc * 9), device="cuda", generator=g) * (2.0 / (Cc * 9)) ** 0.5
    Wc = hbmm.quantize(wc, hbmm.alloc_operand(Nc, Cc * 9, BETA, hbmm.F32))
    geom = hbmm.make_geom(Bc, Cc, Hc, Hc, 3, 3, (1, 1), (1, 1))
    wsc = torch.empty(hbmm.conv_workspace_bytes(geom, 1, hbmm.F32, Wc), dtype=torch.uint8, device="cuda")
    Cc_out = torch.empty((Bc * Hc * Hc, Nc), device="cuda")
    am = torch.empty((Bc * Cc * Hc, Hc), device="cuda", dtype=torch.bfloat16)

    def eq3_conv(flags):
        hbmm.binarize_dense(xm.view(Bc * Cc * Hc, Hc), 8, hbmm.BF16, am)
        hbmm.conv_im2col(am.view(Bc, Cc, Hc, Hc), geom, 1, hbmm.F32, Wc, Cc_out, wsc, flags=flags)

    eq3_conv(0)
    ms3 = time_loop(torch, lambda: eq3_conv(hbmm.CONV_WEIGHTS_PREPARED), iters)
    ach = 2.0 * Bc * Hc * Hc * Nc * Cc * 9 / (ms3 * 1e-3) / 1e12
    out.append({"kernel": "conv2_x_eq3_grouping_beta_a8: hbmm_binarize_dense + hbmm_conv_im2col(beta_a=1)", "shape": [Bc * Hc * Hc, Nc, Cc * 9],
                "ms": round(ms3, 5), "bound": "tensor", "achieved": ach, "peak": bf16_tflops, "unit": "TFLOP/s", "frac": ach / bf16_tflops})
    del xm, am, Cc_out, amap, a, gy, gx
    # Two dense-activation convolutions (conv3_x -> conv3_x) with ReLU and the next block's batch-norm map between them:
    # chained through the epilogue (NHWC bf16 written by layer 1, read directly by layer 2) against the unfused
    # sequence (fp32 NHWC product, the map / rounding / NHWC -> NCHW permutation as torch element-wise kernels, then the
    # second convolution with its own layout copy).
    sh = inputs.resnet18_convs(64)[1]
    xc = torch.randn((sh.B, sh.C, sh.H, sh.W), device="cuda", generator=g).to(torch.bfloat16)
    W1 = hbmm.quantize(torch.randn((sh.N, sh.K), device="cuda", generator=g) * (2.0 / sh.K) ** 0.5, hbmm.alloc_operand(sh.N, sh.K, BETA, hbmm.F32))
    W2 = hbmm.quantize(torch.randn((sh.N, sh.N * 9), device="cuda", generator=g) * (2.0 / (sh.N * 9)) ** 0.5, hbmm.alloc_operand(sh.N, sh.N * 9, BETA, hbmm.F32))
    bs = torch.rand(sh.N, device="cuda", generator=g) + 0.5
    bh = torch.randn(sh.N, device="cuda", generator=g) * 0.2
    geom3 = hbmm.make_geom(sh.B, sh.C, sh.H, sh.W, 3, 3, (1, 1), (1, 1))
    ws1 = torch.empty(hbmm.conv_workspace_bytes(geom3, 1, hbmm.F32, W1), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(hbmm.conv_workspace_bytes(geom3, 1, hbmm.F32, W2), dtype=torch.uint8, device="cuda")
    zc = torch.empty((sh.M, sh.N), device="cuda", dtype=torch.bfloat16)
    c1 = torch.empty((sh.M, sh.N), device="cuda")
    c2 = torch.empty((sh.M, sh.N), device="cuda")
    epc = hbmm.make_epilogue(hbmm.ACT_RELU, bs, bh, out=zc)
    PREPF = hbmm.CONV_WEIGHTS_PREPARED

    def chain_fused(flags):
        hbmm.conv_im2col_fused(xc, geom3, 1, hbmm.F32, W1, epc, ws1, flags=flags)
        hbmm.conv_im2col(zc.view(sh.B, sh.H, sh.W, sh.N), geom3, 1, hbmm.F32, W2, c2, ws2, flags=flags | hbmm.CONV_INPUT_NHWC)

    def chain_unfused(flags):
        hbmm.conv_im2col(xc, geom3, 1, hbmm.F32, W1, c1, ws1, flags=flags)
        zt = (torch.relu(c1) * bs + bh).to(torch.bfloat16).view(sh.B, sh.H, sh.W, sh.N).permute(0, 3, 1, 2).contiguous()
        hbmm.conv_im2col(zt, geom3, 1, hbmm.F32, W2, c2, ws2, flags=flags)

    chain_fused(0)
    ms_f = time_loop(torch, lambda: chain_fused(PREPF), iters)
    chain_unfused(0)
    ms_u = time_loop(torch, lambda: chain_unfused(PREPF), iters)
    out.append({"kernel": "conv3_x -> relu -> bn -> conv3_x (bf16 activations): chained through the epilogue, 2 launches", "ms": round(ms_f, 5),
                "tflops": 4.0 * sh.M * sh.N * sh.K / (ms_f * 1e-3) / 1e12})
    out.append({"kernel": "conv3_x -> relu -> bn -> conv3_x (bf16 activations): unfused (fp32 product, torch element-wise + permute, layout copy)",
                "ms": round(ms_u, 5), "tflops": 4.0 * sh.M * sh.N * sh.K / (ms_u * 1e-3) / 1e12})
    del xc, zc, c1, c2, ws1, ws2
    # Exact-scale variants on the four convolution matrices (seeded device-generated operands of the same shapes):
    # HBMM with integer group dots and a per-group fp32 scale step (HBMM_PATH_TENSOR) beside the default
    # folded-scale kernel, and HBWN on the dense bf16 im2col matrix with three bf16 weight pieces (scales to 2^-26,
    # HBMM_PATH_TENSOR) beside two pieces (HBMM_PATH_FOLDED).
    for sh in inputs.resnet18_convs(64):
        a = torch.randn((sh.M, sh.K), device="cuda", generator=g)
        w = torch.randn((sh.N, sh.K), device="cuda", generator=g) * (2.0 / sh.K) ** 0.5
        A = hbmm.quantize(a, hbmm.alloc_operand(sh.M, sh.K, BETA, hbmm.F32))
        W = hbmm.quantize(w, hbmm.alloc_operand(sh.N, sh.K, BETA, hbmm.F32))
        C = torch.empty((sh.M, sh.N), device="cuda")
        ws = torch.empty(max(hbmm.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
        ops = 2.0 * sh.M * sh.N * sh.K
        for label, first, again in (("hbmm_umma_kernel (e4m3 operands, per-group fp32 scale step)", hbmm.PATH_TENSOR, hbmm.PATH_TENSOR_PREPARED),
                                    ("hbmm_fold_kernel (default)", hbmm.PATH_FOLDED, hbmm.PATH_FOLDED_PREPARED),
                                    ("gemm_popc_kernel (integer pipe, no workspace)", hbmm.PATH_POPC, hbmm.PATH_POPC)):
            hbmm.gemm_ex(A, W, C, first, ws)
            ms = time_loop(torch, lambda: hbmm.gemm_ex(A, W, C, again, ws), iters)
            out.append({"kernel": "%s/%s" % (label, sh.name), "shape": [sh.M, sh.N, sh.K], "ms": round(ms, 5),
                        "tops": ops / (ms * 1e-3) / 1e12, "timing": "L2-warm loop on one operand set"})
        Ad = hbmm.wrap_dense(a.to(torch.bfloat16))
        wsd = torch.empty(max(hbmm.gemm_workspace_bytes(Ad, W), 16), dtype=torch.uint8, device="cuda")
        for label, first, again in (("hbwn_umma_kernel, three weight pieces (dense bf16 rows)", hbmm.PATH_TENSOR, hbmm.PATH_TENSOR_PREPARED),
                                    ("hbwn_umma_kernel, two weight pieces (dense bf16 rows)", hbmm.PATH_FOLDED, hbmm.PATH_FOLDED_PREPARED),
                                    ("hbwn_select_kernel (fp32 sign-select, no workspace)", hbmm.PATH_POPC, hbmm.PATH_POPC)):
            hbmm.gemm_ex(Ad, W, C, first, wsd)
            ms = time_loop(torch, lambda: hbmm.gemm_ex(Ad, W, C, again, wsd), iters if first != hbmm.PATH_POPC else max(2, iters // 4))
            out.append({"kernel": "%s/%s" % (label, sh.name), "shape": [sh.M, sh.N, sh.K], "ms": round(ms, 5),
                        "tflops": ops / (ms * 1e-3) / 1e12, "timing": "L2-warm loop on one operand set"})
        del a, A, C, ws, Ad, wsd
    return out


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (same kernels, same workload); entries are dropped when a kernel changes after its capture.
NCU_DRAM_BYTES = {
    ("hbmm_contraction", "conv2_x"): 32.340e6 + 1.998e6,     # profiles/conv2_x_conv3_x_kernels.md
    ("hbmm_contraction", "conv3_x"): 15.174e6 + 0.314e6,
    ("hbwn_conv", "conv2_x"): 25.998e6 + 3.054e6,            # the contraction kernel of the call (the layout copy is a launch of its own)
    ("hbwn_conv", "conv3_x"): 13.531e6 + 0.005e6,
    ("front_end_pack", "conv2_x"): 51.502e6 + 2.789e6,
    ("front_end_pack", "conv3_x"): 25.837e6,
}


def hbmm_bytes(M, N, K, beta, scale_bytes=4):
    """Algorithmic bytes of a packed x packed product: both packed operands once, the fp32 result once."""
    G = -(-K // beta)
    return M * K / 8.0 + M * G * scale_bytes + N * K / 8.0 + N * G * scale_bytes + 4.0 * M * N


def popc_hbm_roofline(M, N, K, beta, scale_bytes, rates, hbm_gbs):
    """Seconds: the larger of the bytes at the HBM copy bandwidth and one population count per output and
    K-word at the measured population-count rate (and at that rate scaled to the maximum SM clock)."""
    t_hbm = hbmm_bytes(M, N, K, beta, scale_bytes) / (hbm_gbs * 1e9)
    words = M * N * float(-(-K // 32))
    t_popc = words / rates["popc"]["ops_per_s"]
    t_popc_max = words / rates["popc"]["ops_per_s_at_max_clock"]
    return {"t_hbm_us": t_hbm * 1e6, "t_popc_us": t_popc * 1e6, "t_roof_us": max(t_hbm, t_popc) * 1e6,
            "t_roof_us_at_max_clock": max(t_hbm, t_popc_max) * 1e6, "bound": "hbm" if t_hbm > t_popc else "popc"}


def roofline_for(kind: str, li: int, shape, ms: float, peaks, rates):
    """Roofline entry of one kernel launch (layer li) given its measured duration.

    Both contractions run on the tensor cores (HBMM: two fp16 pieces per operand carrying sign and group
    scale; HBWN: bf16 activations x two bf16 weight pieces), so they are set against the measured dense
    16-bit GEMM peak.  `achieved` counts the ALGORITHMIC operations 2 M N K; the HBMM kernel issues three
    times that on the tensor pipe (three cross products of the operands' pieces), the HBWN kernel twice:
    `frac_of_peak_in_issued_tensor_work` is `frac` times that factor, i.e. how busy the tensor pipe is with
    the work the formulation gives it.  Beside it: the fraction of the
    popcount / HBM roofline for HBMM (one population count per output and K-word at the MEASURED rate of the
    integer pipe, or the algorithmic bytes at the HBM copy bandwidth, whichever is slower) and of the fp32-add
    / HBM roofline for HBWN (one addition per output and K-element at the measured rate)."""
    hbm_gbs, bf16_tflops, hbm_src = peaks
    M, N, K = shape.M, shape.N, shape.K
    G = -(-K // BETA)
    if kind == "hbmm_contraction":
        ops = 2.0 * M * N * K
        ach = ops / (ms * 1e-3) / 1e12
        rf = popc_hbm_roofline(M, N, K, BETA, 4, rates, hbm_gbs)
        return {"kernel": "hbmm_fold_kernel/%s" % shape.name, "bound": "tensor", "achieved": ach,
                "peak": bf16_tflops, "unit": "TFLOP/s", "frac": ach / bf16_tflops, "traffic": None,
                "peak_source": "%s bf16 GEMM peak (fp16 operands, same rate)" % hbm_src,
                "tensor_pipe_work_factor": 3, "frac_of_peak_in_issued_tensor_work": 3 * ach / bf16_tflops,
                "frac_of_popcount_hbm_roofline": rf["t_roof_us"] / (ms * 1e3),
                "frac_of_popcount_hbm_roofline_at_max_clock": rf["t_roof_us_at_max_clock"] / (ms * 1e3),
                "popcount_hbm_roofline": rf, "timing": "L2-cold (ring of buffer sets larger than L2), weights already expanded"}
    if kind == "hbwn_conv":
        # the whole HBWN call (layout copy + weight pieces + contraction) set against the contraction's flops
        ops = 2.0 * M * N * K
        ach = ops / (ms * 1e-3) / 1e12
        by = 2.0 * shape.B * shape.C * shape.H * shape.W + N * K / 8.0 + 4.0 * N * G + 4.0 * M * N
        t_roof = max(by / (hbm_gbs * 1e9), M * N * float(K) / rates["fadd"]["ops_per_s"])
        return {"kernel": "hbwn tcgen05 kernels (layout copy + contraction)/%s" % shape.name, "bound": "tensor", "achieved": ach,
                "peak": bf16_tflops, "unit": "TFLOP/s", "frac": ach / bf16_tflops, "traffic": None,
                "peak_source": "%s bf16 GEMM peak" % hbm_src, "tensor_pipe_work_factor": 2,
                "frac_of_peak_in_issued_tensor_work": 2 * ach / bf16_tflops,
                "frac_of_fp32_add_hbm_roofline": t_roof / (ms * 1e-3), "timing": "L2-cold, whole call (layout copy + contraction)"}
    x_bytes = 4.0 * shape.B * shape.C * shape.H * shape.W
    lw = ((K + 31) // 32 + 3) // 4 * 4
    ls = (G + 3) // 4 * 4
    by = x_bytes + M * lw * 4.0 + M * ls * 4.0
    if kind == "hbmm_conv_call":
        by += N * K / 8.0 + 4.0 * N * G + 4.0 * M * N - (M * lw * 4.0 + M * ls * 4.0)   # the packed operand is internal to the call
        rf = popc_hbm_roofline(M, N, K, BETA, 4, rates, hbm_gbs)
        t_roof = max(by / (hbm_gbs * 1e9), rf["t_popc_us"] * 1e-6)
        ach = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        return {"kernel": "hbmm_conv_im2col/%s" % shape.name, "bound": "tensor", "achieved": ach, "peak": bf16_tflops,
                "unit": "TFLOP/s", "frac": ach / bf16_tflops, "traffic": None,
                "frac_of_popcount_hbm_roofline": t_roof / (ms * 1e-3), "timing": "L2-cold, whole call (front end + contraction)"}
    return {"kernel": "%s/%s" % (kind, shape.name), "bound": "hbm", "achieved": by / (ms * 1e-3) / 1e9,
            "peak": hbm_gbs, "unit": "GB/s", "frac": by / (ms * 1e-3) / 1e9 / hbm_gbs, "traffic": None,
            "peak_source": "%s HBM copy bandwidth" % hbm_src, "timing": "L2-cold, front end alone (HBMM_CONV_PACK_ONLY)"}


# ----------------------------------------------------------------------------- the five configurations, one by one
def cublas_context(torch, M, N, K, iters):
    """torch.matmul of the same shape in fp32 (TF32 off: the analogue of the paper's full-precision multiply)
    and in bf16, milliseconds per call; library GEMMs, timed for context only."""
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        a = torch.randn((M, K), device="cuda")
        w = torch.randn((N, K), device="cuda")
        c = torch.empty((M, N), device="cuda")
        for _ in range(2):
            torch.matmul(a, w.t(), out=c)
        ms32 = time_loop(torch, lambda: torch.matmul(a, w.t(), out=c), iters)
        ab, wb = a.to(torch.bfloat16), w.to(torch.bfloat16)
        cb = torch.empty((M, N), device="cuda", dtype=torch.bfloat16)
        for _ in range(2):
            torch.matmul(ab, wb.t(), out=cb)
        msb = time_loop(torch, lambda: torch.matmul(ab, wb.t(), out=cb), iters)
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    return {"fp32_ms": round(ms32, 5), "bf16_ms": round(msb, 5),
            "fp32_tflops": 2.0 * M * N * K / (ms32 * 1e-3) / 1e12, "bf16_tflops": 2.0 * M * N * K / (msb * 1e-3) / 1e12}


def oracle_row_sample(oracle, a_rows, w, beta_a, beta_w, M, hbwn=False):
    """The CPU checker as it stands on a row sample of the shape: seconds for the sample and the time for all M
    rows extrapolated by rows (labelled as such)."""
    t0 = time.perf_counter()
    if hbwn:
        oracle.hbwn(a_rows, w, beta_w, "f32")
    else:
        oracle.hbmm(a_rows, w, beta_a, beta_w, "f32")
    dt = time.perf_counter() - t0
    r = a_rows.shape[0]
    return {"sample_rows": r, "sample_s": round(dt, 4), "full_ms_row_extrapolated": dt * 1e3 * M / r, "cores": oracle.num_threads()}


def sample_rows_for(M, N, K, budget_macs=1.2e9):
    return int(max(1, min(M, budget_macs / (float(N) * K))))


def product_row(torch, hbmm, name, M, N, K, beta, sdt, a_dev, w_dev, rates, peaks, iters, with_quantize=True):
    """One packed x packed product of a configuration: hbmm_quantize of the activation matrix alone, hbmm_gemm
    alone on the packed operands (weights expanded once, outside the timing), against the popcount / HBM
    roofline.  Products whose operands and result fit L2 are timed over a ring of operand / result sets."""
    hbm_gbs, bf16_tflops, _ = peaks
    sb = 4 if sdt == hbmm.F32 else 2
    W = hbmm.quantize(w_dev, hbmm.alloc_operand(N, K, beta, sdt))
    row = {"name": name, "M": M, "N": N, "K": K, "beta": beta, "scale_dtype": "f32" if sdt == hbmm.F32 else "bf16"}
    by = hbmm_bytes(M, N, K, beta, sb)
    n_sets = max(1, min(16, int(2 * L2_BYTES / by) + 1)) if by < 2 * L2_BYTES else 1
    As = [hbmm.quantize(a_dev, hbmm.alloc_operand(M, K, beta, sdt)) for _ in range(n_sets)]
    Cs = [torch.empty((M, (N + 3) // 4 * 4), device="cuda") for _ in range(n_sets)]
    nws = max(hbmm.gemm_workspace_bytes(As[0], W), 16)
    wss = [torch.empty(nws, dtype=torch.uint8, device="cuda") for _ in range(n_sets)]
    gemv = M <= 8
    if gemv:
        # a handful of rows: the matrix-vector kernel reads the packed weights; its ring rotates weight copies too
        Ws = [W] + [hbmm.quantize(w_dev, hbmm.alloc_operand(N, K, beta, sdt)) for _ in range(n_sets - 1)]
        fns = [(lambda i=i: hbmm.gemm(As[i], Ws[i], Cs[i], wss[i])) for i in range(n_sets)]
        path = "gemv_popc_kernel"
    else:
        for i in range(n_sets):
            hbmm.gemm(As[i], W, Cs[i], wss[i])                 # leaves the expanded weights in each workspace
        auto_folded = min(beta, K) <= 128
        prepared = hbmm.PATH_FOLDED_PREPARED if auto_folded else hbmm.PATH_TENSOR_PREPARED
        fns = [(lambda i=i: hbmm.gemm_ex(As[i], W, Cs[i], prepared, wss[i])) for i in range(n_sets)]
        path = "hbmm_fold_kernel" if auto_folded else "hbmm_umma_kernel"
    small = 2.0 * M * N * K < 4e9                      # a few microseconds of work: time inside a CUDA graph
    ms = time_graph(torch, fns, max(2, 40 // n_sets)) if small else time_rotating(torch, fns, max(2, iters // n_sets))
    rf = popc_hbm_roofline(M, N, K, beta, sb, rates, hbm_gbs)
    row.update({"kernel": path, "hbmm_gemm_ms": round(ms, 5), "tops": 2.0 * M * N * K / (ms * 1e-3) / 1e12,
                "gbs": by / (ms * 1e-3) / 1e9, "roofline_bound": rf["bound"], "t_roof_us": round(rf["t_roof_us"], 3),
                "frac_of_popcount_hbm_roofline": rf["t_roof_us"] / (ms * 1e3),
                "frac_of_popcount_hbm_roofline_at_max_clock": rf["t_roof_us_at_max_clock"] / (ms * 1e3),
                "frac_of_bf16_tensor_peak": 2.0 * M * N * K / (ms * 1e-3) / 1e12 / bf16_tflops, "buffer_sets": n_sets,
                "timing": "CUDA graph replay" if small else "stream of launches"})
    if with_quantize:
        qs = [hbmm.alloc_operand(M, K, beta, sdt) for _ in range(n_sets)]
        x_copies = [a_dev] + [a_dev.clone() for _ in range(n_sets - 1)] if 4.0 * M * K < 2 * L2_BYTES else [a_dev] * n_sets
        qfns = [(lambda i=i: hbmm.quantize(x_copies[i], qs[i])) for i in range(n_sets)]
        msq = time_graph(torch, qfns, max(2, 40 // n_sets)) if 4.0 * M * K < 64e6 else time_rotating(torch, qfns, max(2, iters // n_sets))
        G = -(-K // beta)
        byq = 4.0 * M * K + M * K / 8.0 + M * G * sb
        row.update({"hbmm_quantize_ms": round(msq, 5), "quantize_gbs": byq / (msq * 1e-3) / 1e9,
                    "quantize_frac_of_hbm": byq / (msq * 1e-3) / 1e9 / hbm_gbs})
    return row


def config_rows(torch, hbmm, inputs, layers, brk, rates, peaks, iters):
    """Every configuration of the workload list on its own: the 256-cube, the square sweep (two sizes x three
    group sizes x two scale storage types), the four convolution shapes as HBMM and as HBWN (from the kernel
    breakdown), and the fully connected stack at batch 256 and batch 1.  Each row: time, effective binary
    TOPS, algorithmic GB/s, fraction of its roofline, a library GEMM of the same shape in fp32 and bf16, and
    the CPU checker on a row sample of the same shape."""
    import oracle
    oracle.build()
    rows = []
    hbm_gbs, bf16_tflops, _ = peaks
    # --- 256-cube
    a = inputs.normal((256, 256), inputs.SEEDS["square256"][0])
    w = inputs.normal((256, 256), inputs.SEEDS["square256"][1])
    r = product_row(torch, hbmm, "square256", 256, 256, 256, 32, hbmm.F32, torch.from_numpy(a).cuda(), torch.from_numpy(w).cuda(),
                    rates, peaks, 200)
    r["note"] = "0.1 us of roofline time: launch latency decides"
    r["cublas"] = cublas_context(torch, 256, 256, 256, 100)
    r["oracle"] = oracle_row_sample(oracle, a, w, 32, 32, 256)
    rows.append(r)
    # --- square sweep
    for n in (4096, 8192):
        a = inputs.normal((n, n), inputs.SEEDS["square_sweep"][0] + n // 4096)
        w = inputs.normal((n, n), inputs.SEEDS["square_sweep"][1] + n // 4096)
        ad, wd = torch.from_numpy(a).cuda(), torch.from_numpy(w).cuda()
        cub = cublas_context(torch, n, n, n, 5 if n == 4096 else 3)
        sr = sample_rows_for(n, n, n)
        orc = {}
        for beta in (32, 64, 128):
            orc[beta] = oracle_row_sample(oracle, a[:sr], w, beta, beta, n)
            for sdt in (hbmm.F32, hbmm.BF16):
                r = product_row(torch, hbmm, "square%d" % n, n, n, n, beta, sdt, ad, wd, rates, peaks, 10 if n == 4096 else 4)
                r["cublas"] = cub
                r["oracle"] = orc[beta]
                rows.append(r)
        del ad, wd
    # --- the convolution shapes, from the breakdown of the timed step's calls
    for i, L in enumerate(layers):
        sh = L["shape"]
        cub = cublas_context(torch, sh.M, sh.N, sh.K, 10)
        sr = sample_rows_for(sh.M, sh.N, sh.K, 6e8)
        b = max(1, -(-sr // (sh.M // sh.B)))
        sub = inputs.ConvShape(sh.name, b, sh.C, sh.H, sh.W, sh.N)
        xa = oracle.im2col(inputs.conv_activation(sub, inputs.SEEDS["resnet_hbmm"][0] + i), sh.kh, sh.kw, (1, 1), (1, 1))[:sr]
        wh = inputs.he_normal(sh.N, sh.K, inputs.SEEDS["resnet_hbmm"][1] + i)
        rf = popc_hbm_roofline(sh.M, sh.N, sh.K, BETA, 4, rates, hbm_gbs)
        ms = brk["hbmm_contraction"][i]
        rows.append({"name": "resnet18_%s_hbmm" % sh.name, "M": sh.M, "N": sh.N, "K": sh.K, "beta": BETA, "scale_dtype": "f32",
                     "kernel": "hbmm_fold_kernel", "hbmm_gemm_ms": round(ms, 5), "tops": 2.0 * sh.M * sh.N * sh.K / (ms * 1e-3) / 1e12,
                     "gbs": hbmm_bytes(sh.M, sh.N, sh.K, BETA) / (ms * 1e-3) / 1e9, "roofline_bound": rf["bound"],
                     "t_roof_us": round(rf["t_roof_us"], 3), "frac_of_popcount_hbm_roofline": rf["t_roof_us"] / (ms * 1e3),
                     "frac_of_popcount_hbm_roofline_at_max_clock": rf["t_roof_us_at_max_clock"] / (ms * 1e3),
                     "front_end_ms": round(brk["front_end_pack"][i], 5), "conv_call_ms": round(brk["hbmm_conv_call"][i], 5),
                     "conv_call_frac_of_popcount_hbm_roofline": roofline_for("hbmm_conv_call", i, sh, brk["hbmm_conv_call"][i], peaks, rates)["frac_of_popcount_hbm_roofline"],
                     "cublas": cub, "oracle": oracle_row_sample(oracle, xa, wh, BETA, BETA, sh.M)})
        _, xab = inputs.as_bf16(xa)
        msb = brk["hbwn_conv"][i]
        rows.append({"name": "resnet18_%s_hbwn" % sh.name, "M": sh.M, "N": sh.N, "K": sh.K, "beta_w": BETA, "activation_dtype": "bf16",
                     "kernel": "nhwc copy + hbwn_umma_kernel", "conv_call_ms": round(msb, 5),
                     "tops": 2.0 * sh.M * sh.N * sh.K / (msb * 1e-3) / 1e12,
                     "frac_of_fp32_add_hbm_roofline": roofline_for("hbwn_conv", i, sh, msb, peaks, rates)["frac_of_fp32_add_hbm_roofline"],
                     "frac_of_bf16_tensor_peak": 2.0 * sh.M * sh.N * sh.K / (msb * 1e-3) / 1e12 / bf16_tflops,
                     "cublas": cub, "oracle": oracle_row_sample(oracle, xab, wh, 1, BETA, sh.M, hbwn=True)})
    # --- fully connected stack, scale groups of 64
    for batch in (256, 1):
        stack = []
        for i, (K, N) in enumerate(inputs.ALEXNET_FC):
            a = inputs.normal((batch, K), inputs.SEEDS["alexnet_fc"][0] + i)
            w = inputs.he_normal(N, K, inputs.SEEDS["alexnet_fc"][1] + i)
            ad, wd = torch.from_numpy(a).cuda(), torch.from_numpy(w).cuda()
            r = product_row(torch, hbmm, "alexnet_fc%d_b%d" % (6 + i, batch), batch, N, K, 64, hbmm.F32, ad, wd, rates, peaks, 60)
            r["cublas"] = cublas_context(torch, batch, N, K, 30)
            r["oracle"] = oracle_row_sample(oracle, a[:sample_rows_for(batch, N, K)], w, 64, 64, batch)
            rows.append(r)
            A = hbmm.quantize(ad, hbmm.alloc_operand(batch, K, 64, hbmm.F32))
            W = hbmm.quantize(wd, hbmm.alloc_operand(N, K, 64, hbmm.F32))
            ws = torch.empty(max(hbmm.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
            C = torch.empty((batch, (N + 3) // 4 * 4), device="cuda")
            hbmm.gemm(A, W, C, ws)
            stack.append((A, W, C, ws))

        def run_stack():
            for A, W, C, ws in stack:
                if batch <= 8:
                    hbmm.gemm(A, W, C, ws)
                else:
                    hbmm.gemm_ex(A, W, C, hbmm.PATH_FOLDED_PREPARED, ws)

        # the three launches as one CUDA graph, so that they run back to back on the device
        warm = time_graph(torch, [run_stack], 20)
        one = torch.cuda.CUDAGraph()
        with torch.cuda.graph(one):
            run_stack()
        flush = torch.empty(int(2 * L2_BYTES) // 4, dtype=torch.float32, device="cuda")
        cold = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(20):
            flush.zero_()                                   # evicts the weights from L2
            e0.record()
            one.replay()
            e1.record()
            torch.cuda.synchronize()
            cold.append(e0.elapsed_time(e1))
        by = sum(hbmm_bytes(batch, N, K, 64) for K, N in inputs.ALEXNET_FC)
        ops = sum(2.0 * batch * N * K for K, N in inputs.ALEXNET_FC)
        t_roof = sum(popc_hbm_roofline(batch, N, K, 64, 4, rates, hbm_gbs)["t_roof_us"] for K, N in inputs.ALEXNET_FC)
        rows.append({"name": "alexnet_fc_stack_b%d" % batch, "launches": 3, "warm_l2_ms": round(warm, 5),
                     "cold_l2_ms_median": round(statistics.median(cold), 5), "cold_l2_ms_min": round(min(cold), 5),
                     "tops_warm": ops / (warm * 1e-3) / 1e12, "gbs_cold": by / (statistics.median(cold) * 1e-3) / 1e9,
                     "t_roof_us": round(t_roof, 3), "frac_of_popcount_hbm_roofline_cold": t_roof / (statistics.median(cold) * 1e3),
                     "note": "three hbmm_gemm launches back to back in one CUDA graph; products are not chained (each layer has its own seeded input)"})
        del stack
    return rows


# ----------------------------------------------------------------------------- CPU checker timing
def oracle_sample_rows(shapes, frac: float):
    return [max(32, int(s.M * frac)) for s in shapes]


def oracle_inputs(inputs, shapes, rows):
    """Seeded inputs of the row sample: the first ceil(rows / (Ho*Wo)) images of each layer."""
    data = []
    for li, (s, ms) in enumerate(zip(shapes, rows)):
        b = max(1, -(-ms // (s.M // s.B)))
        sub = inputs.ConvShape(s.name, b, s.C, s.H, s.W, s.N)
        data.append((inputs.conv_activation(sub, inputs.SEEDS["resnet_hbmm"][0] + li),
                     inputs.he_normal(s.N, s.K, inputs.SEEDS["resnet_hbmm"][1] + li)))
    return data


def oracle_step(oracle, inputs, shapes, rows, data) -> float:
    """The checker as it stands on a row sample of each layer: HBMM and HBWN of the im2col rows."""
    t0 = time.perf_counter()
    for (s, ms, (x, w)) in zip(shapes, rows, data):
        a = oracle.im2col(x, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))[:ms]
        oracle.hbmm(a, w, BETA, BETA, "f32")
        _, ab = inputs.as_bf16(a)
        oracle.hbwn(ab, w, BETA, "f32")
    return time.perf_counter() - t0


def sample_ops(shapes, rows) -> float:
    return sum(2.0 * 2 * ms * s.N * s.K for s, ms in zip(shapes, rows))


def cpu_baseline(shapes, budget_s: float):
    """Time the checker on a row sample sized (from a small calibration run) to about budget_s seconds."""
    import oracle
    from paper_1905_10759_b200 import inputs
    oracle.build()
    rows = oracle_sample_rows(shapes, 1.0 / 256)
    data = oracle_inputs(inputs, shapes, rows)
    oracle_step(oracle, inputs, shapes, rows, data)
    t = oracle_step(oracle, inputs, shapes, rows, data)
    frac = min(0.5, (1.0 / 256) * budget_s / max(t, 1e-3))
    rows = oracle_sample_rows(shapes, frac)
    data = oracle_inputs(inputs, shapes, rows)
    t = oracle_step(oracle, inputs, shapes, rows, data)
    res = {"value": sample_ops(shapes, rows) / t / 1e12, "unit": "TOPS", "cores": oracle.num_threads(),
           "kind": "oracle",
           "sample": "first %s rows of the im2col matrices of conv2_x..conv5_x (%.4f of each layer), HBMM + HBWN, %.1f s"
                     % (rows, frac, t)}
    return res, rows, data


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    from paper_1905_10759_b200 import inputs
    oracle.build()
    shapes = inputs.resnet18_convs(64)
    total_budget = 150.0
    per_step = max(0.3, min(4.0, total_budget / max(1, args.steps + args.warmup)))
    base, rows, data = cpu_baseline(shapes, per_step)
    for _ in range(args.warmup):
        oracle_step(oracle, inputs, shapes, rows, data)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, inputs, shapes, rows, data)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    val = sample_ops(shapes, rows) / dt / 1e12
    line = {
        "impl": "reference", "metric": "hbmm_effective_binary_tops", "value": val, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "resnet18_conv3x3_b64_hbmm+hbwn_beta32", "sample_rows": rows,
                   "note": "CPU checker (oracle/) on a bounded row sample of each layer per step"},
        "cpu_baseline": {"value": val, "unit": "TOPS", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": "rows %s per layer per step" % rows},
        "e2e": {"value": val, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- main arm
def run_ours(args):
    import torch
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the HBMM path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_1905_10759_b200 import build as _build
    if rank == 0 or world == 1:
        _build.build_lib()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    from paper_1905_10759_b200 import hbmm, inputs

    shapes, layers = build_workload(torch, hbmm, inputs, rank, device, args.profile_layer)
    ops_step = 2.0 * sum(layer_ops(shapes))        # HBMM + HBWN product of every layer
    if args.profile_layer:
        # a small, short run of one layer for profiler captures: no end-to-end leg, no breakdown, no CPU timing
        for _ in range(max(args.warmup, 3) + args.steps):
            run_step(hbmm, layers)
        torch.cuda.synchronize()
        assert hbmm.last_device_error() == 0
        print(json.dumps({"profile_layer": args.profile_layer, "steps": args.steps, "launches_per_step": 4}))
        return 0

    # warm-up: the first step expands the weights into the workspaces, the rest run as the timed steps do
    PREP = hbmm.CONV_WEIGHTS_PREPARED
    run_step(hbmm, layers)
    step2 = TwoStreamStep(torch)
    for _ in range(max(args.warmup, 3) - 1):
        step2(hbmm, layers, PREP)
    torch.cuda.synchronize()
    if args.profile_step:
        # the timed schedule and nothing else (no breakdown, side rows or CPU timing): for a profiler's launch list
        for _ in range(args.steps):
            step2(hbmm, layers, PREP)
        torch.cuda.synchronize()
        assert hbmm.last_device_error() == 0
        print(json.dumps({"profile_step": True, "steps": args.steps, "launches_per_step": LAUNCHES_PER_STEP}))
        return 0

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_ready()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The timed region (exactly `steps` steps between a barrier + synchronize on both sides) is repeated
    # kRepeats times; the reported step time is the median region, the spread is reported beside it.
    kRepeats = 5
    regions = []
    t0 = time.time()
    for _ in range(kRepeats):
        barrier()
        e0.record()
        for _ in range(args.steps):
            step2(hbmm, layers, PREP)
        e1.record()
        barrier()
        regions.append(max_over_ranks(e0.elapsed_time(e1) / args.steps, world, device))
    t1 = time.time()
    ms_step = statistics.median(regions)
    # the same step with all eight calls on one stream
    barrier()
    e0.record()
    for _ in range(args.steps):
        run_step(hbmm, layers, PREP)
    e1.record()
    barrier()
    ms_step_one_stream = max_over_ranks(e0.elapsed_time(e1) / args.steps, world, device)
    # the same step with the weight expansion repeated by every call (plain hbmm_conv_im2col), for comparison
    barrier()
    e0.record()
    for _ in range(args.steps):
        run_step(hbmm, layers)
    e1.record()
    barrier()
    ms_step_expand = max_over_ranks(e0.elapsed_time(e1) / args.steps, world, device)

    # end to end: pinned host inputs -> device, path, results -> pinned host, every step
    pipe = E2EPipeline(torch, layers)
    cur = torch.cuda.current_stream()
    for _ in range(2):
        pipe.step(hbmm, layers, PREP)
    barrier()
    e0.record()
    for s_ in (pipe.up, pipe.comp, pipe.down):
        s_.wait_event(e0)
    for _ in range(args.steps):
        pipe.step(hbmm, layers, PREP)
    pipe.join(cur)
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1) / args.steps, world, device)
    clocks = sampler.stop(t0, t1, time.time())
    err = hbmm.last_device_error()
    if err != 0:
        raise RuntimeError("a kernel reported device error %d during the timed steps: the numbers are void" % err)
    h2d = sum(L["x_host"].numel() * 4 + L["xb_host"].numel() * 2 for L in layers)
    d2h = sum(L["C_host"].numel() * 4 + L["Cb_host"].numel() * 4 for L in layers)

    # measured issue rates of the integer and fp32 pipes: the denominators of the ALU rooflines
    rates = measure_alu_rates(torch, hbmm, lambda: (read_sm_clock(local_rank) or (None,))[0])
    ck = read_sm_clock(local_rank)
    sm_max = ck[1] if ck else None
    for k in ("popc", "fadd", "ffma"):
        r = rates[k]
        scale = (sm_max / r["sm_mhz"]) if (sm_max and r["sm_mhz"]) else 1.0
        r["ops_per_s_at_max_clock"] = r["ops_per_s"] * scale
    rates["sm_max_mhz"] = sm_max
    rates["popcount_roofline_tops"] = rates["popc"]["ops_per_s"] * 64 / 1e12         # 32 binary MACs = 64 ops per count
    rates["planning_figures"] = {"popc_per_clk_per_sm": PLAN_POPC_PER_CLK_SM, "fadd_per_clk_per_sm": PLAN_FADD_PER_CLK_SM}

    # per-kernel durations for the roofline entry (launch configuration of the step, L2-cold)
    brk = kernel_breakdown(torch, hbmm, layers, 3 if args.steps < 50 else 6)
    peaks = measured_peaks()
    hbm_gbs, _, hbm_src = peaks
    families = ("hbmm_contraction", "hbwn_conv", "front_end_pack")       # these three add up to the step's kernels
    totals = {k: sum(brk[k]) for k in families}
    dominant = max(totals, key=totals.get)
    li = int(np.argmax(brk[dominant]))
    roof = roofline_for(dominant, li, shapes[li], brk[dominant][li], peaks, rates)
    roof["traffic"] = NCU_DRAM_BYTES.get((dominant, shapes[li].name))
    roof["share_of_step"] = totals[dominant] / sum(totals.values())
    kernels = {}
    keep = ("bound", "achieved", "peak", "unit", "frac", "frac_of_peak_in_issued_tensor_work", "frac_of_popcount_hbm_roofline",
            "frac_of_popcount_hbm_roofline_at_max_clock",
            "frac_of_fp32_add_hbm_roofline", "timing")
    for kind in families + ("hbmm_conv_call",):
        kernels[kind] = [dict(layer=s.name, ms=round(t, 5), **{k: v for k, v in roofline_for(kind, i, s, t, peaks, rates).items() if k in keep})
                         for i, (s, t) in enumerate(zip(shapes, brk[kind]))]
    kernels["buffer_sets_per_layer"] = brk["sets"]

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()
        return 0

    base = None
    side = None
    configs = None
    if world == 1:
        configs = config_rows(torch, hbmm, inputs, layers, brk, rates, peaks, 10)
        side = side_measurements(torch, hbmm, inputs, peaks, max(5, min(args.steps, 20)))
        base, _, _ = cpu_baseline(shapes, 12.0)
        err = hbmm.last_device_error()
        if err != 0:
            raise RuntimeError("a kernel reported device error %d during the side measurements: the numbers are void" % err)

    line = {
        "metric": "hbmm_effective_binary_tops", "value": aggregate(ops_step, world, ms_step), "unit": "TOPS",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "timed_regions": {"count": len(regions), "steps_each": args.steps, "ms_per_step_median": ms_step,
                          "ms_per_step_min": min(regions), "ms_per_step_max": max(regions)},
        "ms_per_step_one_stream": ms_step_one_stream,
        "ms_per_step_expanding_weights_every_call": ms_step_expand,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {
            "workload": "resnet18_conv3x3_b64_hbmm+hbwn_beta32",
            "layers": [dict(name=s.name, M=s.M, N=s.N, K=s.K) for s in shapes],
            "beta_a": BETA, "beta_w": BETA, "scale_dtype": "f32", "hbwn_activation_dtype": "bf16",
            "tensor_operands": "HBMM: sign x group scale as two fp16 pieces per operand (22-bit scales, exact products); HBWN: bf16 activations x two bf16 weight pieces (scales to 2^-18); fp32 accumulate",
            "weights": "binarized and expanded into the contraction's tile layout once, outside the timed region (HBMM_CONV_WEIGHTS_PREPARED); "
                       "ms_per_step_expanding_weights_every_call repeats the expansion in every call",
            "schedule": "two streams per step: the four HBMM calls on one, the four HBWN calls on the other, joined every step; "
                        "ms_per_step_one_stream runs the eight calls in a row; ms_per_step_expanding_weights_every_call is one stream too",
            "batch_per_gpu": 64, "parallelism": "replicas(batch-sharded)x%d" % world,
            "l2": "per-step inputs+outputs+workspaces (~0.7 GB) exceed the 126 MB L2; no explicit flush",
        },
        "roofline": roof,
        "kernels": kernels,
        "measured_alu_rates": rates,
        "configs": configs,
        "context": {"paper": PAPER_CONTEXT,
                    "cublas": "each row of `configs` carries torch.matmul of the same shape in fp32 (TF32 off) and in bf16"},
        "other_rows": side,
        "e2e": {"value": aggregate(ops_step, world, ms_e2e), "unit": "TOPS", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": LAUNCHES_PER_STEP * args.steps * len(regions), "gpu_launches_per_step": LAUNCHES_PER_STEP,
        "clocks": clocks,
    }
    if base is not None:
        line["cpu_baseline"] = base
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--profile-step", action="store_true",
                    help="run the warm-up and the timed steps only, no measurement: for a profiler's launch list")
    ap.add_argument("--profile-layer", default=None,
                    help="run only this layer (conv2_x .. conv5_x), few launches, no measurement: for profiler captures")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
