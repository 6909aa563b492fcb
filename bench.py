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
SM_COUNT = 148
SM_MAX_MHZ = 1965.0
# Unit counts of one SM (per clock): 16 POPC results, 128 fp32 FMA lanes.
POPC_PER_CLK_SM = 16
FMA_PER_CLK_SM = 128
FALLBACK_HBM_GBS = 6650.0


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


def kernel_breakdown(torch, hbmm, layers, iters: int):
    """Per-kernel average launch durations on the bench's own buffers and launch configuration.
    The packed activation operand of each layer is rebuilt in its workspace by the front end, then
    the contraction kernel is timed alone through hbmm_gemm_ex on exactly that operand; the front end
    (with the weight expansion its launch carries) is the rest of the convolution call."""
    out = {"hbmm_contraction": [], "hbwn_conv": [], "front_end_pack": []}
    for L in layers:
        s = L["shape"]
        PREP = hbmm.CONV_WEIGHTS_PREPARED      # the timed step reuses the expanded weights the warm-up left in the workspaces
        t_conv = time_loop(torch, lambda: hbmm.conv_im2col(L["x"], L["geom"], BETA, hbmm.F32, L["W"], L["C"], L["ws"], flags=PREP), iters)
        _, _, lw, ls = hbmm.operand_bytes(s.M, s.K, BETA, hbmm.F32)
        bits_bytes = (s.M * lw * 4 + 255) // 256 * 256
        bits = L["ws"][: s.M * lw * 4].view(torch.int32).reshape(s.M, lw)
        scales = L["ws"][bits_bytes: bits_bytes + s.M * ls * 4].view(torch.float32).reshape(s.M, ls)
        A = hbmm.wrap_packed(bits, scales, s.K, BETA)
        gws = torch.empty(max(hbmm.gemm_workspace_bytes(A, L["W"]), 16), dtype=torch.uint8, device=L["C"].device)
        # the contraction kernel alone: the weight expansion is part of the front end's launch in the
        # convolution call, so it is left in the workspace once and skipped here
        hbmm.gemm(A, L["W"], L["C"], gws)
        t_gemm = time_loop(torch, lambda: hbmm.gemm_ex(A, L["W"], L["C"], hbmm.PATH_FOLDED_PREPARED, gws), iters)
        out["hbmm_contraction"].append(t_gemm)
        out["front_end_pack"].append(max(t_conv - t_gemm, 1e-3))
        # HBWN: one call = NCHW -> NHWC bf16 copy, weight pieces, implicit-GEMM contraction (no im2col matrix)
        t_convb = time_loop(torch, lambda: hbmm.conv_im2col(L["xb"], L["geom"], 1, hbmm.F32, L["W"], L["Cb"], L["wsb"], flags=PREP), iters)
        out["hbwn_conv"].append(t_convb)
    return out


def side_measurements(torch, hbmm, peaks, iters: int):
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
    for ba, bw in ((16, 16), (4, 4), (2, 16)):
        A = hbmm.quantize(a, hbmm.alloc_operand(M, K, ba, hbmm.F32))
        W = hbmm.quantize(w, hbmm.alloc_operand(N, K, bw, hbmm.F32))
        ws = torch.empty(max(hbmm.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
        C = torch.empty((M, N), device="cuda")
        hbmm.gemm_ex(A, W, C, hbmm.PATH_FOLDED, ws)
        ms = time_loop(torch, lambda: hbmm.gemm_ex(A, W, C, hbmm.PATH_FOLDED_PREPARED, ws), iters)
        ach = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        out.append({"kernel": "hbmm_fold_kernel/beta_a%d_beta_w%d" % (ba, bw), "shape": [M, N, K], "ms": round(ms, 5), "bound": "tensor",
                    "achieved": ach, "peak": bf16_tflops, "unit": "TFLOP/s", "frac": ach / bf16_tflops})
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
    return out


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (same kernels, same workload); entries are dropped when a kernel changes after its capture.
NCU_DRAM_BYTES = {
    ("hbmm_contraction", "conv2_x"): 32.373e6 + 2.103e6,     # profiles/hbmm_fold_kernel_conv2_x.md
    ("front_end_pack", "conv2_x"): 51.511e6 + 2.524e6,       # profiles/im2col_quantize_tma_kernel_conv2_x.md
}


def roofline_for(kind: str, li: int, shape, ms: float, peaks):
    """Roofline entry of one kernel launch (layer li) given its measured duration.

    Both contractions run on the tensor cores (HBMM: two fp16 pieces per operand carrying sign and group
    scale; HBWN: bf16 activations x two bf16 weight pieces), so they are set against the measured dense
    16-bit GEMM peak.  `achieved` counts the ALGORITHMIC operations 2 M N K; the HBMM kernel issues four
    times that on the tensor pipe (2 x 2 pieces), the HBWN kernel twice.  For HBMM the fraction of
    the integer-pipe popcount roofline (one POPC per output and K-word at 16 / clk / SM) is given beside it."""
    hbm_gbs, bf16_tflops, hbm_src = peaks
    M, N, K = shape.M, shape.N, shape.K
    G = -(-K // BETA)
    if kind == "hbmm_contraction":
        ops = 2.0 * M * N * K
        peak = bf16_tflops
        popc_peak = SM_COUNT * POPC_PER_CLK_SM * SM_MAX_MHZ * 1e6 * 64 / 1e12
        ach = ops / (ms * 1e-3) / 1e12
        return {"kernel": "hbmm_fold_kernel/%s" % shape.name, "bound": "tensor", "achieved": ach,
                "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "traffic": None,
                "peak_source": "%s bf16 GEMM peak (fp16 operands, same rate)" % hbm_src,
                "tensor_pipe_work_factor": 4,
                "frac_of_popcount_roofline": ach / popc_peak, "popcount_roofline_tops": popc_peak}
    if kind == "hbwn_conv":
        # the whole HBWN call (layout copy + weight pieces + contraction) set against the contraction's flops
        ops = 2.0 * M * N * K
        ach = ops / (ms * 1e-3) / 1e12
        return {"kernel": "hbwn_umma_kernel(im2col tensor copies)/%s" % shape.name, "bound": "tensor", "achieved": ach,
                "peak": bf16_tflops, "unit": "TFLOP/s", "frac": ach / bf16_tflops, "traffic": None,
                "peak_source": "%s bf16 GEMM peak" % hbm_src}
    x_bytes = 4.0 * shape.B * shape.C * shape.H * shape.W
    lw = ((K + 31) // 32 + 3) // 4 * 4
    ls = (G + 3) // 4 * 4
    by = x_bytes + M * lw * 4.0 + M * ls * 4.0
    return {"kernel": "%s/%s" % (kind, shape.name), "bound": "hbm", "achieved": by / (ms * 1e-3) / 1e9,
            "peak": hbm_gbs, "unit": "GB/s", "frac": by / (ms * 1e-3) / 1e9 / hbm_gbs, "traffic": None,
            "peak_source": "%s HBM copy bandwidth" % hbm_src}


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

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_ready()
    barrier()
    t0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step2(hbmm, layers, PREP)
    e1.record()
    barrier()
    t1 = time.time()
    ms_step = e0.elapsed_time(e1) / args.steps
    ms_step = max_over_ranks(ms_step, world, device)
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

    # per-kernel durations for the roofline entry (same buffers, same launch configuration)
    brk = kernel_breakdown(torch, hbmm, layers, max(5, min(args.steps, 20)))
    peaks = measured_peaks()
    hbm_gbs, _, hbm_src = peaks
    totals = {k: sum(v) for k, v in brk.items()}
    dominant = max(totals, key=totals.get)
    li = int(np.argmax(brk[dominant]))
    roof = roofline_for(dominant, li, shapes[li], brk[dominant][li], peaks)
    roof["traffic"] = NCU_DRAM_BYTES.get((dominant, shapes[li].name))
    roof["share_of_step"] = totals[dominant] / sum(totals.values())
    kernels = {}
    for kind, times in brk.items():
        kernels[kind] = [dict(layer=s.name, ms=round(t, 5), **{k: v for k, v in roofline_for(kind, i, s, t, peaks).items()
                                                                if k in ("bound", "achieved", "peak", "unit", "frac")})
                         for i, (s, t) in enumerate(zip(shapes, times))]

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()
        return 0

    base = None
    side = None
    if world == 1:
        side = side_measurements(torch, hbmm, peaks, max(5, min(args.steps, 20)))
        base, _, _ = cpu_baseline(shapes, 12.0)

    line = {
        "metric": "hbmm_effective_binary_tops", "value": aggregate(ops_step, world, ms_step), "unit": "TOPS",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
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
        "other_rows": side,
        "e2e": {"value": aggregate(ops_step, world, ms_e2e), "unit": "TOPS", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": LAUNCHES_PER_STEP * args.steps,
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
    ap.add_argument("--profile-layer", default=None,
                    help="run only this layer (conv2_x .. conv5_x), few launches, no measurement: for profiler captures")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
