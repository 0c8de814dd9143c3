#!/usr/bin/env python
"""Benchmark of the DyBit hot path on B200.

A step = one pass of the whole path over the ResNet-18-shaped batch-32
workload: for each of its 21 layers, max-abs scale + quantize + pack of the
fp32 NHWC activation to unsigned 4-bit DyBit, then the convolution as an
implicit GEMM against signed 4-bit DyBit weights (quantized once at set-up,
as a deployed model would hold them), dequantised fp32 output.

The layers of this workload are independent (each has its own synthetic
activation, weights and output), so the step issues them round-robin on a few
CUDA streams, one workspace per stream, and the whole step is captured once as
a CUDA graph whose replays are timed.

Prints ONE JSON line (rank 0).  `value` is the whole-job TOPS (2*MACs of all
layers on all ranks / step time, inputs resident in HBM); `e2e` times the
same step with the activations coming from pinned host memory and the outputs
copied back.  Three roofline objects: `roofline` is the tensor-core kernel of
the 8192^3 4-bit GEMM (the configuration the GEMM half of the metric is quoted
on; bound: tensor), `roofline_quantize` the 2^28-element 4-bit quantize/pack
kernel (bound: hbm), `roofline_conv` the convolution kernels of the step's 21
layers against their layer-wise bound.  `peaks_measured_here` holds dense
int8 / fp8 / bf16 library matmuls and a device-to-device copy timed in the
same run; `cpu_baseline` is the plain CPU oracle on a bounded sample of the
same workload.

`--impl reference` times that oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

FMT_W = (4, 1)      # weights: signed 4-bit
FMT_A = (4, 0)      # post-ReLU activations: unsigned 4-bit
NOMINAL = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0, "int8_tops": 4500.0, "fp8_tflops": 4500.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, copied from the ncu summaries under profiles/ (bench.py cannot
# read hardware counters itself); an entry is None while the kernel has changed since its counters were taken
NCU_TRAFFIC = {"gemm_8192": (147033344 + 111412480) * (8192.0 / 6144.0) ** 2, "quantize_2p26_per_element": (268458496 + 8048640) / float(1 << 26),
               "conv_step": (79310336 + 42336512) / 21.0}
NCU_TRAFFIC_HOW = {
    "gemm_8192": "profiles/dybit_gemm_pair_kernel_i8_square6144_and_4096.txt: one launch at M=N=K=6144 (a capture small "
                 "enough to end by itself, whole tiles only as at 8192^3), x (8192 / 6144)^2 for 8192^3 (operand and output "
                 "bytes both grow with the square of the size)",
    "quantize_2p26_per_element": "profiles/quantize_pack_kernel_4bit_signed_2p26.txt: bytes per element of one launch at "
                                 "2^26 elements x the elements of this launch (streaming kernel: traffic is proportional)",
    "conv_step": "profiles/dybit_gemm_kernel_conv_resnet18_b32_dram_traffic.txt: mean over the 21 conv launches of one step",
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        # the busy samples are the upper half (idle samples before/after the region sit at low clocks)
        med = sm[len(sm) // 2] if sm else None
        return {"sm_mhz": med, "sm_max_mhz": smax, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- workload

class LayerwiseStep:
    """Device buffers and the per-step call sequence for a list of independent conv/FC layers.

    bits[i] = (weight bits, activation bits) of layer i; weights are signed, activations unsigned."""

    def __init__(self, dy, wl, device, layers, bits, host_copies=True, two_calls=False, n_streams=1, fold=False):
        self.dy, self.device = dy, device
        self.two_calls = two_calls          # quantize_pack + conv2d as two library calls instead of one
        self.fold = fold                    # max-abs and quantize + expand of ALL layers in two launches, then the convolutions
        self.shared_launches = True         # ... as dybit_conv2d_prepared_layers (False: one launch per layer on the side streams)
        self.n_streams = max(1, int(n_streams))
        self.layers = layers
        self.fw = [(wb, 1) for wb, _ in bits]
        self.fa = [(ab, 0) for _, ab in bits]
        self.x_host, self.x_dev, self.pw, self.sw, self.px, self.sx, self.y, self.y_host = [], [], [], [], [], [], [], []
        self.desc = []
        ws_bytes = 0
        for i, L in enumerate(self.layers):
            if host_copies:
                xh = wl.half_normal((L.n, L.h, L.w, L.c), seed=1000 + i).pin_memory()
                self.x_host.append(xh)
                self.x_dev.append(xh.to(device))
            else:
                self.x_dev.append(wl.half_normal((L.n, L.h, L.w, L.c), seed=1000 + i, device=device))
            w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2000 + i).reshape(L.k, -1).to(device)
            pw, sw = dy.dybit_quantize_pack_2d(w, self.fw[i])
            self.pw.append(pw)
            self.sw.append(sw)
            n = self.x_dev[i].numel()
            self.px.append(torch.empty(dy.dybit_packed_bytes(n, self.fa[i][0]), dtype=torch.uint8, device=device))
            self.sx.append(torch.empty(2, dtype=torch.float32, device=device))
            self.y.append(torch.empty((L.n, L.oh, L.ow, L.k), dtype=torch.float32, device=device))
            d = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
            self.desc.append(d)
            ws_bytes = max(ws_bytes, dy.dybit_conv2d_workspace_bytes(d, self.fa[i], self.fw[i]))
        self.ws = torch.empty(ws_bytes + 1024, dtype=torch.uint8, device=device)
        # one workspace per stream: layers on different streams run at the same time
        self.ws_pool = [self.ws] + [torch.empty_like(self.ws) for _ in range(self.n_streams - 1)]
        self.side = [torch.cuda.Stream(device) for _ in range(self.n_streams)] if self.n_streams > 1 else []
        if fold:
            # same buffers, every layer with a workspace of its own (all of them are in use at once)
            self.folded = dy.ConvLayers([dict(desc=self.desc[i], X=self.x_dev[i], fx=self.fa[i], W=self.pw[i], fw=self.fw[i],
                                              scale_w=self.sw[i], packed=self.px[i], scale_out=self.sx[i], Y=self.y[i])
                                         for i in range(len(self.layers))])
        self.macs = sum(L.macs for L in self.layers)
        self.h2d_bytes = sum(x.numel() * 4 for x in self.x_dev)
        self.d2h_bytes = sum(y.numel() * 4 for y in self.y)
        self.quant_elems = sum(x.numel() for x in self.x_dev)

    def alloc_host_outputs(self):
        self.y_host = [torch.empty(y.shape, dtype=torch.float32).pin_memory() for y in self.y]

    def _layer(self, i, ws):
        dy = self.dy
        if self.two_calls:
            dy.dybit_quantize_pack(self.x_dev[i], self.fa[i], packed=self.px[i], scale_out=self.sx[i])
            dy.dybit_conv2d(self.desc[i], self.px[i], self.fa[i], self.sx[i], self.pw[i], self.fw[i], self.sw[i],
                            Y=self.y[i], ws=ws)
        else:
            # same results (codes, scale, layer output) from one library call that saves a launch per layer
            dy.dybit_quantize_conv2d(self.desc[i], self.x_dev[i], self.fa[i], self.pw[i], self.fw[i], self.sw[i],
                                     scale_out=self.sx[i], packed=self.px[i], Y=self.y[i], ws=ws)

    def step(self, events=None, clocks=None, only=None, serial=False):
        """One pass over the layers.  With several streams (and no per-kernel profiling asked for) layer j goes to
        stream j mod S; the calling stream forks into them and joins them again, so the step is one unit of work
        for whoever times or captures it.  `serial` keeps everything on the calling stream."""
        dy = self.dy
        profiling = events is not None or clocks is not None
        if self.fold and not self.two_calls and only is None and not profiling and not serial:
            # dybit_quantize_expand_layers: one max-abs launch and one quantize + expand launch for all layers; then
            # dybit_conv2d_prepared_layers: the tensor-core work, layers of one kernel configuration sharing launches
            dy.dybit_quantize_expand_layers(self.folded)
            if self.shared_launches:
                dy.dybit_conv2d_prepared_layers(self.folded)
                return
            # one tensor-core launch per layer, round-robin on the side streams
            cur = torch.cuda.current_stream()
            for st in self.side:
                st.wait_stream(cur)
            for j in range(len(self.layers)):
                dy.dybit_conv2d_prepared(self.folded, j, stream=self.side[j % self.n_streams] if self.side else None)
            for st in self.side:
                cur.wait_stream(st)
            return
        if self.n_streams > 1 and only is None and not profiling and not serial:
            cur = torch.cuda.current_stream()
            for st in self.side:
                st.wait_stream(cur)
            for j in range(len(self.layers)):
                with torch.cuda.stream(self.side[j % self.n_streams]):
                    self._layer(j, self.ws_pool[j % self.n_streams])
            for st in self.side:
                cur.wait_stream(st)
            return
        for i in (range(len(self.layers)) if only is None else (only,)):
            if clocks is not None:
                dy.dybit_profile_next_gemm_clock(clocks[i])
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                dy.dybit_profile_next_gemm(e0, e1)
                events[i].append((e0, e1))
            self._layer(i, self.ws)

    def prepare_requant(self, fq=(4, 0)):
        """Output scales for the re-quantizing epilogue: max-abs of each layer's fp32 output from one normal step
        (a stand-in for calibrated scales); packed output buffers."""
        dy = self.dy
        self.fq = fq
        self.step()
        self.sq = [dy.dybit_absmax_scale(y.reshape(-1).clamp_min(0), fq) for y in self.y]
        self.q = [torch.zeros(dy.dybit_packed_bytes(y.numel(), fq[0]), dtype=torch.uint8, device=self.device)
                  for y in self.y]
        self.q_bytes = sum(q.numel() for q in self.q)

    def step_requant(self):
        """The same step with results written back as packed DyBit codes (ReLU + encode in the epilogue)."""
        dy = self.dy
        if self.fold:
            if not hasattr(self, "folded_q"):
                self.folded_q = dy.ConvLayers([dict(desc=self.desc[i], X=self.x_dev[i], fx=self.fa[i], W=self.pw[i],
                                                    fw=self.fw[i], scale_w=self.sw[i], packed=self.px[i], scale_out=self.sx[i],
                                                    fq=self.fq, scale_q=self.sq[i], relu=True, Q=self.q[i])
                                               for i in range(len(self.layers))])
            dy.dybit_quantize_expand_layers(self.folded_q)
            dy.dybit_conv2d_prepared_layers(self.folded_q)
            return

        def layer(i, ws):
            dy.dybit_quantize_conv2d_requant(self.desc[i], self.x_dev[i], self.fa[i], self.pw[i], self.fw[i], self.sw[i],
                                             self.fq, self.sq[i], relu=True, scale_out=self.sx[i], packed=self.px[i],
                                             Q=self.q[i], ws=ws)
        if self.n_streams > 1:
            cur = torch.cuda.current_stream()
            for st in self.side:
                st.wait_stream(cur)
            for j in range(len(self.layers)):
                with torch.cuda.stream(self.side[j % self.n_streams]):
                    layer(j, self.ws_pool[j % self.n_streams])
            for st in self.side:
                cur.wait_stream(st)
            return
        for i in range(len(self.layers)):
            layer(i, self.ws)

    def step_e2e(self):
        """One step with its inputs coming from pinned host memory and its outputs going back there, pipelined layer
        by layer over three streams (host->device copies, the library's kernels, device->host copies), so that the two
        copy directions and the kernels overlap.  Per-buffer events keep a buffer from being refilled before its last
        reader is done; e2e_join() makes the calling stream wait for the copies still in flight."""
        n = len(self.layers)
        cur = torch.cuda.current_stream()
        if not hasattr(self, "_h2d"):
            self._h2d, self._d2h = torch.cuda.Stream(self.device), torch.cuda.Stream(self.device)
            self._in_ready = [torch.cuda.Event() for _ in range(n)]
            self._computed = [torch.cuda.Event() for _ in range(n)]
            self._out_copied = [torch.cuda.Event() for _ in range(n)]
            self._first = True
            self._h2d.wait_stream(cur)
            self._d2h.wait_stream(cur)
        for i in range(n):
            with torch.cuda.stream(self._h2d):
                if not self._first:
                    self._h2d.wait_event(self._computed[i])        # last step's layer i has read x_dev[i]
                self.x_dev[i].copy_(self.x_host[i], non_blocking=True)
                self._in_ready[i].record(self._h2d)
            cur.wait_event(self._in_ready[i])
            if not self._first:
                cur.wait_event(self._out_copied[i])                # last step's y[i] has left the device
            self.step(only=i)
            self._computed[i].record(cur)
            with torch.cuda.stream(self._d2h):
                self._d2h.wait_event(self._computed[i])
                self.y_host[i].copy_(self.y[i], non_blocking=True)
                self._out_copied[i].record(self._d2h)
        self._first = False

    def e2e_join(self):
        cur = torch.cuda.current_stream()
        cur.wait_stream(self._h2d)
        cur.wait_stream(self._d2h)

    def layer_bounds(self, tensor_tops, hbm_gbs):
        """Per layer: (flops, algorithmic bytes of the conv, ideal seconds = max of the two bounds)."""
        out = []
        for L, fa, fw in zip(self.layers, self.fa, self.fw):
            flops = 2.0 * L.macs
            byts = (L.n * L.h * L.w * L.c * fa[0] / 8 + L.k * L.gemm_k * fw[0] / 8 + 4.0 * L.gemm_m * L.k)
            out.append((flops, byts, max(flops / (tensor_tops * 1e12), byts / (hbm_gbs * 1e9))))
        return out


def timed_region(fn, steps, dist, device):
    """barrier + sync, K steps between CUDA events, sync + barrier; returns max-over-ranks ms."""
    torch.cuda.synchronize(device)
    if dist is not None:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize(device)
    if dist is not None:
        dist.barrier()
    return max_over_ranks(e0.elapsed_time(e1), dist, device)


def max_over_ranks(ms, dist, device):
    """The slowest rank's time: every multi-GPU number is reported against it."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def workload_name(batch):
    """The same string in both arms (the product's and the reference's)."""
    return (f"resnet18_b{batch}_w4a4: 20 convs + FC as implicit GEMM, per layer max-abs + quantize/pack of the fp32 "
            "activation then conv; weights pre-quantized")


def whole_job_tops(macs_per_rank, world, ms_step):
    """Replicas: every rank runs the same step on its own GPU, so the job's work is world x one rank's."""
    return world * 2.0 * macs_per_rank / (ms_step * 1e-3) / 1e12


def capture_step(work, device, fn=None):
    """One step captured as a CUDA graph (the library's calls are plain stream work, so they capture)."""
    graph = torch.cuda.CUDAGraph()
    cap_stream = torch.cuda.Stream(device)
    cap_stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap_stream):
        with torch.cuda.graph(graph, stream=cap_stream):
            (fn or work.step)()
    torch.cuda.current_stream().wait_stream(cap_stream)
    return graph


# --------------------------------------------------------------------------- single-kernel targets

def time_calls(fn, iters, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def target_gemm(dy, wl, device, peaks, size=8192, fmt=(4, 1)):
    """Square DyBit GEMM, both operands N(0,1) in the same signed format (4-bit -> int8, 8-bit -> bf16 container)."""
    a = wl.normal((size, size), seed=11, device=device)
    b = wl.normal((size, size), seed=12, device=device)
    pa, sa = dy.dybit_quantize_pack_2d(a, fmt)
    pb, sb = dy.dybit_quantize_pack_2d(b, fmt)
    del a, b
    cont = CONTAINERS[dy.dybit_choose_container(fmt, fmt)[0]]
    c = torch.empty((size, size), dtype=torch.float32, device=device)
    ws = torch.empty(dy.dybit_gemm_workspace_bytes(size, size, size, fmt, fmt) + 1024, dtype=torch.uint8,
                     device=device)
    call = lambda: dy.dybit_gemm(size, size, size, pa, fmt, sa, pb, fmt, sb, C_out=c, ws=ws)  # noqa: E731
    ms_call = time_calls(call, 10)
    # tensor-core kernel alone
    evs = []
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dy.dybit_profile_next_gemm(e0, e1)
        call()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    ms_kernel = sorted(e0.elapsed_time(e1) for e0, e1 in evs)[len(evs) // 2]
    ops = 2.0 * size ** 3
    ratio = 1.0 if cont == "bf16" else 2.0                   # nominal int8 (fp8) : bf16 tensor throughput
    peak_burst = ratio * peaks["bf16_tflops"]
    out = {"M=N=K": size, "formats": f"s{fmt[0]} x s{fmt[0]} -> {cont} container", "container": cont,
           "ms_call": ms_call, "ms_mma_kernel": ms_kernel,
           "tops_call": ops / ms_call / 1e9, "tops_mma_kernel": ops / ms_kernel / 1e9,
           "peak_tops": peak_burst,
           "peak_how": f"{ratio:g} x bf16 burst ({peaks['source']}); int8/fp8 : bf16 = 2 : 1 nominal",
           "frac_call": ops / ms_call / 1e9 / peak_burst, "frac_mma_kernel": ops / ms_kernel / 1e9 / peak_burst,
           "nominal_int8_tops": NOMINAL["int8_tops"]}
    # context: a plain library matmul of the container type and the same shape on this machine
    try:
        if cont == "int8":
            x = torch.randint(-8, 8, (size, size), dtype=torch.int8, device=device)
            y = torch.randint(-8, 8, (size, size), dtype=torch.int8, device=device)
            ms_lib = time_calls(lambda: torch._int_mm(x, y), 10)
        else:
            x = torch.randn((size, size), dtype=torch.bfloat16, device=device)
            y = torch.randn((size, size), dtype=torch.bfloat16, device=device)
            ms_lib = time_calls(lambda: torch.matmul(x, y), 10)
        out["library_matmul_tops"] = ops / ms_lib / 1e9
    except Exception as exc:  # pragma: no cover
        out["library_matmul_tops"] = None
        out["library_matmul_note"] = str(exc)[:80]
    return out


def target_gemm_decode(dy, wl, device, shapes=((128, 28672, 8192), (128, 8192, 8192), (8192, 8192, 8192))):
    """The two ways dybit_gemm can turn packed 4-bit weights into int8: a separate expand launch into the workspace, or
    decode warps inside the GEMM kernel's main loop (dybit_set_gemm_decode).  Per-call time, L2 flushed before each call."""
    fa, fb = (4, 0), (4, 1)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    rows = []
    for (M, N, K) in shapes:
        pa, sa = dy.dybit_quantize_pack_2d(wl.half_normal((M, K), seed=1, device=device), fa)
        pb, sb = dy.dybit_quantize_pack_2d(wl.normal((N, K), seed=2, device=device), fb)
        C = torch.empty((M, N), dtype=torch.float32, device=device)
        ws = torch.empty(dy.dybit_gemm_workspace_bytes(M, N, K, fa, fb) + 1024, dtype=torch.uint8, device=device)
        us = {}
        try:
            for mode, name in ((0, "expand_launch"), (1, "decode_in_main_loop")):
                dy.dybit_set_gemm_decode(mode)
                us[name] = time_calls_flushed(lambda: dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb, C_out=C, ws=ws), 7, flush) * 1e3
        finally:
            dy.dybit_set_gemm_decode(2)
        rows.append({"M": M, "N": N, "K": K, "us_per_call": us,
                     "packed_weight_gbs_decode_in_main_loop": N * K / 2 / us["decode_in_main_loop"] / 1e3})
        del pa, pb, C, ws
        torch.cuda.empty_cache()
    return rows


def target_quantize(dy, wl, device, peaks, log2n=28, bits=4):
    n = 1 << log2n
    x = wl.normal((n,), seed=21, device=device)
    fmt = (bits, 1)
    packed = torch.empty(dy.dybit_packed_bytes(n, bits), dtype=torch.uint8, device=device)
    scale = dy.dybit_absmax_scale(x, fmt)
    ms_given = time_calls(lambda: dy.dybit_quantize_pack(x, fmt, scale=scale, packed=packed), 10)
    so = torch.empty(2, dtype=torch.float32, device=device)
    ms_maxabs = time_calls(lambda: dy.dybit_quantize_pack(x, fmt, packed=packed, scale_out=so), 10)
    bytes_given = n * (4 + bits / 8)
    bytes_maxabs = n * (8 + bits / 8)
    return {"elements": n, "bits": bits,
            "scale_given": {"ms": ms_given, "gbs": bytes_given / ms_given / 1e6,
                            "frac": bytes_given / ms_given / 1e6 / peaks["hbm_gbs"]},
            "with_max_abs": {"ms": ms_maxabs, "gbs": bytes_maxabs / ms_maxabs / 1e6,
                             "frac": bytes_maxabs / ms_maxabs / 1e6 / peaks["hbm_gbs"]},
            "peak_gbs": peaks["hbm_gbs"], "peak_how": f"copy bandwidth ({peaks['source']})",
            "nominal_gbs": NOMINAL["hbm_gbs"]}


def target_quantize_expand(dy, wl, device, peaks, log2n=26):
    """quantize_expand_kernel alone on an activation beyond the L2: fp32 in (4 B), packed 4-bit codes (0.5 B) and int8
    tensor-core elements (1 B) out, scale given.  Reached through dybit_quantize_expand_layers on a single pointwise
    layer (64 channels, 16 filters), whose only launch it then is."""
    n_pix = (1 << log2n) // 64
    desc = dy.ConvDesc(1, n_pix // 128, 128, 64, 16, 1, 1, 1, 0, 1)
    fx, fw = (4, 0), (4, 1)
    x = wl.half_normal((desc.n, desc.h, desc.w, desc.c), seed=23, device=device)
    w = wl.kaiming_normal(16, 1, 1, 64, seed=24).reshape(16, -1).to(device)
    pw, sw = dy.dybit_quantize_pack_2d(w, fw)
    scale = dy.dybit_absmax_scale(x.reshape(-1), fx)
    layer = dy.ConvLayers([dict(desc=desc, X=x, fx=fx, W=pw, fw=fw, scale_w=sw, scale_x=scale, scale_out=scale)])
    n0 = dy.dybit_launch_count()
    dy.dybit_quantize_expand_layers(layer)
    launches = dy.dybit_launch_count() - n0
    ms = time_calls(lambda: dy.dybit_quantize_expand_layers(layer), 10)
    n = x.numel()
    return {"elements": n, "bytes_per_element": 5.5, "launches_per_call": launches, "ms": ms, "gbs": n * 5.5 / ms / 1e6,
            "frac": n * 5.5 / ms / 1e6 / peaks["hbm_gbs"], "peak_gbs": peaks["hbm_gbs"],
            "peak_how": f"copy bandwidth ({peaks['source']})"}


def measure_peaks_here(device, peaks, size=8192):
    """Dense library matmuls of the three container types and a device-to-device copy, timed in this run: context for
    the denominators of MEASURED_PEAKS.json (which holds the copy bandwidth and the bf16 figure only)."""
    out = {"shape": f"{size}^3", "what": "torch (cuBLASLt) dense matmuls, CUDA events over 10 calls after 3 warm-ups"}
    ops = 2.0 * size ** 3
    try:
        x = torch.randint(-8, 8, (size, size), dtype=torch.int8, device=device)
        y = torch.randint(-8, 8, (size, size), dtype=torch.int8, device=device)
        out["int8_matmul_tops"] = ops / time_calls(lambda: torch._int_mm(x, y), 10) / 1e9
        del x, y
    except Exception as exc:  # pragma: no cover
        out["int8_matmul_tops"] = None
        out["int8_note"] = str(exc)[:120]
    try:
        a = torch.randn((size, size), dtype=torch.bfloat16, device=device)
        b = torch.randn((size, size), dtype=torch.bfloat16, device=device)
        out["bf16_matmul_tflops"] = ops / time_calls(lambda: torch.matmul(a, b), 10) / 1e9
        a8 = a.to(torch.float8_e4m3fn)
        b8 = b.to(torch.float8_e4m3fn).t().contiguous().t()            # column-major second operand
        one = torch.ones((), dtype=torch.float32, device=device)
        out["fp8_e4m3_matmul_tflops"] = ops / time_calls(
            lambda: torch._scaled_mm(a8, b8, scale_a=one, scale_b=one, out_dtype=torch.bfloat16), 10) / 1e9
        del a, b, a8, b8
    except Exception as exc:  # pragma: no cover
        out.setdefault("bf16_matmul_tflops", None)
        out["fp8_e4m3_matmul_tflops"] = None
        out["fp8_note"] = str(exc)[:120]
    try:
        src = torch.empty(1 << 30, dtype=torch.uint8, device=device)
        dst = torch.empty_like(src)
        out["copy_gbs"] = 2.0 * src.numel() / time_calls(lambda: dst.copy_(src), 10) / 1e6
        del src, dst
    except Exception as exc:  # pragma: no cover
        out["copy_gbs"] = None
        out["copy_note"] = str(exc)[:120]
    torch.cuda.empty_cache()
    out["measured_peaks_file"] = {k: peaks[k] for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "source")}
    out["nominal"] = NOMINAL
    return out


# --------------------------------------------------------------------------- the other configurations

def time_calls_flushed(fn, iters, flush):
    """Per-call CUDA-event time with L2 overwritten before every call (inputs smaller than L2)."""
    fn()
    torch.cuda.synchronize()
    ms = []
    for _ in range(iters):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    ms.sort()
    return ms[len(ms) // 2]


def time_graph(run, replays):
    """Device time of one replay of `run` captured as a CUDA graph (ms)."""
    run()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        run()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            run()
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / replays


SWEEP_SECTIONS = ("quantize_sweep", "rmse", "rmse_sweep", "fake_quant", "decode", "depthwise", "gemm_batched", "gemm_sweep",
                  "bitwidth_search", "resnet50_b64_mixed")


def run_sweeps(dy, wl, device, peaks, only=None, log2n=28):
    """Configs 3-5 of the workload list (quantize/pack sweep, square GEMM sweep, ResNet-50 mixed bitwidths) and the
    kernels beyond the hot path.  `only`: names from SWEEP_SECTIONS to run (default all); `log2n`: size of the
    streaming-kernel cases (a smaller one keeps a profiler capture short)."""
    want = set(SWEEP_SECTIONS if not only else only)
    unknown = want - set(SWEEP_SECTIONS)
    if unknown:
        raise SystemExit(f"unknown sweep section(s) {sorted(unknown)}; choose from {SWEEP_SECTIONS}")
    out = {"peaks": peaks}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    if "quantize_sweep" in want:
        out["quantize_sweep"] = sweep_quantize(dy, wl, device, flush)
    if want & {"rmse", "rmse_sweep", "fake_quant", "decode"}:
        x = wl.normal((1 << log2n,), seed=5, device=device)
        if "rmse" in want:
            out["rmse"] = sweep_rmse(dy, x, log2n, flush)
        if "rmse_sweep" in want:
            out["rmse_sweep"] = sweep_rmse_candidates(dy, x, log2n, flush)
        if "fake_quant" in want:
            out["fake_quant"] = sweep_fake_quant(dy, x, log2n, flush)
        if "decode" in want:
            out["decode"] = sweep_decode(dy, x, log2n, flush)
        del x
        torch.cuda.empty_cache()
    if "depthwise" in want:
        out["depthwise"] = sweep_depthwise(dy, wl, device, peaks)
    if "gemm_batched" in want:
        out["gemm_batched"] = sweep_gemm_batched(dy, wl, device, peaks, flush)
    if "gemm_sweep" in want:
        out["gemm_sweep"] = []
        for fmt in ((4, 1), (8, 1)):
            for size in (1024, 2048, 4096, 8192):
                r = target_gemm(dy, wl, device, peaks, size=size, fmt=fmt)
                out["gemm_sweep"].append({"size": size, "bits": fmt[0], "container": r["container"],
                                          "tops_call": r["tops_call"], "tops_mma_kernel": r["tops_mma_kernel"],
                                          "library_matmul_tops": r.get("library_matmul_tops")})
    if "bitwidth_search" in want:
        out["bitwidth_search"] = run_search(dy, wl, device)
    if "resnet50_b64_mixed" in want:
        out["resnet50_b64_mixed"] = sweep_resnet50(dy, wl, device)
    return out


def sweep_quantize(dy, wl, device, flush):
    rows = []
    for log2n in (20, 22, 24, 26, 28, 30):
        n = 1 << log2n
        for dist in ("normal", "laplace", "half_normal"):
            x = wl.DISTRIBUTIONS[dist]((n,), seed=log2n, device=device)
            for bits in (2, 3, 4, 6, 8):
                fmt = (bits, 0 if dist == "half_normal" else 1)
                packed = torch.empty(dy.dybit_packed_bytes(n, bits), dtype=torch.uint8, device=device)
                scale = dy.dybit_absmax_scale(x, fmt)
                so = torch.empty(2, dtype=torch.float32, device=device)
                ms_g = time_calls_flushed(lambda: dy.dybit_quantize_pack(x, fmt, scale=scale, packed=packed), 7, flush)
                ms_m = time_calls_flushed(lambda: dy.dybit_quantize_pack(x, fmt, packed=packed, scale_out=so), 7, flush)
                row = {"log2n": log2n, "dist": dist, "bits": bits,
                       "gbs_scale_given": n * (4 + bits / 8) / ms_g / 1e6,
                       "gbs_with_max_abs": n * (8 + bits / 8) / ms_m / 1e6}
                if log2n <= 26 and dist == "normal":
                    # the same launch back to back over buffers that rotate through more than the L2 holds (one CUDA
                    # graph of nbuf launches): what a stream of such tensors sustains, without the per-launch gap of a
                    # lone, event-bracketed call
                    nbuf = min(64, max(4, (512 << 20) // (n * 4)))
                    xs = [x] + [x.clone() for _ in range(nbuf - 1)]
                    outs = [torch.empty_like(packed) for _ in range(nbuf)]

                    def run():
                        for xi, oi in zip(xs, outs):
                            dy.dybit_quantize_pack(xi, fmt, scale=scale, packed=oi)
                    ms_b = time_graph(run, 5) / nbuf
                    row["gbs_scale_given_back_to_back"] = n * (4 + bits / 8) / ms_b / 1e6
                    del xs, outs
                rows.append(row)
            del x
            torch.cuda.empty_cache()
    return rows


def sweep_rmse(dy, x, log2n, flush):
    """Eq. 2 error metric: one streaming pass, 4 B/element."""
    rows = []
    for bits in (2, 4, 8):
        scale = dy.dybit_absmax_scale(x, (bits, 1))
        res = torch.empty(4, dtype=torch.float64, device=x.device)
        ms = time_calls_flushed(lambda: dy.dybit_rmse(x, (bits, 1), scale, out=res), 7, flush)
        rows.append({"log2n": log2n, "bits": bits, "gbs": x.numel() * 4 / ms / 1e6, "rmse": res[0].item()})
    return rows


def sweep_rmse_candidates(dy, x, log2n, flush):
    """The same metric for several candidates in one pass: the 7 signed bitwidths, then 16 scales of one format."""
    rows = []
    fmts7 = [(b, 1) for b in range(2, 9)]
    sc7 = torch.stack([dy.dybit_absmax_scale(x, f) for f in fmts7]).contiguous()
    base = dy.dybit_absmax_scale(x, (4, 1))
    ratios = torch.linspace(1.0, 0.25, 16, device=x.device)
    sc16 = torch.stack([base[0] * ratios, 1.0 / (base[0] * ratios)], dim=1).contiguous()
    for what, fmts, sc in (("bitwidths 2..8 signed", fmts7, sc7), ("16 clipping ratios, 4-bit signed", [(4, 1)] * 16, sc16)):
        holder = {}

        def call():
            holder["r"] = dy.dybit_rmse_sweep(x, fmts, sc)
        ms = time_calls_flushed(call, 5, flush)
        res, best = holder["r"]
        rows.append({"log2n": log2n, "candidates": what, "n_cand": len(fmts), "ms": ms,
                     "gbs": x.numel() * 4 / ms / 1e6, "gelem_cand_per_s": x.numel() * len(fmts) / ms / 1e6,
                     "best": int(best.item()), "rmse": [float(v) for v in res[:, 0].tolist()]})
    return rows


def sweep_fake_quant(dy, x, log2n, flush):
    """QAT pair: quantize-dequantize image (8 B/element) and its clipped straight-through gradient (12 B/element)."""
    rows = []
    y = torch.empty_like(x)
    for fmt in ((4, 1), (8, 1), (2, 0)):
        scale = dy.dybit_absmax_scale(x, fmt)
        ms = time_calls_flushed(lambda: dy.dybit_fake_quant(x, fmt, scale, out=y), 5, flush)
        rows.append({"log2n": log2n, "fmt": list(fmt), "direction": "forward", "ms": ms, "gbs": x.numel() * 8 / ms / 1e6})
    g = torch.empty_like(x).normal_()
    ms = time_calls_flushed(lambda: dy.dybit_fake_quant_backward(x, g, (4, 1), scale, out=y), 5, flush)
    rows.append({"log2n": log2n, "fmt": [4, 1], "direction": "backward", "ms": ms, "gbs": x.numel() * 12 / ms / 1e6})
    return rows


def sweep_decode(dy, x, log2n, flush):
    """dybit_decode: packed codes back to fp32 (bits/8 B read + 4 B written per element)."""
    rows = []
    out = torch.empty_like(x)
    for fmt in ((2, 1), (4, 1), (6, 1), (8, 1)):
        packed, scale = dy.dybit_quantize_pack(x, fmt)
        ms = time_calls_flushed(lambda: dy.dybit_decode(packed, x.numel(), fmt, scale, out=out), 5, flush)
        rows.append({"log2n": log2n, "fmt": list(fmt), "ms": ms, "gbs": x.numel() * (4 + fmt[0] / 8) / ms / 1e6})
        del packed
    return rows


def sweep_depthwise(dy, wl, device, peaks):
    """Depth-wise convolutions of MobileNetV2 at batch 32, 4-bit: one CUDA graph over buffers that rotate through
    more than the L2 holds, so that the output stream goes to HBM."""
    rows = []
    for L in wl.mobilenetv2_depthwise_layers(32):
        if any(r["shape"] == [L.c, L.h, L.stride] for r in rows):
            continue
        fx, fw = (4, 0), (4, 1)
        d = dy.ConvDesc(L.n, L.h, L.w, L.c, L.c, L.r, L.s, L.stride, L.pad, 1)
        out_elems = L.n * L.oh * L.ow * L.c
        nbuf = min(64, max(2, int(300e6 // (out_elems * 4)) + 1))
        xs = [dy.dybit_quantize_pack(wl.half_normal((L.n, L.h, L.w, L.c), seed=i, device=device), fx) for i in range(nbuf)]
        ys = [torch.empty((L.n, L.oh, L.ow, L.c), dtype=torch.float32, device=device) for _ in range(nbuf)]
        pw, sw = dy.dybit_quantize_pack_2d(wl.normal((L.c, 9), seed=2, device=device), fw)

        def run():
            for (px, sx), y in zip(xs, ys):
                dy.dybit_depthwise_conv2d(d, px, fx, sx, pw, fw, sw, Y=y)
        ms = time_graph(run, 5) / nbuf
        nbytes = out_elems * 4 + L.n * L.h * L.w * L.c * fx[0] / 8
        rows.append({"shape": [L.c, L.h, L.stride], "us": ms * 1e3, "gbs": nbytes / ms / 1e6,
                     "frac_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"], "goutputs_per_s": out_elems / ms / 1e6})
        del xs, ys
        torch.cuda.empty_cache()
    return rows


def sweep_gemm_batched(dy, wl, device, peaks, flush):
    """ViT-Base attention products at batch 32 (12 heads): Q K^T and (attention) V as batched GEMMs."""
    rows = []
    for fmt in ((4, 1), (8, 1)):
        for (batch, M, N, K) in ((384, 197, 197, 64), (384, 197, 64, 197)):
            pa, sa = dy.dybit_quantize_pack_2d(wl.normal((batch * M, K), seed=1, device=device), fmt)
            pb, sb = dy.dybit_quantize_pack_2d(wl.normal((batch * N, K), seed=2, device=device), fmt)
            pa, pb = pa.reshape(batch, M, -1), pb.reshape(batch, N, -1)
            C = torch.empty((batch, M, N), dtype=torch.float32, device=device)
            ws = torch.empty(dy.dybit_gemm_batched_workspace_bytes(batch, M, N, K, fmt, fmt) + 1024, dtype=torch.uint8,
                             device=device)
            ms = time_calls_flushed(lambda: dy.dybit_gemm_batched(M, N, K, pa, fmt, sa, pb, fmt, sb, C=C, ws=ws), 7, flush)
            nbytes = batch * (M * N * 4 + (M + N) * K * fmt[0] / 8)
            rows.append({"batch": batch, "M": M, "N": N, "K": K, "bits": fmt[0], "us": ms * 1e3,
                         "tflops": 2 * batch * M * N * K / ms / 1e9, "gbs": nbytes / ms / 1e6,
                         "frac_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"]})
    return rows


def sweep_resnet50(dy, wl, device):
    layers = wl.resnet50_layers(64)
    bits = wl.mixed_bitwidths(len(layers), seed=0)
    work = LayerwiseStep(dy, wl, device, layers, bits, host_copies=False, n_streams=3)
    for _ in range(3):
        work.step()
    graph = capture_step(work, device)
    for _ in range(3):
        graph.replay()
    ms = timed_region(graph.replay, 10, None, device) / 10
    graph1 = capture_step(work, device, lambda: work.step(serial=True))
    for _ in range(3):
        graph1.replay()
    ms1 = timed_region(graph1.replay, 10, None, device) / 10
    del graph, graph1
    # the same step with the streaming launches folded over the layers (dybit_quantize_expand_layers: one max-abs
    # launch per 32 layers, one quantize + expand launch per pair of formats), then the convolutions on three streams
    ms_fold, fold_launches, fold_variants = None, None, {}
    try:
        work.folded = dy.ConvLayers([dict(desc=work.desc[i], X=work.x_dev[i], fx=work.fa[i], W=work.pw[i], fw=work.fw[i],
                                          scale_w=work.sw[i], packed=work.px[i], scale_out=work.sx[i], Y=work.y[i])
                                     for i in range(len(layers))])
        work.fold = True
        best = None
        for shared in (False, True):      # tensor-core launches per layer on three streams / shared, on one stream
            work.shared_launches = shared
            for _ in range(3):
                work.step()
            n0 = dy.dybit_launch_count()
            graph_f = capture_step(work, device)
            launches = dy.dybit_launch_count() - n0
            for _ in range(3):
                graph_f.replay()
            t = timed_region(graph_f.replay, 10, None, device) / 10
            del graph_f
            fold_variants = dict(fold_variants, **{("shared_launches" if shared else "per_layer_launches_3_streams"):
                                                   {"ms_per_step": t, "launches": launches}})
            if best is None or t < best:
                best, fold_launches = t, launches
        ms_fold = best
    except dy.DybitError as exc:        # a layer whose lowering has no fused expand
        ms_fold = None
        fold_note = str(exc)
    work.fold = False
    conts = [CONTAINERS[dy.dybit_choose_container(fa, fw)[0]] for fa, fw in zip(work.fa, work.fw)]
    return {"ms_per_step": ms, "ms_per_step_one_stream": ms1, "streams": 3,
            "ms_per_step_folded": ms_fold, "launches_per_folded_step": fold_launches, "folded_variants": fold_variants,
            "tops": 2.0 * work.macs / (ms * 1e-3) / 1e12, "layers": len(layers), "seed": 0,
            "containers": {c: conts.count(c) for c in sorted(set(conts))}, "bits_w_a": bits}


def run_search(dy, wl, device, batch=32, alpha=3.0, beta=3.0, top_k=4):
    """Algorithm 1 on the ResNet-18 shapes with MEASURED per-layer latencies (quantize + conv on this GPU, in place of
    the paper's accelerator simulator) and Eq. 2 errors (weights' RMSE + activations' RMSE) for a, w in {8, 4, 2}."""
    layers = wl.resnet18_layers(batch)
    levels = (8, 4, 2)
    lat, err = [], []
    for i, L in enumerate(layers):
        x = wl.half_normal((L.n, L.h, L.w, L.c), seed=1000 + i, device=device)
        w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2000 + i).reshape(L.k, -1).to(device)
        d = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
        y = torch.empty((L.n, L.oh, L.ow, L.k), dtype=torch.float32, device=device)
        ra = {a: dy.dybit_rmse(x.reshape(-1), (a, 0), dy.dybit_absmax_scale(x, (a, 0)))[0].item() for a in levels}
        rw = {b: dy.dybit_rmse(w.reshape(-1), (b, 1), dy.dybit_absmax_scale(w, (b, 1)))[0].item() for b in levels}
        for a in levels:
            for b in levels:
                fa, fw = (a, 0), (b, 1)
                pw, sw = dy.dybit_quantize_pack_2d(w, fw)
                px = torch.empty(dy.dybit_packed_bytes(x.numel(), a), dtype=torch.uint8, device=device)
                sx = torch.empty(2, dtype=torch.float32, device=device)
                ws = torch.empty(dy.dybit_conv2d_workspace_bytes(d, fa, fw) + 1024, dtype=torch.uint8, device=device)

                def layer_call():
                    dy.dybit_quantize_pack(x, fa, packed=px, scale_out=sx)
                    dy.dybit_conv2d(d, px, fa, sx, pw, fw, sw, Y=y, ws=ws)
                lat.append(time_calls(layer_call, 5, warmup=2))
                err.append(ra[a] + rw[b])
    n = len(layers)
    base = sum(lat[i * 9] for i in range(n))
    res = {"alpha": alpha, "beta": beta, "top_k": top_k, "latency_ms_all_8bit": base}
    for strategy, c in (("speedup", alpha), ("rmse", beta)):
        W, A = dy.dybit_search_bitwidths(lat, err, n, strategy, c, top_k)
        idx = {8: 0, 4: 1, 2: 2}
        cur = sum(lat[(i * 3 + idx[A[i]]) * 3 + idx[W[i]]] for i in range(n))
        cur_e = sum(err[(i * 3 + idx[A[i]]) * 3 + idx[W[i]]] for i in range(n))
        res[strategy] = {"w_bits": W, "a_bits": A, "latency_ms": cur, "speedup": base / cur,
                         "rmse_ratio": cur_e / sum(err[i * 9] for i in range(n))}
    return res


CONTAINERS = {0: "int8", 1: "e4m3", 2: "bf16"}


# --------------------------------------------------------------------------- CPU oracle legs

def oracle_step(orc, wl, batch):
    """The same step on the CPU oracle at the given batch.  Returns (seconds, MACs)."""
    layers = wl.resnet18_layers(batch)
    inputs = []
    for i, L in enumerate(layers):
        x = wl.half_normal((L.n, L.h, L.w, L.c), seed=1000 + i).numpy()
        w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2000 + i).numpy()
        sw = orc.absmax_scale(w, FMT_W[0], True)
        cw = orc.quantize(w, FMT_W[0], True, sw[1])
        inputs.append((L, x, cw, sw))
    t0 = time.perf_counter()
    for L, x, cw, sw in inputs:
        sx = orc.absmax_scale(x, FMT_A[0], False)
        cx = orc.quantize(x, FMT_A[0], False, sx[1])
        orc.pack(cx, FMT_A[0])
        orc.conv2d(cx, FMT_A, sx[0], cw, FMT_W, sw[0], stride=L.stride, pad=L.pad)
    return time.perf_counter() - t0, sum(L.macs for L in layers)


def cpu_baseline(wl, budget_s=15.0):
    from oracle import dybit_oracle as orc
    t1, macs1 = oracle_step(orc, wl, 1)
    batch = max(1, min(32, int(budget_s / max(t1, 1e-3))))
    if batch > 1:
        t, macs = oracle_step(orc, wl, batch)
    else:
        t, macs = t1, macs1
    r50 = sum(L.macs for L in wl.resnet50_layers(64))
    return {"value": 2.0 * macs / t / 1e12, "unit": "TOPS", "cores": orc.threads(), "kind": "oracle",
            "sample": f"the same 21-layer step at batch {batch} ({t:.1f} s on the host)",
            "resnet50_b64_mixed_extrapolated": {
                "seconds_per_step": r50 / (macs / t), "how": "extrapolated: the multiply-add rate measured on the ResNet-18 "
                "sample x the multiply-adds of the 54-layer batch-64 step (the oracle's convolution loop does the same work "
                "per multiply-add whatever the bitwidths)"}}


def load_workloads_alone():
    """The shape tables and seeded generators without the package around them: importing the package would map
    libdybit.so into this process, and the reference arm runs nothing of the product."""
    import importlib.util
    path = os.path.join(ROOT, "paper_2302_12510_b200", "workloads.py")
    spec = importlib.util.spec_from_file_location("dybit_workloads_standalone", path)
    mod = importlib.util.module_from_spec(spec)
    sys.modules[spec.name] = mod          # dataclasses looks the module up by name
    spec.loader.exec_module(mod)
    return mod


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = load_workloads_alone()
    from oracle import dybit_oracle as orc
    t1, _ = oracle_step(orc, wl, 1)
    per_step_budget = 120.0 / max(1, args.steps + args.warmup)
    batch = max(1, min(args.batch, int(per_step_budget / max(t1, 1e-3))))
    for _ in range(args.warmup):
        oracle_step(orc, wl, batch)
    total_t, total_macs = 0.0, 0
    for _ in range(args.steps):
        t, macs = oracle_step(orc, wl, batch)
        total_t += t
        total_macs += macs
    value = 2.0 * total_macs / total_t / 1e12
    sample = f"21-layer step at batch {batch} per step"
    print(json.dumps({
        "impl": "reference", "metric": "dybit_resnet18_w4a4_step_tops", "value": value, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_t / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": workload_name(args.batch), "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": orc.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dybit", choices=["dybit", "reference"])
    ap.add_argument("--batch", type=int, default=32, help="images per step (32 = the quoted configuration)")
    ap.add_argument("--streams", type=int, default=3,
                    help="streams the step's independent layers are issued on, round-robin (1 = one after the other)")
    ap.add_argument("--per-layer-calls", action="store_true",
                    help="time one dybit_quantize_conv2d call per layer as the step instead of the folded "
                         "dybit_quantize_expand_layers + dybit_conv2d_prepared sequence")
    ap.add_argument("--no-targets", action="store_true", help="skip the single-kernel target measurements")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--step-only", action="store_true",
                    help="only the step itself (graph replays, direct launches, end to end): no device-clock pass, no "
                         "re-quantizing or two-call variants, no targets, no CPU baseline (for profiler captures)")
    ap.add_argument("--conv-layer", default="",
                    help="run only this ResNet-18 layer (e.g. layer1.0.conv1) at --batch, a few calls (for profiler captures)")
    ap.add_argument("--targets-only", action="store_true",
                    help="run only the single-kernel target measurements (small cases for profiler captures)")
    ap.add_argument("--gemm-size", type=int, default=8192, help="M=N=K of the square 4-bit GEMM target")
    ap.add_argument("--quant-log2n", type=int, default=28, help="log2 of the element count of the quantize target")
    ap.add_argument("--quant-bits", type=int, default=4)
    ap.add_argument("--sweeps", action="store_true",
                    help="measure the other configurations instead (quantize sweep, square GEMM sweep, "
                         "ResNet-50 batch 64 with mixed bitwidths) and print them as one JSON object")
    ap.add_argument("--only", default="",
                    help="with --sweeps: comma-separated sections to run (" + ", ".join(SWEEP_SECTIONS) + ")")
    ap.add_argument("--sweep-log2n", type=int, default=28,
                    help="with --sweeps: log2 of the element count of the rmse / fake_quant cases")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the DyBit path has no CPU fallback")
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod

    import paper_2302_12510_b200 as dy
    from paper_2302_12510_b200 import workloads as wl
    peaks = load_peaks()
    warmup = max(3, args.warmup)
    if args.sweeps:
        only = [t for t in args.only.split(",") if t] if args.only else None
        print(json.dumps({"sweeps": run_sweeps(dy, wl, device, peaks, only=only, log2n=args.sweep_log2n)}))
        return
    if args.conv_layer:
        # one layer of the step alone (a small case for a profiler capture): a few dybit_quantize_conv2d calls
        layers = [L for L in wl.resnet18_layers(args.batch) if L.name == args.conv_layer]
        if not layers:
            raise SystemExit(f"no layer named {args.conv_layer}; names: {[L.name for L in wl.resnet18_layers(1)]}")
        work = LayerwiseStep(dy, wl, device, layers, [(FMT_W[0], FMT_A[0])], host_copies=False)
        ms = time_calls(work.step, max(1, args.steps), warmup=warmup)
        print(json.dumps({"conv_layer": args.conv_layer, "batch": args.batch, "us_per_call": ms * 1e3,
                          "device_status": dy.dybit_last_device_status()}))
        return
    if args.targets_only:
        out = {}
        if args.gemm_size > 0:
            out["gemm_w4a4"] = target_gemm(dy, wl, device, peaks, size=args.gemm_size)
        if args.quant_log2n > 0:
            out["quantize_pack"] = target_quantize(dy, wl, device, peaks, log2n=args.quant_log2n, bits=args.quant_bits)
            out["quantize_expand"] = target_quantize_expand(dy, wl, device, peaks, log2n=min(args.quant_log2n, 26))
        print(json.dumps({"targets": out}))
        return

    layers = wl.resnet18_layers(args.batch)
    work = LayerwiseStep(dy, wl, device, layers, [(FMT_W[0], FMT_A[0])] * len(layers), n_streams=args.streams,
                         fold=not args.per_layer_calls)
    for _ in range(warmup):
        work.step()
    torch.cuda.synchronize()
    st, detail = dy.dybit_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} detail {detail:#x}")

    # ---- one step captured as a CUDA graph (the library's calls are plain stream work, so they capture; the side
    #      streams fork from and join the capturing stream)
    launches0 = dy.dybit_launch_count()
    graph = capture_step(work, device)
    launches_per_step = dy.dybit_launch_count() - launches0
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()

    # ---- timed region: K replays, inputs resident in HBM (footprint per step > L2, see config)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms_total = timed_region(graph.replay, args.steps, dist, device)
    launches = launches_per_step * args.steps
    ms_step = ms_total / args.steps
    value = whole_job_tops(work.macs, world, ms_step)

    # ---- the same step as one dybit_quantize_conv2d call per layer on the same streams (three launches per layer)
    ms_per_layer_calls = None
    if work.fold:
        work.fold = False
        graph_pl = capture_step(work, device)
        for _ in range(warmup):
            graph_pl.replay()
        ms_per_layer_calls = timed_region(graph_pl.replay, args.steps, dist, device) / args.steps
        del graph_pl
        work.fold = True
    # ---- the same step with every layer on one stream (what the per-kernel figures below are taken from)
    graph_serial = capture_step(work, device, lambda: work.step(serial=True))
    for _ in range(warmup):
        graph_serial.replay()
    ms_serial = timed_region(graph_serial.replay, args.steps, dist, device) / args.steps
    del graph_serial
    # ---- the same K steps launched directly (host-bound: every launch goes through the Python binding)
    ms_eager = timed_region(work.step, args.steps, dist, device) / args.steps
    # ---- and with events around each layer's tensor-core kernel, one stream.  A spin kernel is queued in front of
    #      every profiled step so that the host has submitted the whole step before the GPU starts it: the event
    #      pairs then bracket the kernel itself, not the wait for its launch to arrive.
    events = [[] for _ in work.layers]
    prof_steps = max(3, min(args.steps, 20))

    def profiled_step():
        torch.cuda._sleep(5_000_000)        # ~2.5 ms at 1965 MHz; one directly launched step takes ~1 ms of host time
        work.step(events)

    timed_region(profiled_step, prof_steps, dist, device)
    st, detail = dy.dybit_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} detail {detail:#x}")
    # ---- and on the device's own clock inside graph replays: per layer, first CTA past the dependency wait to last
    #      CTA retired (the event pairs above also contain the launch latency that the graph's overlapped launches hide)
    clk = torch.empty((len(work.layers), 2), dtype=torch.int64, device=device)
    graph_c = capture_step(work, device, lambda: work.step(clocks=clk))
    clock_us = [0.0] * len(work.layers)
    clock_reps = 1 if args.step_only else 10
    for rep in range(clock_reps + (0 if args.step_only else 2)):
        clk[:, 0] = -1
        clk[:, 1] = 0
        graph_c.replay()
        torch.cuda.synchronize(device)
        if rep >= 2 or args.step_only:
            span = (clk[:, 1] - clk[:, 0]).cpu().tolist()
            clock_us = [a + s * 1e-3 / clock_reps for a, s in zip(clock_us, span)]
    del graph_c
    mma_ms = [sum(e0.elapsed_time(e1) for e0, e1 in ev) / len(ev) for ev in events]
    mma_total_ms = sum(mma_ms)
    peak_tensor = 2.0 * peaks["bf16_tflops_sustained"]      # int8 = 2 x bf16 (nominal ratio), sustained: inside a long step
    bounds = work.layer_bounds(peak_tensor, peaks["hbm_gbs"])
    flops_total = sum(b[0] for b in bounds)
    bytes_total = sum(b[1] for b in bounds)
    ideal_s = sum(b[2] for b in bounds)
    tensor_bound = flops_total / (peak_tensor * 1e12) >= bytes_total / (peaks["hbm_gbs"] * 1e9)
    if tensor_bound:
        achieved, peak, unit = flops_total / (mma_total_ms * 1e-3) / 1e12, peak_tensor, "TFLOP/s"
    else:
        achieved, peak, unit = bytes_total / (mma_total_ms * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s"
    roofline_conv = {
        "kernel": "dybit_conv_halo_kernel<I8> / dybit_gemm_kernel<I8, conv> (21 launches per step, one per layer)",
        "workload": f"resnet18_b{args.batch}_w4a4, the 21 layers of one step",
        "bound": "tensor" if tensor_bound else "hbm", "achieved": achieved, "peak": peak, "unit": unit,
        "frac": achieved / peak,
        "traffic": NCU_TRAFFIC["conv_step"] if args.batch == 32 else None,
        "traffic_how": NCU_TRAFFIC_HOW["conv_step"],
        "peak_how": (f"2 x sustained bf16 ({peaks['source']})" if tensor_bound else f"copy bandwidth ({peaks['source']})"),
        "how": "CUDA events recorded by the library around this kernel alone, in %d directly launched single-stream steps "
               "right after the timed region, each queued behind a spin kernel so that launches never arrive late" % prof_steps,
        "ms_per_step_in_kernel": mma_total_ms, "ms_per_step_one_stream": ms_serial,
        "ms_per_step_direct_launch": ms_eager,
        "layers_us": {L.name: [round(t * 1e3, 1), round(b[2] * 1e6, 1)] for L, t, b in zip(work.layers, mma_ms, bounds)},
        "frac_of_layerwise_bound": ideal_s / (mma_total_ms * 1e-3),
        "device_clock": {
            "what": "the same kernel timed by %%globaltimer inside CUDA-graph replays of the single-stream step "
                    "(dybit_profile_next_gemm_clock): first CTA past its dependency wait to last CTA retired, mean of %d replays" % clock_reps,
            "ms_per_step_in_kernel": sum(clock_us) * 1e-3,
            "achieved": (flops_total / 1e12 if tensor_bound else bytes_total / 1e9) / (sum(clock_us) * 1e-6),
            "frac": (flops_total / 1e12 if tensor_bound else bytes_total / 1e9) / (sum(clock_us) * 1e-6) / peak,
            "frac_of_layerwise_bound": ideal_s / (sum(clock_us) * 1e-6),
            "layers_us": {L.name: round(t, 1) for L, t in zip(work.layers, clock_us)}},
        "algorithmic_flops_per_step": flops_total, "algorithmic_bytes_per_step": bytes_total,
    }
    if work.fold:
        # the two halves of the timed step on their own (graph replays): the folded streaming launches, and the 21
        # tensor-core problems in shared launches against the same layer-wise bound
        g_a = capture_step(work, device, lambda: dy.dybit_quantize_expand_layers(work.folded))
        g_b = capture_step(work, device, lambda: dy.dybit_conv2d_prepared_layers(work.folded))
        for _ in range(3):
            g_a.replay()
            g_b.replay()
        ms_a = timed_region(g_a.replay, args.steps, dist, device) / args.steps
        n0 = dy.dybit_launch_count()
        dy.dybit_conv2d_prepared_layers(work.folded)
        conv_launches = dy.dybit_launch_count() - n0
        ms_b = timed_region(g_b.replay, args.steps, dist, device) / args.steps
        del g_a, g_b
        roofline_conv["shared_launches"] = {
            "what": "dybit_conv2d_prepared_layers alone (the tensor-core part of the timed step: problems of one kernel "
                    "configuration share a launch), CUDA-graph replays",
            "launches": conv_launches, "ms_per_step": ms_b,
            "achieved": (flops_total / 1e12 if tensor_bound else bytes_total / 1e9) / (ms_b * 1e-3),
            "frac": (flops_total / 1e12 if tensor_bound else bytes_total / 1e9) / (ms_b * 1e-3) / peak,
            "frac_of_layerwise_bound": ideal_s / (ms_b * 1e-3),
            "streaming_launches_ms_per_step": ms_a}
        # the figures at the top of this object are those of the configuration the step is timed in (shared launches);
        # the launch-by-launch ones (events and device clock per layer) move one level down
        sl = roofline_conv["shared_launches"]
        roofline_conv["per_layer_launches"] = {k: roofline_conv[k] for k in ("achieved", "frac", "frac_of_layerwise_bound", "how",
                                                                             "ms_per_step_in_kernel")}
        roofline_conv.update({"achieved": sl["achieved"], "frac": sl["frac"], "frac_of_layerwise_bound": sl["frac_of_layerwise_bound"],
                              "ms_per_step_in_kernel": ms_b,
                              "kernel": "dybit_conv_halo_multi_kernel<I8> / dybit_gemm_multi_kernel<I8, conv> (%d launches per step "
                                        "for the 21 layers)" % conv_launches,
                              "how": "CUDA-graph replays of dybit_conv2d_prepared_layers alone, CUDA events around K replays"})
    # whole step against its memory roofline: fp32 activation read twice (max-abs, quantize), codes written, conv traffic
    step_bytes = work.quant_elems * (8.0 + FMT_A[0] / 8.0) + bytes_total
    roofline_conv["whole_step"] = {"algorithmic_bytes": step_bytes, "gbs": step_bytes / (ms_step * 1e-3) / 1e9,
                                   "frac_of_hbm_peak": step_bytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    # ---- end to end: activations from pinned host memory each step, outputs copied back
    work.alloc_host_outputs()
    for _ in range(2):
        work.step_e2e()
    work.e2e_join()
    e2e_steps = max(2, min(args.steps, 10))

    def e2e_run():
        for _ in range(e2e_steps):
            work.step_e2e()
        work.e2e_join()                # the closing event then also covers the copies still in flight

    ms_e2e = timed_region(e2e_run, 1, dist, device) / e2e_steps
    for i in (0, len(work.layers) // 2, len(work.layers) - 1):       # what came back is what the device holds
        if not torch.equal(work.y_host[i], work.y[i].cpu()):
            raise SystemExit(f"end-to-end step: host copy of layer {i}'s output differs from the device tensor")
    clocks = sampler.stop() if rank == 0 else None       # sampled over the timed region, the direct pass and the e2e steps
    e2e = {"value": whole_job_tops(work.macs, world, ms_e2e), "unit": "TOPS",
           "how": "per layer: pinned host -> device copy of the fp32 activation, dybit_quantize_conv2d, device -> pinned "
                  "host copy of the fp32 output; three streams, so both copy directions and the kernels overlap",
           "ms_per_step": ms_e2e, "h2d_bytes_per_step": work.h2d_bytes, "d2h_bytes_per_step": work.d2h_bytes}

    result = {
        "metric": "dybit_resnet18_w4a4_step_tops", "value": value, "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": workload_name(args.batch),
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "launch": ("dybit_quantize_expand_layers for the 21 independent layers (one max-abs launch, one quantize + "
                              "expand launch), then dybit_conv2d_prepared_layers (the 21 tensor-core problems in shared "
                              "launches, one per kernel configuration), all on one stream; " if work.fold else
                              "one dybit_quantize_conv2d call per layer; the 21 independent layers are issued round-robin on "
                              "%d streams (one workspace each) that fork from and join the step's stream; " % work.n_streams)
                             + "one step captured once as a CUDA graph, timed region = K replays",
                   "streams": work.n_streams,
                   "l2": "per-step footprint (fp32 inputs %.0f MB + fp32 outputs %.0f MB) exceeds the 126 MB L2"
                         % (work.h2d_bytes / 1e6, work.d2h_bytes / 1e6)},
        "gpu_launches": launches, "clocks": clocks, "e2e": e2e, "roofline_conv": roofline_conv,
        "quantize_elems_per_step": work.quant_elems,
    }
    if ms_per_layer_calls is not None:
        result["per_layer_call_step"] = {
            "what": "the same step as one dybit_quantize_conv2d call per layer (max-abs, quantize + expand and the "
                    "tensor-core kernel launched layer by layer), round-robin on %d streams" % work.n_streams,
            "ms_per_step": ms_per_layer_calls, "value": whole_job_tops(work.macs, world, ms_per_layer_calls), "unit": "TOPS"}
    if args.step_only:
        result["roofline"] = roofline_conv
        if rank == 0:
            print(json.dumps(result))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    # ---- the same step with the re-quantizing epilogue (results leave as 4-bit codes instead of fp32)
    work.prepare_requant()
    for _ in range(3):
        work.step_requant()
    graph_q = capture_step(work, device, work.step_requant)
    for _ in range(3):
        graph_q.replay()
    ms_q = timed_region(graph_q.replay, args.steps, dist, device) / args.steps
    result["requant_epilogue"] = {
        "what": "same 21 layers, launched the same way, results written back as unsigned 4-bit DyBit codes (ReLU + encode in "
                "the GEMM epilogue, given output scales) instead of fp32",
        "ms_per_step": ms_q, "value": whole_job_tops(work.macs, world, ms_q), "unit": "TOPS",
        "output_bytes_per_step": work.q_bytes, "fp32_output_bytes_per_step": work.d2h_bytes}
    # ---- the same step as two library calls per layer (dybit_quantize_pack, then dybit_conv2d): one more launch each
    work.two_calls = True
    for _ in range(3):
        work.step()
    launches0 = dy.dybit_launch_count()
    graph_2 = capture_step(work, device)
    launches_2 = dy.dybit_launch_count() - launches0
    for _ in range(3):
        graph_2.replay()
    ms_2 = timed_region(graph_2.replay, args.steps, dist, device) / args.steps
    result["two_call_step"] = {"what": "dybit_quantize_pack + dybit_conv2d per layer instead of dybit_quantize_conv2d",
                               "ms_per_step": ms_2, "value": whole_job_tops(work.macs, world, ms_2), "unit": "TOPS",
                               "gpu_launches_per_step": launches_2}
    del work, graph, graph_q, graph_2
    torch.cuda.empty_cache()

    if rank == 0 and not args.no_targets:
        here = measure_peaks_here(device, peaks)
        result["peaks_measured_here"] = here
        g = target_gemm(dy, wl, device, peaks, size=args.gemm_size)
        q = target_quantize(dy, wl, device, peaks, log2n=args.quant_log2n, bits=args.quant_bits)
        result["targets"] = {"gemm_w4a4": g, "quantize_pack": q, "gemm_decode": target_gemm_decode(dy, wl, device),
                             "quantize_expand": target_quantize_expand(dy, wl, device, peaks)}
        # the metric's two figures as roofline objects: the tensor-core kernel of the square GEMM against the int8
        # tensor peak, the quantize/pack kernel (scale given) against the copy bandwidth
        lib_int8 = here.get("int8_matmul_tops")
        ratio_peak = 2.0 * peaks["bf16_tflops"]
        peak_g = max(ratio_peak, lib_int8 or 0.0)
        result["roofline"] = {
            "kernel": "dybit_gemm_pair_kernel<I8> (tcgen05 cta_group::2, 256 x 256 tiles)",
            "workload": f"M=N=K={args.gemm_size}, signed 4-bit x signed 4-bit DyBit codes, int8 container, fp32 output",
            "bound": "tensor", "achieved": g["tops_mma_kernel"], "peak": peak_g, "unit": "TFLOP/s",
            "frac": g["tops_mma_kernel"] / peak_g,
            "traffic": NCU_TRAFFIC["gemm_8192"] if args.gemm_size == 8192 else None,
            "traffic_how": NCU_TRAFFIC_HOW["gemm_8192"],
            "peak_how": "the larger of (a) a dense int8 library matmul of the same shape timed in this run "
                        f"({lib_int8 and round(lib_int8, 1)} TOPS) and (b) 2 x the bf16 burst peak of MEASURED_PEAKS.json "
                        f"({ratio_peak:.1f}; {peaks['source']}; int8 : bf16 = 2 : 1 nominal).  Integer multiply-adds counted as 2 ops",
            "frac_of_int8_library_matmul": (g["tops_mma_kernel"] / lib_int8) if lib_int8 else None,
            "frac_of_2x_bf16_peak": g["tops_mma_kernel"] / ratio_peak,
            "frac_of_nominal_int8": g["tops_mma_kernel"] / NOMINAL["int8_tops"],
            "how": "CUDA events recorded by the library around the tensor-core kernel alone (median of 10 calls); the whole "
                   "call, expand launch included, is `per_call`",
            "ms_kernel": g["ms_mma_kernel"],
            "per_call": {"ms": g["ms_call"], "achieved": g["tops_call"], "frac": g["tops_call"] / peak_g},
            "algorithmic_flops_per_launch": 2.0 * args.gemm_size ** 3,
        }
        n_q = 1 << args.quant_log2n
        result["roofline_quantize"] = {
            "kernel": f"quantize_pack_kernel<{args.quant_bits}, signed>",
            "workload": f"2^{args.quant_log2n} fp32 elements from N(0,1), signed {args.quant_bits}-bit DyBit, scale given",
            "bound": "hbm", "achieved": q["scale_given"]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": q["scale_given"]["frac"],
            "traffic": (NCU_TRAFFIC["quantize_2p26_per_element"] * n_q
                        if args.quant_bits == 4 and NCU_TRAFFIC["quantize_2p26_per_element"] is not None else None),
            "traffic_how": NCU_TRAFFIC_HOW["quantize_2p26_per_element"],
            "peak_how": f"copy bandwidth of MEASURED_PEAKS.json ({peaks['source']}); a device-to-device copy timed in this "
                        f"run: {here.get('copy_gbs') and round(here['copy_gbs'], 1)} GB/s",
            "how": "CUDA events around 10 back-to-back calls (one kernel each); input 1 GiB, far larger than L2",
            "algorithmic_bytes_per_launch": n_q * (4 + args.quant_bits / 8),
            "with_max_abs": q["with_max_abs"],
        }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


if __name__ == "__main__":
    main()
