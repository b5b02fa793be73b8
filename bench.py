#!/usr/bin/env python
"""Benchmark of the NVFP4 W4A4 linear-layer path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mlp|gdn|linear] [--tokens M]
    python bench.py --impl reference ...        # times the CPU oracle instead

Default workload ("mlp"): one step = one pass of the hot path over the MLP prefill
pair of a 27B-class hybrid layer, M = 8192 tokens:
    quantize X1 [8192 x 5120] -> fused gate/up GEMM (N = 2 x 17408, two segments,
    separate global scales) -> quantize X2 [8192 x 17408] -> down GEMM (N = 5120).
The headline value is GEMM FLOPs of the step divided by the WHOLE step time
(quantization included).  Also reported: the GEMM's roofline fraction (events around
each launch inside the timed region), the quantize kernel alone on the heavy-tailed
8192 x 5120 activation tensor ("quantize"), the producer-fused quantizers, an
end-to-end arm with host buffers ("e2e") and the CPU oracle on a sample ("cpu_baseline").

Prints one JSON line (rank 0).  Multi-GPU runs are independent replicas (the path
has no exchange step): every rank runs the same step on its own GPU.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_04098_b200 import synth  # noqa: E402

HIDDEN, INNER = synth.HIDDEN, synth.MLP_INNER
NOMINAL_FP4_TFLOPS = 9000.0
NOMINAL_HBM_GBS = 8000.0
FP4_OVER_BF16 = 4.0          # nominal dense FP4 : bf16 tensor throughput on B200 (9 : 2.25 PFLOP/s)
QUANT_BYTES_PER_ELEM = 2.0 + 0.5 + 1.0 / 16.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def tensor_peak(peaks, timed_seconds: float, clocks: dict):
    """Which measured bf16 figure the FP4 roofline is built on (x 4, the nominal FP4 : bf16 ratio):
    the burst figure when the timed region was short and never power-capped (the clocks then sit
    at their maximum, as they did when the burst figure was taken), the sustained one otherwise."""
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    burst = timed_seconds < 1.0 and not capped
    base = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    basis = "%s bf16 %s %.1f TFLOP/s x %.0f (nominal FP4:bf16 ratio); timed region %.3f s, %s" % (
        peaks["source"], "burst" if burst else "sustained", base, FP4_OVER_BF16, timed_seconds,
        "power cap seen" if capped else "no power cap seen")
    return base * FP4_OVER_BF16, basis


def ncu_traffic(name: str):
    """DRAM bytes per launch from the committed ncu summary (profiles/traffic.json), or None."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        return json.load(f).get(name)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML every few milliseconds while
    the timed region runs (reading only; no setting is touched)."""
    BITS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period = index, period_s
        self.sm, self.power, self.reasons = [], [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self.thread = None
        self.err = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if vis:
                try:
                    idx = int(vis.split(",")[self.index])
                except ValueError:
                    idx = self.index
            h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                      # noqa: BLE001
            self.err = "nvml unavailable: %s" % e
            return

        def loop():
            while not self._stop.is_set():
                try:
                    self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                    self.power.append(pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0)
                    r = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                    for bit, name in self.BITS.items():
                        if r & bit:
                            self.reasons.add(name)
                except Exception as e:              # noqa: BLE001
                    self.err = str(e)
                    return
                time.sleep(self.period)

        self.thread = threading.Thread(target=loop, daemon=True)
        self.thread.start()

    def stop(self):
        self._stop.set()
        if self.thread is not None:
            self.thread.join(timeout=2)
        out = {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
               "sm_mhz_min": min(self.sm) if self.sm else None, "samples": len(self.sm),
               "power_w_max": max(self.power) if self.power else None, "reasons": sorted(self.reasons)}
        if self.err:
            out["note"] = self.err
        return out


# --------------------------------------------------------------------------- workloads
def gemm_flops(M, N, K):
    return 2.0 * M * N * K


class MlpPair:
    """configs[2]: MLP prefill pair, M tokens."""
    name = "mlp_prefill_pair"

    def __init__(self, M=8192):
        self.M = M
        self.seg_gu = synth.make_segments((("gate", INNER, 0.02), ("up", INNER, 0.02)))
        self.seg_d = synth.make_segments((("down", HIDDEN, 0.02),))
        self.flops = gemm_flops(M, 2 * INNER, HIDDEN) + gemm_flops(M, HIDDEN, INNER)
        self.quant_elems = M * HIDDEN + M * INNER
        self.describe = ("configs[2] MLP prefill pair: M=%d, gate/up K=5120->N=2x17408 (2 segments), "
                         "down K=17408->N=5120; activation quantize inside the step" % M)

    def host_inputs(self, seed=0):
        return {"x1": synth.prefill_activations(seed, 301, self.M, HIDDEN),
                "x2": synth.prefill_activations(seed, 303, self.M, INNER),
                "w_gu": synth.weights(seed, 302, self.seg_gu, HIDDEN),
                "w_d": synth.weights(seed, 304, self.seg_d, INNER)}


class GdnProj:
    """configs[3]: fused GDN in-projection, six segments."""
    name = "gdn_in_projection"

    def __init__(self, M=8192):
        self.M = M
        self.segs = synth.make_segments(synth.GDN_SEGMENTS)
        self.N = 16480
        self.flops = gemm_flops(M, self.N, HIDDEN)
        self.quant_elems = M * HIDDEN
        self.describe = "configs[3] fused GDN in-projection: M=%d, K=5120, N=16480 in 6 segments" % M


class OneLinear:
    """configs[4]: one K=5120 -> N=6144 layer at a given M, quantize inside the timed call."""
    name = "linear_5120_6144"

    def __init__(self, M):
        self.M = M
        self.segs = synth.make_segments((("w", 6144, 0.02),))
        self.N = 6144
        self.flops = gemm_flops(M, self.N, HIDDEN)
        self.quant_elems = M * HIDDEN
        self.describe = "configs[4] linear K=5120->N=6144 at M=%d, quantize fused into the timed call" % M


# --------------------------------------------------------------------------- other configs, same JSON line
def measure_configs(torch, nv, dev, peaks, seed):
    """configs[3] (fused GDN in-projection, six segments) and configs[4] (K=5120 -> N=6144 at
    M in {1 .. 32768}, quantize inside the timed call), each timed for a few hundred ms at most.
    Every timed call goes through nvfp4_linear_bf16.  Weights rotate through enough copies to
    exceed L2 (a model streams each layer's weights from HBM; one layer replayed would sit in
    L2); activations and outputs rotate too where they are large.  Decode-sized shapes are timed as
    a CUDA-graph replay, so the host's launch cost is not what is measured."""
    stream = torch.cuda.current_stream()

    def up(bits):
        return synth.to_torch_bf16(bits).to(dev)

    def time_layer(M, segs, hx, w_c, w_sf, g_w, n_wsets, reps, graph):
        N = sum(s.count for s in segs)
        per_set = M * HIDDEN * 2 + M * N * 2
        # activations and outputs rotate through enough buffers to exceed L2 -- except at decode sizes:
        # there the activations of a layer were written by the kernel in front of it a few microseconds
        # earlier and are L2-resident in any real chain, while the rotating weights (17.7 MB per call)
        # would evict a rotated 40 KB input and put an HBM round trip in front of every call
        nset = 1 if graph else max(1, min(6, int(np.ceil(300e6 / per_set))))
        xs = [up(hx) for _ in range(nset)]
        g1 = nv.nvfp4_calibrate(xs[0])
        ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _ in range(nset)]
        ws = nv.alloc_workspace(dev, M, N, HIDDEN, len(segs), fused=True)
        wsets = [(w_c, w_sf)] + [(w_c.clone(), w_sf.clone()) for _ in range(n_wsets - 1)]
        k = [0]

        def call():
            i = k[0]
            k[0] += 1
            wc_, wsf_ = wsets[i % n_wsets]
            # the weights were written long before the timed region: the kernel may fetch them while
            # the previous call's kernel still runs
            nv.nvfp4_linear_bf16(xs[i % nset], g1, wc_, wsf_, segs, g_w, ws, out=ys[i % nset], w_resident=True)

        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if graph:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for _ in range(reps):
                        call()
                g.replay()
                side.synchronize()
                e0.record(side)
                g.replay()
                e1.record(side)
                side.synchronize()
        else:
            e0.record(stream)
            for _ in range(reps):
                call()
            e1.record(stream)
            torch.cuda.synchronize()
        status = nv.device_status(ws)
        if status != 0:
            raise SystemExit("device status %d in the configs block" % status)
        return e0.elapsed_time(e1) / reps * 1e3            # microseconds per call

    out = {}
    # configs[3]
    gdn = GdnProj(8192)
    hx = synth.prefill_activations(seed, 401, gdn.M, HIDDEN)
    w_c, w_sf, g_w = nv.nvfp4_quantize_weight(up(synth.weights(seed, 402, gdn.segs, HIDDEN)), gdn.segs)
    us = time_layer(gdn.M, gdn.segs, hx, w_c, w_sf, g_w, n_wsets=1, reps=40, graph=False)
    tf = gdn.flops / (us * 1e-6) / 1e12
    out["configs[3] fused GDN in-projection M=8192 K=5120 N=16480 (6 segments), quantize inside the call"] = {
        "us_per_call": round(us, 1), "tflops": round(tf, 1), "frac_of_nominal_9pf": round(tf / NOMINAL_FP4_TFLOPS, 4)}
    del w_c, w_sf
    # configs[4]
    lin = OneLinear(1)
    w_c, w_sf, g_w = nv.nvfp4_quantize_weight(up(synth.weights(seed, 402, lin.segs, HIDDEN)), lin.segs)
    weight_bytes = lin.N * HIDDEN * (0.5 + 1.0 / 16.0)
    n_wsets = int(np.ceil(200e6 / weight_bytes))
    hx_all = synth.prefill_activations(seed, 401, 32768, HIDDEN)
    sweep = []
    for M in (1, 4, 8, 16, 128, 1024, 8192, 32768):
        small = M <= 1024
        us = time_layer(M, lin.segs, hx_all[:M], w_c, w_sf, g_w, n_wsets=n_wsets if small else 1,
                        reps=200 if small else (40 if M == 8192 else 12), graph=small)
        row = {"M": M, "us_per_call": round(us, 2), "launch": "cuda graph replay" if small else "stream launches"}
        flops = gemm_flops(M, lin.N, HIDDEN)
        if M <= 128:
            floor_us = weight_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6
            row.update({"weight_gbs": round(weight_bytes / (us * 1e-6) / 1e9, 1),
                        "frac_of_weight_bandwidth_roofline": round(floor_us / us, 4),
                        "roofline_us": round(floor_us, 2)})
        else:
            tf = flops / (us * 1e-6) / 1e12
            row.update({"tflops": round(tf, 1), "frac_of_nominal_9pf": round(tf / NOMINAL_FP4_TFLOPS, 4)})
        sweep.append(row)
    out["configs[4] K=5120 -> N=6144, quantize inside the call, weights flagged resident; they rotate through %d copies (%.0f MB) for M <= 1024" % (
        n_wsets, n_wsets * weight_bytes / 1e6)] = sweep
    return out


# --------------------------------------------------------------------------- GPU arm
def run_gpu(args):
    import torch
    from paper_2609_04098_b200 import binding as nv
    from paper_2609_04098_b200 import build as nvbuild

    from paper_2609_04098_b200.replicas import Replicas

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    group = Replicas(backend="nccl", device=dev)         # independent replicas: barrier + max only
    rank, world = group.rank, group.world
    nvbuild.build()
    nv.lib()
    if args.variant:
        nv.set_gemm_variant(args.variant)
    peaks = measured_peaks()
    stream = torch.cuda.current_stream()

    def up(bits):
        return synth.to_torch_bf16(bits).to(dev)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    result = {}
    if args.workload == "mlp":
        wl = MlpPair(args.tokens)
        host = wl.host_inputs(args.seed)
        cpu_x, cpu_w = host["x1"], host["w_gu"]
        x1, x2 = up(host["x1"]), up(host["x2"])
        w_gu_c, w_gu_sf, g_gu = nv.nvfp4_quantize_weight(up(host["w_gu"]), wl.seg_gu)
        w_d_c, w_d_sf, g_d = nv.nvfp4_quantize_weight(up(host["w_d"]), wl.seg_d)
        w_il_c, w_il_sf, g_il = nv.nvfp4_quantize_weight_gate_up(up(host["w_gu"]))      # rows interleaved 16 by 16
        g1, g2 = nv.nvfp4_calibrate(x1), nv.nvfp4_calibrate(x2)     # static activation scales (offline)
        q1 = nv.alloc_quantized(wl.M, HIDDEN, dev)
        q2 = nv.alloc_quantized(wl.M, INNER, dev)
        y1 = torch.empty((wl.M, 2 * INNER), dtype=torch.bfloat16, device=dev)
        y2 = torch.empty((wl.M, HIDDEN), dtype=torch.bfloat16, device=dev)
        ws = nv.alloc_workspace(dev)
        torch.cuda.synchronize()

        def step(marks=None):
            if marks is not None:
                marks[0].record(stream)
            nv.nvfp4_quantize_act(x1, g1, out=q1)
            if marks is not None:
                marks[1].record(stream)
            nv.nvfp4_linear(q1[0], q1[1], g1, w_gu_c, w_gu_sf, wl.seg_gu, g_gu, ws, out=y1)
            if marks is not None:
                marks[2].record(stream)
            nv.nvfp4_quantize_act(x2, g2, out=q2)
            if marks is not None:
                marks[3].record(stream)
            nv.nvfp4_linear(q2[0], q2[1], g2, w_d_c, w_d_sf, wl.seg_d, g_d, ws, out=y2)
            if marks is not None:
                marks[4].record(stream)

        def fused_step():
            # the MLP as served: the down projection's input is silu(gate)*up, quantized by the
            # producer-fused kernel straight from the gate/up GEMM's output
            nv.nvfp4_quantize_act(x1, g1, out=q1)
            nv.nvfp4_linear(q1[0], q1[1], g1, w_gu_c, w_gu_sf, wl.seg_gu, g_gu, ws, out=y1)
            nv.nvfp4_swiglu_quantize(y1, g2, out=q2)
            nv.nvfp4_linear(q2[0], q2[1], g2, w_d_c, w_d_sf, wl.seg_d, g_d, ws, out=y2)

        def fused_epilogue_step(y_out=None, x_in=None):
            # the same MLP with SwiGLU and the quantization of h inside the gate/up GEMM's epilogue:
            # the 570 MB of gate/up output are never written
            nv.nvfp4_quantize_act(x1 if x_in is None else x_in, g1, out=q1)
            nv.nvfp4_linear_swiglu(q1[0], q1[1], g1, w_il_c, w_il_sf, g_il, g2, ws, out=q2)
            nv.nvfp4_linear(q2[0], q2[1], g2, w_d_c, w_d_sf, wl.seg_d, g_d, ws, out=y2 if y_out is None else y_out)

        gemm_slots, quant_slots, gemm_per_step = ((1, 2), (3, 4)), ((0, 1), (2, 3)), 2
        h2d_tensors = [synth.to_torch_bf16(host["x1"]).pin_memory(), synth.to_torch_bf16(host["x2"]).pin_memory()]
        d_inputs = [x1, x2]
        d_result = y2
        l2_note = "step touches >1 GB of distinct buffers (inputs larger than the 126 MB L2)"
    elif args.workload in ("gdn", "linear"):
        wl = GdnProj(args.tokens) if args.workload == "gdn" else OneLinear(args.tokens)
        hx = synth.prefill_activations(args.seed, 401, wl.M, HIDDEN)
        hw = synth.weights(args.seed, 402, wl.segs, HIDDEN)
        cpu_x, cpu_w = hx, hw
        # rotate through enough distinct activation/output sets to exceed L2
        per_set = wl.M * HIDDEN * 2 + wl.M * wl.N * 2
        nset = max(1, min(8, int(np.ceil(300e6 / per_set))))
        xs = [up(hx) for _ in range(nset)]
        w_c, w_sf, g_w = nv.nvfp4_quantize_weight(up(hw), wl.segs)
        g1 = nv.nvfp4_calibrate(xs[0])
        ys = [torch.empty((wl.M, wl.N), dtype=torch.bfloat16, device=dev) for _ in range(nset)]
        wss = [nv.alloc_workspace(dev, wl.M, wl.N, HIDDEN, len(wl.segs), fused=True) for _ in range(nset)]
        torch.cuda.synchronize()
        counter = [0]

        def step(marks=None):
            i = counter[0] % nset
            counter[0] += 1
            if marks is not None:
                marks[0].record(stream)
            nv.nvfp4_linear_bf16(xs[i], g1, w_c, w_sf, wl.segs, g_w, wss[i], out=ys[i])
            if marks is not None:
                marks[1].record(stream)

        gemm_slots, quant_slots, gemm_per_step = (), (), 1
        h2d_tensors = [synth.to_torch_bf16(hx).pin_memory()]
        d_inputs = [xs[0]]
        d_result = ys[0]
        l2_note = "rotating %d activation/output sets (%.0f MB) between iterations" % (nset, nset * per_set / 1e6)
    else:
        raise SystemExit("unknown workload")

    barrier = group.barrier

    # ---- device-resident timing
    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    nmark = 5 if args.workload == "mlp" else 2
    marks = [[ev() for _ in range(nmark)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    launches0 = nv.launch_count()
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_start, t_end = ev(), ev()
    use_graph = args.workload != "mlp" and args.graph and args.tokens <= 2048
    if use_graph:
        # launch-bound shapes: the K steps are captured once in a CUDA graph (rotating buffers as in
        # the eager loop) and replayed, so that the host's launch cost is not what is timed
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for i in range(args.steps):
                    step()
            graph.replay()                      # one untimed replay
            side.synchronize()
            t_start.record(side)
            graph.replay()
            t_end.record(side)
            side.synchronize()
        for m in marks:                         # per-step marks are not available inside a graph
            m[0].record(stream)
            m[1].record(stream)
    else:
        t_start.record(stream)
        for i in range(args.steps):
            step(marks[i])
        t_end.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    launches = nv.launch_count() - launches0
    # (graph mode: the count is what was captured = what the one timed replay launches)
    total_ms = group.max_over_ranks(t_start.elapsed_time(t_end))
    ms_per_step = total_ms / args.steps
    value = wl.flops * world / (ms_per_step * 1e-3) / 1e12

    # per-kernel durations from the marks (same timed region)
    def span(slots):
        return sum(m[a].elapsed_time(m[b]) for m in marks for (a, b) in slots)
    if args.workload == "mlp":
        gemm_ms = span(gemm_slots) / (args.steps * gemm_per_step)         # average per GEMM launch
        quant_ms = span(quant_slots) / (args.steps * 2)
        gemm_flops_per_launch = wl.flops / gemm_per_step
        achieved = gemm_flops_per_launch / (gemm_ms * 1e-3) / 1e12
        quant_in_step_gbs = wl.quant_elems / 2 * QUANT_BYTES_PER_ELEM / (quant_ms * 1e-3) / 1e9
        gu_ms = span((gemm_slots[0],)) / args.steps
        dn_ms = span((gemm_slots[1],)) / args.steps
        result["gemm_detail"] = {
            "gate_up": {"ms": round(gu_ms, 4), "tflops": round(gemm_flops(wl.M, 2 * INNER, HIDDEN) / gu_ms / 1e9, 1)},
            "down": {"ms": round(dn_ms, 4), "tflops": round(gemm_flops(wl.M, HIDDEN, INNER) / dn_ms / 1e9, 1)},
            "quantize_x1_us": round(span((quant_slots[0],)) / args.steps * 1e3, 2),
            "quantize_x2_us": round(span((quant_slots[1],)) / args.steps * 1e3, 2)}
    else:
        gemm_ms = ms_per_step
        achieved = wl.flops / (gemm_ms * 1e-3) / 1e12
        quant_in_step_gbs = None
    fp4_peak, peak_basis = tensor_peak(peaks, total_ms * 1e-3, clocks)
    # the SM clock the last GEMM of the timed region really ran at, from the kernel's own counters
    # (the management library's samples lag: they still show the idle boost clock after 20 ms of load)
    kernel_mhz, _ = nv.last_gemm_clock(ws if args.workload == "mlp" else wss[(counter[0] - 1) % nset])
    clock_scaled = (148 * 32768 * kernel_mhz * 1e6 / 1e12) if kernel_mhz > 0 else None
    roofline = {"kernel": "gemm_kernel (tcgen05 block-scaled FP4)", "bound": "tensor",
                "achieved": round(achieved, 2), "peak": round(fp4_peak, 1), "unit": "TFLOP/s",
                "frac": round(achieved / fp4_peak, 4), "peak_basis": peak_basis,
                "frac_of_burst_x4": round(achieved / (peaks["bf16_tflops"] * FP4_OVER_BF16), 4),
                "frac_of_sustained_x4": round(achieved / (peaks["bf16_tflops_sustained"] * FP4_OVER_BF16), 4),
                "frac_of_nominal_9pf": round(achieved / NOMINAL_FP4_TFLOPS, 4),
                "frac_of_clock_scaled_peak": None if not clock_scaled else round(achieved / clock_scaled, 4),
                "sm_mhz_in_kernel": round(kernel_mhz, 1),
                "clock_scaled_peak_basis": "148 SMs x 32768 FLOP/clk x the SM clock read inside the last GEMM of the timed region (cycle counter / wall clock)",
                "avg_launch_ms": round(gemm_ms, 4),
                "traffic": ncu_traffic("gemm_kernel")}
    result["roofline"] = roofline

    # Secondary measurements are short bursts with a pause in front of each (the headline region above is
    # a 20 ms burst at full clocks; back-to-back loops would run the later ones under the power cap and
    # make them look slower than they are).  Each reports the SM clock it saw.
    def burst(fn, reps=20, warm=3, pause_s=0.4):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        time.sleep(pause_s)
        smp = ClockSampler(local_rank, 0.002)
        smp.start()
        b0, b1 = ev(), ev()
        b0.record(stream)
        for _ in range(reps):
            fn()
        b1.record(stream)
        torch.cuda.synchronize()
        ck = smp.stop()
        return b0.elapsed_time(b1) / reps, ck.get("sm_mhz")

    # ---- the MLP as served: producer-fused quantize, and SwiGLU + quantize inside the gate/up epilogue
    if args.workload == "mlp" and rank == 0:
        sw_ms, sw_mhz = burst(lambda: nv.nvfp4_swiglu_quantize(y1, g2, out=q2))
        sw_bytes = wl.M * INNER * (4.0 + 0.5 + 1.0 / 16.0)          # read gate and up, write codes and scales
        fused_ms, fused_mhz = burst(fused_step)
        fe_ms, fe_mhz = burst(fused_epilogue_step)
        fe_gemm_ms, fe_gemm_mhz = burst(lambda: nv.nvfp4_linear_swiglu(q1[0], q1[1], g1, w_il_c, w_il_sf, g_il, g2, ws, out=q2))
        plain_ms, plain_mhz = burst(step)
        result["fused_epilogue"] = {
            "what": "gate/up GEMM with SwiGLU + NVFP4 quantization of h in its epilogue (nvfp4_linear_swiglu), then the down GEMM",
            "gate_up_swiglu_ms": round(fe_gemm_ms, 4), "gate_up_swiglu_sm_mhz": fe_gemm_mhz,
            "gate_up_swiglu_tflops": round(gemm_flops(wl.M, 2 * INNER, HIDDEN) / fe_gemm_ms / 1e9, 1),
            "mlp_step_ms": round(fe_ms, 4), "mlp_step_sm_mhz": fe_mhz,
            "mlp_step_tflops": round(wl.flops / (fe_ms * 1e-3) / 1e12, 1),
            "same_burst_protocol": {"headline_step_ms": round(plain_ms, 4), "headline_step_sm_mhz": plain_mhz,
                                    "mlp_step_with_fused_producer_ms": round(fused_ms, 4),
                                    "mlp_step_with_fused_producer_sm_mhz": fused_mhz}}
        result["swiglu_quantize"] = {
            "workload": "silu(gate)*up -> NVFP4 in one pass, [8192 x 2x17408] bf16 in (570 MB, larger than L2)",
            "us_per_call": round(sw_ms * 1e3, 1), "sm_mhz": sw_mhz,
            "value": round(sw_bytes / (sw_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
            "frac_of_measured_hbm": round(sw_bytes / (sw_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
            "mlp_step_with_fused_producer_ms": round(fused_ms, 4),
            "mlp_step_with_fused_producer_tflops": round(wl.flops / (fused_ms * 1e-3) / 1e12, 1)}

    # ---- the quantize kernel alone on the heavy-tailed activation tensor (configs[1])
    if rank == 0 and not args.skip_quantize:
        hq = synth.config2_activations(args.seed)
        nbuf = 6                                           # 6 x 84 MB inputs: larger than L2
        xq = [up(hq) for _ in range(nbuf)]
        gq = nv.nvfp4_calibrate(xq[0])
        outs = [nv.alloc_quantized(8192, HIDDEN, dev) for _ in range(nbuf)]
        for i in range(2 * nbuf):
            nv.nvfp4_quantize_act(xq[i % nbuf], gq, out=outs[i % nbuf])
        torch.cuda.synchronize()
        reps = 10 * nbuf
        e0, e1 = ev(), ev()
        e0.record(stream)
        for i in range(reps):
            nv.nvfp4_quantize_act(xq[i % nbuf], gq, out=outs[i % nbuf])
        e1.record(stream)
        torch.cuda.synchronize()
        q_ms = e0.elapsed_time(e1) / reps
        q_bytes = 8192 * HIDDEN * QUANT_BYTES_PER_ELEM
        q_gbs = q_bytes / (q_ms * 1e-3) / 1e9
        c0, c1 = ev(), ev()
        c0.record(stream)
        for i in range(reps):
            nv.nvfp4_calibrate(xq[i % nbuf], g=gq)
        c1.record(stream)
        torch.cuda.synchronize()
        cal_ms = c0.elapsed_time(c1) / reps
        # the same tensor through the RMSNorm-fused quantizer (norm gain ~ 1)
        wn = torch.ones(HIDDEN, dtype=torch.bfloat16, device=dev)
        for i in range(nbuf):
            nv.nvfp4_rmsnorm_quantize(xq[i % nbuf], wn, 1e-6, gq, out=outs[i % nbuf])
        torch.cuda.synchronize()
        n0, n1 = ev(), ev()
        n0.record(stream)
        for i in range(reps):
            nv.nvfp4_rmsnorm_quantize(xq[i % nbuf], wn, 1e-6, gq, out=outs[i % nbuf])
        n1.record(stream)
        torch.cuda.synchronize()
        rms_ms = n0.elapsed_time(n1) / reps
        result["quantize"] = {
            "workload": "configs[1] activation quantize 8192x5120 bf16, heavy-tailed; %d rotating buffers" % nbuf,
            "metric": "act_quantize_gbs", "value": round(q_gbs, 1), "unit": "GB/s", "us_per_call": round(q_ms * 1e3, 2),
            "roofline": {"kernel": "quantize_kernel", "bound": "hbm", "achieved": round(q_gbs, 1),
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(q_gbs / peaks["hbm_gbs"], 4),
                         "peak_basis": "%s copy bandwidth" % peaks["source"],
                         "frac_of_nominal_8tbs": round(q_gbs / NOMINAL_HBM_GBS, 4),
                         "traffic": ncu_traffic("quantize_kernel")},
            "calibrate_gbs": round(8192 * HIDDEN * 2 / (cal_ms * 1e-3) / 1e9, 1),
            "rmsnorm_quantize": {"us_per_call": round(rms_ms * 1e3, 2), "value": round(q_bytes / (rms_ms * 1e-3) / 1e9, 1),
                                 "unit": "GB/s", "note": "RMSNorm fused in front: same HBM bytes, the row stays in registers between the sum of squares and the quantization"},
            "in_step_gbs": None if quant_in_step_gbs is None else round(quant_in_step_gbs, 1)}
        del xq, outs

    # ---- end to end: host buffers in, result back, through the same calls
    e2e_steps = max(4, min(args.steps, 20))
    if args.workload == "mlp":
        # The MLP as a caller runs it: X1 arrives from pinned host memory, the down projection's
        # input is produced on the device (silu(gate)*up fused into the quantizer), Y comes back.
        # Copies and compute are double-buffered over three streams, as a serving loop would do.
        h_in = h2d_tensors[0]
        xin = [x1, torch.empty_like(x1)]
        yout = [y2, torch.empty_like(y2)]
        h_outs = [torch.empty_like(y2, device="cpu").pin_memory() for _ in range(2)]
        s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        h2d_bytes = h_in.numel() * h_in.element_size()
        d2h_bytes = h_outs[0].numel() * h_outs[0].element_size()

        def pipelined(n):
            for i in range(n):
                b = i & 1
                with torch.cuda.stream(s_in):
                    s_in.wait_event(ev_cmp[b])                 # compute of step i-2 has read xin[b]
                    xin[b].copy_(h_in, non_blocking=True)
                    ev_in[b].record(s_in)
                with torch.cuda.stream(s_cmp):
                    s_cmp.wait_event(ev_in[b])
                    s_cmp.wait_event(ev_out[b])                # the copy-out of step i-2 has read yout[b]
                    fused_epilogue_step(y_out=yout[b], x_in=xin[b])
                    ev_cmp[b].record(s_cmp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_cmp[b])
                    h_outs[b].copy_(yout[b], non_blocking=True)
                    ev_out[b].record(s_out)

        torch.cuda.synchronize()
        pipelined(2)
        torch.cuda.synchronize()
        barrier()
        s0, s1 = ev(), ev()
        s0.record(stream)
        for st_ in (s_in, s_cmp, s_out):
            st_.wait_stream(stream)
        pipelined(e2e_steps)
        for st_ in (s_in, s_cmp, s_out):
            stream.wait_stream(st_)
        s1.record(stream)
        torch.cuda.synchronize()
        e2e_note = ("MLP with SwiGLU + quantization in the gate/up epilogue (X1 from pinned host memory, Y back to host "
                    "every step), copies and compute double-buffered over three streams")
    else:
        h_out = torch.empty_like(d_result, device="cpu").pin_memory()
        h2d_bytes = sum(t.numel() * t.element_size() for t in h2d_tensors)
        d2h_bytes = h_out.numel() * h_out.element_size()

        def e2e_step():
            for src, dst in zip(h2d_tensors, d_inputs):
                dst.copy_(src, non_blocking=True)
            step()
            h_out.copy_(d_result, non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        barrier()
        s0, s1 = ev(), ev()
        s0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        s1.record(stream)
        torch.cuda.synchronize()
        e2e_note = "host input in, fused call, result back, on one stream"
    e2e_ms = group.max_over_ranks(s0.elapsed_time(s1) / e2e_steps)
    result["e2e"] = {"value": round(wl.flops * world / (e2e_ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
                     "ms_per_step": round(e2e_ms, 3), "h2d_bytes_per_step": h2d_bytes,
                     "d2h_bytes_per_step": d2h_bytes, "what": e2e_note}
    status = nv.device_status(ws if args.workload == "mlp" else wss[0])
    if status != 0:
        raise SystemExit("device status %d after the timed region" % status)

    if rank == 0 and not args.skip_configs and args.workload == "mlp":
        del x1, x2, y1, y2, q1, q2
        torch.cuda.empty_cache()
        result["configs"] = measure_configs(torch, nv, dev, peaks, args.seed)

    if rank == 0:
        if not args.skip_cpu:
            result["cpu_baseline"] = cpu_baseline(wl, target_s=args.cpu_seconds, seed=args.seed,
                                                  x_bits=cpu_x, w_bits=cpu_w)
        line = {"metric": "nvfp4_w4a4_linear_tflops", "value": round(value, 2), "unit": "TFLOP/s",
                "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
                "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "nvfp4 (e2m1 x e4m3 block scales, f32 accumulate, bf16 out)",
                "data": "synthetic (seeded; shapes and statistics of the paper's 27B hybrid model)",
                "config": {"workload": wl.describe, "tokens": wl.M, "l2": l2_note,
                           "parallelism": "replicas only" if world > 1 else "single GPU",
                           "gemm_variant": args.variant or "auto",
                           "launch": "cuda graph replay" if use_graph else "stream launches"},
                "gpu_launches": int(launches), "clocks": clocks}
        line.update(result)
        print(json.dumps(line))
    group.close()


# --------------------------------------------------------------------------- CPU oracle arm
def cpu_baseline(wl, target_s=15.0, seed=0, x_bits=None, w_bits=None):
    """The oracle as it stands, timed on a bounded sample of the same workload: quantize R
    activation rows of the first layer's input and run the exact GEMM of those rows against
    ALL of that layer's (oracle-quantized) weight rows.  R is sized for about `target_s`
    seconds from a small trial.  Weight quantization is setup (offline in the path), untimed."""
    import oracle
    K = HIDDEN
    segs = wl.seg_gu if hasattr(wl, "seg_gu") else wl.segs
    N = sum(s.count for s in segs)
    if w_bits is None:
        w_bits = synth.weights(seed, 302 if hasattr(wl, "seg_gu") else 402, segs, K)
    if x_bits is None:
        x_bits = synth.prefill_activations(seed, 301 if hasattr(wl, "seg_gu") else 401, min(wl.M, 8192), K)
    gs = [oracle.calibrate(w_bits[s.begin:s.begin + s.count])[1] for s in segs]
    wc, wsf = oracle.quantize(w_bits, oracle.row_scales(N, segs, gs))
    gcol = oracle.col_scales(N, segs, gs)

    def run(rows):
        x = x_bits[:rows]
        t0 = time.perf_counter()
        _, ga = oracle.calibrate(x)
        ac, asf = oracle.quantize(x, oracle.row_scales(rows, g=ga))
        oracle.gemm(ac, asf, ga, wc, wsf, gcol)
        return time.perf_counter() - t0

    trial = min(32, x_bits.shape[0])
    t_trial = run(trial)
    rows = int(max(trial, min(x_bits.shape[0], trial * target_s / max(t_trial, 1e-3))))
    t = run(rows) if rows > trial else t_trial
    flops = gemm_flops(rows, N, K)
    return {"value": round(flops / t / 1e12, 6), "unit": "TFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(t, 2),
            "sample": "quantize + exact GEMM of %d token rows x all %d weight rows (K=%d) of the step's first layer" % (
                rows, N, K)}


def run_reference(args):
    """The reference arm: the CPU oracle on the same metric and workload, each step a
    bounded sample.  Rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = {"mlp": MlpPair, "gdn": GdnProj, "linear": OneLinear}[args.workload](args.tokens)
    per_step_s = max(1.0, min(15.0, 100.0 / max(1, args.steps + args.warmup)))
    segs = wl.seg_gu if hasattr(wl, "seg_gu") else wl.segs
    mlp = hasattr(wl, "seg_gu")
    w_bits = synth.weights(args.seed, 302 if mlp else 402, segs, HIDDEN)
    x_bits = synth.prefill_activations(args.seed, 301 if mlp else 401, min(wl.M, 8192), HIDDEN)
    for _ in range(args.warmup):
        cpu_baseline(wl, target_s=per_step_s / 4, seed=args.seed, x_bits=x_bits, w_bits=w_bits)
    vals, secs, last = [], [], None
    for _ in range(args.steps):
        last = cpu_baseline(wl, target_s=per_step_s, seed=args.seed, x_bits=x_bits, w_bits=w_bits)
        vals.append(last["value"])
        secs.append(last["seconds"])
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": "nvfp4_w4a4_linear_tflops", "value": round(value, 6), "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(1e3 * float(np.mean(secs)), 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64/f64 (exact)", "data": "synthetic (seeded)",
            "config": {"workload": wl.describe, "tokens": wl.M},
            "cpu_baseline": {"value": round(value, 6), "unit": "TFLOP/s", "kind": "oracle",
                             "cores": last["cores"], "sample": last["sample"]},
            "e2e": {"value": round(value, 6), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mlp", choices=["mlp", "gdn", "linear"])
    ap.add_argument("--tokens", type=int, default=8192)
    ap.add_argument("--variant", type=int, default=0, help="GEMM tile variant (0 = auto)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="time small-M workloads with plain stream launches instead of a CUDA graph")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-quantize", action="store_true")
    ap.add_argument("--skip-configs", action="store_true", help="leave out the configs[3] / configs[4] block")
    args = ap.parse_args()
    ref = args.impl == "reference"
    if args.steps is None:
        args.steps = 3 if ref else 200
    if args.warmup is None:
        args.warmup = 1 if ref else 10
    if args.impl == "reference":
        run_reference(args)
        return
    from paper_2609_04098_b200.replicas import launched_by_a_launcher, spawn_replicas
    if args.gpus > 1 and not launched_by_a_launcher():
        # nobody started the ranks for us: one process per GPU, each an independent replica
        sys.exit(spawn_replicas(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    run_gpu(args)


if __name__ == "__main__":
    main()
