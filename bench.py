#!/usr/bin/env python
"""Benchmark of the SegLinear + DualScale W8A8 layer path on B200.

A step = one pass of the per-call hot path (activation quantize -> tcgen05 GEMM -> dequant epilogue)
over every layer of one workload, on seeded synthetic inputs that are already resident in HBM.
Calibration and weight quantization are offline by the method's definition and run once at set-up.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` = executed tensor TOPS of the whole job (dual layers execute
two GEMMs: 4*M*N*K ops; single-scale layers 2*M*N*K), `e2e` = the same metric with pinned-host inputs
and outputs copied inside the timed region, `roofline` = the GEMM kernel against the dense int8/fp8
tensor peak, `cpu_baseline` = the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "SegLinear+DualScale W8A8 TOPS per layer shape, % of B200 dense int8/fp8 peak"
NOMINAL_8BIT_TOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 << 20
L2_FLUSH_BYTES = 256 << 20
COOL_DOWN_S = 1.0          # idle time in front of every burst measurement


def measured_peaks():
    """Driver-written measured peaks; fallback figures if the file is absent."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def layer_ops(spec, M=None):
    M = spec.M if M is None else M
    useful = 2.0 * M * spec.N * spec.K
    return useful * (2 if spec.dual else 1), useful


def gemm_bytes(spec, M=None):
    """Algorithmic HBM bytes of one GEMM launch: code matrices + weight codes + bf16 output."""
    M = spec.M if M is None else M
    return M * spec.K * (2 if spec.dual else 1) + spec.N * spec.K + 2 * M * spec.N


def quant_bytes(spec, M=None):
    M = spec.M if M is None else M
    xb = 4 if spec.x_dtype == "f32" else 2
    return M * spec.K * (xb + (2 if spec.dual else 1))


# ------------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) during the timed region."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, device_index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report that no clocks were sampled
            self.nv, self.err = None, repr(e)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr:
            self._stop.set()
            self._thr.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------ our arm

class BenchLayer:
    def __init__(self, spec, device, M=None):
        from paper_2507_14811_b200 import binding as B
        from paper_2507_14811_b200 import workloads as WL
        from paper_2507_14811_b200.layer import SegQuantLinear
        self.B = B
        self.spec = spec
        self.M = spec.M if M is None else M
        data = WL.make_layer(spec, M=self.M)
        t0 = time.perf_counter()
        self.layer = SegQuantLinear(data.W, data.bias, spec.kb, spec.nb, spec.dual, spec.code, device)
        self.layer.calibrate(data.X_cal)
        torch.cuda.synchronize()
        self.offline_s = time.perf_counter() - t0
        self.X_host = data.X.pin_memory()
        self.X = data.X.to(device)
        self.x_stage = torch.empty_like(self.X)
        self.c_pos = B.new_codes(self.M, spec.K, device)
        self.c_neg = B.new_codes(self.M, spec.K, device) if spec.dual else None
        self.Y = torch.empty((self.M, spec.N), dtype=torch.bfloat16, device=device)
        self.y_stage = torch.empty_like(self.Y)
        self.Y_host = torch.empty((self.M, spec.N), dtype=torch.bfloat16).pin_memory()
        self.layer.scratch_for(self.M)
        # comparison variants of DualScale layers: the zero-point scheme (int8) and the fused activation
        self.act = spec.x_kind.partition("+")[2] or None
        self.zp = None
        if spec.dual and spec.code == "int8":
            L = self.layer
            s_x, z_x = B.segquant_calib_zero_point(data.X_cal.to(device), L.seg, L.workspace)
            self.zp = {"s_x": s_x, "z_x": z_x, "codes": B.new_codes(self.M, spec.K, device),
                       "bias": B.segquant_fold_zero_point(L.Wq, L.seg, s_x, z_x, L.s_w, L.bias)}
        self.a_stage = torch.empty_like(self.X) if (spec.dual and self.act) else None
        self.ws_split = None
        # gated GELU: the pre-activation row holds a value half and a gate half (timing only: any values do)
        self.H2 = torch.cat([self.X, self.X], dim=1).contiguous() if self.act == "geglu" else None
        self.g_stage = torch.empty_like(self.X) if self.act == "geglu" else None
        # the same layer as W4A8: per-channel 4-bit weights (kept packed), per-token activation scales
        self.w4 = None
        if spec.code == "int8" and spec.K <= 16384:
            seg4 = B.SegTable(spec.kb, [0, spec.N])
            s_w4, _, w8, _ = B.segquant_quantize_per_row(data.W.to(device), seg4, False, bits=4)
            self.w4 = {"s_w": s_w4, "packed": B.segquant_pack_w4(w8), "w8": w8,
                       "s_pos": torch.empty((self.M, spec.P), dtype=torch.float32, device=device),
                       "s_neg": torch.empty((self.M, spec.P), dtype=torch.float32, device=device) if spec.dual else None}
            self.seg4 = seg4

    def quantize(self):
        L = self.layer
        self.B.segquant_quantize_act(self.X, L.seg, L.s_pos, L.s_neg, L.code, L.flags, self.c_pos, self.c_neg)

    def gemm(self):
        L = self.layer
        if L.dual:
            self.B.segquant_dualscale_gemm(self.c_pos, self.c_neg, L.Wq, L.seg, L.code, L.s_pos, L.s_neg, L.s_w,
                                           L.bias, L.workspace, Y=self.Y)
        else:
            self.B.segquant_seglinear_gemm(self.c_pos, L.Wq, L.seg, L.code, L.s_pos, L.s_w, L.bias, L.workspace,
                                           Y=self.Y)

    def quantize_plain(self):
        """Single-scale codes of the same input (the plain W8A8 layer's quantize pass).  Timing only."""
        L = self.layer
        self.B.segquant_quantize_act(self.X, L.seg, L.s_pos, None, L.code, L.flags, self.c_pos, None)

    def quantize_zero_point(self):
        self.B.segquant_quantize_act_zero_point(self.X, self.layer.seg, self.zp["s_x"], self.zp["z_x"], self.zp["codes"])

    def gemm_zero_point(self):
        """The zero-point layer: its codes and the folded bias through the single-scale GEMM."""
        L = self.layer
        self.B.segquant_seglinear_gemm(self.zp["codes"], L.Wq, L.seg, L.code, self.zp["s_x"], L.s_w, self.zp["bias"],
                                       L.workspace, Y=self.Y)

    def quantize_fused_act(self):
        """Pre-activation -> activation -> codes in one pass.  Timing only: the layer's input stands in for the
        pre-activation (the cost does not depend on the values)."""
        L = self.layer
        H = self.H2 if self.act == "geglu" else self.X
        self.B.segquant_quantize_act_fused(H, L.seg, L.s_pos, L.s_neg, L.code, act=self.act, c_pos=self.c_pos,
                                           c_neg=self.c_neg)

    def act_unfused(self):
        """The activation as its own elementwise pass (a library kernel, comparison only): reads the
        pre-activation, writes the activation that the quantize pass then reads."""
        if self.act == "geglu":                                  # two library kernels: GELU of the gate half, the product
            K = self.spec.K
            torch.ops.aten.gelu.out(self.H2[:, K:], out=self.g_stage)
            torch.mul(self.H2[:, :K], self.g_stage, out=self.a_stage)
        elif self.act == "silu":
            torch.nn.functional.silu(self.X, inplace=False) if self.a_stage is None else torch.ops.aten.silu.out(self.X, out=self.a_stage)
        else:
            torch.ops.aten.gelu.out(self.X, out=self.a_stage)

    def w4_unpack(self):
        self.B.segquant_unpack_w4(self.w4["packed"], out=self.w4["w8"])

    def w4_quantize(self):
        """Per-token scales and codes (one kernel)."""
        L, w = self.B.lib(), self.w4
        import ctypes as C
        from paper_2507_14811_b200.binding import _ptr, _dt, _stream, _check
        st = L.segquant_quantize_per_row(_ptr(self.X), C.c_int(_dt(self.X)), C.c_int64(self.M), C.c_int64(self.spec.K),
                                         C.c_int64(self.X.stride(0)), self.seg4.ref(), C.c_int(8), C.c_uint32(0),
                                         _ptr(w["s_pos"]), _ptr(w["s_neg"]), _ptr(self.c_pos), _ptr(self.c_neg),
                                         C.c_int64(self.c_pos.stride(0)), _stream())
        _check(st, "segquant_quantize_per_row")

    def w4_gemm(self):
        w = self.w4
        self.B.segquant_w4a8_gemm(self.c_pos, self.c_neg, w["w8"], self.seg4, w["s_pos"], w["s_neg"], w["s_w"],
                                  self.layer.bias, self.layer.workspace, Y=self.Y)

    def gemm_split(self):
        """The layer's GEMM with tiles split along K across CTA pairs (the larger workspace; forced, whatever the
        automatic choice would be).  Timing only."""
        if self.ws_split is None:
            self.ws_split = self.B.new_workspace(self.X.device, split_for=(self.M, self.spec.N, self.spec.dual))
        L = self.layer
        self.B.segquant_set_tuning(0, 0, 0, 6)
        try:
            if L.dual:
                self.B.segquant_dualscale_gemm(self.c_pos, self.c_neg, L.Wq, L.seg, L.code, L.s_pos, L.s_neg, L.s_w,
                                               L.bias, self.ws_split, Y=self.Y)
            else:
                self.B.segquant_seglinear_gemm(self.c_pos, L.Wq, L.seg, L.code, L.s_pos, L.s_w, L.bias, self.ws_split,
                                               Y=self.Y)
        finally:
            self.B.segquant_set_tuning(0, 0, 0, 0)

    def gemm_plain(self):
        """The same shape as a plain single-scale W8A8 layer (one code matrix): the denominator of the
        DualScale overhead.  Timing only; its output is not checked."""
        L = self.layer
        self.B.segquant_seglinear_gemm(self.c_pos, L.Wq, L.seg, L.code, L.s_pos, L.s_w, L.bias, L.workspace, Y=self.Y)

    def gemm_unsegmented(self):
        """The same shape and polarity handling with ONE segment (P = Q = 1): the denominator of the SegLinear
        overhead (the paper reports +37..50 % for its own kernels).  Timing only; its output is not checked."""
        L = self.layer
        if not hasattr(self, "_unseg"):
            self._unseg = self.B.SegTable([0, self.spec.K], [0, self.spec.N])
        if L.dual:
            self.B.segquant_dualscale_gemm(self.c_pos, self.c_neg, L.Wq, self._unseg, L.code, L.s_pos[:1], L.s_neg[:1],
                                           L.s_w[:1], L.bias, L.workspace, Y=self.Y)
        else:
            self.B.segquant_seglinear_gemm(self.c_pos, L.Wq, self._unseg, L.code, L.s_pos[:1], L.s_w[:1], L.bias,
                                           L.workspace, Y=self.Y)

    def device_copy(self):
        """A second instance of the layer whose device buffers (weight codes, scale tables, input, code
        matrices, output, workspace) are fresh allocations with the same contents: the members of the
        rotating buffer sets of time_steps_back_to_back."""
        import copy
        other = copy.copy(self)
        other.layer = copy.copy(self.layer)
        for name in ("Wq", "s_w", "bias", "s_pos", "s_neg", "workspace"):
            t = getattr(self.layer, name)
            setattr(other.layer, name, None if t is None else t.clone())
        for name in ("X", "c_pos", "c_neg", "Y", "a_stage", "H2", "g_stage", "ws_split"):
            t = getattr(self, name)
            setattr(other, name, None if t is None else t.clone())
        if self.zp is not None:
            other.zp = {k: v.clone() for k, v in self.zp.items()}
        if self.w4 is not None:
            other.w4 = {k: (None if v is None else v.clone()) for k, v in self.w4.items()}
        return other

    def device_bytes(self):
        ts = [self.layer.Wq, self.X, self.c_pos, self.c_neg, self.Y]
        return sum(t.numel() * t.element_size() for t in ts if t is not None)

    def forward_e2e(self, chunks=0, stream_in=None, stream_out=None):
        """Pinned-host X -> pinned-host Y through the C ABI; chunks > 1 overlaps the copies with the kernels."""
        if chunks > 1:
            self.layer.forward_pipelined(self.X_host, self.Y_host, self.x_stage, self.y_stage, chunks, stream_in, stream_out)
        else:
            self.layer.forward(self.X_host, Y=self.Y_host, x_stage=self.x_stage, y_stage=self.y_stage)


def graph_time_per_launch(calls, rounds):
    """Mean device time of one call: `rounds` passes over the list `calls` (one launch each, every one on its own
    copy of the layer's buffers) are captured into a CUDA graph; the graph is replayed once untimed and once
    between a pair of CUDA events on its stream.  Returns microseconds per launch."""
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for c in calls:                       # eager once: loads the kernels, sets their attributes
            c()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream, capture_error_mode="relaxed"):
            for _ in range(rounds):
                for c in calls:
                    c()
        graph.replay()
        stream.synchronize()
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        stream.synchronize()
    torch.cuda.current_stream().wait_stream(stream)
    return e0.elapsed_time(e1) * 1e3 / (rounds * len(calls))


def library_gemm_same_shape(spec, M, n_copies, rounds, dev):
    """Context only: the vendor library's plain dense GEMM on the layer's shape (int8 -> int32, or e4m3 -> bf16 with
    unit scales; no segment scales, no bias, one code matrix), timed like the product's kernels: a CUDA graph of
    launches over rotating operand copies.  M is rounded up to a multiple of 8 for the library.  Returns
    microseconds per launch, or None where the library refuses the shape."""
    Mp = -(-M // 8) * 8
    try:
        if spec.code == "int8":
            sets = [(torch.randint(-127, 128, (Mp, spec.K), dtype=torch.int8, device=dev),
                     torch.randint(-127, 128, (spec.N, spec.K), dtype=torch.int8, device=dev).t()) for _ in range(n_copies)]
            calls = [(lambda a=a, b=b: torch._int_mm(a, b)) for a, b in sets]
        else:
            one = torch.ones((), device=dev)
            sets = [(torch.randn((Mp, spec.K), device=dev).to(torch.float8_e4m3fn),
                     torch.randn((spec.N, spec.K), device=dev).to(torch.float8_e4m3fn).t()) for _ in range(n_copies)]
            calls = [(lambda a=a, b=b: torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16))
                     for a, b in sets]
        t = graph_time_per_launch(calls, rounds)
    except Exception:
        t = None
    torch.cuda.empty_cache()
    return t


def time_kernels(layers, launches=48, max_copies=96, with_w4a8=True, with_split=False, with_library=True):
    """Per-layer device time of each kernel, timed alone: a CUDA graph of >= `launches` launches of that one
    kernel, launch i on copy i mod C of the layer's device buffers, C chosen so that the copies the kernel walks
    through are at least twice the L2 capacity (every launch finds its operands in HBM).  A single launch between
    its own pair of events cannot be used for this: the event timer of these GPUs ticks in steps of 2 us and an
    event pair around one small kernel reads 6-8 us more than the kernel's own span.
    Returns lists (quantize_us, gemm_us, plain_us | None, unsegmented_us | None, copies)."""
    out = {"q": [], "g": [], "plain": [], "unseg": [], "copies": [], "q_plain": [], "q_zp": [], "g_zp": [], "q_fused": [],
           "act": [], "w4_q": [], "w4_unpack": [], "w4_g": [], "g_split": [], "lib": []}
    for bl in layers:
        s = bl.spec
        foot = min(quant_bytes(s, bl.M), gemm_bytes(s, bl.M))
        n = int(min(max_copies, max(2, -(-2 * L2_BYTES // foot))))
        copies = [bl] + [bl.device_copy() for _ in range(n - 1)]
        rounds = max(1, -(-launches // n))
        out["copies"].append(n)
        out["q"].append(graph_time_per_launch([c.quantize for c in copies], rounds))
        out["g"].append(graph_time_per_launch([c.gemm for c in copies], rounds))
        out["plain"].append(graph_time_per_launch([c.gemm_plain for c in copies], rounds) if s.dual else None)
        out["unseg"].append(graph_time_per_launch([c.gemm_unsegmented for c in copies], rounds)
                            if (s.P > 1 or s.Q > 1) else None)
        out["q_plain"].append(graph_time_per_launch([c.quantize_plain for c in copies], rounds) if s.dual else None)
        out["q_zp"].append(graph_time_per_launch([c.quantize_zero_point for c in copies], rounds) if bl.zp else None)
        out["g_zp"].append(graph_time_per_launch([c.gemm_zero_point for c in copies], rounds) if bl.zp else None)
        fused = s.dual and bl.act
        out["q_fused"].append(graph_time_per_launch([c.quantize_fused_act for c in copies], rounds) if fused else None)
        out["act"].append(graph_time_per_launch([c.act_unfused for c in copies], rounds) if fused else None)
        split = with_split and s.P == 1 and bl.M > 128
        out["g_split"].append(graph_time_per_launch([c.gemm_split for c in copies], rounds) if split else None)
        w4 = bl.w4 is not None and with_w4a8
        out["w4_q"].append(graph_time_per_launch([c.w4_quantize for c in copies], rounds) if w4 else None)
        out["w4_unpack"].append(graph_time_per_launch([c.w4_unpack for c in copies], rounds) if w4 else None)
        out["w4_g"].append(graph_time_per_launch([c.w4_gemm for c in copies], rounds) if w4 else None)
        del copies
        torch.cuda.empty_cache()
        out["lib"].append(library_gemm_same_shape(s, bl.M, min(n, 24), max(1, -(-launches // min(n, 24))), bl.X.device)
                          if with_library else None)
    return out


def time_steps_back_to_back(layer_sets, steps, warmup, min_region_s=0.0):
    """K whole steps (quantize + GEMM of every layer) issued back to back, one CUDA-event pair around all of
    them.  Step i works on buffer set i mod R; the sets together are several times the L2 capacity, so every
    step finds its inputs and weights in HBM without a flush between steps.  The K steps are captured once
    into a CUDA graph (the launches keep their programmatic-dependent-launch edges) and the timed region is
    `reps` replays of that graph (as many as the region needs to last min_region_s), so the host's launch rate
    is not part of the measurement.  Returns (ms per step, mode, kernel launches per replay, reps)."""
    from paper_2507_14811_b200 import binding as B
    R = len(layer_sets)
    stream = torch.cuda.Stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def issue(n):
        for i in range(n):
            for bl in layer_sets[i % R]:
                bl.quantize()
                bl.gemm()

    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        issue(max(warmup, R))
        stream.synchronize()
        mode = "cuda graph of K steps"
        try:
            graph = torch.cuda.CUDAGraph()
            n0 = B.segquant_launch_count()
            with torch.cuda.graph(graph, stream=stream, capture_error_mode="relaxed"):
                issue(steps)
            launches = B.segquant_launch_count() - n0        # kernel nodes of the graph = launches per replay
            run = graph.replay
        except Exception as e:      # capture refused: issue the same launches from the host
            torch.cuda.synchronize()
            mode = f"launched from the host back to back (graph capture failed: {type(e).__name__})"
            run = lambda: issue(steps)
            launches = None
        run()                                  # untimed: graph upload, and warm-up of every buffer set
        stream.synchronize()
        e0.record(stream)
        run()
        e1.record(stream)
        stream.synchronize()
        # the K-step graph is replayed back to back until the region lasts min_region_s (at least once)
        reps = max(1, int(np.ceil(min_region_s / max(e0.elapsed_time(e1) * 1e-3, 1e-9))))
        n0 = B.segquant_launch_count()
        e0.record(stream)
        for _ in range(reps):
            run()
        e1.record(stream)
        stream.synchronize()
        if launches is None:
            launches = (B.segquant_launch_count() - n0) // reps
    torch.cuda.current_stream().wait_stream(stream)
    return e0.elapsed_time(e1) / (steps * reps), mode, launches, reps


def time_steps_planned(layer_sets, steps, min_region_s=0.02):
    """The same whole steps issued from the host through prepared calls (one plan per layer and buffer set, built
    outside the timed region; a step's host cost is one call per layer = two kernel launches each), no CUDA graph.
    Returns ms per step."""
    R = len(layer_sets)
    plans = [[bl.layer.plan(bl.X, bl.Y) for bl in layers] for layers in layer_sets]
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        def issue(n):
            for i in range(n):
                for p in plans[i % R]:
                    p.run()
        issue(max(R, 3))
        stream.synchronize()
        e0.record(stream); issue(steps); e1.record(stream)
        stream.synchronize()
        n = max(steps, int(np.ceil(steps * min_region_s / max(e0.elapsed_time(e1) * 1e-3, 1e-9))))
        e0.record(stream); issue(n); e1.record(stream)
        stream.synchronize()
    torch.cuda.current_stream().wait_stream(stream)
    return e0.elapsed_time(e1) / n


def time_e2e(layers, steps, warmup, flush, chunks=0):
    nl = len(layers)
    s_in, s_out = (torch.cuda.Stream(), torch.cuda.Stream()) if chunks > 1 else (None, None)
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(nl)] for _ in range(steps)]
    for _ in range(min(warmup, 3)):
        for bl in layers:
            bl.forward_e2e(chunks, s_in, s_out)
    torch.cuda.synchronize()
    for s in range(steps):
        for i, bl in enumerate(layers):
            flush()
            ev[s][i][0].record()
            bl.forward_e2e(chunks, s_in, s_out)
            ev[s][i][1].record()
    torch.cuda.synchronize()
    ms = np.array([[ev[s][i][0].elapsed_time(ev[s][i][1]) for i in range(nl)] for s in range(steps)])
    return ms.mean(axis=0)


def time_e2e_step(layers, steps, warmup, flush, chunks):
    """Whole end-to-end steps: every layer's call (pinned-host X -> pinned-host Y) is issued on its own set of
    streams, so that one layer's output copy (device to host) overlaps another layer's input copy (host to
    device) on the full-duplex link; the layers of the workload are independent batches.  One event pair
    around each step on the current stream, which the layers' streams fork from and join into."""
    cur = torch.cuda.current_stream()
    sets = [(torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()) for _ in layers]
    order = sorted(range(len(layers)), key=lambda i: -layers[i].spec.M * layers[i].spec.N)   # largest output first

    def step():
        for i in order:
            main, s_in, s_out = sets[i]
            main.wait_stream(cur)
            with torch.cuda.stream(main):
                layers[i].forward_e2e(max(chunks, 2), s_in, s_out)
        for main, _, _ in sets:
            cur.wait_stream(main)

    for _ in range(min(warmup, 3)):
        step()
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
    for s in range(steps):
        flush()
        ev[s][0].record()
        step()
        ev[s][1].record()
    torch.cuda.synchronize()
    return float(np.mean([a.elapsed_time(b) for a, b in ev]))


def oracle_sample(specs, target_s=12.0, probe_rows=8):
    """Times the CPU oracle (as it stands) on the first rows of every layer of the workload: a short
    probe fixes the row count so that the sample costs about `target_s` seconds."""
    import oracle as O
    from paper_2507_14811_b200 import workloads as WL

    def run(rows):
        total_ops, total_t = 0.0, 0.0
        for spec in specs:
            data = WL.make_layer(spec, M=rows)
            qmax, qmin = (127.0, 128.0) if spec.code == "int8" else (448.0, 448.0)
            Wn = data.W.numpy()
            s_pos, s_neg = O.calib_act(data.X_cal.float().numpy(), spec.kb, spec.dual, q_max=qmax, q_min_abs=qmin)
            s_w = O.calib_weight(Wn, spec.kb, spec.nb, w_max=qmax)
            Wq = O.quantize_weight(Wn, spec.kb, spec.nb, s_w, code=spec.code, w_max=qmax)
            Xn = data.X.float().numpy()
            t0 = time.perf_counter()
            O.layer_forward(Xn, Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w, data.bias.numpy(),
                            code=spec.code, q_max=qmax, q_min_abs=qmin)
            total_t += time.perf_counter() - t0
            total_ops += layer_ops(spec, rows)[0]
        return total_ops, total_t

    _, t_probe = run(probe_rows)
    max_rows = min(s.M for s in specs)
    rows = int(max(probe_rows, min(max_rows, probe_rows * target_s / max(t_probe, 1e-6))))
    ops, t, reps = 0.0, 0.0, 0
    while reps < 1 or (t < 0.8 * target_s and reps < 20):      # a whole small workload is repeated up to the target
        o, dt = run(rows)
        ops, t, reps = ops + o, t + dt, reps + 1
    what = "every row" if rows == max_rows else f"the first {rows} rows"
    return {"value": ops / t / 1e12, "unit": "TOPS", "cores": O.num_threads(), "kind": "oracle",
            "sample": f"{what} of every layer of the workload (steps quantize+accumulate+dequant), "
                      f"{reps} pass(es), {t:.1f} s of CPU time"}, rows, t


def library_8bit_peaks(dev):
    """Context for the peak: what the vendor library's own dense int8 and fp8 GEMMs reach on this GPU (8192^3, best
    of 10 single launches after warm-up, CUDA events; these are 1-2 ms kernels, far above the event timer's
    resolution).  Denominator context only: nothing of the product path calls these."""
    out = {}
    n = 8192
    ops = 2.0 * n * n * n

    def best(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return ops / (min(ts) * 1e-3) / 1e12

    try:
        a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev)
        b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev).t()
        out["int8_tops"] = round(best(lambda: torch._int_mm(a, b)), 1)
    except Exception as e:
        out["int8_tops"] = None
        out["int8_error"] = f"{type(e).__name__}: {str(e)[:120]}"
    try:
        a8 = torch.randn((n, n), device=dev).to(torch.float8_e4m3fn)
        b8 = torch.randn((n, n), device=dev).to(torch.float8_e4m3fn).t()
        one = torch.ones((), device=dev)
        out["fp8_tops"] = round(best(lambda: torch._scaled_mm(a8, b8, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)), 1)
    except Exception as e:
        out["fp8_tops"] = None
        out["fp8_error"] = f"{type(e).__name__}: {str(e)[:120]}"
    torch.cuda.empty_cache()
    return out


def eight_bit_peaks(peaks):
    """Dense 8-bit tensor peaks (TOPS): measured bf16 burst and sustained figures x the nominal 8-bit : bf16
    ratio of 2, and the nominal figure itself."""
    sustained = peaks.get("bf16_tflops_sustained")
    return {"burst": peaks["bf16_tflops"] * 2.0, "sustained": None if sustained is None else sustained * 2.0,
            "nominal": NOMINAL_8BIT_TOPS}


def fractions(tops, p8):
    """A throughput against the three 8-bit peaks."""
    return {"of_measured_burst": round(tops / p8["burst"], 4),
            "of_measured_sustained": None if p8["sustained"] is None else round(tops / p8["sustained"], 4),
            "of_nominal_4500": round(tops / p8["nominal"], 4)}


def layer_table(specs, kt, peaks):
    """Per-layer figures from the kernels timed alone (time_kernels: burst peaks)."""
    q_ms, g_ms = [t * 1e-3 for t in kt["q"]], [t * 1e-3 for t in kt["g"]]
    plain_ms = [None if t is None else t * 1e-3 for t in kt["plain"]]
    unseg_ms = [None if t is None else t * 1e-3 for t in kt["unseg"]]
    p8 = eight_bit_peaks(peaks)
    rows = []
    for s, q, g, pl, un in zip(specs, q_ms, g_ms, plain_ms, unseg_ms):
        eo, uo = layer_ops(s)
        t_tensor = eo / (p8["burst"] * 1e12)
        t_hbm = gemm_bytes(s) / (peaks["hbm_gbs"] * 1e9)
        tops = eo / (g * 1e-3) / 1e12
        rows.append({
            "layer": s.name, "M": s.M, "K": s.K, "N": s.N, "P": s.P, "Q": s.Q, "dual": s.dual, "code": s.code,
            "quant_us": round(float(q) * 1e3, 2), "gemm_us": round(float(g) * 1e3, 2),
            "gemm_exec_tops": round(tops, 1), "gemm_useful_tops": round(uo / (g * 1e-3) / 1e12, 1),
            "gemm_frac_of_measured_8bit_peak": round(tops / p8["burst"], 4),
            "gemm_frac_of_sustained_8bit_peak": None if p8["sustained"] is None else round(tops / p8["sustained"], 4),
            "gemm_frac_of_nominal_4500": round(tops / NOMINAL_8BIT_TOPS, 4),
            "gemm_bound": "tensor" if t_tensor >= t_hbm else "hbm",
            "gemm_roofline_frac": round(max(t_tensor, t_hbm) / (g * 1e-3), 4),
            "layer_roofline_frac": round((max(t_tensor, t_hbm) + quant_bytes(s) / (peaks["hbm_gbs"] * 1e9)) /
                                         ((q + g) * 1e-3), 4),
            "quant_gbs": round(quant_bytes(s) / (q * 1e-3) / 1e9, 1),
            "quant_frac_of_measured_hbm": round(quant_bytes(s) / (q * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
            "quant_frac_of_nominal_8000": round(quant_bytes(s) / (q * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
            "plain_w8a8_gemm_us": None if pl is None else round(pl * 1e3, 2),
            "dual_gemm_time_over_plain": None if pl is None else round(float(g) / pl, 3),
            "unsegmented_gemm_us": None if un is None else round(un * 1e3, 2),
            "seglinear_gemm_time_over_unsegmented": None if un is None else round(float(g) / un, 3),
        })
        i = len(rows) - 1
        r, us = rows[-1], lambda v: None if v is None else round(v, 2)
        layer_us = (q + g) * 1e3
        if kt["q_plain"][i] is not None:
            plain_us = kt["q_plain"][i] + kt["plain"][i]
            r.update({"plain_w8a8_quant_us": us(kt["q_plain"][i]),
                      "dual_layer_time_over_plain_layer": round(layer_us / plain_us, 3)})
            if kt["q_zp"][i] is not None:
                zp_us = kt["q_zp"][i] + kt["g_zp"][i]
                r.update({"asym_quant_us": us(kt["q_zp"][i]), "asym_gemm_us": us(kt["g_zp"][i]),
                          "dual_layer_time_over_asym_layer": round(layer_us / zp_us, 3),
                          "asym_layer_time_over_plain_layer": round(zp_us / plain_us, 3)})
        if kt["w4_q"][i] is not None:
            w4_us = kt["w4_q"][i] + kt["w4_unpack"][i] + kt["w4_g"][i]
            r["w4a8"] = {"per_token_quant_us": us(kt["w4_q"][i]), "unpack_us": us(kt["w4_unpack"][i]),
                         "gemm_us": us(kt["w4_g"][i]), "layer_time_over_w8a8_layer": round(w4_us / layer_us, 3),
                         "note": "per-channel 4-bit weights kept packed and unpacked in front of the GEMM, per-token "
                                 "activation scales; the GEMM runs the variant with per-(token, channel) factors"}
        if kt["lib"][i] is not None:
            ours = kt["plain"][i] if s.dual else g * 1e3           # the single-code-matrix GEMM of this shape
            r["library_gemm_same_shape"] = {
                "us": us(kt["lib"][i]), "ours_single_scale_us": us(ours), "ours_over_library": round(ours / kt["lib"][i], 3),
                "note": "vendor library's plain dense GEMM of this M, K, N (int8 -> int32 or e4m3 -> bf16, no segment "
                        "scales, no bias), same timing method; ours is the single-scale GEMM with its dequantizing "
                        "epilogue; context, not part of the product path"}
        if kt["g_split"][i] is not None:
            r["split_tiles"] = {"gemm_us": us(kt["g_split"][i]), "time_over_whole_tiles": round(kt["g_split"][i] / (g * 1e3), 3),
                                "note": "K loops cut across CTA pairs with the partial sums exchanged through the larger "
                                        "workspace, forced for this measurement; the automatic choice is the other column"}
        if kt["q_fused"][i] is not None:
            r["fused_act"] = {"act": s.x_kind.partition("+")[2], "fused_quant_us": us(kt["q_fused"][i]),
                              "unfused_act_us": us(kt["act"][i]), "unfused_pair_us": us(kt["act"][i] + q * 1e3),
                              "fused_time_over_unfused_pair": round(kt["q_fused"][i] / (kt["act"][i] + q * 1e3), 3),
                              # unfused: the activation is written and read again (gated: so is GELU(gate))
                              "hbm_bytes_saved": (8 if s.x_kind.endswith("geglu") else 4) * s.M * s.K,
                              "note": "the unfused activation is a library elementwise kernel (comparison only)"}
    return rows


def buffer_sets(layers):
    """Rotating buffer sets for the back-to-back timing: together at least three times the L2 capacity."""
    set_bytes = sum(bl.device_bytes() for bl in layers)
    n_sets = max(2, -(-3 * L2_BYTES // set_bytes))
    return [layers] + [[bl.device_copy() for bl in layers] for _ in range(n_sets - 1)], set_bytes, n_sets


def measure_side_workload(name, dev, args, peaks):
    """One of the further workloads of the report: the per-layer table (kernels timed alone) and whole steps
    back to back; no end-to-end leg, no CPU baseline."""
    from paper_2507_14811_b200 import workloads as WL
    specs = WL.WORKLOADS[name]
    layers = [BenchLayer(s, dev) for s in specs]
    time.sleep(COOL_DOWN_S)                    # the power state of the previous long region must not leak in
    kt = time_kernels(layers, with_w4a8=name in ("dit_xl2", "sd3_heads"), with_split=name in ("dit_xl2", "sdxl_geglu"))
    for bl in layers:
        bl.layer.check_status()
    sets, set_bytes, n_sets = buffer_sets(layers)
    steps = max(3, min(args.steps, 50))
    step_ms, mode, launches, reps = time_steps_back_to_back(sets, steps, max(3, min(args.warmup, 5)), 0.05)
    planned_ms = time_steps_planned(sets, steps)
    del sets
    exec_ops = sum(layer_ops(s)[0] for s in specs)
    tops = exec_ops / (step_ms * 1e-3) / 1e12
    out = {"ms_per_step": round(step_ms, 5), "ms_per_step_planned_calls_from_host": round(planned_ms, 5),
           "exec_tops": round(tops, 1),
           "whole_step": fractions(tops, eight_bit_peaks(peaks)),
           "timed_region": f"{reps} replay(s) of a CUDA graph of {steps} steps over {n_sets} buffer sets "
                           f"({n_sets * set_bytes / 2**20:.0f} MiB)",
           "dtype": specs[0].code,
           "per_layer": layer_table(specs, kt, peaks)}
    del layers
    torch.cuda.empty_cache()
    return out


SIDE_WORKLOADS = ["flux", "dit_xl2", "sdxl_skip", "sdxl_sweep", "sd3_heads", "sdxl_geglu", "modulation_small_m", "sd3_qkv_768x2"]


def run_ours(args):
    from paper_2507_14811_b200 import binding as B
    from paper_2507_14811_b200 import workloads as WL

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    B.lib()

    specs = WL.WORKLOADS[args.workload]
    layers = [BenchLayer(s, dev) for s in specs]
    if args.profile_steps:
        # For captures with a profiler: nothing but eager whole steps over the rotating buffer sets (launch order per
        # step: quantize, GEMM of layer 0, quantize, GEMM of layer 1, ...).  Prints no measurement.
        layer_sets, _, n_sets = buffer_sets(layers)
        for i in range(args.profile_steps):
            for bl in layer_sets[i % n_sets]:
                bl.quantize()
                bl.gemm()
        torch.cuda.synchronize()
        for bl in layers:
            bl.layer.check_status()
        return {"profile_steps": args.profile_steps, "workload": args.workload, "buffer_sets": n_sets}
    flush_w = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_r = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)

    def flush():
        """Evicts the layer's inputs from L2: a write larger than L2, then a read larger than L2 so that
        the cache is left holding clean lines (dirty lines of the write would otherwise be written back
        during the timed kernel and be charged to it)."""
        flush_w.zero_()
        flush_r.sum()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    peaks = measured_peaks()
    p8 = eight_bit_peaks(peaks)

    # ---- every kernel timed alone (burst conditions), before anything heats the chip
    barrier()
    sampler_k = ClockSampler(local)
    sampler_k.start()
    kt = time_kernels(layers)
    clocks_k = sampler_k.stop()
    for bl in layers:
        bl.layer.check_status()
    # ---- whole steps back to back: the graph of K steps is replayed until the region lasts args.min_region_s
    layer_sets, set_bytes, n_sets = buffer_sets(layers)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()                            # SM clock and throttle reasons DURING the long timed region
    step_ms, step_mode, launches, reps = time_steps_back_to_back(layer_sets, args.steps, args.warmup, args.min_region_s)
    clocks = sampler.stop()
    barrier()
    time.sleep(COOL_DOWN_S)
    planned_ms = time_steps_planned(layer_sets, args.steps)
    del layer_sets
    torch.cuda.empty_cache()
    time.sleep(COOL_DOWN_S)
    e2e_steps = max(3, min(args.steps, 50) // 4)
    e2e_ms = time_e2e(layers, e2e_steps, args.warmup, flush, args.e2e_chunks)
    e2e_step_ms = time_e2e_step(layers, e2e_steps, args.warmup, flush, args.e2e_chunks)
    barrier()

    split_ms = (sum(kt["q"]) + sum(kt["g"])) * 1e-3     # the step's kernels timed alone, summed
    e2e_layers_ms = float(e2e_ms.sum())        # the layers' end-to-end calls timed one after the other
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([step_ms, e2e_step_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        step_ms, e2e_step_ms = float(t[0]), float(t[1])

    exec_ops = sum(layer_ops(s)[0] for s in specs)
    useful_ops = sum(layer_ops(s)[1] for s in specs)
    gemm_ms = sum(kt["g"]) * 1e-3
    quant_ms = sum(kt["q"]) * 1e-3
    achieved = exec_ops / (gemm_ms * 1e-3) / 1e12
    per_layer = layer_table(specs, kt, peaks)
    # roofline of the dominant kernel (the GEMM launches of one step): per launch the slower of tensor time and
    # HBM time, summed, over the measured time
    t_roof = sum(max(layer_ops(s)[0] / (p8["burst"] * 1e12), gemm_bytes(s) / (peaks["hbm_gbs"] * 1e9)) for s in specs)
    bounds = sorted({r["gemm_bound"] for r in per_layer})
    traffic, traffic_note = gemm_dram_traffic(args.workload)
    step_tops = exec_ops / (step_ms * 1e-3) / 1e12
    region_s = step_ms * 1e-3 * args.steps * reps

    lib_peaks = None
    if world == 1 and rank == 0 and not args.only_headline:
        time.sleep(COOL_DOWN_S)
        lib_peaks = library_8bit_peaks(dev)
    side = {}
    if world == 1 and rank == 0 and not args.only_headline:
        del layers
        torch.cuda.empty_cache()
        for name in SIDE_WORKLOADS:
            if name != args.workload:
                side[name] = measure_side_workload(name, dev, args, peaks)

    out = None
    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu, _, _ = oracle_sample(specs)
        h2d = sum(s.M * s.K * (4 if s.x_dtype == "f32" else 2) for s in specs)
        d2h = sum(s.M * s.N * 2 for s in specs)
        out = {
            "metric": METRIC, "value": round(world * step_tops, 2), "unit": "TOPS",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(step_ms, 5),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "e4m3" if specs[0].code == "e4m3" else "int8", "data": "synthetic",
            "config": {"workload": args.workload,
                       "layers": [f"{s.name} M={s.M} K={s.K} N={s.N} P={s.P} Q={s.Q} {'dual' if s.dual else 'single'} {s.code}"
                                  for s in specs],
                       "step": "every layer: quantize_act -> dual/seg GEMM + dequant epilogue (bf16 out); steps run "
                               "back to back between one pair of CUDA events",
                       "timed_region": f"{step_mode}: {reps} replay(s) x {args.steps} steps = {reps * args.steps} steps, "
                                       f"{region_s:.3f} s between one pair of CUDA events",
                       "ops": "executed tensor ops: 4MNK for dual layers, 2MNK for single-scale layers",
                       "l2": f"inputs larger than L2: step i uses buffer set i mod {n_sets} (weights, inputs, codes, outputs; "
                             f"{set_bytes / 2**20:.0f} MiB per set, {n_sets * set_bytes / 2**20:.0f} MiB in all, L2 = {L2_BYTES >> 20} MiB); "
                             "the per-kernel timings rotate over copies of one layer's buffers the same way",
                       "parallelism": f"{world} independent row-sharded replicas, no collective" if world > 1 else "1 GPU"},
            "timed_region_s": round(region_s, 4), "graph_replays": reps,
            "useful_tops": round(world * useful_ops / (step_ms * 1e-3) / 1e12, 2),
            "whole_step": dict(fractions(step_tops, p8),
                               note="quantize + GEMM of every layer inside a long back-to-back region: the sustained "
                                    "peak is the fair denominator; the quantize passes are HBM work inside it"),
            "ms_per_step_kernels_timed_alone": round(split_ms, 5),
            "ms_per_step_planned_calls_from_host": round(planned_ms, 5),
            "planned_calls_note": "the same steps without a CUDA graph: every layer issued from the host through its "
                                  "prepared call (segquant_plan_run: two launches, no checks or queries), short region",
            "frac_of_nominal_4500_tops": round(step_tops / NOMINAL_8BIT_TOPS, 4),
            "e2e": {"value": round(world * exec_ops / (e2e_step_ms * 1e-3) / 1e12, 2), "unit": "TOPS",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_step_ms, 4),
                    "ms_per_step_layers_one_by_one": round(e2e_layers_ms, 4),
                    "call": f"segquant_layer_forward_pipelined per layer, {max(args.e2e_chunks, 2)} row chunks, copies on their own "
                            "streams; the layers of a step run on separate streams so that their copies in opposite "
                            "directions overlap"},
            "gpu_launches": int(launches) * reps,
            "roofline": {"bound": bounds[0] if len(bounds) == 1 else "tensor+hbm (per layer, see per_layer.gemm_bound)",
                         "achieved": round(achieved, 1), "peak": round(p8["burst"], 1),
                         "unit": "TFLOP/s", "frac": round(t_roof / (gemm_ms * 1e-3), 4),
                         "frac_of_sustained_peak": None if p8["sustained"] is None else round(achieved / p8["sustained"], 4),
                         "frac_of_nominal_4500": round(achieved / NOMINAL_8BIT_TOPS, 4),
                         "traffic": traffic, "traffic_note": traffic_note,
                         "traffic_unit": "bytes per step (all GEMM launches of the step, like achieved)",
                         "algorithmic_bytes_per_step": int(sum(gemm_bytes(s) for s in specs)),
                         "kernel": "segquant_gemm_kernel", "launches_per_step": len(specs),
                         "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} TFLOP/s x 2 (nominal 8-bit : bf16 "
                                        "ratio); burst because each launch is timed alone between its own events with L2 flushed",
                         "frac_definition": "sum over the step's GEMM launches of max(executed ops / peak, algorithmic bytes / "
                                            "measured HBM bandwidth), over their summed CUDA-event time",
                         "library_gemm_8192": lib_peaks,
                         "library_gemm_note": "the vendor library's dense int8 / fp8 GEMM at 8192^3 on this GPU (burst), for "
                                              "context beside the derived peak; not part of the product path",
                         "algorithmic_ops_per_step": exec_ops, "avg_launch_us": round(gemm_ms * 1e3 / len(specs), 2),
                         "note": "8-bit integer / fp8 tensor ops counted as flops"},
            "quantize_roofline": {"bound": "hbm",
                                  "achieved": round(sum(quant_bytes(s) for s in specs) / (quant_ms * 1e-3) / 1e9, 1),
                                  "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": round(sum(quant_bytes(s) for s in specs) / (quant_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                                  "frac_of_nominal_8000": round(sum(quant_bytes(s) for s in specs) / (quant_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
                                  "kernel": "quantize_kernel"},
            "cpu_baseline": cpu,
            "clocks": clocks,
            "clocks_kernels_timed_alone": clocks_k,
            "kernel_timing": "each kernel alone: a CUDA graph of >= 48 launches of that kernel over copies of the layer's "
                             "buffers that together exceed twice the L2 capacity, one replay between a pair of events",
            "per_layer": per_layer,
            "workloads": side,
        }
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return out


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the GEMM launches of one step, from ncu captures of
# these workloads whose summaries are kept among the committed profile summaries.  Each entry carries the SHA-256
# prefix of the GEMM kernel source the counters were taken with; once that file has changed the figure is stale
# and the bench prints null.
GEMM_DRAM_TRAFFIC = {
    "sd3_mmdit": {"bytes": 41489920 + 39200512 + 23266048 + 59767040 + 122890496 + 14484224, "source_tag": "377849a5a34f92d9",
                  "from": "ncu --set full of the three GEMM launches of one eager step (bench.py --workload sd3_mmdit "
                          "--profile-steps 4); below the algorithmic bytes because part of Y is still in L2 when a kernel ends"},
    "dit_xl2": {"bytes": 12758272 + 15872 + 24237312 + 0, "source_tag": "377849a5a34f92d9",
                "from": "ncu --set full of the two GEMM launches of one eager step (bench.py --workload dit_xl2 "
                        "--profile-steps 4); operands partly L2-resident from the quantize pass, Y stays in L2"},
}


def gemm_source_tag():
    import hashlib
    path = os.path.join(ROOT, "paper_2507_14811_b200", "csrc", "gemm_tcgen05.cu")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def gemm_dram_traffic(workload):
    entry = GEMM_DRAM_TRAFFIC.get(workload)
    if entry is None:
        return None, "no ncu capture of this workload's GEMM launches is on file"
    if entry["source_tag"] != gemm_source_tag():
        return None, "the GEMM kernel source has changed since the counters were taken"
    return entry["bytes"], entry["from"]


# ------------------------------------------------------------------------------------ reference arm

def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    import oracle as O
    from paper_2507_14811_b200 import workloads as WL
    specs = WL.WORKLOADS[args.workload]
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    rows = 128 if args.workload != "tiny_qkv" else 16      # per layer and step: the whole run stays within a minute or two
    prepared = []
    for spec in specs:
        data = WL.make_layer(spec, M=rows)
        qmax, qmin = (127.0, 128.0) if spec.code == "int8" else (448.0, 448.0)
        Wn = data.W.numpy()
        s_pos, s_neg = O.calib_act(data.X_cal.float().numpy(), spec.kb, spec.dual, q_max=qmax, q_min_abs=qmin)
        s_w = O.calib_weight(Wn, spec.kb, spec.nb, w_max=qmax)
        Wq = O.quantize_weight(Wn, spec.kb, spec.nb, s_w, code=spec.code, w_max=qmax)
        prepared.append((spec, data.X.float().numpy(), Wq, s_pos, s_neg, s_w, data.bias.numpy(), qmax, qmin))

    def step():
        for spec, Xn, Wq, s_pos, s_neg, s_w, b, qmax, qmin in prepared:
            O.layer_forward(Xn, Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w, b, code=spec.code,
                            q_max=qmax, q_min_abs=qmin)

    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    ops = sum(layer_ops(s, rows)[0] for s in specs)
    val = round(ops / dt / 1e12, 5)
    sample = f"each step = first {rows} rows of every layer of the workload through the CPU oracle"
    return {"impl": "reference", "metric": METRIC, "value": val, "unit": "TOPS", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "e4m3" if specs[0].code == "e4m3" else "int8", "data": "synthetic",
            "config": {"workload": args.workload,
                       "layers": [f"{s.name} M={s.M} K={s.K} N={s.N} P={s.P} Q={s.Q} {'dual' if s.dual else 'single'} {s.code}"
                                  for s in specs],
                       "ops": "executed tensor ops: 4MNK for dual layers, 2MNK for single-scale layers",
                       "sample": sample},
            "cpu_baseline": {"value": val, "unit": "TOPS", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="sd3_mmdit")
    ap.add_argument("--min-region-s", type=float, default=0.5,
                    help="the K-step graph is replayed until the timed region lasts this long")
    ap.add_argument("--profile-steps", type=int, default=0,
                    help="run this many eager steps of the workload and exit (for profiler captures; no timing)")
    ap.add_argument("--only-headline", action="store_true", help="skip the per-layer tables of the other workloads")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tile-n", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--cta-group", type=int, default=0)
    ap.add_argument("--segment-mode", type=int, default=0)
    ap.add_argument("--e2e-chunks", type=int, default=4, help="row chunks of the end-to-end call (1 = no overlap of copies and kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        out = run_reference(args)
    else:
        if args.tile_n or args.stages or args.cta_group or args.segment_mode:
            from paper_2507_14811_b200 import binding as B
            B.segquant_set_tuning(args.tile_n, args.stages, args.cta_group, args.segment_mode)
        out = run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
