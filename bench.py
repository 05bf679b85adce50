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
L2_BYTES = 126 << 20
L2_FLUSH_BYTES = 256 << 20


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
        for name in ("X", "c_pos", "c_neg", "Y"):
            t = getattr(self, name)
            setattr(other, name, None if t is None else t.clone())
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


def time_workload(layers, steps, warmup, flush, sampler=None):
    """Returns per-layer mean (quantize_ms, gemm_ms) over `steps` timed steps, each layer starting
    with a flushed L2; events are recorded on the launching (current) stream."""
    nl = len(layers)
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(nl)] for _ in range(steps)]
    for _ in range(warmup):
        for bl in layers:
            flush()
            bl.quantize()
            bl.gemm()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    for s in range(steps):
        for i, bl in enumerate(layers):
            flush()
            ev[s][i][0].record()
            bl.quantize()
            ev[s][i][1].record()
            bl.gemm()
            ev[s][i][2].record()
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    q_ms = np.array([[ev[s][i][0].elapsed_time(ev[s][i][1]) for i in range(nl)] for s in range(steps)])
    g_ms = np.array([[ev[s][i][1].elapsed_time(ev[s][i][2]) for i in range(nl)] for s in range(steps)])
    return q_ms.mean(axis=0), g_ms.mean(axis=0), clocks


def time_layers(layers, steps, warmup, flush):
    """Per-layer mean time of quantize + GEMM issued back to back (one event pair per layer, L2 flushed before)."""
    nl = len(layers)
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(nl)] for _ in range(steps)]
    for _ in range(warmup):
        for bl in layers:
            flush()
            bl.quantize()
            bl.gemm()
    torch.cuda.synchronize()
    for s in range(steps):
        for i, bl in enumerate(layers):
            flush()
            ev[s][i][0].record()
            bl.quantize()
            bl.gemm()
            ev[s][i][1].record()
    torch.cuda.synchronize()
    return np.array([[ev[s][i][0].elapsed_time(ev[s][i][1]) for i in range(nl)] for s in range(steps)]).mean(axis=0)


def time_steps_back_to_back(layer_sets, steps, warmup):
    """K whole steps (quantize + GEMM of every layer) issued back to back, one CUDA-event pair around all of
    them.  Step i works on buffer set i mod R; the sets together are several times the L2 capacity, so every
    step finds its inputs and weights in HBM without a flush between steps.  The K steps are captured once
    into a CUDA graph (the launches keep their programmatic-dependent-launch edges) and the timed region is
    one replay, so the host's launch rate is not part of the measurement.  Returns (ms per step, mode,
    kernel launches inside the timed region)."""
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
        mode = "cuda graph of K steps, one replay timed"
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
        n0 = B.segquant_launch_count()
        e0.record(stream)
        run()
        e1.record(stream)
        stream.synchronize()
        if launches is None:
            launches = B.segquant_launch_count() - n0
    torch.cuda.current_stream().wait_stream(stream)
    return e0.elapsed_time(e1) / steps, mode, launches


def time_variant(layers, steps, flush, pick, call):
    """Mean GEMM time of a comparison variant (`call`) on the layers selected by `pick`; None for the others."""
    out = []
    for bl in layers:
        if not pick(bl.spec):
            out.append(None)
            continue
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        for _ in range(3):
            call(bl)
        for s in range(steps):
            flush()
            bl.quantize()
            ev[s][0].record()
            call(bl)
            ev[s][1].record()
        torch.cuda.synchronize()
        out.append(float(np.mean([a.elapsed_time(b) for a, b in ev])))
    return out


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
    flush_w = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_r = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)

    def flush():
        """Evicts the layer's inputs from L2: a write larger than L2, then a read larger than L2 so that
        the cache is left holding clean lines (dirty lines of the write would otherwise be written back
        during the timed kernel and be charged to it)."""
        flush_w.zero_()
        flush_r.sum()
    sampler = ClockSampler(local)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # buffer sets for the back-to-back timing: together at least three times the L2 capacity
    set_bytes = sum(bl.device_bytes() for bl in layers)
    n_sets = max(2, -(-3 * L2_BYTES // set_bytes))
    layer_sets = [layers] + [[bl.device_copy() for bl in layers] for _ in range(n_sets - 1)]

    barrier()
    sampler.start()                            # SM clock and throttle reasons over both timed passes
    step_ms, step_mode, launches = time_steps_back_to_back(layer_sets, args.steps, args.warmup)
    barrier()
    q_ms, g_ms, _ = time_workload(layers, args.steps, args.warmup, flush, None)
    clocks = sampler.stop()
    barrier()
    for bl in layers:
        bl.layer.check_status()
    layer_ms = time_layers(layers, args.steps, 3, flush)
    cmp_steps = max(3, min(args.steps, 20))
    plain_ms = time_variant(layers, cmp_steps, flush, lambda sp: sp.dual, lambda bl: bl.gemm_plain())
    unseg_ms = time_variant(layers, cmp_steps, flush, lambda sp: sp.P > 1 or sp.Q > 1, lambda bl: bl.gemm_unsegmented())
    e2e_ms = time_e2e(layers, max(3, args.steps // 4), args.warmup, flush, args.e2e_chunks)
    e2e_step_ms = time_e2e_step(layers, max(3, args.steps // 4), args.warmup, flush, args.e2e_chunks)
    barrier()

    layers_ms = float(layer_ms.sum())          # quantize + GEMM of a layer between one event pair, L2 flushed before
    split_ms = float((q_ms + g_ms).sum())      # the same kernels timed one by one (an event between them)
    e2e_layers_ms = float(e2e_ms.sum())        # the layers' end-to-end calls timed one after the other
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([step_ms, e2e_step_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        step_ms, e2e_step_ms = float(t[0]), float(t[1])

    exec_ops = sum(layer_ops(s)[0] for s in specs)
    useful_ops = sum(layer_ops(s)[1] for s in specs)
    peaks = measured_peaks()
    # dense 8-bit tensor peak = measured bf16 burst peak x nominal ratio (4.5 / 2.25 PFLOP/s)
    peak8 = peaks["bf16_tflops"] * 2.0
    gemm_ops = exec_ops
    gemm_ms = float(g_ms.sum())
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12

    per_layer = []
    for s, q, g, pl, un in zip(specs, q_ms, g_ms, plain_ms, unseg_ms):
        eo, uo = layer_ops(s)
        t_tensor = eo / (peak8 * 1e12)
        t_hbm = gemm_bytes(s) / (peaks["hbm_gbs"] * 1e9)
        per_layer.append({
            "layer": s.name, "M": s.M, "K": s.K, "N": s.N, "P": s.P, "Q": s.Q, "dual": s.dual, "code": s.code,
            "quant_us": round(float(q) * 1e3, 2), "gemm_us": round(float(g) * 1e3, 2),
            "gemm_exec_tops": round(eo / (g * 1e-3) / 1e12, 1), "gemm_useful_tops": round(uo / (g * 1e-3) / 1e12, 1),
            "gemm_frac_of_measured_8bit_peak": round(eo / (g * 1e-3) / 1e12 / peak8, 4),
            "gemm_frac_of_nominal_4500": round(eo / (g * 1e-3) / 1e12 / NOMINAL_8BIT_TOPS, 4),
            "gemm_roofline_frac": round(max(t_tensor, t_hbm) / (g * 1e-3), 4),
            "quant_gbs": round(quant_bytes(s) / (q * 1e-3) / 1e9, 1),
            "quant_frac_of_measured_hbm": round(quant_bytes(s) / (q * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
            "plain_w8a8_gemm_us": None if pl is None else round(pl * 1e3, 2),
            "dual_gemm_time_over_plain": None if pl is None else round(float(g) / pl, 3),
            "unsegmented_gemm_us": None if un is None else round(un * 1e3, 2),
            "seglinear_gemm_time_over_unsegmented": None if un is None else round(float(g) / un, 3),
        })

    out = None
    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu, _, _ = oracle_sample(specs)
        h2d = sum(s.M * s.K * (4 if s.x_dtype == "f32" else 2) for s in specs)
        d2h = sum(s.M * s.N * 2 for s in specs)
        out = {
            "metric": METRIC, "value": round(world * exec_ops / (step_ms * 1e-3) / 1e12, 2), "unit": "TOPS",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(step_ms, 5),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "e4m3" if specs[0].code == "e4m3" else "int8", "data": "synthetic",
            "config": {"workload": args.workload,
                       "layers": [f"{s.name} M={s.M} K={s.K} N={s.N} P={s.P} Q={s.Q} {'dual' if s.dual else 'single'} {s.code}"
                                  for s in specs],
                       "step": "every layer: quantize_act -> dual/seg GEMM + dequant epilogue (bf16 out); the K steps run "
                               "back to back between one pair of CUDA events",
                       "timed_region": step_mode,
                       "ops": "executed tensor ops: 4MNK for dual layers, 2MNK for single-scale layers",
                       "l2": f"inputs larger than L2: step i uses buffer set i mod {n_sets} (weights, inputs, codes, outputs; "
                             f"{set_bytes / 2**20:.0f} MiB per set, {n_sets * set_bytes / 2**20:.0f} MiB in all, L2 = {L2_BYTES >> 20} MiB); "
                             f"the per-kernel and per-layer timings flush L2 instead ({L2_FLUSH_BYTES >> 20} MiB write, then read)",
                       "parallelism": f"{world} independent row-sharded replicas, no collective" if world > 1 else "1 GPU"},
            "useful_tops": round(world * useful_ops / (step_ms * 1e-3) / 1e12, 2),
            "ms_per_step_layers_timed_one_by_one": round(layers_ms, 5),
            "ms_per_step_kernels_timed_one_by_one": round(split_ms, 5),
            "frac_of_nominal_4500_tops": round(exec_ops / (step_ms * 1e-3) / 1e12 / NOMINAL_8BIT_TOPS, 4),
            "e2e": {"value": round(world * exec_ops / (e2e_step_ms * 1e-3) / 1e12, 2), "unit": "TOPS",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_step_ms, 4),
                    "ms_per_step_layers_one_by_one": round(e2e_layers_ms, 4),
                    "call": f"segquant_layer_forward_pipelined per layer, {max(args.e2e_chunks, 2)} row chunks, copies on their own "
                            "streams; the layers of a step run on separate streams so that their copies in opposite "
                            "directions overlap"},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "achieved": round(achieved, 1), "peak": round(peak8, 1),
                         "unit": "TFLOP/s", "frac": round(achieved / peak8, 4),
                         "traffic": GEMM_DRAM_TRAFFIC.get(args.workload),
                         "traffic_unit": "bytes per step (all GEMM launches of the step, like achieved)",
                         "kernel": "segquant_gemm_kernel", "launches_per_step": len(specs),
                         "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} TFLOP/s x 2 (nominal 8-bit : bf16 ratio)",
                         "algorithmic_ops_per_step": gemm_ops, "avg_launch_us": round(gemm_ms * 1e3 / len(specs), 2),
                         "note": "8-bit integer / fp8 tensor ops counted as flops"},
            "cpu_baseline": cpu,
            "clocks": clocks,
            "per_layer": per_layer,
            "offline_setup_s": round(sum(bl.offline_s for bl in layers), 3),
        }
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return out


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the GEMM launches of one step, from the ncu
# capture of these workloads (its summary is kept among the committed profile summaries); None = not captured.
GEMM_DRAM_TRAFFIC = {"dit_xl2": 12758528 + 12544 + 24237568 + 1792,
                     "sd3_mmdit": 41489152 + 38824960 + 23200512 + 56566784 + 123355648 + 13652992}


# ------------------------------------------------------------------------------------ reference arm

def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    import oracle as O
    from paper_2507_14811_b200 import workloads as WL
    specs = WL.WORKLOADS[args.workload]
    steps, warmup = max(1, min(args.steps, 3)), max(0, min(args.warmup, 1))
    rows = 16
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
            "config": {"workload": args.workload, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "TOPS", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="dit_xl2")
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
