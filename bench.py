#!/usr/bin/env python
"""Benchmark of the HGF linear-layer forward pass on B200.

A step is one pass of the whole hot path (activation quantisation, LoRA down-projection, packed
ternary GEMV/GEMM, fused dequantisation + gated correction) over every layer of the workload.

Headline workload (N = 1): decode, M = 1, over the seven projections of a 1.2B-class block
(d = 2048, FFN 5632, r = 32) replicated over enough distinct weight copies that the working set
is > 4x the 126 MB L2, so the weight stream really comes from HBM.  The layers are independent
problems (each has its own seeded x), served by one hgf_group_forward per step: one prologue
launch and one GEMV launch that streams all packed weights.  The metric is algorithmic bytes per
second (packed W + A + B + gate + x + y).  Further lines of evidence (the same layers issued as one
hgf_linear_forward per layer, other token counts, the 7B-class stack, prefill TOPS) are reported
under "extra".

`--impl reference` times the CPU oracle (test infrastructure, as it stands) on the same metric.
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

import numpy as np  # noqa: E402

METRIC = "HGF layer HBM GB/s (M=1 decode) & int8 TOPS (prefill), % of B200 peak"
UNIT = "GB/s"
L2_BYTES = 126e6


def layer_bytes(K, N, r, M, out_bytes=4, base3=False):
    """Algorithmic bytes one layer call must move: packed W (2 bits per weight, or 1.6 in the base-3
    layout), A, B, gate, x, y."""
    return (K * N // 5 if base3 else K * N // 4) + 2 * r * (K + N) + 4 * N + 2 * M * K + out_bytes * M * N


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d.get("hbm_gbs", 6650.0), "bf16_tflops": d.get("bf16_tflops", 1590.0),
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", 1400.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def wait_first_sample(self, timeout_s=10.0):
        """nvidia-smi takes a second or so to print its first line: wait for it, so that a short timed
        region is never over before the sampling has begun."""
        t0 = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t0 < timeout_s:
            time.sleep(0.02)

    def mark(self):
        return len(self.lines)

    def stop(self, first=0, last=None):
        """Summary of the samples [first, last) (marks taken with mark()); the sampler keeps running
        until the process ends if `last` is given."""
        if last is not None:
            return self._summary(self.lines[first:last])
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self._summary(self.lines[first:])

    @staticmethod
    def _summary(lines):
        if not lines:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": []}
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------ GPU arm
class Workload:
    """A list of independent layer problems with everything resident on the device."""

    def __init__(self, hgf, torch, shapes, M, copies, flags=0, seed=0, host_io=False, own_ws=False):
        self.hgf, self.torch, self.M, self.flags = hgf, torch, M, flags
        base3 = bool(flags & hgf.FLAG_BASE3)
        self.base3 = base3
        dev = torch.device("cuda")
        g = torch.Generator(device=dev)
        g.manual_seed(seed)
        out_dt = torch.bfloat16 if flags & hgf.FLAG_OUT_BF16 else torch.float32
        self.layers = []
        x_elems = sum(M * s.d_in for s in shapes) * copies
        y_elems = sum(M * s.d_out for s in shapes) * copies
        self.x_all = torch.empty(x_elems, dtype=torch.bfloat16, device=dev)
        self.y_all = torch.empty(y_elems, dtype=out_dt, device=dev)
        xo = yo = 0
        self.bytes = 0
        self.ops = 0
        ws_bytes = max(hgf.workspace_bytes(M, s.d_in, s.d_out, s.r, flags) for s in shapes)
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        self.ws_of = []   # own_ws: a workspace per layer, so that a layer's prologue results stay put
        for c in range(copies):
            for s in shapes:
                if own_ws:
                    self.ws_of.append(torch.empty(hgf.workspace_bytes(M, s.d_in, s.d_out, s.r, flags), dtype=torch.uint8, device=dev))
                W = torch.randn((s.d_out, s.d_in), generator=g, device=dev, dtype=torch.float32) * 0.02
                packed, gamma = hgf.pack_ternary(W, base3=base3)
                del W
                At = (torch.randn((s.r, s.d_in), generator=g, device=dev) / s.d_in ** 0.5).to(torch.float16)
                Bt = (torch.randn((s.d_out, s.r), generator=g, device=dev) / s.r ** 0.5).to(torch.float16)
                gate = torch.rand(s.d_out, generator=g, device=dev)
                x = self.x_all[xo:xo + M * s.d_in].view(M, s.d_in)
                xf = torch.randn((M, s.d_in), generator=g, device=dev)
                ch = torch.randperm(s.d_in, generator=g, device=dev)[: int(0.02 * s.d_in)]
                xf[:, ch] *= 20.0
                x.copy_(xf.to(torch.bfloat16))
                y = self.y_all[yo:yo + M * s.d_out].view(M, s.d_out)
                xo += M * s.d_in
                yo += M * s.d_out
                self.layers.append((s, x, packed, gamma, At, Bt, gate, y))
                self.bytes += layer_bytes(s.d_in, s.d_out, s.r, M, 2 if flags & hgf.FLAG_OUT_BF16 else 4, base3)
                self.ops += 2 * M * s.d_in * s.d_out
        self.weight_bytes = sum(l[2].numel() + l[4].numel() * 2 + l[5].numel() * 2 for l in self.layers)
        self.graph = None
        self.group = None
        self.launches_per_step = 0
        if host_io:
            self.x_host = torch.empty(x_elems, dtype=torch.bfloat16).pin_memory()
            self.x_host.copy_(self.x_all)
            self.y_host = torch.empty(y_elems, dtype=out_dt).pin_memory()

    def enqueue(self, stream, phases=None):
        for i, (s, x, packed, gamma, At, Bt, gate, y) in enumerate(self.layers):
            self.hgf.linear_forward(x, packed, gamma, s.d_in, s.d_out, At, Bt, gate, y=y,
                                    workspace=self.ws_of[i] if self.ws_of else self.ws,
                                    flags=self.flags, stream=stream, phases=phases)

    def time_phase(self, stream, phases, steps, warmup):
        """Milliseconds per pass over the layers of one launch of each layer call (hgf_linear_forward_phases),
        CUDA events on the launching stream.  Needs own_ws (the contraction reads its layer's prologue results)."""
        torch = self.torch
        assert self.ws_of
        with torch.cuda.stream(stream):
            self.enqueue(stream)
            for _ in range(warmup):
                self.enqueue(stream, phases)
            stream.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for _ in range(steps):
                self.enqueue(stream, phases)
            t1.record(stream)
            stream.synchronize()
        return t0.elapsed_time(t1) / steps

    def make_group(self):
        """All layers as one group of independent problems (hgf_group_forward: two launches)."""
        probs = [dict(x=x, packed=p, gamma=g, d_in=s.d_in, d_out=s.d_out, At=At, Bt=Bt, gate=gate, y=y)
                 for (s, x, p, g, At, Bt, gate, y) in self.layers]
        self.group = self.hgf.Group(probs, flags=self.flags)
        self.launches_per_step = 2

    def make_second_buffers(self):
        """A second set of x / y device buffers and a second group on the same weights, for the
        end-to-end loop: while one step computes, the next step's inputs arrive and the previous
        step's results leave."""
        torch = self.torch
        self.x_all2 = torch.empty_like(self.x_all)
        self.y_all2 = torch.empty_like(self.y_all)
        self.y_host2 = torch.empty_like(self.y_host).pin_memory()
        probs, xo, yo = [], 0, 0
        for (s, x, p, g, At, Bt, gate, y) in self.layers:
            x2 = self.x_all2[xo:xo + self.M * s.d_in].view(self.M, s.d_in)
            y2 = self.y_all2[yo:yo + self.M * s.d_out].view(self.M, s.d_out)
            xo += self.M * s.d_in
            yo += self.M * s.d_out
            probs.append(dict(x=x2, packed=p, gamma=g, d_in=s.d_in, d_out=s.d_out, At=At, Bt=Bt, gate=gate, y=y2))
        self.group2 = self.hgf.Group(probs, flags=self.flags)

    def time_steps_e2e_pipelined(self, stream, steps, warmup):
        """Milliseconds per step with host buffers: every step copies its x from pinned host memory and
        its y back, on copy streams of their own, double-buffered against the kernels."""
        torch = self.torch
        bufs = [(self.x_all, self.y_all, self.group, self.y_host), (self.x_all2, self.y_all2, self.group2, self.y_host2)]
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_comp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def one(i):
            b = i & 1
            x, y, group, y_host = bufs[b]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_comp[b])      # the forward that read this x buffer two steps ago
                x.copy_(self.x_host, non_blocking=True)
                ev_in[b].record(s_in)
            stream.wait_event(ev_in[b])
            stream.wait_event(ev_out[b])         # this y buffer has left for the host
            group.forward(stream)
            ev_comp[b].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[b])
                y_host.copy_(y, non_blocking=True)
                ev_out[b].record(s_out)

        for i in range(warmup):
            one(i)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for i in range(steps):
            one(warmup + i)
        stream.wait_event(ev_out[0])
        stream.wait_event(ev_out[1])
        t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / steps

    def gemv_bytes(self):
        """Algorithmic bytes of the GEMV launch alone: packed W, B, gate, x~ (int8), y."""
        ob = 2 if self.flags & self.hgf.FLAG_OUT_BF16 else 4
        wdiv = 5 if self.base3 else 4
        return sum(s.d_in * s.d_out // wdiv + 2 * s.r * s.d_out + 4 * s.d_out + self.M * s.d_in + ob * self.M * s.d_out
                   for (s, *_rest) in self.layers)

    def time_gemv_only(self, stream, steps, warmup):
        """Average duration of the group's GEMV launch alone, CUDA events on the launching stream."""
        torch = self.torch
        with torch.cuda.stream(stream):
            self.group.forward(stream)
            for _ in range(warmup):
                self.group.forward_phases(self.hgf.PHASE_GEMV, stream)
            stream.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for _ in range(steps):
                self.group.forward_phases(self.hgf.PHASE_GEMV, stream)
            t1.record(stream)
            stream.synchronize()
        return t0.elapsed_time(t1) / steps

    def capture(self, stream):
        torch = self.torch
        with torch.cuda.stream(stream):
            self.enqueue(stream)           # first call outside capture: one-time set-up happens here
            stream.synchronize()
            before = self.hgf.launch_count()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=stream):
                self.enqueue(stream)
            self.launches_per_step = self.hgf.launch_count() - before
        stream.synchronize()

    def time_steps(self, stream, steps, warmup, e2e=False):
        """Milliseconds per step, CUDA events on the launching stream."""
        torch = self.torch
        with torch.cuda.stream(stream):
            def one():
                if e2e:
                    self.x_all.copy_(self.x_host, non_blocking=True)
                if self.group is not None:
                    self.group.forward(stream)
                else:
                    self.graph.replay()
                if e2e:
                    self.y_host.copy_(self.y_all, non_blocking=True)
            for _ in range(warmup):
                one()
            stream.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for _ in range(steps):
                one()
            t1.record(stream)
            stream.synchronize()
        return t0.elapsed_time(t1) / steps


def reduce_max_over_ranks(ms, world, dist, device):
    """The step time of the job = the slowest rank's (every rank runs its own replica of the workload)."""
    if world == 1:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2602_05269_b200 import hgf, inputs as syn

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    hgf.lib()
    stream = torch.cuda.Stream()
    peaks = measured_peaks()
    sampler = ClockSampler(local)     # read-only queries; started before the workload is built
    sampler.start()

    def max_over_ranks(ms):
        return reduce_max_over_ranks(ms, world, dist, "cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- headline: config 1 decode, M = 1 -------------------------------------------------------
    shapes1 = syn.CONFIGS[1]["layers"]
    block_bytes = sum(layer_bytes(s.d_in, s.d_out, s.r, 1) for s in shapes1)
    copies = int(np.ceil(4.4 * L2_BYTES / block_bytes))
    main = Workload(hgf, torch, shapes1, 1, copies, host_io=True)
    main.make_group()
    sampler.wait_first_sample()
    barrier()
    mark0 = sampler.mark()
    t_wall = time.perf_counter()
    ms = main.time_steps(stream, args.steps, args.warmup)
    while time.perf_counter() - t_wall < 0.5:       # a short timed region: keep the same step running until the
        main.time_steps(stream, args.steps, 0)      # sampler (one line per 50 ms) has seen the GPU under this load
    mark1 = sampler.mark()
    barrier()
    ms = max_over_ranks(ms)
    ms_e2e_serial = max_over_ranks(main.time_steps(stream, max(args.steps // 4, 1), args.warmup, e2e=True))
    main.make_second_buffers()
    barrier()
    ms_e2e = max_over_ranks(main.time_steps_e2e_pipelined(stream, max(args.steps // 4, 1), args.warmup))
    gemv_ms = main.time_gemv_only(stream, args.steps, args.warmup)
    clocks = sampler.stop(mark0, max(mark1, mark0 + 1))
    hgf.check_status(stream)
    value = world * main.bytes / (ms * 1e-3) / 1e9
    value_e2e = world * main.bytes / (ms_e2e * 1e-3) / 1e9
    n_layers = len(main.layers)
    gemv_bytes = main.gemv_bytes()

    roofline = {"bound": "hbm", "kernel": "decode_gemv_kernel<1> (the GEMV launch of hgf_group_forward, timed alone)",
                "achieved": gemv_bytes / (gemv_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": None, "traffic": decode_traffic(gemv_bytes), "peak_source": peaks["source"],
                "traffic_note": "ncu dram bytes per algorithmic byte of the captured launch x this launch's bytes; null "
                                "when hgf_decode.cu differs from the captured source (sha1 %s)" % DECODE_TRAFFIC["source_sha1"][:12],
                "bytes_per_launch": gemv_bytes, "us_per_launch": gemv_ms * 1e3,
                "frac_of_nominal_8000": None,
                "whole_step": {"GB/s": value, "frac": value / peaks["hbm_gbs"], "launches": 2,
                               "note": "prologue launch (reads x and A) + GEMV launch, all algorithmic bytes"}}
    roofline["frac"] = roofline["achieved"] / roofline["peak"]
    roofline["frac_of_nominal_8000"] = roofline["achieved"] / 8000.0

    # ---- the prefill half of the metric: 2048 -> 5632, r = 32, M = 8192 (config 3) ----------------
    main.group.close()
    main.group2.close()
    del main.group, main.group2
    main_summary = {"bytes": main.bytes, "weight_bytes": main.weight_bytes, "x_bytes": main.x_host.numel() * 2,
                    "y_bytes": main.y_host.numel() * main.y_host.element_size(), "launches_per_step": main.launches_per_step}
    del main
    torch.cuda.empty_cache()
    roofline_prefill = None
    if rank == 0:
        roofline_prefill = measure_prefill_headline(hgf, torch, syn, stream, args, peaks)
    prefill_clocks = sampler.stop(mark1, sampler.mark())

    extra = {}
    if rank == 0 and not args.quick:
        extra = run_extra(hgf, torch, syn, stream, args, peaks, roofline_prefill["peak"] if roofline_prefill else None)
    sampler.stop()

    cpu = cpu_baseline(10.0) if (rank == 0 and world == 1 and not args.no_cpu) else None

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x ternary (int32 accumulate) + fp16 correction",
            "data": "synthetic",
            "config": {"workload": "config1: 1.2B-class block (d=2048, FFN 5632, r=32), 7 projections x "
                                   f"{copies} distinct weight copies = {n_layers} independent layer problems, decode M=1, "
                                   "one hgf_group_forward per step",
                       "why_this_workload": "the metric's decode half is quoted at M=1 on the 1.2B-class layer shapes "
                                            "(configs[1]); its prefill half is measured on configs[3]'s largest case "
                                            "(roofline_prefill); configs 2 and 4 (faster per byte: longer rows) are under "
                                            "extra, config 4 with tokens/s against T_max",
                       "layers_per_step": n_layers, "weight_bytes": main_summary["weight_bytes"],
                       "l2_policy": "inputs larger than L2 (weight working set %.0f MB > 4 x 126 MB)"
                                    % (main_summary["weight_bytes"] / 1e6),
                       "parallelism": "replicas" if world > 1 else "single"},
            "e2e": {"value": value_e2e, "unit": UNIT, "h2d_bytes_per_step": main_summary["x_bytes"],
                    "d2h_bytes_per_step": main_summary["y_bytes"],
                    "ms_per_step": ms_e2e,
                    "how": "every step: x from pinned host memory, hgf_group_forward, y to pinned host memory; two "
                           "sets of device buffers, copies on their own streams, so a step's copies overlap its "
                           "neighbours' kernels",
                    "one_stream_value": world * main_summary["bytes"] / (ms_e2e_serial * 1e-3) / 1e9},
            "gpu_launches": main_summary["launches_per_step"] * args.steps,
            "clocks": clocks, "roofline": roofline, "roofline_prefill": roofline_prefill,
            "value_prefill": None if roofline_prefill is None else
            {"value": roofline_prefill["layer"]["TOPS"], "unit": "int8 TOPS (2*M*K*N per layer call: prologue, rounding and GEMM launches)",
             "frac_of_measured_int8_peak": roofline_prefill["layer"]["frac"], "clocks": prefill_clocks},
            "cpu_baseline": cpu, "extra": extra,
        }
        print(json.dumps(out))
    if world > 1:
        dist.barrier()      # rank 0 alone runs the secondary measurements; the others wait here
        dist.destroy_process_group()


# DRAM traffic of the decode GEMV launch from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum
# of a config-1, M = 1 group launch): bytes moved per algorithmic byte.  It is only reported while the
# kernel source is the one that was captured.
DECODE_TRAFFIC = {"source_sha1": "7b2cc479563a0d062a4c3a356e67630e5471a690",
                  "dram_bytes_per_algorithmic_byte": (517.347072e6 + 7.010560e6) / 518805504.0}


# DRAM traffic of the prefill GEMM launch from one ncu capture of the very shape the bench times
# (2048 -> 5632, r = 32, M = 8192, bf16 y): dram__bytes_read.sum + dram__bytes_write.sum of one launch.  Below
# the launch's algorithmic bytes because most of y is still in L2 when the kernel ends.
PREFILL_TRAFFIC = {"source_sha1": "8ff95e068f9752902d0b321377a47b0986601768", "dram_bytes_per_launch": 21.581312e6 + 43.126016e6}


def prefill_traffic():
    import hashlib
    srcs = [os.path.join(ROOT, "paper_2602_05269_b200", "csrc", f) for f in ("hgf_prefill.cu", "hgf_tc.cuh")]
    if not all(os.path.exists(f) for f in srcs):
        return None
    if hashlib.sha1(b"".join(open(f, "rb").read() for f in srcs)).hexdigest() != PREFILL_TRAFFIC["source_sha1"]:
        return None
    return PREFILL_TRAFFIC["dram_bytes_per_launch"]


def decode_traffic(gemv_bytes):
    import hashlib
    src = os.path.join(ROOT, "paper_2602_05269_b200", "csrc", "hgf_decode.cu")
    if DECODE_TRAFFIC["source_sha1"] is None or not os.path.exists(src):
        return None
    if hashlib.sha1(open(src, "rb").read()).hexdigest() != DECODE_TRAFFIC["source_sha1"]:
        return None
    return DECODE_TRAFFIC["dram_bytes_per_algorithmic_byte"] * gemv_bytes


def measure_int8_ceiling(torch, stream, M, K, N, copies, steps, warmup):
    """A library int8 GEMM (torch._int_mm, int32 out) as the measuring stick for the int8 tensor peak
    of this GPU: on the prefill workload's own shape (rotating over `copies` operand sets, like the
    workload) and on a large square problem.  Returns TOPS figures; None where the call is unavailable."""
    out = {"same_shape_TOPS": None, "square_8192_TOPS": None, "how": "torch._int_mm (cuBLASLt int8 x int8 -> int32), CUDA events"}

    def run(m, k, n, nsets, reps):
        a = [torch.randint(-127, 128, (m, k), dtype=torch.int8, device="cuda") for _ in range(nsets)]
        b = [torch.randint(-1, 2, (k, n), dtype=torch.int8, device="cuda") for _ in range(nsets)]
        c = [torch.empty((m, n), dtype=torch.int32, device="cuda") for _ in range(nsets)]
        with torch.cuda.stream(stream):
            for i in range(warmup):
                torch._int_mm(a[i % nsets], b[i % nsets], out=c[i % nsets])
            stream.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for i in range(reps):
                torch._int_mm(a[i % nsets], b[i % nsets], out=c[i % nsets])
            t1.record(stream)
            stream.synchronize()
        return 2.0 * m * k * n * reps / (t0.elapsed_time(t1) * 1e-3) / 1e12

    try:
        out["same_shape_TOPS"] = run(M, K, N, copies, steps)
        out["square_8192_TOPS"] = run(8192, 8192, 8192, 1, max(steps // 4, 5))
    except Exception as e:  # noqa: BLE001 - the stick is optional, the fallback is stated in the output
        out["error"] = f"{type(e).__name__}: {e}"[:200]
    torch.cuda.empty_cache()
    return out


def measure_prefill_headline(hgf, torch, syn, stream, args, peaks):
    """The prefill half of the metric: hgf_linear_forward on the 2048 -> 5632 projection of config 3
    (r = 32, M = 8192 tokens, bf16 y), rotating over three distinct layers (x, weights, y: 430 MB, larger
    than L2).  Reports the layer call (prologue and rounding launches + tcgen05 GEMM), the GEMM launch and the prologue phase timed alone,
    against a measured int8 ceiling."""
    s = syn.CONFIGS[3]["layers"][4]
    M, copies = 8192, 3
    w = Workload(hgf, torch, [s], M, copies, flags=hgf.FLAG_OUT_BF16, own_ws=True)
    steps = max(20, min(200, args.steps))
    w.capture(stream)
    ms_layer = w.time_steps(stream, steps, args.warmup) / copies
    ms_gemm = w.time_phase(stream, hgf.PHASE_GEMV, steps, args.warmup) / copies
    ms_prol = w.time_phase(stream, hgf.PHASE_PROLOGUE, steps, args.warmup) / copies
    hgf.check_status(stream)
    ops = 2.0 * M * s.d_in * s.d_out
    del w
    torch.cuda.empty_cache()
    stick = measure_int8_ceiling(torch, stream, M, s.d_in, s.d_out, copies, steps, args.warmup)
    cands = [v for v in (stick["same_shape_TOPS"], stick["square_8192_TOPS"]) if v]
    if cands:
        peak, peak_source = max(cands), "measured: library int8 GEMM (the better of the same shape and 8192^3)"
    else:
        peak, peak_source = 2.0 * peaks["bf16_tflops"], "2 x measured bf16 burst (%s; the library int8 GEMM was unavailable)" % peaks["source"]
    tops_gemm, tops_layer = ops / (ms_gemm * 1e-3) / 1e12, ops / (ms_layer * 1e-3) / 1e12
    prol_bytes = 2 * M * s.d_in + M * s.d_in + 2 * s.r * s.d_in      # x read, x~ written, A read
    return {"bound": "tensor", "kernel": "prefill_gemm_kernel (the contraction launch of hgf_linear_forward, timed alone)",
            "workload": f"config3 {s.d_in}->{s.d_out}, r={s.r}, M={M}, bf16 y, {copies} distinct layers in rotation (inputs larger than L2)",
            "achieved": tops_gemm, "peak": peak, "unit": "TOPS (int8, 2*M*K*N)", "frac": tops_gemm / peak, "traffic": prefill_traffic(),
            "traffic_note": "ncu dram bytes of one launch of this shape (x~ 16.8 MB + W 2.9 MB read, y 92 MB written, of which "
                            "about half is still in L2 at kernel end); null when hgf_prefill.cu or hgf_tc.cuh differs from the captured source",
            "algorithmic_bytes_per_launch": M * s.d_in + s.d_in * s.d_out // 4 + 2 * M * s.d_out + 2 * 64 * (M + s.d_out),
            "peak_source": peak_source, "int8_stick": stick,
            "ops_per_launch": ops, "us_per_launch": ms_gemm * 1e3,
            "frac_of_2x_measured_bf16": tops_gemm / (2.0 * peaks["bf16_tflops"]), "frac_of_nominal_4500": tops_gemm / 4500.0,
            "layer": {"us": ms_layer * 1e3, "TOPS": tops_layer, "frac": tops_layer / peak,
                      "frac_of_2x_measured_bf16": tops_layer / (2.0 * peaks["bf16_tflops"]),
                      "frac_of_nominal_4500": tops_layer / 4500.0, "launches": 3,
                      "note": "prologue launch (per-token maxima + LoRA down-projection), rounding launch, GEMM launch, "
                              "chained by programmatic dependent launch"},
            "prologue": {"us": ms_prol * 1e3, "bytes": prol_bytes, "GB/s": prol_bytes / (ms_prol * 1e-3) / 1e9,
                         "frac_of_hbm_peak": prol_bytes / (ms_prol * 1e-3) / 1e9 / peaks["hbm_gbs"]}}


def run_extra(hgf, torch, syn, stream, args, peaks, int8_peak_measured=None):
    """Secondary measurements, same timing rules, each with its own workload."""
    extra = {"decode_group": [], "decode_per_call": [], "prefill": []}
    steps = max(args.steps // 4, 10)

    def decode_case(cfg, shapes, M, label, min_copies=1, group=True, base3=False):
        block = sum(layer_bytes(s.d_in, s.d_out, s.r, M, 4, base3) for s in shapes)
        copies = max(min_copies, int(np.ceil(4.4 * L2_BYTES / block)))
        w = Workload(hgf, torch, shapes, M, copies, flags=hgf.FLAG_BASE3 if base3 else 0)
        if group:
            w.make_group()
        else:
            w.capture(stream)
        ms = w.time_steps(stream, steps, args.warmup)
        gbs = w.bytes / (ms * 1e-3) / 1e9
        row = {"workload": label, "M": M, "bits_per_weight": 1.6 if base3 else 2.0, "layers": len(w.layers), "ms_per_step": ms, "GB/s": gbs,
               "frac_measured_peak": gbs / peaks["hbm_gbs"], "frac_nominal_8000": gbs / 8000.0,
               "launches_per_step": w.launches_per_step}
        if group:
            gms = w.time_gemv_only(stream, steps, args.warmup)
            row["gemv_launch"] = {"us": gms * 1e3, "GB/s": w.gemv_bytes() / (gms * 1e-3) / 1e9,
                                  "frac_measured_peak": w.gemv_bytes() / (gms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
            w.group.close()
        del w
        torch.cuda.empty_cache()
        return row

    for M in (4, 16):
        extra["decode_group"].append(decode_case(1, syn.CONFIGS[1]["layers"], M, "config1 1.2B-class block"))
    for M in (1, 8):
        extra["decode_group"].append(decode_case(2, syn.CONFIGS[2]["layers"], M, "config2 3B-class block"))
    extra["decode_group"].append(decode_case(2, syn.CONFIGS[2]["layers"], 1, "config2 3B-class block", base3=True))
    extra["decode_group"].append(decode_case(1, syn.CONFIGS[1]["layers"], 1, "config1 1.2B-class block", base3=True))
    # config 4: the 7B-class stack, 32 blocks x 7 projections, decode M = 1 -> tokens/s
    params = 32 * sum(s.d_in * s.d_out for s in syn.CONFIGS[4]["layers"])
    for group, base3 in ((True, False), (True, True), (False, False)):
        row = decode_case(4, syn.CONFIGS[4]["layers"], 1, "config4 7B-class stack (32 blocks)", min_copies=32, group=group, base3=base3)
        tok_s = 1e3 / row["ms_per_step"] * (32 * 7 / row["layers"])
        row.update({"tokens_per_s": tok_s, "params": params,
                    "tmax_2bit_measured_bw": hgf.tmax_tokens_per_s(peaks["hbm_gbs"] * 1e9, params, 2.0),
                    "tmax_1p58bit_measured_bw": hgf.tmax_tokens_per_s(peaks["hbm_gbs"] * 1e9, params, 1.58),
                    "tmax_1p6bit_measured_bw": hgf.tmax_tokens_per_s(peaks["hbm_gbs"] * 1e9, params, 1.6),
                    "tmax_2bit_8TBs": hgf.tmax_tokens_per_s(8e12, params, 2.0),
                    "tmax_1p58bit_8TBs": hgf.tmax_tokens_per_s(8e12, params, 1.58)})
        extra["decode_group" if group else "decode_per_call"].append(row)
    # the headline layers issued one hgf_linear_forward per layer (CUDA-graph chained, PDL): launch-bound
    extra["decode_per_call"].append(decode_case(1, syn.CONFIGS[1]["layers"], 1, "config1 1.2B-class block", group=False))

    # prefill: config 3 shapes, bf16 output
    int8_peak_nominal = 4500.0
    int8_peak_2x_bf16 = 2.0 * peaks["bf16_tflops"]
    for M in (512, 2048, 8192):
        for s in syn.distinct_shapes(3):
            w = Workload(hgf, torch, [s], M, 1, flags=hgf.FLAG_OUT_BF16)
            w.capture(stream)
            psteps = max(10, min(200, int(2e11 / w.ops) * 10))
            ms = w.time_steps(stream, psteps, args.warmup)
            tops = w.ops / (ms * 1e-3) / 1e12
            extra["prefill"].append({"shape": f"{s.d_in}->{s.d_out}", "r": s.r, "M": M, "ms": ms, "TOPS": tops,
                                     "frac_measured_int8": tops / int8_peak_measured if int8_peak_measured else None,
                                     "frac_nominal_4500": tops / int8_peak_nominal,
                                     "frac_2x_measured_bf16": tops / int8_peak_2x_bf16})
            del w
            torch.cuda.empty_cache()
    # differential attention forward on projection-shaped inputs (1.2B-class block: 16 heads of 64), causal
    B_, L_, h_, dh_ = 4, 4096, 16, 64
    gq = torch.Generator(device="cuda")
    gq.manual_seed(5)
    qa = torch.randn((B_ * L_, 2 * h_ * dh_), generator=gq, device="cuda").to(torch.bfloat16)
    ka = torch.randn((B_ * L_, 2 * h_ * dh_), generator=gq, device="cuda").to(torch.bfloat16)
    va = torch.randn((B_ * L_, h_ * dh_), generator=gq, device="cuda").to(torch.bfloat16)
    oa = torch.empty((B_ * L_, h_ * dh_), dtype=torch.bfloat16, device="cuda")
    with torch.cuda.stream(stream):
        for _ in range(3):
            hgf.diff_attention_forward(qa, ka, va, B_, L_, h_, dh_, 0.8, out=oa, flags=hgf.FLAG_OUT_BF16, stream=stream)
        stream.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(10):
            hgf.diff_attention_forward(qa, ka, va, B_, L_, h_, dh_, 0.8, out=oa, flags=hgf.FLAG_OUT_BF16, stream=stream)
        t1.record(stream)
        stream.synchronize()
    ms = t0.elapsed_time(t1) / 10
    at_flops = 4.0 * L_ * L_ * dh_ * B_ * h_ * 0.5 * 2   # two streams x (Q K^T and P V) x the causal half
    extra["diff_attention"] = {"workload": f"causal differential attention forward, B={B_}, L={L_}, {h_} heads of {dh_}, bf16",
                               "ms": ms, "TFLOP/s": at_flops / (ms * 1e-3) / 1e12,
                               "frac_measured_bf16": at_flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                               "note": "tcgen05 kernel (a 'next' row): scores and outputs in tensor memory, one softmax thread per row and stream"}
    del qa, ka, va, oa
    torch.cuda.empty_cache()

    # straight-through backward pass of one layer (2048 -> 5632, r = 32, M = 8192): all five gradients
    sb = syn.CONFIGS[3]["layers"][4]
    Mb = 8192
    wb = Workload(hgf, torch, [sb], Mb, 1)
    (_s, xb, pb, gb, Ab, Bb, gateb, _y) = wb.layers[0]
    dyb = torch.randn((Mb, sb.d_out), generator=gq, device="cuda").to(torch.bfloat16)
    hgf.linear_backward(xb, pb, gb, sb.d_in, sb.d_out, dyb, Ab, Bb, gateb, stream=stream)
    stream.synchronize()
    with torch.cuda.stream(stream):
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        keep = hgf.linear_backward(xb, pb, gb, sb.d_in, sb.d_out, dyb, Ab, Bb, gateb, stream=stream)
        t0.record(stream)
        for _ in range(5):
            keep = hgf.linear_backward(xb, pb, gb, sb.d_in, sb.d_out, dyb, Ab, Bb, gateb, stream=stream, out=keep)
        t1.record(stream)
        stream.synchronize()
    ms = t0.elapsed_time(t1) / 5
    bw_flops = 2.0 * Mb * sb.d_in * sb.d_out * 2 + 2.0 * Mb * sb.r * (sb.d_in + sb.d_out) * 3
    extra["ste_backward"] = {"workload": f"straight-through backward of one layer {sb.d_in}->{sb.d_out}, r={sb.r}, M={Mb}: dX, dW, dA, dB, dgate",
                             "ms": ms, "TFLOP/s": bw_flops / (ms * 1e-3) / 1e12,
                             "frac_measured_bf16": bw_flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                             "note": "tcgen05 bf16 GEMMs reading every operand in its stored form (a 'next' row); "
                                     "includes the operand preparation kernels; gradients and workspace preallocated"}
    del wb, keep, dyb
    torch.cuda.empty_cache()

    # config 4 prefill: the whole 7B-class stack, 32 blocks x 7 projections = 224 layers, each with its own
    # weights (generated and packed layer by layer) and its own seeded x, M = 4096, bf16 y
    stack = Workload(hgf, torch, syn.CONFIGS[4]["layers"], 4096, 32, flags=hgf.FLAG_OUT_BF16)
    stack.capture(stream)
    ms = stack.time_steps(stream, 5, 3)
    tops = stack.ops / (ms * 1e-3) / 1e12
    extra["prefill_config4_stack"] = {"workload": "config4 7B-class stack: 224 layers (32 blocks x 7 projections, r=64), "
                                                  "prefill M=4096, bf16 y, one hgf_linear_forward per layer",
                                      "layers": len(stack.layers), "ms_per_pass": ms, "int8_ops": stack.ops, "TOPS": tops,
                                      "frac_measured_int8": tops / int8_peak_measured if int8_peak_measured else None,
                                      "frac_nominal_4500": tops / int8_peak_nominal,
                                      "frac_2x_measured_bf16": tops / int8_peak_2x_bf16,
                                      "prefill_tokens_per_s": 4096 / (ms * 1e-3)}
    del stack
    torch.cuda.empty_cache()
    return extra


# ----------------------------------------------------------------------------------- CPU arms
def cpu_baseline(budget_s: float):
    """The oracle, as it stands, on this host's cores, on a bounded sample of the headline workload."""
    import oracle
    from paper_2602_05269_b200 import inputs as syn

    shapes = syn.distinct_shapes(1)
    probs = []
    for i, s in enumerate(shapes):
        L = syn.make_layer(s, 1, config=1, layer=i)
        g = oracle.gamma_w(L["W"])
        probs.append((s, L, oracle.ternarise(L["W"], g), g))
    nbytes = 0
    reps = 0
    t0 = time.perf_counter()
    while True:
        for s, L, T, g in probs:
            oracle.forward(L["x"], T, g, L["At"], L["Bt"], L["gate"])
            nbytes += layer_bytes(s.d_in, s.d_out, s.r, 1)
        reps += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "host_cores": os.cpu_count(),
            "sample": f"{reps} passes over one layer of each distinct config-1 shape "
                      "(2048->2048, 2048->5632, 5632->2048, r=32) at M=1; bytes are the same algorithmic "
                      "bytes as the GPU metric (the oracle itself reads unpacked int8 codes)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warm = max(args.steps, 1), max(args.warmup, 0)
    per_step = max(0.05, min(2.0, 90.0 / (steps + warm)))
    for _ in range(warm):
        cpu_baseline(per_step)
    vals = []
    t0 = time.perf_counter()
    for _ in range(steps):
        vals.append(cpu_baseline(per_step))
    dt = time.perf_counter() - t0
    v = float(np.mean([c["value"] for c in vals]))
    cb = dict(vals[-1])
    cb["value"] = v
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 / int64 (CPU oracle)", "data": "synthetic",
        "config": {"workload": "config1 decode M=1, bounded sample: one layer of each distinct shape per pass"},
        "cpu_baseline": cb,
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_profile_case(spec: str, reps: int):
    """Plain launches of one layer problem, for use under a profiler: `kind:KxNxM[xr][:bf16]`.
    The printed time is wall-clock context only, never a benchmark value."""
    import torch

    from paper_2602_05269_b200 import hgf, inputs as syn

    parts = spec.split(":")
    dims = [int(v) for v in parts[1].split("x")]
    if parts[0] in ("attention", "backward"):
        return run_profile_next_rows(parts[0], dims, reps)
    K, N, M = dims[:3]
    r = dims[3] if len(dims) > 3 else 32
    flags = hgf.FLAG_OUT_BF16 if (len(parts) > 2 and parts[2] == "bf16") else 0
    copies = int(parts[3]) if len(parts) > 3 else 1
    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    w = Workload(hgf, torch, [syn.LayerShape("p", K, N, r)], M, copies, flags=flags)
    with torch.cuda.stream(stream):
        for _ in range(reps):
            w.enqueue(stream)
        stream.synchronize()
    hgf.check_status(stream)
    print(json.dumps({"profile_case": spec, "reps": reps, "launches": hgf.launch_count()}))


def run_profile_next_rows(kind, dims, reps):
    """`attention:BxLxhxdh` (differential attention forward, bf16 output) or `backward:KxNxMxr` (straight-through
    backward of one layer, all five gradients): plain launches for use under a profiler."""
    import torch

    from paper_2602_05269_b200 import hgf, inputs as syn

    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    if kind == "attention":
        B, L, h, dh = dims
        q = torch.randn((B * L, 2 * h * dh), generator=g, device="cuda").to(torch.bfloat16)
        k = torch.randn((B * L, 2 * h * dh), generator=g, device="cuda").to(torch.bfloat16)
        v = torch.randn((B * L, h * dh), generator=g, device="cuda").to(torch.bfloat16)
        o = torch.empty((B * L, h * dh), dtype=torch.bfloat16, device="cuda")
        with torch.cuda.stream(stream):
            for _ in range(reps):
                hgf.diff_attention_forward(q, k, v, B, L, h, dh, 0.8, out=o, flags=hgf.FLAG_OUT_BF16, stream=stream)
            stream.synchronize()
    else:
        K, N, M, r = dims
        w = Workload(hgf, torch, [syn.LayerShape("p", K, N, r)], M, 1)
        (_s, x, packed, gamma, At, Bt, gate, _y) = w.layers[0]
        dy = torch.randn((M, N), generator=g, device="cuda").to(torch.bfloat16)
        keep = None
        with torch.cuda.stream(stream):
            for _ in range(reps):
                keep = hgf.linear_backward(x, packed, gamma, K, N, dy, At, Bt, gate, stream=stream, out=keep)
            stream.synchronize()
    hgf.check_status(stream)
    print(json.dumps({"profile_case": kind, "dims": dims, "reps": reps, "launches": hgf.launch_count()}))


def run_profile_group(spec: str, reps: int):
    """A few grouped decode steps of one configuration, for use under a profiler (never a benchmark value)."""
    import torch

    from paper_2602_05269_b200 import hgf, inputs as syn

    cfg, M = (int(v) for v in spec.split(","))
    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    shapes = syn.CONFIGS[cfg]["layers"]
    block = sum(layer_bytes(s.d_in, s.d_out, s.r, M) for s in shapes)
    copies = max(32 if cfg == 4 else 1, int(np.ceil(4.4 * L2_BYTES / block)))
    w = Workload(hgf, torch, shapes, M, copies)
    w.make_group()
    with torch.cuda.stream(stream):
        for _ in range(reps + 5):
            w.group.forward(stream)
        stream.synchronize()
    hgf.check_status(stream)
    print(json.dumps({"profile_group": spec, "layers": len(w.layers), "steps": reps + 5, "launches": hgf.launch_count()}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline measurement only")
    ap.add_argument("--no-cpu", action="store_true", help="skip the cpu_baseline leg")
    ap.add_argument("--profile", default=None,
                    help="run plain launches of one case for a profiler, e.g. prefill:2048x5632x8192x32:bf16")
    ap.add_argument("--profile-group", default=None,
                    help="run a few hgf_group_forward steps of one decode workload for a profiler: CONFIG,M (e.g. 1,1)")
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    if args.profile:
        run_profile_case(args.profile, args.reps)
        return
    if args.profile_group:
        run_profile_group(args.profile_group, args.reps)
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
