#!/usr/bin/env python
"""Benchmark of the FGMP linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Default workload: Llama-2-7B FC1 at decode (M=16 tokens, K=4096, N=11008, 10% FP8 blocks in
weights and activations); metric = packed-weight GB/s.  One step = the online path: quantize
the step's activations (bf16 -> mixed NVFP4/FP8) and run the mixed-precision GEMM against
offline-packed weights -- one fused launch at decode, two calls at prefill.  Weight packing is
offline in the method and is timed separately (reported under "offline").  The step rotates
over several weight copies so that the working set exceeds L2.  `value` is the median of
--replays timed runs of exactly --steps steps.  The default run adds the 70B decode layer and
a prefill layer as side objects ("decode_70b", "prefill").  Prints ONE JSON line (rank 0).

With N > 1 (torchrun) every rank runs an independent replica of the same workload on its own
GPU ("weak" scaling, no data-path collective); the time is the max over ranks.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import fgmp_inputs as gi  # noqa: E402

L2_BYTES = 126e6


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def algorithmic_weight_bytes(N, K, p):
    B = N * K // 16
    n8 = int(np.floor(p * B + 0.5))
    return (B - n8) * 9 + n8 * 16 + B / 8.0


def algorithmic_act_bytes(M, K, p):
    B = M * K // 16
    n8 = int(np.floor(p * B + 0.5))
    return (B - n8) * 9 + n8 * 16 + B / 8.0


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU while the timed region runs.

    NVML is polled from a background thread as fast as it answers (a timed region of a few
    milliseconds still gets samples); if NVML is not importable, `nvidia-smi -lms` is used."""
    REASONS = (("hw_slowdown", 0x8), ("sw_power_cap", 0x4), ("sw_thermal_slowdown", 0x20),
               ("hw_thermal_slowdown", 0x40))

    def __init__(self, index: int):
        self.index, self.sm, self.mx, self.reasons = index, [], None, set()
        self.stop = threading.Event()
        self.thread = None
        self.proc = None

    def _poll_nvml(self):
        import pynvml
        pynvml.nvmlInit()
        try:
            # the visible device order may differ from NVML's: map through the PCI bus id
            bus = torch.cuda.get_device_properties(self.index).pci_bus_id if hasattr(
                torch.cuda.get_device_properties(self.index), "pci_bus_id") else None
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            if bus is not None:
                for i in range(pynvml.nvmlDeviceGetCount()):
                    hi = pynvml.nvmlDeviceGetHandleByIndex(i)
                    if pynvml.nvmlDeviceGetPciInfo(hi).bus == bus:
                        h = hi
                        break
            self.mx = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while True:
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                bits = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                for name, bit in self.REASONS:
                    if bits & bit:
                        self.reasons.add(name)
                if self.stop.is_set():
                    break
                time.sleep(0.001)
        finally:
            pynvml.nvmlShutdown()

    def _poll_smi(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.sw_power_cap,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.hw_thermal_slowdown")
        self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}",
                                      "--format=csv,noheader,nounits", "-lms", "50"],
                                     stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        for line in self.proc.stdout:
            c = [x.strip() for x in line.split(",")]
            try:
                self.sm.append(float(c[0])); self.mx = float(c[1])
                for (name, _), v in zip(self.REASONS, c[2:6]):
                    if v.lower().startswith("active"):
                        self.reasons.add(name)
            except Exception:
                pass

    def _run(self):
        try:
            self._poll_nvml()
        except Exception:
            try:
                self._poll_smi()
            except Exception:
                pass

    def __enter__(self):
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        if self.proc:
            self.proc.terminate()
        self.thread.join(timeout=5)

    def summary(self):
        if not self.sm:
            return None
        return {"sm_mhz": statistics.median(self.sm), "sm_max_mhz": self.mx, "reasons": sorted(self.reasons),
                "samples": len(self.sm)}


def dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def barrier_and_sync(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x: float, world: int) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device="cuda" if torch.cuda.is_available() else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


WORKLOADS = {
    # name: (M, N, K, fp8 fraction, kind)
    "llama2-7b-fc1-decode": (16, 11008, 4096, 0.10, "decode"),
    "llama2-70b-fc1-decode": (16, 28672, 8192, 0.10, "decode"),
    "llama2-7b-qkvo-prefill": (4096, 4096, 4096, 0.10, "prefill"),
    "llama2-7b-fc1-prefill": (4096, 11008, 4096, 0.10, "prefill"),
    "llama2-7b-fc2-prefill": (4096, 4096, 11008, 0.10, "prefill"),
    # Section 5.1's other model sizes: Llama-2-13B (config 4: M = 2048) and Llama-2-70B (config 5)
    "llama2-13b-fc1-prefill": (2048, 13824, 5120, 0.10, "prefill"),
    "llama2-13b-fc2-prefill": (2048, 5120, 13824, 0.10, "prefill"),
    "llama2-70b-fc1-prefill": (8192, 28672, 8192, 0.10, "prefill"),
    "llama2-70b-fc2-decode": (16, 8192, 28672, 0.10, "decode"),
    "llama2-13b-fc1-decode": (16, 13824, 5120, 0.10, "decode"),
    # the other families Section 5.1 names (hidden / feed-forward widths of the models' public descriptions)
    "gpt3-1.3b-fc1-decode": (16, 8192, 2048, 0.10, "decode"),
    "gpt3-8.3b-fc1-decode": (16, 12288, 3072, 0.10, "decode"),
    "gpt3-8.3b-fc1-prefill": (2048, 12288, 3072, 0.10, "prefill"),
    "gpt3-22b-fc1-decode": (16, 24576, 6144, 0.10, "decode"),
    "nemotron4-15b-fc1-decode": (16, 24576, 6144, 0.10, "decode"),
    "nemotron4-15b-fc2-decode": (16, 6144, 24576, 0.10, "decode"),
    "nemotron4-15b-fc1-prefill": (4096, 24576, 6144, 0.10, "prefill"),
    "tiny": (64, 256, 256, 0.10, "decode"),
}


class Workload:
    """Device-resident inputs of one workload: packed weight copies (packed offline, timed), the step's
    activations, threshold, workspace and output."""

    def __init__(self, fg, dev, name, m_override=0, fp8=None):
        self.fg, self.dev, self.name = fg, dev, name
        M, N, K, p, kind = WORKLOADS[name]
        if m_override:
            M = m_override
        if fp8 is not None:
            p = fp8
        self.M, self.N, self.K, self.p, self.kind = M, N, K, p, kind
        self.wl = gi.llama(name, M, N, K, p, seed=0) if name != "tiny" else gi.tiny(0)
        x_cpu, w_cpu = self.wl.x(), self.wl.w()
        self.x_cpu = x_cpu
        self.fx, fw = self.wl.fx().to(dev), self.wl.fw().to(dev)
        self.s4 = gi.tensor_scale(x_cpu)
        self.wbytes = algorithmic_weight_bytes(N, K, p)
        # enough distinct weight copies that the weights alone exceed L2
        n_copies = max(2, int(np.ceil(1.5 * L2_BYTES / self.wbytes))) if kind == "decode" else 2
        self.n_copies = min(n_copies, 16)
        w_dev = w_cpu.to(dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        self.packed_w, self.pack_ms = [], []
        for _ in range(self.n_copies):
            ev[0].record()
            self.packed_w.append(fg.quantize_weights(w_dev, fw, clip_mode=fg.CLIP_SW_BRUTE, fp8_fraction=p))
            ev[1].record()
            torch.cuda.synchronize()
            self.pack_ms.append(ev[0].elapsed_time(ev[1]))
        del w_dev, fw
        self.x_dev = x_cpu.to(dev)
        # offline: activation threshold for the target fraction (Eq. 9 on this batch)
        self.tau = float(fg.calibrate_tau(self.x_dev, self.fx, scale_fp4=self.s4, fp8_fraction=p).item())
        self.acts_buf = fg.binding._alloc_aligned(fg.acts_bytes(M, K), dev)
        self.ws = fg.alloc_workspace(fg.binding.OP_LINEAR_FUSED, M, N, K, dev)
        self.y = torch.empty(M, N, dtype=torch.float32, device=dev)
        self.n_x = 4
        self.xs = [self.x_dev] + [self.x_dev.clone() for _ in range(self.n_x - 1)]
        self.flops = 2.0 * M * N * K
        self.alg_bytes = self.wbytes + algorithmic_act_bytes(M, K, p) + M * N * 4

    def step(self, i, x=None, y=None):
        """One pass of the online path: quantize the step's activations and multiply them with the packed
        weights.  Decode-sized batches: one launch (fgmp_linear_fused); else the two calls."""
        fg = self.fg
        x = self.xs[i % self.n_x] if x is None else x
        y = self.y if y is None else y
        if self.kind == "decode":
            fg.linear_fused(x, self.fx, self.packed_w[i % self.n_copies], scale_fp4=self.s4, tau=self.tau, out=y, workspace=self.ws)
        else:
            pa = fg.quantize_activations(x, self.fx, scale_fp4=self.s4, tau=self.tau, out=self.acts_buf)
            fg.linear(pa, self.packed_w[i % self.n_copies], out=y, workspace=self.ws)

    @property
    def units_per_step(self):
        return self.wbytes / 1e9 if self.kind == "decode" else self.flops / 1e12

    @property
    def metric_unit(self):
        return (("FGMP linear weight GB/s (decode)", "GB/s") if self.kind == "decode"
                else ("FGMP linear TFLOP/s (prefill)", "TFLOP/s"))


def capture(fn, steps, use_graph=True):
    """The K steps as one CUDA graph (None if capture is off or fails)."""
    if not use_graph:
        return None, "eager launches"
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(steps):
                    fn(i)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g.replay()                                      # untimed: uploads the graph
        torch.cuda.synchronize()
        return g, f"one CUDA graph of {steps} steps"
    except Exception as e:      # capture is an optimisation of the launch path, not of the kernels
        torch.cuda.synchronize()
        return None, f"eager launches (graph capture failed: {type(e).__name__})"


def timed_runs(fn, graph, steps, replays, world):
    """`replays` timings of exactly `steps` steps each (CUDA events on the launch stream, barrier and
    synchronize on both sides, max over ranks): milliseconds per run."""
    out = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(replays):
        barrier_and_sync(world)
        e0.record()
        if graph is not None:
            graph.replay()
        else:
            for i in range(steps):
                fn(i)
        e1.record()
        barrier_and_sync(world)
        out.append(max_over_ranks(e0.elapsed_time(e1), world))
    return out


def kernel_pass(fg, wk, steps, world):
    """The same steps launched eagerly with CUDA events around every launch of the library's kernels (recorded
    by the library on the launch stream): launch counts and per-kernel durations."""
    timed = ("expand_acts", "expand_weights", "gemm_bf16_tcgen05", "gemm_nvfp4_tcgen05", "decode_gemm", "quant_act")
    timed = tuple(k for k in timed if k in fg.kernel_names())
    fg.profile_begin(timed)
    for i in range(steps):
        wk.step(i)
    barrier_and_sync(world)
    prof = fg.profile_end()
    fg.check(wk.ws)
    return prof


def roofline_of(fg, wk, prof, step_ms, dev, peaks):
    """Roofline of the dominant kernel.  Decode: the step is one launch of the weight-streaming kernel, so its
    average duration over the timed region is the step time itself.  Prefill: per-launch events."""
    if wk.kind == "decode":
        avg_s = step_ms / 1e3
        ach = wk.alg_bytes / avg_s / 1e9
        ev_us = None
        if "decode_gemm" in prof and prof["decode_gemm"][1]:
            ev_us = prof["decode_gemm"][1] / prof["decode_gemm"][0] * 1e3
        return {"kernel": "decode_gemm", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": traffic_bytes("decode_gemm", wk.name),
                "traffic_from_profile": load_traffic("decode_gemm", wk.name),
                "peak_source": peaks["source"], "avg_kernel_us": avg_s * 1e6,
                "avg_kernel_us_note": "timed region / launches: the step is one launch of this kernel (activation quantizer inside)",
                "eager_event_timed_kernel_us": ev_us,
                "algorithmic_bytes_per_launch": wk.alg_bytes}
    dom = max(((k, v) for k, v in prof.items() if v[1] > 0 and k.startswith("gemm")), key=lambda kv: kv[1][1], default=None)
    if dom is None:
        return None
    name, (n_l, tot_ms) = dom
    avg_s = tot_ms / n_l / 1e3
    ach = wk.flops / avg_s / 1e12
    # the roofline of the mix: FP4 x FP4 pairs at the NVFP4 rate, every other pair at the FP8 rate (rates
    # measured here with MMA-only loops); beside it the bf16 reading of the container path
    f4 = (1 - wk.p) * (1 - wk.p)
    tp = tensor_peaks(fg, dev)
    p4, p8 = tp["nvfp4"], tp["e4m3"]
    blended_s = wk.flops * (f4 / p4 + (1 - f4) / p8) / 1e12
    blended_peak = wk.flops / blended_s / 1e12
    return {"kernel": name, "bound": "tensor", "achieved": ach, "peak": blended_peak, "unit": "TFLOP/s",
            "frac": ach / blended_peak, "traffic": traffic_bytes(name, wk.name), "traffic_from_profile": load_traffic(name, wk.name),
            "peak_source": "blend of the NVFP4 and E4M3 tcgen05 rates measured in this run for this FP8 fraction",
            "avg_kernel_us": avg_s * 1e6,
            "frac_of_fp8_roofline": (wk.flops / p8 / 1e12) / avg_s,
            "frac_of_measured_bf16_sustained": ach / peaks["bf16_tflops_sustained"],
            "tensor_peaks_tflops": tp}


def side_measurement(fg, dev, name, steps, replays, world, peaks, use_graph, fp8=None, m=0):
    """A shorter measurement of another workload for the same JSON line."""
    wk = Workload(fg, dev, name, m, fp8=fp8)
    for i in range(3):
        wk.step(i)
    fg.check(wk.ws)
    g, note = capture(wk.step, steps, use_graph)
    runs = timed_runs(wk.step, g, steps, replays, world)
    fg.check(wk.ws)
    ms = statistics.median(runs)
    prof = kernel_pass(fg, wk, steps, world)
    metric, unit = wk.metric_unit
    out = {"workload": name, "M": wk.M, "N": wk.N, "K": wk.K, "fp8_fraction": wk.p, "metric": metric, "unit": unit,
           "value": world * wk.units_per_step * steps / (ms / 1e3), "step_us": ms / steps * 1e3,
           "steps": steps, "replays": replays, "launch": note,
           "kernels": {k: {"launches": v[0], "avg_us": (v[1] / v[0] * 1e3 if v[1] else None)} for k, v in prof.items()},
           "roofline": roofline_of(fg, wk, prof, ms / steps, dev, peaks)}
    del wk
    torch.cuda.empty_cache()
    return out


def run_ours(args, world, rank, local):
    import paper_2504_14152_b200 as fg
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = measured_peaks()
    wk = Workload(fg, dev, args.workload, args.m, args.fp8)
    M, N, K, p, kind = wk.M, wk.N, wk.K, wk.p, wk.kind
    use_graph = not args.no_graph

    for i in range(max(args.warmup, 3)):
        wk.step(i)
    fg.check(wk.ws)

    # ---- the timed region: exactly K steps, replayed from one CUDA graph when capture works (a decode step is
    # one short kernel: launched from Python it would be the launch that is timed).  The K steps are timed
    # `replays` times; the reported time is the median run.
    graph, graph_note = capture(wk.step, args.steps, use_graph)
    with ClockSampler(local) as clk:
        runs = timed_runs(wk.step, graph, args.steps, args.replays, world)
    fg.check(wk.ws)
    ms = statistics.median(runs)
    clocks = clk.summary()
    prof = kernel_pass(fg, wk, args.steps, world)

    # ---- end to end: host buffers, H2D of the step's activations and D2H of its result inside.  Every step copies
    # its input from pinned host memory and its output back; the copies of neighbouring steps overlap the kernels
    # (two buffers each, copy streams beside the compute stream), as a serving loop would run it.  The strictly
    # serial order (copy in, compute, copy out, next step) is reported beside it.
    x_host = wk.x_cpu.pin_memory()
    e2e = {}
    for tag, dt in (("fp32", torch.float32), ("bf16", torch.bfloat16)):
        nb = 2
        x_in = [torch.empty_like(wk.x_dev) for _ in range(nb)]
        y_dev = [torch.empty(M, N, dtype=dt, device=dev) for _ in range(nb)]
        y_host = [torch.empty(M, N, dtype=dt).pin_memory() for _ in range(nb)]
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        def run_pipelined(K):
            cur = torch.cuda.current_stream()
            s_in.wait_stream(cur)
            s_out.wait_stream(cur)
            ev_c, ev_out = [None] * nb, [None] * nb
            for i in range(K):
                b = i % nb
                with torch.cuda.stream(s_in):
                    if ev_c[b] is not None:
                        s_in.wait_event(ev_c[b])            # the step that read this input buffer is done
                    x_in[b].copy_(x_host, non_blocking=True)
                    ev_in = torch.cuda.Event()
                    ev_in.record(s_in)
                cur.wait_event(ev_in)
                if ev_out[b] is not None:
                    cur.wait_event(ev_out[b])               # this output buffer has been copied out
                wk.step(i, x=x_in[b], y=y_dev[b])
                ev_c[b] = torch.cuda.Event()
                ev_c[b].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_c[b])
                    y_host[b].copy_(y_dev[b], non_blocking=True)
                    ev_out[b] = torch.cuda.Event()
                    ev_out[b].record(s_out)
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)

        def step_serial(i):
            x_in[0].copy_(x_host, non_blocking=True)
            wk.step(i, x=x_in[0], y=y_dev[0])
            y_host[0].copy_(y_dev[0], non_blocking=True)

        run_pipelined(4)
        torch.cuda.synchronize()
        n_rep = max(3, args.replays // 5)
        g2, note2 = capture(lambda i: run_pipelined(args.steps) if i == 0 else None, 1, use_graph)
        note2 = note2.replace("of 1 steps", f"of {args.steps} steps")
        r2 = timed_runs(lambda i: run_pipelined(args.steps) if i == 0 else None, g2, 1, n_rep, world)
        fg.check(wk.ws)
        g3, _ = capture(step_serial, args.steps, use_graph)
        r3 = timed_runs(step_serial, g3, args.steps, n_rep, world)
        fg.check(wk.ws)
        e2e[tag] = (statistics.median(r2), note2 + ", copies of neighbouring steps overlapped (2 buffers)",
                    M * N * (4 if dt == torch.float32 else 2), statistics.median(r3))
        del g2, g3

    metric, unit = wk.metric_unit
    per_step_units = wk.units_per_step
    value = world * per_step_units * args.steps / (ms / 1e3)
    e2e_ms, e2e_note, e2e_d2h, e2e_serial_ms = e2e["fp32"]
    launches = sum(v[0] for v in prof.values())
    out = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "nvfp4+fp8e4m3/f32acc", "data": "synthetic",
        "config": {"workload": args.workload, "M": M, "N": N, "K": K, "fp8_fraction_weights": p,
                   "fp8_fraction_activations": p, "score_mode": "lp_error(Eq.6)", "clip": "sw_brute(Eq.11)",
                   "l2": f"rotating {wk.n_copies} packed weight copies ({wk.n_copies * wk.wbytes / 1e6:.0f} MB > 126 MB L2)"
                   if kind == "decode" else "operands + bf16 planes exceed L2",
                   "step": ("fgmp_linear_fused: activation quantizer + GEMM in one launch" if kind == "decode"
                            else "quantize_activations + linear (online path)") + "; weight packing is offline",
                   "launch": graph_note,
                   "timing": f"median of {args.replays} runs of exactly {args.steps} steps (min {min(runs) / args.steps * 1e3:.2f}, "
                             f"max {max(runs) / args.steps * 1e3:.2f} us per step)"},
        "clocks": clocks,
        "e2e": {"value": world * per_step_units * args.steps / (e2e_ms / 1e3), "unit": unit,
                "h2d_bytes_per_step": wk.x_cpu.numel() * 2, "d2h_bytes_per_step": e2e_d2h,
                "ms_per_step": e2e_ms / args.steps, "launch": e2e_note,
                "serial": {"value": world * per_step_units * args.steps / (e2e_serial_ms / 1e3), "ms_per_step": e2e_serial_ms / args.steps,
                           "note": "copy in, compute, copy out, then the next step"},
                "bf16_output": {"value": world * per_step_units * args.steps / (e2e["bf16"][0] / 1e3),
                                "ms_per_step": e2e["bf16"][0] / args.steps, "d2h_bytes_per_step": e2e["bf16"][2]}},
        "gpu_launches": launches,
        "kernels": {k: {"launches": v[0], "avg_us": (v[1] / v[0] * 1e3 if v[1] else None)} for k, v in prof.items()},
        "roofline": roofline_of(fg, wk, prof, ms / args.steps, dev, peaks),
        "offline": {"quantize_weights_ms": statistics.median(wk.pack_ms), "weights_shape": [N, K],
                    "packed_MB": fg.weights_bytes(N, K, int(p * N * K / 16 + 0.5) + 1) / 1e6,
                    "algorithmic_MB": wk.wbytes / 1e6},
    }
    wl = wk.wl
    del wk, graph
    torch.cuda.empty_cache()
    # ---- the other halves of the metric, measured the same way in the same run (shorter)
    if not args.no_extras and args.workload == "llama2-7b-fc1-decode" and not args.m:
        out["decode_70b"] = side_measurement(fg, dev, "llama2-70b-fc1-decode", 20, 11, world, peaks, use_graph)
        out["decode_70b_m1"] = side_measurement(fg, dev, "llama2-70b-fc1-decode", 20, 11, world, peaks, use_graph, m=1)
        out["prefill"] = side_measurement(fg, dev, "llama2-7b-fc1-prefill", 5, 7, world, peaks, use_graph)
    if args.sweep:
        # the FP8 fraction of both operands swept over the given points (config 4: 0 / 10 / 20 / 30 %), each point
        # measured like the side objects above: step time, kernel times and the roofline of the mix at that point
        out["sweep"] = [side_measurement(fg, dev, args.workload, 5, 7, world, peaks, use_graph, fp8=float(f))
                        for f in args.sweep.split(",")]
    if rank == 0 and not args.no_cpu_baseline and world >= 1:
        out["cpu_baseline"] = cpu_baseline(args, wl, p, kind, per_step_units, unit)
        out["cpu_baseline"]["single_thread"] = cpu_baseline_single_thread(args)
    return out


# DRAM bytes (read + write) per launch from the committed ncu captures (profiles/*.md).  An entry is
# removed when its kernel changes after the capture.
NCU_TRAFFIC = {
    ("llama2-7b-fc1-decode", "decode_gemm"): {"bytes": 29184000, "file": "profiles/decode_kernel_llama2-7b-fc1-decode.md"},
    ("llama2-13b-fc1-prefill", "gemm_nvfp4_tcgen05"): {"bytes": 109814016, "file": "profiles/gemm_nvfp4_kernel_llama2-13b-fc1-prefill.md"},
    ("llama2-7b-fc2-prefill", "gemm_bf16_tcgen05"): {"bytes": 536672512, "file": "profiles/gemm_bf16_pair_kernel_llama2-7b-fc2-prefill.md"},
}


def load_traffic(kernel: str, workload: str):
    return NCU_TRAFFIC.get((workload, kernel))


def traffic_bytes(kernel: str, workload: str):
    e = load_traffic(kernel, workload)
    return e["bytes"] if e else None


def cpu_baseline(args, wl, p, kind, per_step_units, unit, budget_s=20.0, max_steps=None):
    """The oracle, as it stands, on the host cores: the same online step (activation quantizer +
    fp64 GEMM over decoded operands), on a bounded sample of the workload."""
    import oracle
    x, w, fx, fw = wl.x(), wl.w(), wl.fx().numpy(), wl.fw().numpy()
    M, N, K = wl.M, wl.N, wl.K
    # bound the sample: a slice of the weight rows (and of the tokens at prefill)
    n_rows = min(N, 1024 if kind == "decode" else 256)
    m_rows = min(M, 16 if kind == "decode" else 64)
    s4 = gi.tensor_scale(x)
    xb = gi.bf16_bits(x)[:m_rows].copy()
    qw = oracle.quantize_weights(gi.bf16_bits(w)[:n_rows].copy(), fw[:n_rows].copy(), clip=False, fp8_fraction=p)
    scores = oracle.quantize_activations(xb, fx, s4, tau=np.inf).scores
    k = int(np.floor(p * scores.size + 0.5))
    srt = np.sort(scores)[::-1]
    tau = float(np.float32(0.5) * (srt[k - 1] + srt[k])) if 0 < k < scores.size else float("inf")
    frac = (n_rows / N) * (m_rows / M)
    t0 = time.perf_counter()
    steps = 0
    while True:
        qa = oracle.quantize_activations(xb, fx, s4, tau=tau)
        oracle.linear(qa, qw)
        steps += 1
        el = time.perf_counter() - t0
        if el > budget_s or (max_steps and steps >= max_steps):
            break
    sec_per_full_step = el / steps / frac
    return {"value": per_step_units / sec_per_full_step, "unit": unit, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{steps} steps of tokens[:{m_rows}] x weight rows[:{n_rows}] (fraction {frac:.4g} of one step, "
                      f"scaled linearly); weights pre-packed by the oracle without clip search (untimed)",
            "seconds_per_full_step": sec_per_full_step}


def cpu_baseline_single_thread(args):
    """The same oracle sample on one thread (a child process with OMP_NUM_THREADS=1, a few seconds)."""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        env.pop(k, None)
    cmd = [sys.executable, os.path.abspath(__file__), "--impl", "reference", "--workload", args.workload, "--steps", "1", "--warmup", "1"]
    if args.m:
        cmd += ["--m", str(args.m)]
    try:
        line = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600).stdout.strip().splitlines()[-1]
        d = json.loads(line)
        return {"value": d["value"], "unit": d["unit"], "cores": d["cpu_baseline"]["cores"], "sample": d["cpu_baseline"]["sample"]}
    except Exception as e:
        return {"unavailable": f"{type(e).__name__}"}


def run_reference(args, world, rank):
    """The CPU oracle as the reference arm (there is no reference implementation to install)."""
    if rank != 0:
        return None
    M, N, K, p, kind = WORKLOADS[args.workload]
    if args.m:
        M = args.m
    wl = gi.llama(args.workload, M, N, K, p, seed=0) if args.workload != "tiny" else gi.tiny(0)
    flops = 2.0 * M * N * K
    if kind == "decode":
        metric, unit, units = "FGMP linear weight GB/s (decode)", "GB/s", algorithmic_weight_bytes(N, K, p) / 1e9
    else:
        metric, unit, units = "FGMP linear TFLOP/s (prefill)", "TFLOP/s", flops / 1e12
    # warm-up (also builds the oracle) then K bounded-sample steps
    cpu_baseline(args, wl, p, kind, units, unit, budget_s=0.0, max_steps=max(1, min(args.warmup, 1)))
    cb = cpu_baseline(args, wl, p, kind, units, unit, budget_s=1e9, max_steps=max(1, args.steps))
    return {
        "impl": "reference", "metric": metric, "value": cb["value"], "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": cb["seconds_per_full_step"] * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64 accumulate over decoded nvfp4/e4m3 operands",
        "data": "synthetic",
        "config": {"workload": args.workload, "M": M, "N": N, "K": K, "fp8_fraction_weights": p,
                   "fp8_fraction_activations": p},
        "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": cb["value"], "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


_TENSOR_PEAKS = None


def tensor_peaks(fg, dev):
    """TFLOP/s of MMA-only tcgen05 loops (operands resident in shared memory) per operand kind, as single CTAs
    (M = 128, N = 256) and as CTA pairs (M = 256, N = 256): the higher of the two sustained figures (a run of
    about 0.2 s) is the rate the roofline uses."""
    global _TENSOR_PEAKS
    if _TENSOR_PEAKS is not None:
        return _TENSOR_PEAKS
    ws = fg.binding._alloc_aligned(1024, dev)
    ws.zero_()
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    out = {"method": "MMA-only tcgen05 loops, operands in shared memory: one CTA per SM (M128 N256) and CTA pairs (M256 N256)"}
    for kind, (nm, k) in enumerate((("bf16", 16), ("e4m3", 32), ("nvfp4", 64))):
        best = 0.0
        for pair in (0, 1):
            code = kind + 4 * pair
            try:
                fg.tensor_peak(code, 2000, ws)
            except Exception:
                continue
            for tag, n in (("burst", 100_000), ("sustained", 1_500_000)):
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record()
                fg.tensor_peak(code, n, ws)
                e1.record()
                torch.cuda.synchronize()
                ctas = sms if not pair else (sms // 2) * 2
                tf = 2.0 * 128 * 256 * k * n * ctas / (e0.elapsed_time(e1) * 1e-3) / 1e12
                out[f"{nm}_{'pair_' if pair else ''}{tag}"] = tf
                if tag == "sustained":
                    best = max(best, tf)
        out[nm] = best
    fg.check(ws)
    _TENSOR_PEAKS = out
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b-fc1-decode", choices=sorted(WORKLOADS))
    ap.add_argument("--m", type=int, default=0, help="override the token count M")
    ap.add_argument("--sweep", default="", help="comma-separated FP8 fractions: adds a measurement of the workload at each (e.g. 0,0.1,0.2,0.3)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the timed steps eagerly")
    ap.add_argument("--replays", type=int, default=25, help="how often the K steps are timed (the median run is reported)")
    ap.add_argument("--fp8", type=float, default=None, help="override the FP8 fraction of weights and activations")
    ap.add_argument("--no-extras", action="store_true", help="skip the decode_70b and prefill objects of the default run")
    args = ap.parse_args()

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        if rank != 0:
            return 0
        if args.steps == 100:
            args.steps = 3
        out = run_reference(args, int(os.environ.get("WORLD_SIZE", "1")), rank)
        print(json.dumps(out))
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the FGMP kernels have no CPU fallback")
    world, rank, local = dist_setup(args.gpus)
    out = run_ours(args, world, rank, local)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
