#!/usr/bin/env python
"""Benchmark of the FGMP linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Default workload: Llama-2-7B FC1 at decode (M=16 tokens, K=4096, N=11008, 10% FP8 blocks in
weights and activations); metric = packed-weight GB/s.  One step = the online path: quantize
the step's activations (bf16 -> mixed NVFP4/FP8) and run the mixed-precision GEMM against
offline-packed weights.  Weight packing is offline in the method and is timed separately
(reported under "offline").  The step rotates over several weight copies so that the working
set exceeds L2.  Prints ONE JSON line (rank 0).

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
    "tiny": (64, 256, 256, 0.10, "decode"),
}


def run_ours(args, world, rank, local):
    import paper_2504_14152_b200 as fg
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    M, N, K, p, kind = WORKLOADS[args.workload]
    if args.m:
        M = args.m
    wl = gi.llama(args.workload, M, N, K, p, seed=0) if args.workload != "tiny" else gi.tiny(0)
    x_cpu, w_cpu, fx, fw = wl.x(), wl.w(), wl.fx().to(dev), wl.fw().to(dev)
    s4 = gi.tensor_scale(x_cpu)
    wbytes = algorithmic_weight_bytes(N, K, p)
    # enough distinct weight copies that weights alone exceed L2
    n_copies = max(2, int(np.ceil(1.5 * L2_BYTES / wbytes))) if kind == "decode" else 2
    n_copies = min(n_copies, 16)

    # ---- offline: pack the weights (timed, reported separately)
    w_dev = w_cpu.to(dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    packed_w = []
    pw_ms = []
    for i in range(n_copies):
        ev[0].record()
        packed_w.append(fg.quantize_weights(w_dev, fw, clip_mode=fg.CLIP_SW_BRUTE, fp8_fraction=p))
        ev[1].record()
        torch.cuda.synchronize()
        pw_ms.append(ev[0].elapsed_time(ev[1]))
    # ---- offline: activation threshold for the target fraction (Eq. 9 on this batch)
    x_dev = x_cpu.to(dev)
    tau = float(fg.calibrate_tau(x_dev, fx, scale_fp4=s4, fp8_fraction=p).item())

    acts_buf = fg.binding._alloc_aligned(fg.acts_bytes(M, K), dev)
    ws = fg.alloc_workspace(fg.binding.OP_LINEAR, M, N, K, dev)
    y = torch.empty(M, N, dtype=torch.float32, device=dev)
    # distinct activation copies as well (small at decode, > L2 in total at prefill with the planes)
    n_x = 4
    xs = [x_dev] + [x_dev.clone() for _ in range(n_x - 1)]

    def step(i):
        pa = fg.quantize_activations(xs[i % n_x], fx, scale_fp4=s4, tau=tau, out=acts_buf)
        fg.linear(pa, packed_w[i % n_copies], out=y, workspace=ws)

    for i in range(max(args.warmup, 3)):
        step(i)
    fg.check(ws)

    # ---- the timed region: K steps, replayed from one CUDA graph when capture works (the step is
    # launch-bound at decode sizes: two short kernels), else launched eagerly
    graph, graph_note = None, "eager launches"
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for i in range(args.steps):
                        step(i)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph, graph_note = g, f"one CUDA graph of {args.steps} steps"
        except Exception as e:  # capture is an optimisation of the launch path, not of the kernels
            graph_note = f"eager launches (graph capture failed: {type(e).__name__})"
            torch.cuda.synchronize()
    if graph is not None:
        graph.replay()                                  # untimed: uploads the graph
    barrier_and_sync(world)
    with ClockSampler(local) as clk:
        ev[0].record()
        if graph is not None:
            graph.replay()
        else:
            for i in range(args.steps):
                step(i)
        ev[1].record()
        barrier_and_sync(world)
    ms = ev[0].elapsed_time(ev[1])
    fg.check(ws)
    ms = max_over_ranks(ms, world)
    clocks = clk.summary()

    # ---- the same K steps once more, launched eagerly with CUDA events around every launch of the
    # kernels below (recorded by the library on the launch stream): launch counts and kernel durations
    timed = ("expand_acts", "expand_weights", "gemm_bf16_tcgen05", "decode_gemm", "quant_act")
    fg.profile_begin(timed)
    for i in range(args.steps):
        step(i)
    barrier_and_sync(world)
    prof = fg.profile_end()
    fg.check(ws)

    # ---- end to end: host buffers, H2D of the step's activations and D2H of its result inside
    x_host = x_cpu.pin_memory()
    y_host = torch.empty(M, N, dtype=torch.float32).pin_memory()
    x_in = torch.empty_like(x_dev)

    def step_e2e(i):
        x_in.copy_(x_host, non_blocking=True)
        pa = fg.quantize_activations(x_in, fx, scale_fp4=s4, tau=tau, out=acts_buf)
        fg.linear(pa, packed_w[i % n_copies], out=y, workspace=ws)
        y_host.copy_(y, non_blocking=True)

    for i in range(3):
        step_e2e(i)
    barrier_and_sync(world)
    # the same K end-to-end steps as one CUDA graph (copy nodes and kernels) when capture works: at decode
    # sizes four Python calls per step would otherwise be what is timed
    e2e_graph = None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                g2 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g2, stream=side):
                    for i in range(args.steps):
                        step_e2e(i)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g2.replay()                                 # untimed: uploads the graph
            e2e_graph = g2
        except Exception:
            torch.cuda.synchronize()
    barrier_and_sync(world)
    t0 = time.perf_counter()
    ev[0].record()
    if e2e_graph is not None:
        e2e_graph.replay()
    else:
        for i in range(args.steps):
            step_e2e(i)
    ev[1].record()
    barrier_and_sync(world)
    e2e_wall_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = max(ev[0].elapsed_time(ev[1]), 0.0)
    e2e_ms = max_over_ranks(max(e2e_ms, e2e_wall_ms if args.steps else 0.0), world)

    flops = 2.0 * M * N * K
    if kind == "decode":
        metric, unit = "FGMP linear weight GB/s (decode)", "GB/s"
        per_step_units = wbytes / 1e9
    else:
        metric, unit = "FGMP linear TFLOP/s (prefill)", "TFLOP/s"
        per_step_units = flops / 1e12
    value = world * per_step_units * args.steps / (ms / 1e3)
    e2e_value = world * per_step_units * args.steps / (e2e_ms / 1e3)

    peaks = measured_peaks()
    launches = sum(v[0] for v in prof.values())
    # dominant kernel = the timed kernel with the largest share
    dom = max(((k, v) for k, v in prof.items() if v[1] > 0), key=lambda kv: kv[1][1], default=None)
    roofline = None
    if dom:
        name, (n_l, tot_ms) = dom
        avg_s = tot_ms / n_l / 1e3
        if kind == "decode":
            alg = wbytes + algorithmic_act_bytes(M, K, p) + M * N * 4
            ach = alg / avg_s / 1e9
            roofline = {"kernel": name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / peaks["hbm_gbs"], "traffic": load_traffic(name, args.workload),
                        "peak_source": peaks["source"], "avg_kernel_us": avg_s * 1e6,
                        "algorithmic_bytes_per_launch": alg,
                        # the graph-timed step (quantizer + this kernel, overlapped where the launch allows)
                        # is shorter than the event-timed launch alone: the same bytes over the whole step
                        "step_us": ms / args.steps * 1e3,
                        "frac_over_step_time": alg / (ms / args.steps / 1e3) / 1e9 / peaks["hbm_gbs"]}
        else:
            ach = flops / avg_s / 1e12
            pk = peaks["bf16_tflops_sustained"]
            # other readings of the roofline for the same launch: the mix at the FP4/FP8 rates measured
            # here with an MMA-only loop, and FP8 only
            pa = pw = p
            f4 = (1 - pa) * (1 - pw)
            tp = tensor_peaks(fg, dev)
            p4, p8 = tp["nvfp4_sustained"], tp["e4m3_sustained"]
            blended_s = flops * (f4 / p4 + (1 - f4) / p8) / 1e12
            roofline = {"kernel": name, "bound": "tensor", "achieved": ach, "peak": pk, "unit": "TFLOP/s",
                        "frac": ach / pk, "traffic": load_traffic(name, args.workload),
                        "peak_source": peaks["source"] + " bf16 sustained (common-container path runs at the f16 rate)",
                        "avg_kernel_us": avg_s * 1e6,
                        "frac_of_blended_fp4_fp8_roofline": blended_s / avg_s,
                        "frac_of_fp8_roofline": (flops / p8 / 1e12) / avg_s,
                        "tensor_peaks_tflops": tp}
    out = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "nvfp4+fp8e4m3/f32acc", "data": "synthetic",
        "config": {"workload": args.workload, "M": M, "N": N, "K": K, "fp8_fraction_weights": p,
                   "fp8_fraction_activations": p, "score_mode": "lp_error(Eq.6)", "clip": "sw_brute(Eq.11)",
                   "l2": f"rotating {n_copies} packed weight copies ({n_copies * wbytes / 1e6:.0f} MB > 126 MB L2)"
                   if kind == "decode" else "operands + bf16 planes exceed L2",
                   "step": "quantize_activations + linear (online path); weight packing is offline",
                   "launch": graph_note,
                   "kernel_times": "second pass of the same steps, CUDA events around each launch"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": x_cpu.numel() * 2,
                "d2h_bytes_per_step": M * N * 4, "ms_per_step": e2e_ms / args.steps,
                "launch": "one CUDA graph (copies and kernels)" if e2e_graph is not None else "eager launches"},
        "gpu_launches": launches,
        "kernels": {k: {"launches": v[0], "avg_us": (v[1] / v[0] * 1e3 if v[1] else None)} for k, v in prof.items()},
        "roofline": roofline,
        "offline": {"quantize_weights_ms": statistics.median(pw_ms), "weights_shape": [N, K],
                    "packed_MB": fg.weights_bytes(N, K, int(p * N * K / 16 + 0.5) + 1) / 1e6,
                    "algorithmic_MB": wbytes / 1e6},
    }
    if rank == 0 and not args.no_cpu_baseline and world >= 1:
        out["cpu_baseline"] = cpu_baseline(args, wl, p, kind, per_step_units, unit)
    return out


# DRAM bytes (read + write) per launch from the committed ncu captures (profiles/*.md).  An entry is
# removed when its kernel changes after the capture.
NCU_TRAFFIC = {
    ("llama2-7b-fc1-decode", "decode_gemm"): 30531328,          # profiles/decode_kernel_llama2-7b-fc1-decode.md
    ("llama2-7b-fc2-prefill", "gemm_bf16_tcgen05"): 535152896,   # profiles/gemm_bf16_pair_kernel_llama2-7b-fc2-prefill.md
}


def load_traffic(kernel: str, workload: str):
    return NCU_TRAFFIC.get((workload, kernel))


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


def tensor_peaks(fg, dev):
    """TFLOP/s of an MMA-only tcgen05 loop (operands in shared memory, M = 128, N = 256, one CTA per SM)
    per operand kind: a burst of about 20 ms and a run of about 0.3 s."""
    ws = fg.binding._alloc_aligned(1024, dev)
    ws.zero_()
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    out = {"method": "MMA-only tcgen05 loop, M128 N256, operands in shared memory, one CTA per SM"}
    for kind, (nm, k) in enumerate((("bf16", 16), ("e4m3", 32), ("nvfp4", 64))):
        fg.tensor_peak(kind, 2000, ws)
        for tag, n in (("burst", 200_000), ("sustained", 3_000_000)):
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            fg.tensor_peak(kind, n, ws)
            e1.record()
            torch.cuda.synchronize()
            out[f"{nm}_{tag}"] = 2.0 * 128 * 256 * k * n * sms / (e0.elapsed_time(e1) * 1e-3) / 1e12
    fg.check(ws)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b-fc1-decode", choices=sorted(WORKLOADS))
    ap.add_argument("--m", type=int, default=0, help="override the token count M")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the timed steps eagerly")
    args = ap.parse_args()

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        if rank != 0:
            return 0
        if args.steps == 200:
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
