#!/usr/bin/env python
"""Benchmark of the fused-linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path: the five benchmark configurations, one call
each, back to back on one stream (tiled fused linear, SwiGLU, linear + logsumexp,
split-K skinny linear).  The metric is TFLOP/s (algorithmic FLOPs of all calls / device
time); per-configuration times, TFLOP/s or GB/s and roofline fractions ride along in
the same JSON line.  Inputs are seeded synthetic tensors resident in HBM; a step touches
about 1 GB of distinct operands, far more than the 126 MB L2, so every call starts
L2-cold.  With N > 1 (torchrun) every rank runs an independent replica of the same
step on its own GPU -- the path does not shard and there is no data-path collective.

`--impl reference` times the fp64 CPU oracle (as it stands, never tuned) on the host
cores on a bounded row-sample of the same five configurations.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2511_20100_b200 import inputs

ORDER = ["C1", "C2", "C3", "C4", "C5"]
# rows of X the CPU reference arm computes per step and per configuration (bounded sample: about a second per step)
REF_ROWS = {"C1": 256, "C2": 64, "C3": 32, "C4": 32, "C5": 16}
# rows for the cpu_baseline leg of our own arm, run once: C1, C2 and C5 in full, C3 and C4 on a row sample
# (about 15 s of CPU work on 16 cores); --full-cpu-baseline runs all five in full (about two minutes)
CPU_BASELINE_ROWS = {"C1": 256, "C2": 4096, "C3": 512, "C4": 512, "C5": 16}


def flops(c) -> float:
    f = 2.0 * c["M"] * c["N"] * c["K"]
    return 2.0 * f if c["op"] == "swiglu" else f


def algorithmic_bytes(c) -> float:
    """Each operand read once, each output written once."""
    M, N, K = c["M"], c["N"], c["K"]
    if c["op"] == "swiglu":
        return 2.0 * (M * K + 2 * N * K) + 2.0 * M * N
    if c["op"] == "fused_linear_fp8":
        return 1.0 * (M * K + N * K) + 4.0 * N + 2.0 * M * N
    if c["op"] == "fused_linear_mxfp8":
        return (1.0 + 1.0 / 32) * (M * K + N * K) + 4.0 * N + 2.0 * M * N
    if c["op"] in ("linear_lse", "linear_rowmax", "linear_cross_entropy"):
        extra = {"linear_lse": 0.0, "linear_rowmax": 4.0 * M, "linear_cross_entropy": 8.0 * M}[c["op"]]
        return 2.0 * (M * K + N * K) + 4.0 * N + 4.0 * M + extra
    out_b = 2.0 if c["out_dtype"] == "bf16" else 4.0
    if c["op"] == "linear_softmax":         # the probabilities are written, read back and written again by the finishing pass
        return 2.0 * (M * K + N * K) + 4.0 * N + 3.0 * out_b * M * N
    res = out_b * M * N if c["op"] == "fused_linear_residual" else 0.0
    return 2.0 * (M * K + N * K) + 4.0 * N + out_b * M * N + res


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            p = json.load(open(path))
            return {"hbm_gbs": float(p["hbm_gbs"]), "tflops_burst": float(p["bf16_tflops"]),
                    "tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def reduce_max(dist, value: float, device) -> float:
    """Max over ranks of a per-rank time (identity without a process group)."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# --------------------------------------------------------------------------------------- our arm
def make_device_problem(name, device):
    c = inputs.CONFIGS.get(name) or inputs.EXTRA_CONFIGS[name]
    if c["op"] == "fused_linear_fp8":
        fi = inputs.fp8_linear_inputs(c["M"], c["N"], c["K"], c["seed"])
        dev = [fi.X.to(device), fi.W.to(device), fi.b.to(device)]
        out = torch.empty((c["M"], c["N"]), dtype=torch.bfloat16, device=device)
        return {"name": name, "cfg": c, "host": [], "dev": dev, "out": out, "scales": (fi.scale_x, fi.scale_w)}
    if c["op"] == "fused_linear_mxfp8":
        mi = inputs.mx_linear_inputs(c["M"], c["N"], c["K"], c["seed"], spread=3)
        dev = [mi.X.to(device), mi.SX.to(device), mi.W.to(device), mi.SW.to(device), mi.b.to(device)]
        out = torch.empty((c["M"], c["N"]), dtype=torch.bfloat16, device=device)
        return {"name": name, "cfg": c, "host": [], "dev": dev, "out": out}
    if c["op"] == "swiglu":
        si = inputs.swiglu_inputs(c["M"], c["N"], c["K"], c["seed"])
        host = [si.X, si.Wg, si.Wu]
    else:
        li = inputs.linear_inputs(c["M"], c["N"], c["K"], c["seed"])
        host = [li.X, li.W, li.b]
    if c["op"] == "linear_cross_entropy":
        host.append(inputs.targets(c["M"], c["N"], c["seed"]))
    if c["op"] == "fused_linear_residual":
        host.append(inputs.residual(c["M"], c["N"], c["seed"]))
    dev = [t.to(device) for t in host]
    if c["op"] in ("linear_lse", "linear_rowmax", "linear_cross_entropy"):
        out = torch.empty((c["M"],), dtype=torch.float32, device=device)
    else:
        odt = torch.bfloat16 if c.get("out_dtype", "bf16") == "bf16" else torch.float32
        out = torch.empty((c["M"], c["N"]), dtype=odt, device=device)
    return {"name": name, "cfg": c, "host": host, "dev": dev, "out": out}


def call_device(B, pr):
    c, d = pr["cfg"], pr["dev"]
    if c["op"] == "swiglu":
        B.mtmc_swiglu(d[0], d[1], d[2], out=pr["out"])
    elif c["op"] == "linear_lse":
        B.mtmc_linear_lse(d[0], d[1], d[2], lse_out=pr["out"])
    elif c["op"] == "linear_rowmax":
        B.mtmc_linear_rowmax(d[0], d[1], d[2], max_out=pr["out"], want_argmax=False)
    elif c["op"] == "linear_cross_entropy":
        B.mtmc_linear_cross_entropy(d[0], d[1], d[2], d[3], loss_out=pr["out"])
    elif c["op"] == "linear_softmax":
        B.mtmc_linear_softmax(d[0], d[1], d[2], c["out_dtype"], prob_out=pr["out"])
    elif c["op"] == "fused_linear_residual":
        B.mtmc_fused_linear_residual(d[0], d[1], d[2], d[3], c["act"], c["out_dtype"], out=pr["out"])
    elif c["op"] == "fused_linear_fp8":
        B.mtmc_fused_linear_fp8(d[0], d[1], d[2], pr["scales"][0], pr["scales"][1], c["act"], c["out_dtype"], out=pr["out"])
    elif c["op"] == "fused_linear_mxfp8":
        B.mtmc_fused_linear_mxfp8(d[0], d[1], d[2], d[3], d[4], c["act"], c["out_dtype"], out=pr["out"])
    else:
        B.mtmc_fused_linear(d[0], d[1], d[2], c["act"], c["out_dtype"], out=pr["out"])


def call_host(B, pr, pinned, dev_index, blocking=True):
    c = pr["cfg"]
    if c["op"] == "swiglu":
        B.mtmc_swiglu_host(pinned["in"][0], pinned["in"][1], pinned["in"][2], out=pinned["out"], device=dev_index, blocking=blocking)
    elif c["op"] == "linear_lse":
        B.mtmc_linear_lse_host(pinned["in"][0], pinned["in"][1], pinned["in"][2], lse_out=pinned["out"], device=dev_index,
                               blocking=blocking)
    else:
        B.mtmc_fused_linear_host(pinned["in"][0], pinned["in"][1], pinned["in"][2], c["act"], c["out_dtype"],
                                 out=pinned["out"], device=dev_index, blocking=blocking)


def eager_call(pr, dev):
    """The unfused PyTorch-eager sequence of the same operator (context only: it rounds the GEMM
    result to bf16 before the epilogue, and it is not on the product path)."""
    c = pr["cfg"]
    if c["op"] == "swiglu":
        return torch.nn.functional.silu(dev[0] @ dev[1].T) * (dev[0] @ dev[2].T)
    if c["op"] == "linear_lse":
        return torch.logsumexp((dev[0] @ dev[1].T).float() + dev[2], dim=-1)
    if c["op"] == "linear_rowmax":
        return ((dev[0] @ dev[1].T).float() + dev[2]).max(dim=-1).values
    if c["op"] == "linear_cross_entropy":
        return torch.nn.functional.cross_entropy((dev[0] @ dev[1].T).float() + dev[2], dev[3], reduction="none")
    z = (dev[0] @ dev[1].T).float() + dev[2]
    if c["op"] == "linear_softmax":
        return torch.softmax(z, dim=-1).to(torch.bfloat16)
    if c["op"] == "fused_linear_residual":
        return (z + dev[3].float()).to(torch.bfloat16)
    z = torch.relu(z) if c["act"] == "relu" else torch.nn.functional.gelu(z, approximate="tanh")
    return z if c["out_dtype"] == "fp32" else z.to(torch.bfloat16)


def cpu_baseline_sample(rows_by_cfg):
    """The oracle, as it stands, timed on the first rows_by_cfg[c] rows of X of every configuration.  Returns the
    TFLOP/s of one step (all five configurations) with the time of a sampled configuration scaled to all its rows,
    the thread count, the names of the scaled configurations and the per-configuration seconds (scaled)."""
    from oracle import ref
    step_s, scaled, secs = 0.0, [], {}
    for name in ORDER:
        c = inputs.CONFIGS[name]
        t, _ = reference_step_one(ref, name, prepared_reference_inputs(name, rows_by_cfg))
        r = min(rows_by_cfg[name], c["M"])
        if r < c["M"]:
            scaled.append("%s %d/%d" % (name, r, c["M"]))
        secs[name] = t * c["M"] / r
        step_s += secs[name]
    fl = sum(flops(inputs.CONFIGS[n]) for n in ORDER)
    return fl / step_s / 1e12, ref.get_threads(), scaled, secs


_ref_cache = {}


def prepared_reference_inputs(name, rows_by_cfg=None):
    rows_by_cfg = rows_by_cfg or REF_ROWS
    key = (name, rows_by_cfg[name])
    if key not in _ref_cache:
        c = inputs.CONFIGS[name]
        r = min(rows_by_cfg[name], c["M"])
        if c["op"] == "swiglu":
            si = inputs.swiglu_inputs(c["M"], c["N"], c["K"], c["seed"])
            _ref_cache[key] = (inputs.bf16_bits(si.X[:r].contiguous()), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu))
        else:
            li = inputs.linear_inputs(c["M"], c["N"], c["K"], c["seed"])
            _ref_cache[key] = (inputs.bf16_bits(li.X[:r].contiguous()), inputs.bf16_bits(li.W), inputs.f32(li.b))
    return _ref_cache[key]


def reference_step_one(ref, name, arrs):
    c = inputs.CONFIGS[name]
    r = arrs[0].shape[0]
    t0 = time.perf_counter()
    if c["op"] == "swiglu":
        ref.swiglu(arrs[0], arrs[1], arrs[2])
    elif c["op"] == "linear_lse":
        ref.linear_lse(arrs[0], arrs[1], arrs[2])
    else:
        ref.fused_linear(arrs[0], arrs[1], arrs[2], {"none": 0, "relu": 1, "gelu_tanh": 2, "silu": 3}[c["act"]])
    dt = time.perf_counter() - t0
    return dt, flops(c) * r / c["M"]


def sample_description(rows_by_cfg=None):
    rows_by_cfg = rows_by_cfg or REF_ROWS
    return "first rows of X: " + ", ".join("%s %d/%d" % (n, min(rows_by_cfg[n], inputs.CONFIGS[n]["M"]),
                                                          inputs.CONFIGS[n]["M"]) for n in ORDER)


def run_ours(args, rank, world, local_rank):
    from paper_2511_20100_b200 import binding as B   # raises if the CUDA library is missing: no fallback
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)
    B.load()
    # W, Wg, Wu are the weights of a layer: created once below and never written again, which is what this switch promises
    B.mtmc_set_static_weights(True)
    if args.cta_pair:
        B.mtmc_set_tuning(cta_pair=args.cta_pair)
    problems = [make_device_problem(n, device) for n in ORDER]
    peaks = measured_peaks()

    def step():
        for pr in problems:
            call_device(B, pr)

    for _ in range(max(args.warmup, 3)):
        step()
    B.mtmc_check_status()
    torch.cuda.synchronize()

    # ---- timed region: K steps back to back, events at the step boundaries only
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = B.mtmc_launch_count()
    ev[0].record()
    for k in range(args.steps):
        step()
        ev[k + 1].record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    launches = B.mtmc_launch_count() - launches0
    B.mtmc_check_status()
    total_ms = reduce_max(dist, ev[0].elapsed_time(ev[args.steps]), device)
    ms_per_step = total_ms / args.steps

    # ---- per configuration: the same call back to back, rotating over enough copies of the
    # operands that their total exceeds twice the L2 (so every launch reads its operands from HBM);
    # one event pair around the loop, so launch overhead is amortised as it is inside a step.
    #   burst     : 8 launches right after `settle_s` of idle (boost clocks, before the power cap bites) -> compared
    #               with the measured burst peak
    #   sustained : tensor-bound configurations run back to back for `sustain_s` seconds -> compared with the measured
    #               sustained peak; the short ones (C1, C5) loop for `loop_ms`
    L2_BYTES = 126e6
    per_cfg_ms, per_cfg_reps, per_cfg_copies, per_cfg_eager, per_cfg_burst, per_cfg_warm = {}, {}, {}, {}, {}, {}
    per_cfg_kernel, per_cfg_enqueue = {}, {}
    extras = [make_device_problem(n, device) for n in inputs.EXTRA_CONFIGS] if (args.extras and ORDER == list(inputs.CONFIGS)) else []
    for pr in problems + extras:
        n, c = pr["name"], pr["cfg"]
        tensor_bound = c["M"] > 128 and n != "C1"
        nbytes = sum(t.numel() * t.element_size() for t in pr["dev"] if t is not None)
        copies = 1 if n == "C1" else max(1, min(4, int(-(-2 * L2_BYTES // nbytes))))
        variants = [pr] + [dict(pr, dev=[None if t is None else t.clone() for t in pr["dev"]]) for _ in range(copies - 1)]
        for v in variants:
            call_device(B, v)
        per_cfg_kernel[n] = B.mtmc_last_kernel_name()       # the library's own account of what it launched
        torch.cuda.synchronize()
        time.sleep(args.settle_s)      # let the power/clock state left by the previous loop settle: each loop describes its own kernel
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for r in range(8):
            call_device(B, variants[r % copies])
        e1.record()
        torch.cuda.synchronize()
        per_cfg_burst[n] = e0.elapsed_time(e1) / 8
        est = max(per_cfg_burst[n], 1e-3)
        target_ms = args.sustain_s * 1e3 if tensor_bound else args.loop_ms
        reps = int(max(10, min(20000, target_ms / est)))
        e0.record()
        for r in range(reps):
            call_device(B, variants[r % copies])
        e1.record()
        torch.cuda.synchronize()
        per_cfg_ms[n] = e0.elapsed_time(e1) / reps
        per_cfg_reps[n], per_cfg_copies[n] = reps, copies
        if not tensor_bound:
            # launch-latency sized calls: host time to enqueue one call (argument checks, cached tensor maps, launch),
            # measured on an empty queue in batches short enough never to fill it
            t_host = 0.0
            for _ in range(5):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                for r in range(50):
                    call_device(B, variants[r % copies])
                t_host += time.perf_counter() - t0
            torch.cuda.synchronize()
            per_cfg_enqueue[n] = t_host / 250 * 1e6
        if c["M"] <= 128 and n != "C1" and copies > 1:
            # weight-streaming shapes: also the same call on ONE copy of the operands, i.e. with whatever part of W
            # the 126 MB L2 keeps from the launch before (labelled warm; the headline figure above is the cold one)
            e0.record()
            for r in range(reps):
                call_device(B, variants[0])
            e1.record()
            torch.cuda.synchronize()
            per_cfg_warm[n] = e0.elapsed_time(e1) / reps
        if not args.no_eager and c["op"] not in ("fused_linear_fp8", "fused_linear_mxfp8"):
            # context: the unfused torch sequence (cuBLAS GEMM + elementwise kernels), same rotation
            for v in variants:
                eager_call(pr, v["dev"])
            torch.cuda.synchronize()
            ereps = max(5, min(reps // 4, int(300.0 / est)))
            e0.record()
            for r in range(ereps):
                eager_call(pr, variants[r % copies]["dev"])
            e1.record()
            torch.cuda.synchronize()
            per_cfg_eager[n] = e0.elapsed_time(e1) / ereps
        del variants
    B.mtmc_check_status()
    clocks = sampler.stop()
    step_flops = sum(flops(inputs.CONFIGS.get(n) or inputs.EXTRA_CONFIGS[n]) for n in ORDER)
    value = world * step_flops / (ms_per_step * 1e-3) / 1e12

    # DRAM bytes per launch from the committed ncu summaries (a pointer to a capture, not something this run measured)
    traffic = {}
    prof = os.path.join(ROOT, "profiles", "traffic.txt")
    if os.path.exists(prof):
        for ln in open(prof):
            tok = ln.split()
            if len(tok) == 2 and tok[0].endswith("_dram_bytes_per_launch"):
                traffic[tok[0].split("_")[0]] = int(tok[1])

    def describe(n, full):
        """Per-configuration entry; `full` adds the fields that only the detailed (stderr) record carries."""
        c = inputs.CONFIGS.get(n) or inputs.EXTRA_CONFIGS[n]
        ms = per_cfg_ms[n]
        tf, gb = flops(c) / (ms * 1e-3) / 1e12, algorithmic_bytes(c) / (ms * 1e-3) / 1e9
        e = {"ms": round(ms, 5), "kernel": per_cfg_kernel[n]}
        hbm_bound = n == "C5" or (n in inputs.EXTRA_CONFIGS and c["M"] <= 128)
        if n == "C1":
            e.update({"tflops": round(tf, 2), "bound": "launch latency"})
        elif hbm_bound:
            e.update({"gbs": round(gb, 1), "bound": "hbm", "frac": round(gb / peaks["hbm_gbs"], 4), "frac_of_8000": round(gb / 8000.0, 4)})
        else:
            scale = 2.0 if c["op"] in ("fused_linear_fp8", "fused_linear_mxfp8") else 1.0        # E4M3: measured bf16 peak x the nominal 2:1 ratio
            btf = flops(c) / (per_cfg_burst[n] * 1e-3) / 1e12
            e.update({"tflops": round(tf, 1), "bound": "tensor", "burst_ms": round(per_cfg_burst[n], 5),
                      "frac_burst": round(btf / (scale * peaks["tflops_burst"]), 4),
                      "frac_sustained": round(tf / (scale * peaks["tflops_sustained"]), 4),
                      "frac_of_nominal": round(tf / (scale * 2250.0), 4), "loop_s": round(ms * per_cfg_reps[n] * 1e-3, 2)})
        if n in per_cfg_enqueue:
            e["host_enqueue_us"] = round(per_cfg_enqueue[n], 2)
        if n in per_cfg_eager:
            e["eager_ms"] = round(per_cfg_eager[n], 5)
        if full:
            e.update({"call": c["op"], "M": c["M"], "N": c["N"], "K": c["K"], "launches_timed": per_cfg_reps[n],
                      "operand_copies_rotated": per_cfg_copies[n], "tflops": round(tf, 3), "gbs": round(gb, 2),
                      "algorithmic_bytes": int(algorithmic_bytes(c)), "flops": flops(c)})
            if n in per_cfg_warm:
                e["l2_warm_ms"] = round(per_cfg_warm[n], 5)
            if n in traffic:
                e["dram_bytes_per_launch_ncu"] = traffic[n]
        return e

    per_config = {n: describe(n, False) for n in ORDER}

    # dominant kernel of the step: the one with the longest launch (C3's SwiGLU kernel when all five run)
    dom_name = max(ORDER, key=lambda n: per_cfg_ms[n])
    dc = inputs.CONFIGS.get(dom_name) or inputs.EXTRA_CONFIGS[dom_name]
    if dom_name == "C5" or dc["M"] <= 128:
        gb = algorithmic_bytes(dc) / (per_cfg_ms[dom_name] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": round(gb, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": round(gb / peaks["hbm_gbs"], 4), "peak_source": peaks["source"] + " copy bandwidth"}
    else:
        # frac compares like with like: the kernel timed alone in a burst after idle against the burst peak; the
        # seconds-long loop against the sustained peak rides along
        btf = flops(dc) / (per_cfg_burst[dom_name] * 1e-3) / 1e12
        stf = flops(dc) / (per_cfg_ms[dom_name] * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": round(btf, 1), "peak": peaks["tflops_burst"], "unit": "TFLOP/s",
                    "frac": round(btf / peaks["tflops_burst"], 4),
                    "peak_source": peaks["source"] + " cuBLAS bf16 burst; 8 launches after %.1f s idle" % args.settle_s,
                    "sustained": {"achieved": round(stf, 1), "peak": peaks["tflops_sustained"],
                                  "frac": round(stf / peaks["tflops_sustained"], 4),
                                  "loop_s": round(per_cfg_ms[dom_name] * per_cfg_reps[dom_name] * 1e-3, 2)},
                    "frac_of_nominal_2250": round(stf / 2250.0, 4)}
    roofline["kernel"] = per_cfg_kernel[dom_name] + " on " + dom_name
    roofline["traffic"] = traffic.get(dom_name)
    roofline["traffic_source"] = "profiles/traffic.txt (ncu capture of one launch, not this run)"

    # ------------------------------------------------------------------ end to end through the host-pointer C ABI
    e2e = None
    if not args.no_e2e:
        pinned = []
        h2d = d2h = 0
        for pr in problems:
            ins = [None if t is None else t.pin_memory() for t in pr["host"]]
            out = torch.empty(pr["out"].shape, dtype=pr["out"].dtype).pin_memory()
            pinned.append({"in": ins, "out": out})
            h2d += sum(t.numel() * t.element_size() for t in ins if t is not None)
            d2h += out.numel() * out.element_size()
        for _ in range(3):                          # warm-up: three steps size the device copies of every pipeline slot
            for pr, pn in zip(problems, pinned):
                call_host(B, pr, pn, local_rank, blocking=False)
            B.mtmc_host_sync()
        e2e_steps = max(2, min(args.steps, 5))
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        # each step: the five calls issued without waiting, then one wait for all five results on the host -- the
        # library overlaps a call's copy in with the previous call's kernels and copy out (three streams)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            for pr, pn in zip(problems, pinned):
                call_host(B, pr, pn, local_rank, blocking=False)
            B.mtmc_host_sync()
        torch.cuda.synchronize()
        e2e_s = reduce_max(dist, time.perf_counter() - t0, device)
        # the same with every call waiting for its own result (no overlap between calls)
        t0 = time.perf_counter()
        for _ in range(2):
            for pr, pn in zip(problems, pinned):
                call_host(B, pr, pn, local_rank)
        torch.cuda.synchronize()
        blocking_s = reduce_max(dist, time.perf_counter() - t0, device) / 2
        e2e = {"value": round(world * step_flops * e2e_steps / e2e_s / 1e12, 3), "unit": "TFLOP/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
               "ms_per_step": round(e2e_s / e2e_steps * 1e3, 3),
               "ms_per_step_blocking_calls": round(blocking_s * 1e3, 3),
               "api": "mtmc_*_host_async x5 + mtmc_host_sync per step; pinned host buffers, copies inside the timed region"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rows = {n: inputs.CONFIGS[n]["M"] for n in ORDER} if args.full_cpu_baseline else CPU_BASELINE_ROWS
        v, cores, scaled, secs = cpu_baseline_sample(rows)
        cpu = {"value": round(v, 6), "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
               "sample": "full " + "+".join(n for n in ORDER if not any(x.startswith(n) for x in scaled)) +
                         ("; first rows of X, time scaled to all rows: " + ", ".join(scaled) if scaled else ""),
               "extrapolated": bool(scaled), "seconds": {n: round(t, 3) for n, t in secs.items()}}

    if rank == 0:
        if extras or args.details:
            detail = {"detail": "per-configuration record of the same run (not the bench line)",
                      "per_config": {n: describe(n, True) for n in ORDER + [e["name"] for e in extras]}}
            print(json.dumps(detail), file=sys.stderr, flush=True)
        line = {
            "metric": "TFLOP/s over one pass of the fused-linear hot path (C1-C5, one call each)",
            "value": round(value, 3), "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "+".join(ORDER), "l2": "inputs > L2: a step reads ~1 GB of distinct operands; per_config loops rotate operand copies > 2x L2",
                       "static_weights": 1, "parallelism": "replicas only" if world > 1 else "single GPU"},
            "per_config": per_config, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line, separators=(",", ":")), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------- reference arm
def run_reference(args, rank, world):
    if rank != 0:
        return
    from oracle import ref
    arrs = {n: prepared_reference_inputs(n) for n in ORDER}
    steps, warm = args.steps, max(args.warmup, 1)
    for _ in range(warm):
        for n in ORDER:
            reference_step_one(ref, n, arrs[n])
    t_total, fl_total = 0.0, 0.0
    for _ in range(steps):
        for n in ORDER:
            t, fl = reference_step_one(ref, n, arrs[n])
            t_total += t
            fl_total += fl
    value = fl_total / t_total / 1e12
    line = {
        "impl": "reference",
        "metric": "TFLOP/s over one pass of the fused-linear hot path (C1-C5, one call each)",
        "value": round(value, 6), "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warm,
        "ms_per_step": round(t_total / steps * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "C1+C2+C3+C4+C5", "sample": sample_description()},
        "cpu_baseline": {"value": round(value, 6), "unit": "TFLOP/s", "cores": ref.get_threads(), "kind": "oracle",
                         "sample": sample_description()},
        "e2e": {"value": round(value, 6), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    global ORDER
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--settle-s", type=float, default=0.5, help="idle time before each per-configuration loop")
    ap.add_argument("--loop-ms", type=float, default=150.0, help="target length of each per-configuration timing loop")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the timed CPU oracle leg")
    ap.add_argument("--sustain-s", type=float, default=2.0, help="length of the back-to-back loop of each tensor-bound configuration")
    ap.add_argument("--extras", action="store_true", help="also measure the further operators X1.. (detailed record on stderr)")
    ap.add_argument("--details", action="store_true", help="print the detailed per-configuration record on stderr")
    ap.add_argument("--full-cpu-baseline", action="store_true", help="time the oracle on all rows of every configuration (minutes)")
    ap.add_argument("--no-eager", action="store_true", help="skip the PyTorch-eager context timings")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-pointer end-to-end leg")
    ap.add_argument("--cta-pair", type=int, default=0, help="tuning hook for every call (profiling aid): 1 forces the 256 x 256 pair tiles, "
                    "2 the 512 x 256 pair tiles, -1 single-CTA tiles; 0 leaves the choice to the library")
    ap.add_argument("--configs", default=",".join(ORDER), help="comma-separated subset of C1..C5, or of the further operators X1.. (profiling aid)")
    args = ap.parse_args()
    ORDER = [c for c in args.configs.split(",") if c in inputs.CONFIGS or c in inputs.EXTRA_CONFIGS]
    if any(c in inputs.EXTRA_CONFIGS for c in ORDER):     # an operator beside the five (profiling aid): device-timed legs only
        args.no_e2e = args.no_cpu_baseline = True
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
