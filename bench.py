#!/usr/bin/env python
"""Benchmark of the budgeted MoE-layer forward (tokens/s and fraction of roofline on B200).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c1] [--budget-mult M]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

A step is one moe_layer_forward call (gate GEMM + softmax + Top-K, Alloc-T selection,
permutation, grouped SwiGLU expert GEMMs + shared experts, combine) over one batch of seeded
synthetic tokens.  The headline workload is the DeepSeek-V2-Lite-shaped decode layer (c2); on one
GPU the same line also carries the prefill layer (c3 at 3xT), the large-expert layer (c5) and the
26-layer stack (c4) under "workloads", each timed the same way.

Timing: W warm-up steps, then blocks of exactly K steps, each block bracketed by a barrier and a
device synchronisation and timed with CUDA events (max over ranks); blocks are repeated until at
least 5 have run and they add up to half a second, and the median block gives ms_per_step.
One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "budgeted MoE-layer tokens/s"
UNIT = "tokens/s"
MIN_BLOCKS = 5            # timed blocks per figure, at least
MIN_REGION_S = 0.5        # and at least this much timed work in total
MAX_BLOCKS = 400


def kernel_source_sha16():
    """Fingerprint of the expert-GEMM kernels' source: ncu counters are only quoted for the code they were taken on."""
    h = hashlib.sha256()
    for f in ("ffn.cu", "common.cuh"):
        with open(os.path.join(ROOT, "paper_2604_08133_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic_bytes(kernel, workload, budget):
    """dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of `kernel` on this workload, from the table of
    ncu captures kept with the profile summaries (tab-separated: kernel, workload, budget, bytes per launch, source
    fingerprint, commit, how it was taken).  None when there is no capture of the kernel source as it stands."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    if not os.path.exists(path):
        return None
    sha = kernel_source_sha16()
    with open(path) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            c = ln.rstrip("\n").split("\t")
            if len(c) >= 5 and kernel.startswith(c[0]) and c[1] == workload and int(c[2]) == int(budget) and c[4] == sha:
                return float(c[3])
    return None


GATHER_ROWS_PER_EXPERT = 32     # the library's default: up to this many rows per routed expert GEMM-1 reads x by index


def kernels_per_layer(cfg, budget):
    """Launches of one moe_layer_forward call: gate, routing (one fused launch up to 8192 tokens, else
    select + permute count/scan/place), row gather (none where the expert GEMM fetches the rows of x
    itself), 2 expert GEMMs, combine."""
    routing = 1 if cfg.T <= 8192 else 4
    gather = 0 if budget <= GATHER_ROWS_PER_EXPERT * cfg.N else 1
    return 1 + routing + gather + 2 + 1


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--budget-mult", type=float, default=None, help="budget as a multiple of T")
    ap.add_argument("--k-base", type=int, default=None, help="override K_base (the guaranteed experts per token)")
    ap.add_argument("--stack-budgets", default="dirichlet", choices=["dirichlet", "alloc-l"],
                    help="layer stack only: per-layer budgets from the seeded Dirichlet split, or from alloc_l_solve "
                         "on a seeded synthetic sensitivity matrix (same total)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the stage profile / full-Top-K / e2e passes")
    ap.add_argument("--no-workloads", action="store_true", help="headline workload only (no c3 / c5 / c4 entries)")
    ap.add_argument("--blocks", type=int, default=None,
                    help="time exactly this many blocks of --steps steps instead of repeating blocks to half a second "
                         "(short runs for a profiler; such a run's numbers are not benchmark figures)")
    ap.add_argument("--global-alloc-t", action="store_true",
                    help="also time the batch-wide Alloc-T path (gate, all-gather of the score rows, selection over "
                         "the whole pool, routed layer call); always on with more than one GPU")
    return ap.parse_args()


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def workload_cfg(args):
    from paper_2604_08133_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    if args.k_base is not None:
        cfg = cfg.with_(K_base=args.k_base)
    budget = cfg.budget if args.budget_mult is None else int(round(args.budget_mult * cfg.T))
    budget = max(budget, cfg.K_base * cfg.T)
    return cfg, budget


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, torch_device_index: int):
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def start(self):
        if self._h is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
        s = sorted(self.samples)
        med = s[len(s) // 2] if s else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s)}


# ------------------------------------------------------------------------------------------ CPU oracle arm
def oracle_sample(cfg, budget, target_tokens=None):
    """A bounded sample of the workload for the CPU oracle: the first Ts tokens of the batch with
    the budget scaled to them (the whole batch when it is small)."""
    Ts = cfg.T if target_tokens is None else min(cfg.T, target_tokens)
    b = int(round(budget * Ts / cfg.T))
    b = max(cfg.K_base * Ts, min(cfg.K_orig * Ts, b))
    return Ts, b


def time_oracle(cfg, budget, steps=1, warmup=0, target_tokens=None):
    import numpy as np
    import torch
    from oracle import alloc_moe_oracle as orc
    from paper_2604_08133_b200 import synth
    Ts, b = oracle_sample(cfg, budget, target_tokens)
    d = synth.make_layer(cfg)
    f = lambda t: None if t is None else t.float().numpy()
    x = f(d["x"])[:Ts]
    a = (x, f(d["W_gate"]), f(d["gate_bias"]), f(d["W13"]), f(d["W2"]), f(d["Wsh13"]), f(d["Wsh2"]),
         cfg.K_orig, cfg.K_base, b)
    for _ in range(warmup):
        orc.layer_forward(*a)
    t0 = time.perf_counter()
    for _ in range(steps):
        last = orc.layer_forward(*a)
    dt = (time.perf_counter() - t0) / steps
    cores = torch.get_num_threads()
    try:
        from threadpoolctl import threadpool_info
        cores = max([int(i.get("num_threads", 1)) for i in threadpool_info()] + [1])
    except Exception:
        pass
    sample = (f"oracle layer_forward on the first {Ts} of {cfg.T} tokens, budget {b}"
              if Ts < cfg.T else f"oracle layer_forward on the whole batch (T={cfg.T}, budget {b})")
    return dict(value=Ts / dt, unit=UNIT, cores=int(cores), kind="oracle", sample=sample, s_per_step=dt, tokens=Ts,
                budget=b, result=last)


def oracle_tokens_for(cfg):
    # about 10-30 s of CPU work: the small layers whole, the large ones on a token subset
    flops_per_token = 6.0 * cfg.H * cfg.I * (3 + cfg.S)
    weight_elems = (cfg.N + cfg.S) * 3.0 * cfg.H * cfg.I
    if cfg.T * flops_per_token < 2e11 and weight_elems < 1e9:
        return None
    return 64 if weight_elems > 1e9 else 256


def run_reference(args):
    """The oracle as it stands, timed on the host cores; every step is one oracle layer call on a
    bounded sample (the first Ts tokens), Ts sized so that warmup + steps end within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, budget = workload_cfg(args)
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    steps, warmup = max(1, steps), max(0, warmup)
    cap = oracle_tokens_for(cfg) or cfg.T
    probe = min(cap, 2)
    t_probe = time_oracle(cfg, budget, steps=1, warmup=0, target_tokens=probe)["s_per_step"]
    per_token = t_probe / probe
    Ts = max(1, min(cap, int(150.0 / (steps + warmup) / per_token)))
    r = time_oracle(cfg, budget, steps=steps, warmup=warmup, target_tokens=Ts)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": r["s_per_step"] * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(cfg, budget), "note": "CPU oracle as it stands, bounded sample per step"},
        "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": r["cores"], "kind": "oracle", "sample": r["sample"]},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def describe(cfg, budget):
    return (f"{cfg.name}: T={cfg.T} H={cfg.H} N={cfg.N} S={cfg.S} I={cfg.I} K_orig={cfg.K_orig} "
            f"K_base={cfg.K_base} budget={budget} ({budget / cfg.T:g}xT)")


# ------------------------------------------------------------------------------------------ our arm
def algorithmic_work(cfg, budget, touched):
    """FLOPs and bytes of one layer call: weights of touched experts once, activations once per use."""
    Wb = 6.0 * cfg.H * cfg.I                        # bytes of one expert's weights (3 matrices, bf16)
    flops = (budget + cfg.S * cfg.T) * 6.0 * cfg.H * cfg.I + 2.0 * cfg.T * cfg.H * cfg.N
    by = (touched + cfg.S) * Wb + cfg.T * cfg.H * 2 + budget * cfg.H * 2 + 2 * budget * cfg.H * 2 + cfg.T * cfg.H * 2
    if cfg.S:
        by += cfg.T * cfg.H * 2
    return flops, by


def gemm1_work(cfg, budget, touched):
    """Dominant kernel (expert GEMM-1 with the SwiGLU epilogue, routed + shared groups in one launch)."""
    flops = (budget + cfg.S * cfg.T) * 4.0 * cfg.H * cfg.I
    by = (touched + cfg.S) * 4.0 * cfg.H * cfg.I            # W13 of touched experts, bf16
    by += budget * cfg.H * 2 + (cfg.T * cfg.H * 2 if cfg.S else 0)       # A rows
    by += budget * cfg.I * 2 + cfg.S * cfg.T * cfg.I * 2                 # h written
    return flops, by


SECONDARY = (("c3", None), ("c5", None), ("c4", None))     # (workload, budget multiple; None = the workload's own)


class Env:
    """Process-group facts and the timing primitives shared by every measurement of a run."""

    def __init__(self, blocks=None):
        import torch
        import torch.distributed as dist
        self.torch, self.dist = torch, dist
        self.blocks = blocks
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def time_block(self, fn, k):
        """k calls of fn between a barrier + synchronize on both sides, CUDA events, max over ranks; ms."""
        from paper_2604_08133_b200 import dist as pdist
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record()
        for _ in range(k):
            fn()
        e1.record()
        self.barrier()
        return pdist.max_over_ranks(e0.elapsed_time(e1), device="cuda")

    def time_blocks(self, fn, k, call_is_k_steps=False):
        """Blocks of exactly k steps until MIN_BLOCKS have run and they add up to MIN_REGION_S.  Returns the
        per-step ms of every block.  call_is_k_steps: fn() itself runs the k steps (a pipelined loop)."""
        one = (lambda: self.time_block(fn, 1)) if call_is_k_steps else (lambda: self.time_block(fn, k))
        first = one()
        n = max(MIN_BLOCKS, int(math.ceil(MIN_REGION_S * 1e3 / max(first, 1e-3))))
        n = min(n, MAX_BLOCKS)
        if self.blocks is not None:
            n = max(1, self.blocks)
        ms = [first] + [one() for _ in range(n - 1)]
        return [m / k for m in ms]


def median(v):
    s = sorted(v)
    return s[len(s) // 2] if len(s) % 2 else 0.5 * (s[len(s) // 2 - 1] + s[len(s) // 2])


def default_steps(cfg):
    """Steps per block when --steps is not given: blocks of roughly 0.1 s."""
    if cfg.n_layers > 1:
        return 10, 3
    if cfg.T <= 256:
        return 500, 50
    return (25, 5) if cfg.H * cfg.I > 2e7 else (200, 20)


def bench_workload(env, args, name, budget_mult, steps_arg, warmup_arg, full=True):
    """All figures of one workload on this rank's GPU; `full` adds the CUDA-graph and end-to-end passes."""
    import torch
    from paper_2604_08133_b200 import binding as B
    from paper_2604_08133_b200 import synth

    class A:      # the argument view workload_cfg() expects
        pass
    a = A()
    a.workload, a.budget_mult = name, budget_mult
    a.k_base = args.k_base if name == args.workload else None
    cfg, budget = workload_cfg(a)
    # every rank works on its own batch (independent problems, replicated weights): weak scaling
    cfg = cfg.with_(seed=cfg.seed + env.rank)
    n_layers = cfg.n_layers
    dsteps, dwarm = default_steps(cfg)
    steps = steps_arg if steps_arg is not None else dsteps
    warmup = max(3, warmup_arg if warmup_arg is not None else dwarm)

    shape = B.shape_of(cfg)
    layers = [synth.make_layer(cfg, l, device="cuda", with_x=(l == 0)) for l in range(n_layers)]
    if n_layers > 1:
        ks = synth.stack_budgets(cfg)
        if args.stack_budgets == "alloc-l":
            # Alloc-L (Sec. 3.2) on a seeded synthetic sensitivity matrix: the same total as the Dirichlet split
            ks, _ = B.alloc_l_solve(synth.sensitivity_matrix(cfg), sum(ks))
            ks = [max(k, cfg.K_base) for k in ks]
        budgets = [k * cfg.T for k in ks]
    else:
        budgets = [budget]
    x0 = layers[0]["x"]
    ws = B.new_workspace(shape, max(budgets))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bufsets = [[torch.empty_like(x0), torch.empty_like(x0)] for _ in range(2)]   # second set: end-to-end pipeline
    xn = torch.empty_like(x0)
    stack = n_layers > 1     # the stack runs pre-norm: x_{l+1} = x_l + MoE_l(rmsnorm(x_l))

    def layer(l, x, profile=None, p=0):
        d = layers[l]
        out = bufsets[p][l & 1]
        xin = x
        if stack:
            B.moe_rmsnorm(shape, x, xn)
            xin = xn
        B.moe_layer_forward(shape, xin, d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"],
                            budgets[l], out, status, ws, residual=(x if stack else None))
        if profile is not None:
            for k, v in B.moe_profile_read().items():
                profile[k] += v
        return out

    def step(x_in=None, p=0):
        x = x0 if x_in is None else x_in
        for l in range(n_layers):
            x = layer(l, x, p=p)
        return x

    for _ in range(warmup):
        step()
    sampler = ClockSampler(env.local)
    env.barrier()
    sampler.start()
    per_step = env.time_blocks(step, steps)
    clocks = sampler.stop()
    assert int(status.item()) == 0, "device status %d" % int(status.item())
    ms_per_step = median(per_step)
    tokens_per_step = cfg.T * env.world
    per_step_launches = sum(kernels_per_layer(cfg, b) + (1 if stack else 0) for b in budgets)
    res = {
        "value": tokens_per_step / (ms_per_step * 1e-3), "unit": UNIT, "ms_per_step": ms_per_step,
        "steps": steps, "warmup": warmup, "blocks": len(per_step),
        "timed_region_s": sum(per_step) * steps * 1e-3, "ms_per_step_min": min(per_step), "ms_per_step_max": max(per_step),
        "config": {"workload": describe(cfg, budgets[0] if n_layers == 1 else sum(budgets) // n_layers),
                   "layers": n_layers, "parallelism": "independent batches per GPU, replicated weights, no collective",
                   "l2": "weights exceed L2 (no flush)" if (cfg.N + cfg.S) * 6 * cfg.H * cfg.I > 126e6 else
                         "L2-resident workload, no flush (latency-bound case)"},
        "clocks": clocks, "gpu_launches": per_step_launches * steps * len(per_step),
        "launches_per_step": per_step_launches,
    }
    peaks = load_peaks()
    if not args.no_extras:
        # ---- touched experts (data dependent) from the last call's offsets
        inter = B.moe_layer_intermediates(shape, budgets[-1], ws)
        off = inter["expert_offsets"].cpu()
        touched = int((off[1:] > off[:-1]).sum())

        # ---- stage profile: the same steps again with events at the stage boundaries (the dominant kernel's
        # average launch duration, measured live on the stream it is launched on)
        B.moe_profile_enable(True)
        acc = {k: 0.0 for k in B.PROFILE_STAGES}
        nprof = max(3, min(steps * len(per_step), int(0.25e3 / max(ms_per_step, 1e-3)), 400))
        for _ in range(3):
            step()
        for _ in range(nprof):
            x = x0
            for l in range(n_layers):
                x = layer(l, x, profile=acc)
        B.moe_profile_enable(False)
        stage_ms = {k: v / (nprof * n_layers) for k, v in acc.items()}
        b_mean = sum(budgets) / len(budgets)
        g_flops, g_bytes = gemm1_work(cfg, b_mean, touched)
        t_g1 = stage_ms["ffn_gemm1"] * 1e-3
        flops, by = algorithmic_work(cfg, b_mean, touched)
        t_flop = flops / (peaks["bf16_tflops_sustained"] * 1e12)
        t_byte = by / (peaks["hbm_gbs"] * 1e9)
        g_tflop = g_flops / (peaks["bf16_tflops_sustained"] * 1e12)
        g_tbyte = g_bytes / (peaks["hbm_gbs"] * 1e9)
        if g_tbyte >= g_tflop:
            roof = {"bound": "hbm", "achieved": g_bytes / t_g1 / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": g_flops / t_g1 / 1e12, "peak": peaks["bf16_tflops_sustained"],
                    "unit": "TFLOP/s"}
            roof["frac_of_burst_peak"] = roof["achieved"] / peaks["bf16_tflops"]
        roof["frac"] = roof["achieved"] / roof["peak"]
        pair = 128 * cfg.N < b_mean <= 256 * cfg.N      # the library's own rule for CTA-pair tiles
        kname = "ffn_gemm_pair_kernel<true>" if pair else "ffn_gemm_kernel<true, 256>"
        roof["traffic"] = ncu_traffic_bytes(kname, cfg.name, int(budgets[0])) if n_layers == 1 else None
        roof["kernel"] = kname + " (expert GEMM-1 + SwiGLU, routed and shared groups)"
        roof["peak_source"] = peaks["source"] + (" (sustained bf16)" if roof["bound"] == "tensor" else " (copy)")
        roof["avg_launch_ms"] = stage_ms["ffn_gemm1"]
        roof["launches_timed"] = nprof * n_layers
        roof["algorithmic_bytes"] = g_bytes
        roof["algorithmic_flops"] = g_flops
        res["roofline"] = roof
        res["stage_ms"] = stage_ms
        res["touched_experts"] = touched
        res["layer_roofline"] = {"flops": flops, "bytes": by, "t_flop_us": t_flop * 1e6, "t_byte_us": t_byte * 1e6,
                                 "bound": "tensor" if t_flop > t_byte else "hbm",
                                 "frac": max(t_flop, t_byte) / (ms_per_step * 1e-3 / n_layers),
                                 "tokens_per_s_at_roofline": cfg.T / max(t_flop, t_byte) / n_layers}

        # ---- the same kernels at the full Top-K_orig budget (budgeted-vs-full speedup)
        if n_layers == 1 and budget < cfg.K_orig * cfg.T:
            full_b = cfg.K_orig * cfg.T
            ws_full = B.new_workspace(shape, full_b)
            out_f = bufsets[0][0]
            d = layers[0]

            def step_full():
                B.moe_layer_forward(shape, x0, d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"],
                                    full_b, out_f, status, ws_full)
            for _ in range(warmup):
                step_full()
            ms_full = median(env.time_blocks(step_full, steps))
            res["full_topk"] = {"budget": full_b, "ms_per_step": ms_full, "speedup_budgeted_vs_full": ms_full / ms_per_step,
                                "paper_context": "paper reports 1.15x prefill / 1.34x decode at half budget, "
                                                 "whole DeepSeek-V2-Lite model, 1x H100 80GB, vLLM"}
            del ws_full

    if full and not args.no_extras:
        # ---- the same step replayed from a CUDA graph (one host call per step instead of one per kernel)
        cur0 = torch.cuda.current_stream()
        cap = torch.cuda.Stream()
        cap.wait_stream(cur0)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(cap):
            with torch.cuda.graph(graph, stream=cap):
                step()
        cur0.wait_stream(cap)
        for _ in range(warmup):
            graph.replay()
        ms_graph = median(env.time_blocks(graph.replay, steps))
        res["cuda_graph"] = {"ms_per_step": ms_graph, "value": tokens_per_step / (ms_graph * 1e-3), "unit": UNIT}
        assert int(status.item()) == 0

        # ---- end to end: every step's x comes from pinned host memory and its out goes back to pinned host
        # memory.  Steps are independent batches, so the copies run on streams of their own and overlap the
        # neighbouring steps' compute (two x buffers, two output sets); every step still pays both copies
        # inside the timed region.
        x_host = x0.cpu().pin_memory()
        out_host = [torch.empty_like(x_host).pin_memory() for _ in range(2)]
        x_dev = [torch.empty_like(x0) for _ in range(2)]
        cur = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def run_e2e(k):
            s_in.wait_stream(cur)
            s_out.wait_stream(cur)
            for i in range(k):
                p = i & 1
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_cmp[p])      # step i-2 has consumed x_dev[p]
                    x_dev[p].copy_(x_host, non_blocking=True)
                    ev_in[p].record(s_in)
                cur.wait_event(ev_in[p])
                if i >= 2:
                    cur.wait_event(ev_out[p])           # step i-2's result has left output set p
                y = step(x_dev[p], p)
                ev_cmp[p].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_cmp[p])
                    out_host[p].copy_(y, non_blocking=True)
                    ev_out[p].record(s_out)
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)
        run_e2e(4)
        ms_e2e = median(env.time_blocks(lambda: run_e2e(steps), steps, call_is_k_steps=True))
        nbytes = x0.numel() * 2
        res["e2e"] = {"value": tokens_per_step / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": nbytes,
                      "d2h_bytes_per_step": nbytes, "ms_per_step": ms_e2e,
                      "note": "x copied from pinned host memory and out copied back every step on copy streams that "
                              "overlap the neighbouring steps' compute; weights resident"}
        assert int(status.item()) == 0

    if full and not args.no_extras and n_layers == 1:
        res["select_kernels_us"] = bench_select_rules(env, cfg, shape, inter["topk_score"], budget, steps)

    if (args.global_alloc_t or env.world > 1) and n_layers == 1 and name == args.workload:
        res["global_alloc_t"] = bench_global_alloc_t(env, cfg, shape, layers[0], budget, steps, warmup)
    res["_cfg"], res["_budget"] = cfg, budgets[0]
    return res


def bench_select_rules(env, cfg, shape, topk_score, budget, steps):
    """Alloc-T's selection kernel next to the two token-level rules the paper compares it with (Top-P count, skipping
    relative to the top-1 score; thresholds calibrated off line to the same budget), on this workload's own scores:
    device time per call in microseconds.  Speed only; the paper's accuracy comparison is out of scope."""
    import torch
    from paper_2604_08133_b200 import binding as B
    from paper_2604_08133_b200 import token_baselines as TB
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    n_sel = torch.empty(cfg.T, dtype=torch.int32, device="cuda")
    r = {}
    fn = lambda: B.alloc_t_select(shape, topk_score, budget, n_sel, st, None)
    fn()
    r["alloc_t_select"] = median(env.time_blocks(fn, steps)) * 1e3
    for rule, inc, hi in (("top_p", True, 2.0), ("rel", False, 1.5)):
        thr, tot = TB.calibrate(TB.library_selector(rule, shape, st), topk_score, budget, increasing=inc, lo=0.0, hi=hi)
        f = B.moe_select_top_p if rule == "top_p" else B.moe_select_rel_threshold
        fn = lambda: f(shape, topk_score, thr, n_sel, None, st)
        fn()
        key = "top_p_count" if rule == "top_p" else "rel_threshold"
        r[key] = median(env.time_blocks(fn, steps)) * 1e3
        r[key + "_threshold"], r[key + "_kept"] = thr, tot
    assert int(st.item()) == 0
    return r


def bench_global_alloc_t(env, cfg, shape, d, budget, steps, warmup):
    """The batch-wide Alloc-T (Sec. 3.3 pools the scores of ALL tokens) with the batch sharded over the ranks:
    gate -> all-gather of the score rows -> selection over the whole pool on every rank -> routed layer call.
    Reports the whole layer and, separately, what the exchange adds: (gate + all-gather + selection) - gate."""
    import torch
    from paper_2604_08133_b200 import binding as B
    from paper_2604_08133_b200 import dist as pdist
    lay = pdist.GlobalAllocTLayer(shape, "cuda", always_collective=True)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty_like(d["x"])
    budget_global = budget * env.world

    def layer_step():
        lay.forward(d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"], budget_global, out, st)

    def route_step():
        lay.route(d["x"], d["W_gate"], d["gate_bias"], budget_global, st)

    def gate_step():
        B.moe_gate(shape, d["x"], d["W_gate"], d["gate_bias"], None, lay.topk_idx, lay.topk_score)

    r = {}
    for key, fn in (("layer_ms", layer_step), ("gate_exchange_select_ms", route_step), ("gate_ms", gate_step)):
        for _ in range(warmup):
            fn()
        r[key] = median(env.time_blocks(fn, steps))
    assert int(st.item()) == 0, "device status %d" % int(st.item())
    r["exchange_select_ms"] = r["gate_exchange_select_ms"] - r["gate_ms"]
    r["value"] = cfg.T * env.world / (r["layer_ms"] * 1e-3)
    r["unit"] = UNIT
    r["pool_keys"] = cfg.T * env.world * (cfg.K_orig - cfg.K_base)
    r["exchange"] = ("all_gather_into_tensor of %d fp32 score rows per rank over NCCL" % cfg.T) if \
        (env.world > 1 or env.dist.is_initialized()) else "one rank, no process group: the collective is skipped"
    return r


def parity_on_sample(cfg, budget, ref):
    """The GPU path against the oracle on the sample the CPU baseline timed (ref: the oracle's layer_forward
    result on the first Ts tokens): tokens whose selection differs (near-ties between the GPU's fp32 and the
    oracle's fp64 scores) and the output error measures on all other tokens."""
    import numpy as np
    import torch
    from paper_2604_08133_b200 import binding as B
    from paper_2604_08133_b200 import synth
    Ts = ref["out"].shape[0]
    scfg = cfg.with_(T=Ts)
    d = synth.make_layer(cfg, device="cuda")
    x = d["x"][:Ts].contiguous()
    shape = B.shape_of(scfg)
    ws = B.new_workspace(shape, budget)
    out = torch.empty_like(x)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.moe_layer_forward(shape, x, d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"], budget, out, st, ws)
    torch.cuda.synchronize()
    inter = B.moe_layer_intermediates(shape, budget, ws)
    same = (ref["n_sel"] == inter["n_sel"].cpu().numpy()) & (ref["topk_idx"] == inter["topk_idx"].cpu().numpy()).all(axis=1)
    got = out.float().cpu().numpy().astype(np.float64)[same]
    want = np.asarray(ref["out"], np.float64)[same]
    dlt = np.abs(got - want)
    rms = max(float(np.sqrt((want * want).mean())), 1e-30)
    return {"tokens": int(Ts), "flips": int((~same).sum()), "dev_status": int(st.item()),
            "max_rel": float(dlt.max() / max(np.abs(want).max(), 1e-30)),
            "elementwise": float((dlt / (np.abs(want) + rms)).max()),
            "rms_rel": float(np.sqrt((dlt * dlt).mean()) / rms),
            "note": "GPU vs the fp64 oracle on the CPU baseline's sample; flips = tokens whose kept set differs "
                    "(score near-ties), outputs compared on the others"}


def run_ours(args):
    import torch
    from paper_2604_08133_b200 import binding as B
    env = Env(args.blocks)
    B.lib()   # fails loudly when the CUDA library is missing

    res = bench_workload(env, args, args.workload, args.budget_mult, args.steps, args.warmup, full=True)
    cfg, budget0 = res.pop("_cfg"), res.pop("_budget")
    line = {"metric": METRIC, "value": res.pop("value"), "unit": res.pop("unit"), "n_gpus": env.world,
            "steps": res.pop("steps"), "warmup": res.pop("warmup"), "ms_per_step": res.pop("ms_per_step"),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
    line.update(res)

    if env.world == 1 and not args.no_workloads and not args.no_extras and args.workload == "c2" \
            and args.budget_mult is None and args.k_base is None:
        line["workloads"] = {}
        for name, mult in SECONDARY:
            torch.cuda.empty_cache()
            r = bench_workload(env, args, name, mult, None, None, full=False)
            r.pop("_cfg"), r.pop("_budget")
            line["workloads"][name] = r

    if env.rank == 0 and env.world == 1 and not args.no_cpu_baseline:
        torch.cuda.empty_cache()
        r = time_oracle(cfg, budget0, steps=1, warmup=0, target_tokens=oracle_tokens_for(cfg))
        line["cpu_baseline"] = {"value": r["value"], "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                                "sample": r["sample"]}
        line["parity"] = parity_on_sample(cfg, r["budget"], r["result"])
    if env.rank == 0:
        print(json.dumps(line), flush=True)
    if env.world > 1:
        env.dist.barrier()
        env.dist.destroy_process_group()




def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
