#!/usr/bin/env python
"""Benchmark of the BigMac DCCA MoE layer on B200: tokens/s of one training step (forward + backward,
all weight gradients) of one layer, and the fraction of the tensor-core roofline its contractions reach.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config large] [--impl ours|reference]

A step is one pass of the whole hot path (routing, descend, dispatch, expert GEMMs, combine, ascend and
the matching backward) over one batch of synthetic input.  The default workload is the largest
configuration (T=32768, d=4096, r=512, E=128, k=8, h=2048, GELU, BF16), which is the one the layer's
target is stated on.  With N > 1 (launched by torch.distributed.run) every rank runs its own batch on
its own GPU - the layer has no exchange step on one GPU per rank, so there is no data-path collective -
and the reported value is the total over ranks divided by the slowest rank's device time ("weak").

`--impl reference` times the CPU oracle (plain fp64 loops, as it stands) on a bounded token sample of the
same workload on the host cores; it is the reported baseline, not a target.
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

import numpy as np

from paper_2502_16927_b200 import workloads as wl

METRIC = "bigmac_layer_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------------------ counts
def forward_flops(w) -> float:
    """Algorithmic forward FLOPs of one call: gate logits + descend + ascend + the two expert GEMMs over the
    N = T*k routed rows (no padding rows, no dense every-expert work)."""
    return 2.0 * w.T * w.d * (w.E + 2 * w.r) + 4.0 * w.N * w.r * w.h


GEMM_FLOPS = {   # per launch, algorithmic (unpadded rows)
    "gemm_logits": lambda w: 2.0 * w.T * w.d * w.E, "gemm_descend": lambda w: 2.0 * w.T * w.d * w.r,
    "gemm_expert1": lambda w: 2.0 * w.N * w.r * w.h, "gemm_expert2": lambda w: 2.0 * w.N * w.r * w.h,
    "gemm_ascend": lambda w: 2.0 * w.T * w.d * w.r, "gemm_dy_lo": lambda w: 2.0 * w.T * w.d * w.r,
    "gemm_dw_up": lambda w: 2.0 * w.T * w.d * w.r, "gemm_dz": lambda w: 2.0 * w.N * w.r * w.h,
    "gemm_dw2": lambda w: 2.0 * w.N * w.r * w.h, "gemm_dxg": lambda w: 2.0 * w.N * w.r * w.h,
    "gemm_dw1": lambda w: 2.0 * w.N * w.r * w.h, "gemm_dx": lambda w: 2.0 * w.T * w.d * w.r,
    "gemm_dx_gate": lambda w: 2.0 * w.T * w.d * w.E, "gemm_dw_down": lambda w: 2.0 * w.T * w.d * w.r,
    "gemm_dw_gate": lambda w: 2.0 * w.T * w.d * w.E,
}
ROW_MOVE_BYTES = {   # per launch, algorithmic: rows read + rows written (+ the 4-byte tables)
    "dispatch": lambda w, b: (w.T * w.r + w.N * w.r) * b + 4.0 * w.N,
    "combine": lambda w, b: (w.N * w.r + w.T * w.r) * b + 8.0 * w.N,
    "dxlo_gather": lambda w, b: (w.N * w.r + w.T * w.r) * b + 4.0 * w.N,
    "combine_bwd": lambda w, b: (2.0 * w.N * w.r + w.N * w.r) * b + 12.0 * w.N,
}


def _e64(w):
    return (w.E + 63) // 64 * 64


# Algorithmic operand + output bytes per launch of every contraction (b = bytes per element; the saved sigma' is one
# byte per element on the BF16 path, logits are fp32): what the launch has to read and write once, with no re-reads.
GEMM_BYTES = {
    "gemm_logits": lambda w, b: (w.T * w.d + w.E * w.d) * b + 4.0 * w.T * w.E,
    "gemm_descend": lambda w, b: (w.T * w.d + w.r * w.d + w.T * w.r) * b,
    "gemm_expert1": lambda w, b: (w.N * w.r + w.E * w.h * w.r + w.N * w.h) * b + w.N * w.h * (1 if b == 2 else b),
    "gemm_expert2": lambda w, b: (w.N * w.h + w.E * w.h * w.r + w.N * w.r) * b,
    "gemm_ascend": lambda w, b: (w.T * w.r + w.r * w.d + w.T * w.d) * b,
    "gemm_dy_lo": lambda w, b: (w.T * w.d + w.r * w.d + w.T * w.r) * b,
    "gemm_dw_up": lambda w, b: (w.T * w.d + w.T * w.r + w.r * w.d) * b,
    "gemm_dz": lambda w, b: (w.N * w.r + w.E * w.h * w.r + w.N * w.h) * b + w.N * w.h * (1 if b == 2 else b),
    "gemm_dw2": lambda w, b: (w.N * w.r + w.N * w.h + w.E * w.h * w.r) * b,
    "gemm_dxg": lambda w, b: (w.N * w.h + w.E * w.h * w.r + w.N * w.r) * b,
    "gemm_dw1": lambda w, b: (w.N * w.h + w.N * w.r + w.E * w.h * w.r) * b,
    "gemm_dx": lambda w, b: (w.T * w.r + w.r * w.d + w.T * w.d) * b,
    "gemm_dx_gate": lambda w, b: (w.T * _e64(w) + w.E * w.d) * b,
    "gemm_dw_down": lambda w, b: (w.T * w.r + w.T * w.d + w.r * w.d) * b,
    "gemm_dw_gate": lambda w, b: (w.T * _e64(w) + w.E * w.d) * b,
}

# DRAM bytes per launch of the two output-heavy contractions as ncu counted them (dram__bytes_read.sum +
# dram__bytes_write.sum) on a SMALL case of the large workload's widths (T = 8192, N = 65536 routed rows, one launch
# each; the capture's summary is kept with the other profiler summaries): expert GEMM1 343.17 MB read + 393.99 MB written, dz
# 492.26 MB + 264.03 MB.  Split into the bytes that do not depend on the batch (the experts' weights, E h r
# elements of bf16 = 268.44 MB) and bytes per routed row (the rest / 65536); a full launch is scaled from that by
# its rows (traffic grows in proportion: operands and outputs are far larger than L2 at both sizes).
MEASURED_DRAM = {
    ("gemm_expert1", 4096, 512, 2048, 128, 8): (268435456, (343169280 + 393989376 - 268435456) / 65536),
    ("gemm_dz", 4096, 512, 2048, 128, 8): (268435456, (492259072 + 264026112 - 268435456) / 65536),
}


def measured_traffic(stage, w):
    key = (stage, w.d, w.r, w.h, w.E, w.k)
    if key not in MEASURED_DRAM:
        return None
    fixed, per_row = MEASURED_DRAM[key]
    return fixed + per_row * w.N


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "tflops_burst": p["bf16_tflops"],
                "tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while the timed regions run (reading only: no
    setting of the GPU is touched).  NVML is polled every 5 ms from a thread, so that a region of a few tens of
    milliseconds still gets samples; without the NVML module nvidia-smi is polled every 100 ms instead."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, index: int, uuid: str = ""):
        self.rows, self.proc, self.thread, self.nvml, self.max_mhz = [], None, None, None, None   # rows: (time, mhz, watts, reasons)
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid) if uuid else None
            except Exception:
                self.handle = None
            if self.handle is None:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll_nvml(self):
        n = self.nvml
        while not self._stop.is_set():
            try:
                mhz = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                watts = n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
                mask = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                self.rows.append((time.time(), mhz, watts, {name for name, bit in self.REASONS if mask & bit}))
            except Exception:
                pass
            time.sleep(0.005)

    def _read_smi(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                mhz, self.max_mhz, watts = float(parts[0]), float(parts[1]), float(parts[2])
            except ValueError:
                continue
            names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
            self.rows.append((time.time(), mhz, watts, {n for n, v in zip(names, parts[3:7]) if v.lower().startswith("active")}))

    def window(self, t0, t1):
        """Median SM MHz (and the rest) of the samples taken between two host times."""
        inside = [r for r in self.rows if t0 <= r[0] <= t1 + 0.01]
        if not inside:
            return None
        reasons = set()
        for r in inside:
            reasons |= r[3]
        return {"sm_mhz": float(np.median([r[1] for r in inside])), "watts": float(np.median([r[2] for r in inside])),
                "reasons": sorted(reasons), "samples": len(inside)}

    def stop(self, t0=None, t1=None):
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        win, label = (self.window(t0, t1) if t0 is not None else None), "timed region"
        if win is None and self.rows:                    # region shorter than the sampling period: use the loaded run
            win, label = self.window(self.rows[0][0], self.rows[-1][0]), "warm-up and timed region"
        if win is None:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "window": label}
        return {"sm_mhz": win["sm_mhz"], "sm_max_mhz": self.max_mhz, "reasons": win["reasons"], "samples": win["samples"],
                "power_w": round(win["watts"], 1), "window": label, "source": "nvml" if self.nvml else "nvidia-smi"}


# ------------------------------------------------------------------------------------------------ oracle leg
def oracle_sample_rate(w, inp, sample_tokens: int):
    """tokens/s of the CPU oracle (routing + forward + backward with every gradient) on the first
    `sample_tokens` tokens of the workload; cost is linear in T, so the rate carries over."""
    import oracle

    S = min(sample_tokens, w.T)
    sub = dict(inp, x=np.ascontiguousarray(inp["x"][:S]), dy=np.ascontiguousarray(inp["dy"][:S]))
    t0 = time.perf_counter()
    rt = oracle.route(sub, w.k)
    oracle.backward_full(sub, rt, w.act)
    dt = time.perf_counter() - t0
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    threads = int(os.environ.get("OMP_NUM_THREADS", cores))
    return S / dt, dt, S, min(threads, cores)


def sample_size_for(w, inp, seconds: float, repeats: int = 1, cap: int = 0) -> int:
    """Tokens per oracle run so that `repeats` runs take about `seconds` in total (calibrated on 32 tokens)."""
    rate, _, _, _ = oracle_sample_rate(w, inp, 32)
    s = int(seconds * rate / max(repeats, 1))
    s = max(8, min(w.T, s))
    return min(s, cap) if cap else s


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = wl.make_inputs(w)
    S = args.ref_tokens or sample_size_for(w, inp, 90.0, repeats=args.warmup + args.steps)
    rates = []
    for i in range(args.warmup + args.steps):
        rate, dt, S_used, cores = oracle_sample_rate(w, inp, S)
        if i >= args.warmup:
            rates.append((rate, dt))
    total_t = sum(dt for _, dt in rates)
    value = S_used * len(rates) / total_t
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / len(rates),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"first {S_used} tokens of the workload, all experts and gradients, per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(w, args):
    return {"workload": w.name, "T": w.T, "d": w.d, "r": w.r, "h": w.h, "E": w.E, "k": w.k,
            "act": {0: "relu", 1: "gelu_erf", 2: "gelu_tanh", 3: "identity"}[w.act],
            "gate_bias": w.gate_bias, "tokens_per_gpu": w.T, "l2": l2_note(w)}


def l2_note(w) -> str:
    """What the timing-hygiene rule asks to be stated: how the step's inputs compare with the 126 MB L2."""
    esz = 2 if w.dtype == wl.DTYPE_BF16 else 4
    io_mb = w.T * w.d * esz / 1e6                                        # each of x, dy, y, dx
    weights_mb = (w.E * w.d + 2 * w.r * w.d + 2 * w.E * w.h * w.r) * esz / 1e6
    routed_mb = w.T * w.k * (w.h * (esz + 1) + 2 * w.r * esz) / 1e6      # a, sigma' bytes, xg, u kept for the backward
    total = 4 * io_mb + weights_mb + routed_mb
    if 2 * io_mb + weights_mb > 126:
        return (f"inputs larger than L2 (x, dy {io_mb:.0f} MB each, weights {weights_mb:.0f} MB, "
                f"{total:.0f} MB touched per step)")
    if total > 126:
        return (f"x, dy {io_mb:.0f} MB each and weights {weights_mb:.0f} MB fit L2, the {total:.0f} MB a step touches do not: "
                "every step streams its routed rows through L2, no separate flush")
    return f"the {total:.0f} MB a step touches fit the 126 MB L2: no flush, a warm-L2 number (not the headline workload)"


# ------------------------------------------------------------------------------------------------ ranks
def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own batch (independent data-parallel replicas, replicated shapes)."""
    return base_seed + 1000 * rank


def slowest_rank_ms(ms_local: float, device: str = "cpu") -> float:
    """Device time of the slowest rank (MAX all-reduce); the identity without a process group."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Weak scaling: every rank processes tokens_per_rank tokens per step; the job is as fast as its slowest rank."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def run_cdac_twin(w, x, dy, dev, ms_step, ms_fwd, steps, peaks, esz):
    """The conventional fine-grained layer (Eq. 3) with the same E, k, d and expert parameter count (experts
    d -> m -> d, m = r h / d), same x, dy, gate and routing, through the same entry points and kernels: what one
    GPU pays for the layer when tokens travel at width d and there are no shared projections."""
    import torch
    from paper_2502_16927_b200 import binding

    if w.dtype != wl.DTYPE_BF16 or (w.r * w.h) % w.d or (w.r * w.h // w.d) % 64:
        return None
    t = w.cdac_twin()
    gen = torch.Generator(device="cuda").manual_seed(w.seed)
    tw = {"w_gate": dev["w_gate"],
          "w1": (torch.randn((t.E, t.h, t.d), generator=gen, device="cuda") * t.d ** -0.5).to(torch.bfloat16),
          "w2": (torch.randn((t.E, t.d, t.h), generator=gen, device="cuda") * t.h ** -0.5).to(torch.bfloat16)}
    if "b_gate" in dev:
        tw["b_gate"] = dev["b_gate"]
    G = {"dw_gate": torch.empty_like(tw["w_gate"]), "dw1": torch.empty_like(tw["w1"]), "dw2": torch.empty_like(tw["w2"]),
         "db_gate": torch.empty(t.E, dtype=torch.float32, device="cuda")}
    y, dx = torch.empty_like(x), torch.empty_like(x)
    layer = binding.Layer(t.d, t.r, t.h, t.E, t.k, t.T, t.dtype, t.act, wl.FLAG_CDAC)

    def step():
        layer.forward(x, tw, y=y, training=True)
        layer.backward(x, dy, tw, G, dx=dx)

    def timed(fn, n):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(n):
            fn()
        stop.record()
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / n

    for _ in range(3):
        step()
    ms = timed(step, steps)
    binding.bigmac_profile_enable(layer.handle, True)       # a second pass with per-stage events, for the stage rates
    timed(step, steps)
    prof = binding.bigmac_profile_read(layer.handle)
    binding.bigmac_profile_enable(layer.handle, False)
    fwd = lambda: layer.forward(x, tw, y=y, training=False)
    for _ in range(3):
        fwd()
    ms_f = timed(fwd, steps)
    if layer.status() != 0:
        raise RuntimeError("device status word reports a timed-out wait")
    stages = {}
    for name, (tot, calls) in prof["stages"].items():
        per = tot / calls
        entry = {"ms": round(per, 4)}
        if name in GEMM_FLOPS:
            entry["tflops"] = round(GEMM_FLOPS[name](t) / (per * 1e-3) / 1e12, 1)
        elif name in ROW_MOVE_BYTES:
            entry["gbs"] = round(ROW_MOVE_BYTES[name](t, esz) / (per * 1e-3) / 1e9, 1)
        stages[name] = entry
    layer.close()
    return {"config": {"workload": t.name, "T": t.T, "d": t.d, "expert_hidden_m": t.h, "E": t.E, "k": t.k,
                       "expert_parameters": 2 * t.E * t.d * t.h, "bigmac_expert_parameters": 2 * w.E * w.r * w.h},
            "ms_per_step": ms, "tokens_per_s": t.T / (ms * 1e-3), "forward_ms": ms_f,
            "bigmac_over_cdac_time": {"fwd_bwd": round(ms_step / ms, 3), "fwd": round(ms_fwd / ms_f, 3)},
            "stages": stages}


def run_recipe_variant(w, x, dy, dev, G, y, dx, base_step, steps):
    """The same layer and inputs under the paper's pre-training settings (Table 5: capacity factor 1.2,
    load-balancing loss with coefficient 0.001) instead of dropless routing: forward + backward time, the share of
    slots dropped and the loss value."""
    import torch
    from paper_2502_16927_b200 import binding

    f, alpha = 1.2, 0.001
    layer = binding.Layer(w.d, w.r, w.h, w.E, w.k, w.T, w.dtype, w.act, capacity_factor=f, aux_loss_coef=alpha)

    def step():
        layer.forward(x, dev, y=y, training=True)
        layer.backward(x, dy, dev, G, dx=dx)

    def timed(fn):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(steps):
            fn()
        stop.record()
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / steps

    for _ in range(3):
        step()
    # the dropless layer is timed again right beside it (alternating), so that both see the same clocks
    ms_pairs = [(timed(base_step), timed(step)) for _ in range(2)]
    ms_base, ms = (sum(p[i] for p in ms_pairs) / len(ms_pairs) for i in (0, 1))
    _, R = layer.forward(x, dev, y=y, training=True, want_routing=True)
    torch.cuda.synchronize()
    if layer.status() != 0:
        raise RuntimeError("device status word reports a timed-out wait")
    kept = int(R["counts"].sum().item())
    out = {"capacity_factor": f, "aux_loss_coef": alpha, "ms_per_step": ms, "tokens_per_s": w.T / (ms * 1e-3),
           "dropless_ms_per_step_beside_it": ms_base, "over_dropless_time": round(ms / ms_base, 3), "dropped_slot_share": round(1.0 - kept / (w.T * w.k), 5),
           "rows_per_expert_limit": int(np.ceil(f * (w.T * w.k) / w.E)), "aux_loss": float(R["aux_loss"].item())}
    layer.close()
    return out


def run_small_variants(w, x, dy, dev, G, y, dx, base_step, steps):
    """The two small variants of the layer on the same inputs, each timed alternately with the plain layer: the gate
    reading the low-width token x' (w_gate [E,r]) and experts with biases (fp32 b1 [E,h], b2 [E,r])."""
    import torch
    from paper_2502_16927_b200 import binding

    def timed(fn):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(steps):
            fn()
        stop.record()
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / steps

    gen = torch.Generator(device="cuda").manual_seed(w.seed + 7)
    out = {}
    cases = {
        "gate_on_low_width_token": (wl.FLAG_GATE_LOW,
                                    {"w_gate": (torch.randn((w.E, w.r), generator=gen, device="cuda") * w.r ** -0.5).to(x.dtype)},
                                    {"dw_gate": torch.empty((w.E, w.r), dtype=x.dtype, device="cuda")}),
        "expert_biases": (wl.FLAG_EXPERT_BIAS,
                          {"b1": torch.randn((w.E, w.h), generator=gen, device="cuda") * 0.5,
                           "b2": torch.randn((w.E, w.r), generator=gen, device="cuda") * 0.5},
                          {"db1": torch.empty((w.E, w.h), dtype=torch.float32, device="cuda"),
                           "db2": torch.empty((w.E, w.r), dtype=torch.float32, device="cuda")}),
    }
    for name, (flag, extra_w, extra_g) in cases.items():
        Wv, Gv = dict(dev, **extra_w), dict(G, **extra_g)
        layer = binding.Layer(w.d, w.r, w.h, w.E, w.k, w.T, w.dtype, w.act, flag)

        def step():
            layer.forward(x, Wv, y=y, training=True)
            layer.backward(x, dy, Wv, Gv, dx=dx)

        for _ in range(3):
            step()
        pairs = [(timed(base_step), timed(step)) for _ in range(2)]
        ms_base, ms = (sum(p[i] for p in pairs) / len(pairs) for i in (0, 1))
        if layer.status() != 0:
            raise RuntimeError("device status word reports a timed-out wait")
        layer.close()
        out[name] = {"ms_per_step": ms, "plain_layer_ms_per_step_beside_it": ms_base, "over_plain_layer_time": round(ms / ms_base, 3)}
    return out


def run_decode_latencies(peaks, tokens=(1, 8, 16, 64, 512), calls=200):
    """Inference forward at the decode-shaped configuration for a few batch sizes: latency per call (CUDA events over
    `calls` back-to-back calls after 20 warm-up calls; the 70 MB a call touches stay in L2, so a warm number), next to
    the time the touched weights would take from HBM at the measured copy bandwidth."""
    import torch
    from paper_2502_16927_b200 import binding

    base = wl.WORKLOADS["decode"]
    out = {}
    for T in tokens:
        w = base.with_tokens(T)
        inp = wl.make_inputs(w)

        def dev_of(a):
            return torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).view(torch.bfloat16).cuda()

        dev = {k: dev_of(inp[k]) for k in ("w_gate", "w_down", "w1", "w2", "w_up")}
        if inp["b_gate"] is not None:
            dev["b_gate"] = torch.from_numpy(inp["b_gate"]).cuda()
        x = dev_of(inp["x"])
        y = torch.empty_like(x)
        layer = binding.Layer(w.d, w.r, w.h, w.E, w.k, w.T, w.dtype, w.act)
        for _ in range(20):
            layer.forward(x, dev, y=y, training=False)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(calls):
            layer.forward(x, dev, y=y, training=False)
        stop.record()
        torch.cuda.synchronize()
        us = start.elapsed_time(stop) * 1e3 / calls
        # touched weights: both projections, the gate, and the experts at least one token chose (expected number for a
        # uniform gate: E (1 - (1 - k/E)^T))
        experts = w.E * (1.0 - (1.0 - w.k / w.E) ** T)
        weight_bytes = 2.0 * (2 * w.d * w.r + w.E * w.d + experts * 2 * w.r * w.h)
        floor_us = weight_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6
        out[str(T)] = {"us_per_call": round(us, 1), "weight_streaming_floor_us": round(floor_us, 1),
                       "times_floor": round(us / floor_us, 1), "tokens_per_s": round(T / (us * 1e-6))}
        if layer.status() != 0:
            raise RuntimeError("device status word reports a timed-out wait")
        layer.close()
        del dev, x, y
    return {"workload": "decode (d 2048, r 256, h 1024, E 64, k 8), inference forward", "l2": "warm: a call's 70 MB fit L2",
            "by_tokens": out}


def run_ep_on_one_gpu(w, x, dy, dev, ms_step, steps, esz, size=4):
    """The expert-parallel layer (Fig. 2c) with `size` ranks driven on this one GPU: every rank brings T/size of the
    step's tokens and owns E/size experts; rows travel between the ranks' buffers at width r through the same put /
    get kernels a multi-GPU job runs, here within one memory.  What this measures is the cost of the phase structure
    and of the exchange kernels against the one-GPU layer on the same tokens; link time it cannot show.  Beside it the
    conventional layer of Eq. 3 with equal E, k and expert parameters runs the same way, its rows travelling at width d:
    the exchange kernels' times and the bytes that would cross the links per rank and exchange (Eq. 1) are set against
    each other."""
    import torch
    from paper_2502_16927_b200 import binding, ep

    if w.E % size or w.T % size:
        return None
    if not w.cdac:                                   # beside it: the parameter-parity twin of Eq. 3, rows at width d
        twin = None
        if w.dtype == wl.DTYPE_BF16 and (w.r * w.h) % w.d == 0 and (w.r * w.h // w.d) % 64 == 0:
            t = w.cdac_twin()
            gen = torch.Generator(device="cuda").manual_seed(w.seed + 11)
            tw = {"w_gate": dev["w_gate"],
                  "w1": (torch.randn((t.E, t.h, t.d), generator=gen, device="cuda") * t.d ** -0.5).to(torch.bfloat16),
                  "w2": (torch.randn((t.E, t.d, t.h), generator=gen, device="cuda") * t.h ** -0.5).to(torch.bfloat16)}
            if "b_gate" in dev:
                tw["b_gate"] = dev["b_gate"]
            twin = run_ep_on_one_gpu(t, x, dy, tw, None, steps, esz, size)
    Tq = w.T // size
    Ws = [ep.shard_weights(dev, q, size) for q in range(size)]
    xs = [x[q * Tq:(q + 1) * Tq] for q in range(size)]
    dys = [dy[q * Tq:(q + 1) * Tq] for q in range(size)]
    ys, dxs = [torch.empty_like(v) for v in xs], [torch.empty_like(v) for v in xs]
    per = w.E // size
    Gs = [{"dw_gate": torch.empty_like(dev["w_gate"]), "dw1": torch.empty_like(Ws[q]["w1"]), "dw2": torch.empty_like(Ws[q]["w2"]),
           "db_gate": torch.empty(w.E, dtype=torch.float32, device="cuda")} for q in range(size)]
    if not w.cdac:
        for G in Gs:
            G.update(dw_down=torch.empty_like(dev["w_down"]), dw_up=torch.empty_like(dev["w_up"]))
    group = ep.EpLocalGroup(w.d, w.r, w.h, w.E, w.k, Tq, w.dtype, w.act, ["cuda"] * size, wl.FLAG_CDAC if w.cdac else 0)

    def step():
        group.forward(xs, Ws, ys)
        group.backward(xs, dys, Ws, Gs, dxs)

    for _ in range(3):
        step()

    def timed_steps():
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(steps):
            step()
        stop.record()
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / steps

    ms = timed_steps()
    for rk in group.ranks:                                   # a second pass with per-stage events, for the exchange kernels
        binding.bigmac_profile_enable(rk.handle, True)
    timed_steps()
    moves = {}
    for rk in group.ranks:
        prof = binding.bigmac_profile_read(rk.handle)
        for name in ("dispatch", "combine", "combine_bwd", "dxlo_gather"):
            tot, calls = prof["stages"].get(name, (0.0, 1))
            moves[name] = moves.get(name, 0.0) + tot / steps
    if group.status() != 0:
        raise RuntimeError("device status word reports a timed-out wait")
    group.close()
    out = {"ranks_on_this_gpu": size, "tokens_per_rank": Tq, "experts_per_rank": per, "row_width": w.r, "ms_per_step_all_ranks": ms,
           "tokens_per_s": w.T / (ms * 1e-3),
           "exchange_kernels_ms_all_ranks": {name: round(v, 4) for name, v in moves.items()},
           "exchange_kernels_ms_total": round(sum(moves.values()), 4),
           "link_bytes_per_rank_per_exchange": ep.exchange_bytes_per_rank(Tq, w.k, w.r, size, esz)}
    if w.cdac:
        return out
    out["over_one_gpu_layer_time"] = round(ms / ms_step, 3)
    out["eq3_twin_rows_at_width_d"] = twin
    if twin:
        out["bigmac_over_twin"] = {"step_time": round(ms / twin["ms_per_step_all_ranks"], 3),
                                   "exchange_kernel_time": round(out["exchange_kernels_ms_total"] / twin["exchange_kernels_ms_total"], 3),
                                   "link_bytes": round(out["link_bytes_per_rank_per_exchange"] / twin["link_bytes_per_rank_per_exchange"], 4)}
    out["note"] = "ranks share one GPU: no link is crossed; exchanges per step: 2 forward, 2 backward"
    return out


def run_expert_parallel_ranks(w, x, dy, dev, steps, esz, rank, world, timed):
    """One expert-parallel rank per process (Fig. 2c) over the job's NCCL group: every rank keeps its batch of T tokens
    and owns E / N experts; rows cross the links at width r through the library's put / get kernels over symmetric
    memory (plain peer loads and stores).  Beside it the Eq. 3 twin with equal E, k and expert parameters, whose rows
    travel at width d.  Returns, on every rank, the whole-job tokens/s, the slowest rank's step time, this rank's
    exchange-kernel times and the bytes a rank sends per exchange (Eq. 1).  Called after the headline number is final."""
    import torch
    from paper_2502_16927_b200 import binding, ep

    if w.E % world:
        return {"skipped": f"E = {w.E} is not a multiple of {world} ranks"}

    def one(wv, Wfull, flags):
        Ws = ep.shard_weights(Wfull, rank, world)
        G = {"dw_gate": torch.empty_like(Wfull["w_gate"]), "dw1": torch.empty_like(Ws["w1"]), "dw2": torch.empty_like(Ws["w2"]),
             "db_gate": torch.empty(wv.E, dtype=torch.float32, device="cuda")}
        if not wv.cdac:
            G.update(dw_down=torch.empty_like(Wfull["w_down"]), dw_up=torch.empty_like(Wfull["w_up"]))
        epr = ep.EpProcessRank(wv.d, wv.r, wv.h, wv.E, wv.k, wv.T, wv.dtype, wv.act, flags=flags)
        y, dx = torch.empty_like(x), torch.empty_like(x)

        def step():
            epr.forward(x, Ws, y=y)
            epr.backward(x, dy, Ws, G, dx=dx)

        for _ in range(3):
            step()
        ms = timed(step, steps) / steps
        binding.bigmac_profile_enable(epr.rk.handle, True)
        timed(step, steps)
        prof = binding.bigmac_profile_read(epr.rk.handle)
        binding.bigmac_profile_enable(epr.rk.handle, False)
        status = epr.status()
        epr.close()
        if status != 0:
            raise RuntimeError(f"device status word: {status}")
        moves = {name: round(prof["stages"].get(name, (0.0, 1))[0] / steps, 4)
                 for name in ("dispatch", "combine", "combine_bwd", "dxlo_gather")}
        nbytes = ep.exchange_bytes_per_rank(wv.T, wv.k, wv.r, world, esz)
        return {"row_width": wv.r, "ms_per_step": ms, "tokens_per_s": world * wv.T / (ms * 1e-3),
                "exchange_kernels_ms_this_rank": moves, "exchange_kernels_ms_total": round(sum(moves.values()), 4),
                "link_bytes_per_rank_per_exchange": nbytes,
                "exchange_gbs_per_direction": {name: round(nbytes / (v * 1e-3) / 1e9, 1) for name, v in moves.items() if v > 0}}

    out = {"ranks": world, "tokens_per_rank": w.T, "experts_per_rank": w.E // world,
           "exchanges_per_step": "2 forward, 2 backward; peer puts / gets of rows, NCCL only for the count all-gather, "
                                 "the barriers and the shared-gradient sums"}
    out["bigmac_rows_at_width_r"] = one(w, dev, 0)
    if w.dtype == wl.DTYPE_BF16 and (w.r * w.h) % w.d == 0 and (w.r * w.h // w.d) % 64 == 0:
        t = w.cdac_twin()
        need = 4 * world * t.T * t.k * t.r * esz                       # the four exchange buffers, worst case
        if need < 0.5 * torch.cuda.mem_get_info()[0]:
            gen = torch.Generator(device="cuda").manual_seed(w.seed + 11)
            tw = {"w_gate": dev["w_gate"],
                  "w1": (torch.randn((t.E, t.h, t.d), generator=gen, device="cuda") * t.d ** -0.5).to(torch.bfloat16),
                  "w2": (torch.randn((t.E, t.d, t.h), generator=gen, device="cuda") * t.h ** -0.5).to(torch.bfloat16)}
            if "b_gate" in dev:
                tw["b_gate"] = dev["b_gate"]
            out["eq3_twin_rows_at_width_d"] = one(t, tw, wl.FLAG_CDAC)
            a, b = out["bigmac_rows_at_width_r"], out["eq3_twin_rows_at_width_d"]
            ratio = lambda u, v, nd: round(u / v, nd) if v else None
            out["bigmac_over_twin"] = {"step_time": ratio(a["ms_per_step"], b["ms_per_step"], 3),
                                       "exchange_kernel_time": ratio(a["exchange_kernels_ms_total"], b["exchange_kernels_ms_total"], 3),
                                       "link_bytes": ratio(a["link_bytes_per_rank_per_exchange"], b["link_bytes_per_rank_per_exchange"], 4)}
        else:
            out["eq3_twin_rows_at_width_d"] = {"skipped": "exchange buffers at width d would not fit beside the rest"}
    return out


def nccl_communicator_line(path_pattern: str):
    """The line of NCCL's own log that names the communicator's rank count (evidence of how many ranks took part)."""
    import glob
    import re

    for path in sorted(glob.glob(path_pattern)):
        try:
            for line in open(path, errors="replace"):
                if re.search(r"nranks\s+\d+", line):
                    return line.strip()[-240:]
        except OSError:
            continue
    return None


# ------------------------------------------------------------------------------------------------ ours
def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2502_16927_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local)
    want_ep = world > 1 or args.expert_parallel
    nccl_log = None
    if want_ep:
        # NCCL's communicator log goes to a file of its own (its default, stdout, would break the one-line contract)
        import tempfile
        nccl_dir = tempfile.mkdtemp(prefix="bigmac_nccl_")
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(nccl_dir, "rank%p.log"))
        nccl_log = os.environ["NCCL_DEBUG_FILE"].replace("%p", "*").replace("%h", "*")
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    elif want_ep:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(29600 + os.getpid() % 1000))
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    for item in args.debug_set:
        name, _, val = item.partition("=")
        binding.bigmac_debug_set(name, int(val or 0))

    wr = w.with_tokens(w.T, seed=rank_seed(w.seed, rank))
    inp = wl.make_inputs(wr)
    tdt = torch.bfloat16 if w.dtype == wl.DTYPE_BF16 else torch.float32

    def host(a):
        if w.dtype == wl.DTYPE_BF16:
            t = torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).view(torch.bfloat16)
        else:
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        return t.pin_memory()

    hx, hdy = host(inp["x"]), host(inp["dy"])
    dev = {k: host(inp[k]).cuda() for k in ("w_gate", "w_down", "w1", "w2", "w_up")}
    if inp["b_gate"] is not None:
        dev["b_gate"] = torch.from_numpy(inp["b_gate"]).cuda()
    x, dy = hx.cuda(), hdy.cuda()
    y, dx = torch.empty_like(x), torch.empty_like(x)
    G = {"dw_gate": torch.empty_like(dev["w_gate"]), "dw_down": torch.empty_like(dev["w_down"]),
         "dw1": torch.empty_like(dev["w1"]), "dw2": torch.empty_like(dev["w2"]), "dw_up": torch.empty_like(dev["w_up"]),
         "db_gate": torch.empty(w.E, dtype=torch.float32, device="cuda")}
    hy, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
    layer = binding.Layer(w.d, w.r, w.h, w.E, w.k, w.T, w.dtype, w.act)
    if rank != 0:
        del inp

    # the decode-shaped configuration is an inference forward (no backward exists for it in the metric)
    forward_only_workload = w.name == "decode"

    def step():
        if forward_only_workload:
            layer.forward(x, dev, y=y, training=False)
            return
        layer.forward(x, dev, y=y, training=True)
        layer.backward(x, dy, dev, G, dx=dx)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        start.record()
        for _ in range(steps):
            fn()
        stop.record()
        barrier()
        return slowest_rank_ms(start.elapsed_time(stop), device="cuda")

    if args.profile_run:                    # bare loop for a profiler: warm-up and K steps, nothing else
        binding.bigmac_debug_set("overlap", 0)   # one stream: launches reach the profiler in program order
        for _ in range(args.warmup + args.steps):
            step()
        torch.cuda.synchronize()
        if layer.status() != 0:
            raise RuntimeError("device status word reports a timed-out wait")
        print(json.dumps({"profile_run": True, "config": config_dict(w, args), "steps": args.steps,
                          "warmup": args.warmup}))
        return
    sampler = ClockSampler(local, str(torch.cuda.get_device_properties(local).uuid)) if rank == 0 else None
    t_warm = time.time()
    for _ in range(max(args.warmup, 3)):
        step()
    if layer.status() != 0:
        raise RuntimeError("device status word reports a timed-out wait")
    while sampler and not sampler.rows and time.time() - t_warm < 3.0:   # let nvidia-smi come up, under load
        step()
        torch.cuda.synchronize()

    # ---- timed region: K steps as a caller runs them, device-timed, max over ranks; and the same K steps with a
    # CUDA-event pair around every stage (what the roofline and the per-stage rates below come from).  The events cost
    # time of their own (27 pairs per step), and while they are recorded the backward pass keeps all launches on one
    # stream so that a stage's time is its own.  Under the power cap the clocks drift over the first seconds of load, so
    # the two kinds of steps alternate in halves (K/2 plain, K/2 with events, the rest plain, the rest with events) and
    # see the same clocks; each half is bracketed by barrier + synchronize like a whole region.
    halves = [args.steps // 2, args.steps - args.steps // 2]
    ms_total = ms_events_total = 0.0
    prof = {"launches": 0, "dropped": 0, "stages": {}}
    t0 = time.time()
    def plain_half(n):
        nonlocal ms_total
        ms_total += timed(step, n)

    def events_half(n):
        nonlocal ms_events_total
        binding.bigmac_profile_enable(layer.handle, True)
        ms_events_total += timed(step, n)
        part = binding.bigmac_profile_read(layer.handle)
        binding.bigmac_profile_enable(layer.handle, False)
        prof["launches"] += part["launches"]
        prof["dropped"] += part["dropped"]
        for name, (ms, calls) in part["stages"].items():
            old_ms, old_calls = prof["stages"].get(name, (0.0, 0))
            prof["stages"][name] = (old_ms + ms, old_calls + calls)

    # plain, events, events, plain: whichever kind follows a pause (reading the events back) meets a rested GPU
    for i, n in enumerate(halves):
        if n == 0:
            continue
        for half in ((plain_half, events_half) if i == 0 else (events_half, plain_half)):
            half(n)
    t1 = time.time()
    ms_step = ms_total / args.steps
    ms_step_events = ms_events_total / args.steps
    value = whole_job_tokens_per_s(w.T, world, ms_step)

    # ---- the same K plain steps again as separate regions, each with the SM clock seen while it ran: median and
    # minimum over the regions, and time x clock (million SM cycles per step), which tells a faster kernel from a
    # GPU that happened to clock higher under the power cap.  The headline stays the region above.
    n_regions = 5 if ms_step * args.steps < 2000.0 else 2
    regions = []
    for _ in range(n_regions):
        ta = time.time()
        ms_r = timed(step, args.steps) / args.steps
        tb = time.time()
        win = sampler.window(ta, tb) if sampler else None
        regions.append({"ms_per_step": round(ms_r, 4), "sm_mhz": win["sm_mhz"] if win else None,
                        "mcycles_per_step": round(ms_r * win["sm_mhz"] / 1e3, 3) if win else None})
    clocks = sampler.stop(t0, t1) if sampler else None
    r_ms = [r["ms_per_step"] for r in regions]
    r_mc = [r["mcycles_per_step"] for r in regions if r["mcycles_per_step"] is not None]
    repeats = {"regions": n_regions, "steps_per_region": args.steps, "ms_per_step_median": float(np.median(r_ms)),
               "ms_per_step_min": float(np.min(r_ms)),
               "mcycles_per_step_median": float(np.median(r_mc)) if r_mc else None, "each": regions}
    if clocks and clocks.get("sm_mhz"):
        clocks["mcycles_per_step"] = round(ms_step * clocks["sm_mhz"] / 1e3, 3)

    # forward only (inference forward: nothing saved)
    def fwd_only():
        layer.forward(x, dev, y=y, training=False)
    for _ in range(3):
        fwd_only()
    ms_fwd = timed(fwd_only, args.steps) / args.steps

    # small batches are launch-bound: also time the same forward replayed from a CUDA graph (the C ABI neither
    # allocates nor synchronises, so a caller can capture it)
    ms_fwd_graph = None
    if w.T <= 1024:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fwd_only()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fwd_only()
        for _ in range(3):
            graph.replay()
        ms_fwd_graph = timed(graph.replay, args.steps) / args.steps

    # ---- the exchange stage alone at width r (BigMac) and at width d (a fine-grained CDAC layer of equal E, k
    # dispatches and combines full-width rows, Eq. 1): same kernels, same routing, rank 0's GPU only
    exchange = None
    touched_bytes, n_distinct = None, None
    if forward_only_workload:
        _, Rt = layer.forward(x, dev, y=y, training=False, want_routing=True)
        torch.cuda.synchronize()
        n_distinct = int((Rt["counts"] > 0).sum().item())
        esz_ = 2 if w.dtype == wl.DTYPE_BF16 else 4
        touched_bytes = float((2 * w.T * w.d + w.E * w.d + 2 * w.r * w.d + 2 * n_distinct * w.r * w.h) * esz_)
    if rank == 0 and not forward_only_workload:
        layer.forward(x, dev, y=y, training=True)                  # leaves the routing tables in `saved`
        P = ((w.N + 127) // 128 + w.E) * 128
        exchange = {}
        for label, width, src in (("bigmac_width_r", w.r, x[:, : w.r].contiguous()), ("cdac_width_d", w.d, x)):
            grouped = torch.empty((P, width), dtype=tdt, device="cuda")
            dst = torch.empty((w.T, width), dtype=tdt, device="cuda")
            run = lambda: binding.bigmac_exchange_rows(layer.handle, layer._saved, w.T, width, src, grouped, dst, 2)
            for _ in range(3):
                run()
            start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            start.record()
            for _ in range(10):
                run()
            stop.record()
            torch.cuda.synchronize()
            ms = start.elapsed_time(stop) / 10
            nbytes = 2 * (w.T + w.N) * width * (2 if w.dtype == wl.DTYPE_BF16 else 4)
            exchange[label] = {"bytes": nbytes, "ms": round(ms, 4), "gbs": round(nbytes / ms / 1e6, 1)}
            del grouped, dst
        exchange["time_ratio_d_over_r"] = round(exchange["cdac_width_d"]["ms"] / exchange["bigmac_width_r"]["ms"], 2)

    # ---- end to end through the same calls with HOST buffers: every step copies its x, dy in from pinned host memory
    # and its y, dx out again.  The copies run on their own streams over two sets of device buffers, so step i's
    # transfers overlap step i-1's / i+1's kernels (the way a training loop feeds a layer); the timed region ends
    # when the last step's outputs are in host memory.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    main = torch.cuda.current_stream()
    bufs = [(x, dy, y, dx), (torch.empty_like(x), torch.empty_like(x), torch.empty_like(x), torch.empty_like(x))]
    ev_in = [torch.cuda.Event(), torch.cuda.Event()]
    ev_comp = [torch.cuda.Event(), torch.cuda.Event()]
    ev_out = [torch.cuda.Event(), torch.cuda.Event()]

    def e2e_run(n):
        for ev in ev_comp + ev_out:
            ev.record(main)
        for i in range(n):
            bx, bdy, by, bdx = bufs[i & 1]
            s_in.wait_event(ev_comp[i & 1])                 # the step that last read these input buffers is done
            with torch.cuda.stream(s_in):
                bx.copy_(hx, non_blocking=True)
                if not forward_only_workload:
                    bdy.copy_(hdy, non_blocking=True)
                ev_in[i & 1].record(s_in)
            main.wait_event(ev_in[i & 1])
            main.wait_event(ev_out[i & 1])                  # ... and its outputs have left the output buffers
            if forward_only_workload:
                layer.forward(bx, dev, y=by, training=False)
            else:
                layer.forward(bx, dev, y=by, training=True)
                layer.backward(bx, bdy, dev, G, dx=bdx)
            ev_comp[i & 1].record(main)
            s_out.wait_event(ev_comp[i & 1])
            with torch.cuda.stream(s_out):
                hy.copy_(by, non_blocking=True)
                if not forward_only_workload:
                    hdx.copy_(bdx, non_blocking=True)
                ev_out[i & 1].record(s_out)
        main.wait_event(ev_out[0])
        main.wait_event(ev_out[1])

    e2e_run(3)
    e2e_steps = max(4, min(args.steps, 10))
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    e2e_run(e2e_steps)
    stop.record()
    barrier()
    ms_e2e = slowest_rank_ms(start.elapsed_time(stop), device="cuda") / e2e_steps
    del bufs
    if layer.status() != 0:
        raise RuntimeError("device status word reports a timed-out wait")

    # ---- expert parallelism over the job's ranks (N > 1, or on request with a group of one): after everything the
    # headline needs, on all ranks together.  A failure here is recorded, not raised; should a rank hang in a
    # collective, rank 0's watchdog prints the headline without this section before the process group's own time-out
    # can take the process down.
    ep_ranks = None
    if want_ep and w.dtype == wl.DTYPE_BF16 and not forward_only_workload:
        esz_ep = 2
        bytes_io_ep = 2 * w.T * w.d * esz_ep
        minimal = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                   "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                   "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config_dict(w, args), "clocks": clocks,
                   "e2e": {"value": world * w.T / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": bytes_io_ep,
                           "d2h_bytes_per_step": bytes_io_ep, "ms_per_step": ms_e2e},
                   "gpu_launches": prof["launches"], "repeats": repeats,
                   "expert_parallel": {"error": "timed out: a rank did not reach a collective; side measurements skipped"}}

        def print_minimal_and_leave():
            print(json.dumps(minimal), flush=True)
            os._exit(0)

        watchdog = None
        if rank == 0:
            watchdog = threading.Timer(300.0, print_minimal_and_leave)
            watchdog.daemon = True
            watchdog.start()
        try:
            ep_ranks = run_expert_parallel_ranks(w, x, dy, dev, max(3, min(args.steps, 10)), esz_ep, rank, world, timed)
            ep_ranks["nccl_communicator"] = nccl_communicator_line(nccl_log) if nccl_log else None
        except Exception as err:                       # the headline must survive whatever happens here
            ep_ranks = {"error": f"{type(err).__name__}: {err}"[:300]}
        if watchdog:
            watchdog.cancel()

    if rank != 0:
        if dist.is_initialized():
            try:
                dist.destroy_process_group()
            except Exception:
                pass
        return

    peaks = measured_peaks()
    esz = 2 if w.dtype == wl.DTYPE_BF16 else 4
    twin = ep_line = variants = recipe = None
    if not forward_only_workload and not args.headline_only:
        twin = run_cdac_twin(w, x, dy, dev, ms_step, ms_fwd, max(3, min(args.steps, 10)), peaks, esz)
        ep_line = run_ep_on_one_gpu(w, x, dy, dev, ms_step, max(3, min(args.steps, 10)), esz) if w.dtype == wl.DTYPE_BF16 else None
        variants = run_small_variants(w, x, dy, dev, G, y, dx, step, max(3, min(args.steps, 10)))
        recipe = run_recipe_variant(w, x, dy, dev, G, y, dx, step, max(3, min(args.steps, 10)))
    decode_lat = run_decode_latencies(peaks) if (rank == 0 and not args.headline_only and w.dtype == wl.DTYPE_BF16
                                                 and not forward_only_workload) else None
    stages = {}
    gemm_ms = gemm_flops = 0.0
    flops_of = {name: fn(w) for name, fn in GEMM_FLOPS.items()}
    if "gemm_logits" not in prof["stages"]:         # gate logits computed by the descend launch
        flops_of["gemm_descend"] += flops_of["gemm_logits"]
    if "gemm_dx_gate" not in prof["stages"]:        # gate part fused into the dx contraction
        flops_of["gemm_dx"] += flops_of["gemm_dx_gate"]
    if "gemm_dw_gate" not in prof["stages"]:        # dW_gate computed together with dW_down
        flops_of["gemm_dw_down"] += flops_of["gemm_dw_gate"]
    bytes_of = {name: fn(w, esz) for name, fn in GEMM_BYTES.items()}
    if "gemm_logits" not in prof["stages"]:
        bytes_of["gemm_descend"] += esz * w.E * w.d + 4.0 * w.T * w.E
    if "gemm_dx_gate" not in prof["stages"]:
        bytes_of["gemm_dx"] += bytes_of["gemm_dx_gate"]
    if "gemm_dw_gate" not in prof["stages"]:
        bytes_of["gemm_dw_down"] += bytes_of["gemm_dw_gate"]
    gemm_bytes = 0.0
    for name, (ms, calls) in prof["stages"].items():
        per = ms / calls
        entry = {"ms": round(per, 4), "launches_per_step": calls // args.steps}
        if name in GEMM_FLOPS:
            fl = flops_of[name]
            entry["tflops"] = round(fl / (per * 1e-3) / 1e12, 1)
            entry["frac_of_measured_sustained"] = round(entry["tflops"] / peaks["tflops_sustained"], 3)
            gemm_ms += ms
            gemm_flops += fl * calls
            gemm_bytes += bytes_of[name] * calls
            entry["algorithmic_bytes"] = bytes_of[name]
            entry["hbm_gbs"] = round(bytes_of[name] / (per * 1e-3) / 1e9, 1)
            entry["frac_of_measured_hbm"] = round(entry["hbm_gbs"] / peaks["hbm_gbs"], 3)
        elif name in ROW_MOVE_BYTES:
            by = ROW_MOVE_BYTES[name](w, esz)
            entry["gbs"] = round(by / (per * 1e-3) / 1e9, 1)
            entry["frac_of_measured_hbm"] = round(entry["gbs"] / peaks["hbm_gbs"], 3)
        stages[name] = entry
    # the two groups the target names: the per-expert (grouped) contractions together, the row-move kernels together
    grouped = [n for n in ("gemm_expert1", "gemm_expert2", "gemm_dz", "gemm_dw2", "gemm_dxg", "gemm_dw1") if n in stages]
    g_ms = sum(stages[n]["ms"] for n in grouped)
    g_tf = sum(flops_of[n] for n in grouped) / (g_ms * 1e-3) / 1e12 if g_ms > 0 else 0.0
    moves = [n for n in ROW_MOVE_BYTES if n in stages]
    m_ms = sum(stages[n]["ms"] for n in moves)
    m_gbs = sum(ROW_MOVE_BYTES[n](w, esz) for n in moves) / (m_ms * 1e-3) / 1e9 if m_ms > 0 else 0.0
    groups = {"grouped_expert_gemms": {"ms": round(g_ms, 4), "tflops": round(g_tf, 1),
                                       "frac_of_measured_sustained": round(g_tf / peaks["tflops_sustained"], 3),
                                       "frac_of_measured_burst": round(g_tf / peaks["tflops_burst"], 3)},
              "dispatch_combine_and_their_backward": {"ms": round(m_ms, 4), "gbs": round(m_gbs, 1),
                                                      "frac_of_measured_hbm": round(m_gbs / peaks["hbm_gbs"], 3)}}
    achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    fwd_fl = forward_flops(w)
    all_gemms = {"kernels": "every tcgen05 contraction launch of a step", "launches_per_step": sum(stages[n]["launches_per_step"] for n in stages if n in GEMM_FLOPS),
                 "achieved": round(achieved, 1), "unit": "TFLOP/s", "frac": round(achieved / peaks["tflops_sustained"], 4),
                 "frac_of_burst_peak": round(achieved / peaks["tflops_burst"], 4), "ms_per_step": round(gemm_ms / args.steps, 4),
                 "algorithmic_bytes_per_step": gemm_bytes / args.steps}
    gemm_stages = [n for n in stages if n in GEMM_FLOPS]
    if forward_only_workload:
        # decode-shaped batches stream the touched weights once: the bound is HBM, not the tensor pipe
        roofline = {"bound": "hbm", "kernel": "inference forward (every launch of a call)",
                    "achieved": round(touched_bytes / (ms_fwd * 1e-3) / 1e9, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": round(touched_bytes / (ms_fwd * 1e-3) / 1e9 / peaks["hbm_gbs"], 4), "traffic": None,
                    "algorithmic_bytes": touched_bytes, "distinct_experts": n_distinct,
                    "peak_source": f"{peaks['source']}: copy bandwidth", "floor_us": round(touched_bytes / peaks["hbm_gbs"] / 1e3, 2)}
    elif gemm_stages:
        # the dominant kernel = the single launch that takes the most time of a step; all contractions together follow
        top = max(gemm_stages, key=lambda n: stages[n]["ms"])
        t = stages[top]
        roofline = {"bound": "tensor", "kernel": f"{top}: the longest launch of a step (tcgen05 contraction)",
                    "achieved": t["tflops"], "peak": peaks["tflops_sustained"], "unit": "TFLOP/s",
                    "frac": round(t["tflops"] / peaks["tflops_sustained"], 4),
                    "traffic": measured_traffic(top, w),
                    "traffic_source": ("ncu dram bytes of one launch on a small case of the same widths, scaled by rows"
                                       if measured_traffic(top, w) else None),
                    "algorithmic_bytes": t["algorithmic_bytes"], "ms": t["ms"], "hbm_gbs": t["hbm_gbs"],
                    "frac_of_measured_hbm": t["frac_of_measured_hbm"],
                    "peak_source": f"{peaks['source']}: sustained bf16 (kernels timed inside a long step)",
                    "frac_of_burst_peak": round(t["tflops"] / peaks["tflops_burst"], 4),
                    "all_gemm_launches": all_gemms,
                    "step_frac": round(3.0 * fwd_fl / (ms_step * 1e-3) / 1e12 / peaks["tflops_sustained"], 4)}
    else:
        roofline = {"bound": "alu", "kernel": "fp32 FMA path (correctness configuration, not a performance point)",
                    "achieved": None, "peak": None, "unit": "TFLOP/s", "frac": None, "traffic": None}

    rate, dt, S_used, cores = oracle_sample_rate(w, inp, args.ref_tokens or sample_size_for(w, inp, 15.0))
    bytes_io = (1 if forward_only_workload else 2) * w.T * w.d * esz
    line = {"metric": "bigmac_layer_fwd_tokens_per_s" if forward_only_workload else METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == wl.DTYPE_BF16 else "f32", "data": "synthetic",
            "config": config_dict(w, args), "clocks": clocks,
            "e2e": {"value": world * w.T / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": bytes_io,
                    "d2h_bytes_per_step": bytes_io, "ms_per_step": ms_e2e},
            "gpu_launches": prof["launches"],
            "repeats": repeats,
            "with_stage_events": {"ms_per_step": ms_step_events, "value": whole_job_tokens_per_s(w.T, world, ms_step_events), "unit": UNIT},
            "forward_only": {"tokens_per_s": world * w.T / (ms_fwd * 1e-3), "ms": ms_fwd,
                             "frac_of_tensor_roofline": round(fwd_fl / (ms_fwd * 1e-3) / 1e12 / peaks["tflops_sustained"], 4),
                             "cuda_graph_ms": ms_fwd_graph},
            "roofline": roofline,
            "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"first {S_used} tokens of the workload, routing + forward + backward with "
                                       f"every gradient, {dt:.1f} s"},
            "exchange": exchange,
            "cdac_twin": twin,
            "recipe_variant": recipe,
            "small_variants": variants,
            "decode_forward": decode_lat,
            "expert_parallel_on_one_gpu": ep_line,
            "groups": groups,
            "stages": stages}
    if ep_ranks is not None:
        line["expert_parallel"] = ep_ranks
    print(json.dumps(line), flush=True)
    if dist.is_initialized():
        try:
            dist.destroy_process_group()
        except Exception:
            pass


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="large", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--tokens", type=int, default=0, help="override T (per GPU)")
    ap.add_argument("--debug-set", action="append", default=[], metavar="NAME=VALUE",
                    help="measurement aid: set a kernel-choice switch of the library (bigmac_debug_set) before anything runs")
    ap.add_argument("--expert-parallel", action="store_true",
                    help="also run the expert-parallel layer over the job's ranks when there is only one (N > 1: always)")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the side measurements (Eq. 3 twin, expert-parallel ranks on one GPU, variants, recipe)")
    ap.add_argument("--profile-run", action="store_true",
                    help="only run warm-up + K steps (for a kernel-list or counter capture); prints no bench line")
    ap.add_argument("--ref-tokens", type=int, default=0,
                    help="token sample of the CPU-oracle leg (0: sized for about 15 s; reference arm: about 90 s in total)")
    args = ap.parse_args()
    w = wl.WORKLOADS[args.config]
    if args.tokens:
        w = w.with_tokens(args.tokens)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
