#!/usr/bin/env python
"""Benchmark of the MoDA attention operator on B200: one JSON line on stdout.

A "step" is one pass of the whole hot path for one attention layer over one batch of
synthetic inputs that are already resident in HBM: the forward kernel, which also does the
depth-cache "write" of the layer's own K, V (one slot), and the three backward launches (row-local part:
row terms, depth gradients, depth share of dQ; sequence part: dK, dV and the dQ tiles; dQ
finish).  `value` is forward+backward TFLOP/s with the FLOP convention of
paper_2603_15619_b200/flops.py (causal-halved sequence part + depth part, backward =
2.5 x forward).  Default workload: c4 (B=1, T=65536, H=16, d=128, l=24), the largest
configured workload at d = 128 and the one the 64K ratio target is stated on.

`roofline.targets` carries the numbers the targets are stated on: forward % of the measured
burst bf16 peak at T = 8192 for the six depths of c3, at c4 and at c5, and the ratio of the
MoDA kernels to the same kernels with l = 0 at c4.  Sweep rows go to stderr.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl moda|reference]
                    [--sweeps gqa,decode,prefill]

For N > 1 launch with torch.distributed.run, or let `--gpus N` spawn N local ranks itself;
every rank runs the same workload on its own GPU (independent batch shards, no collective
on the data path: weak scaling).
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

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_15619_b200 import flops, synthetic  # noqa: E402

METRIC = "MoDA fwd+bwd TFLOP/s (fwd and % of B200 BF16 peak vs T, ratio to own l=0 kernel: roofline.targets)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (bytes); keyed by (workload, kernel).  None where no capture exists.
NCU_SEQ_C3_L0_B1 = 202.45e6 + 92.27e6   # dram__bytes_read.sum + dram__bytes_write.sum of that one launch
NCU_TRAFFIC_BYTES = {
    # c2 captured at B=1 and scaled x4 (traffic is proportional to B): profiles/ncu_full_c2_B1_fwd_bwd_kernels.md
    ("c2", "fwd_append"): 4 * (822.179e6 + 6.956e6) + 4 * 33554432 * 2,   # + the slot written (not in that capture)
    # row-local part of the backward at c2, B = 1, scaled x4: profiles/ncu_full_c2_B1_bwd_rows_kernel.md
    ("c2", "bwd_rows"): 4 * (822.39e6 + 746.92e6),
    # sequence part of the backward, captured at c3 with l = 0 and B = 1 (T = 8192) and scaled by the number of
    # elements B T H d (every tensor crosses HBM once, re-reads are served by L2):
    # profiles/ncu_full_c3_l0_B1_bwd_fused_kernel.md
    ("c4", "bwd_seq"): 8 * NCU_SEQ_C3_L0_B1,
    ("c3_l0", "bwd_seq"): 2 * NCU_SEQ_C3_L0_B1,
}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        ident = str(device_index)
        try:
            ident = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid).replace("GPU-", "")
        except Exception:
            pass
        self.cmd = ["nvidia-smi", "-i", ident, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"]
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = [l for (t, l) in self.lines if t_begin - 0.05 <= t <= t_end + 0.15] or [l for (_, l) in self.lines]
        for l in rows:
            parts = [x.strip() for x in l.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def ev():
    return torch.cuda.Event(enable_timing=True)


# ---- multi-GPU plumbing: ranks work on independent shards (no collective on the data path) ----
def shard_seed(rank: int) -> int:
    """Seed of the synthetic shard that rank `rank` generates and processes (weak scaling: every
    rank holds one full per-GPU workload of its own)."""
    return int(rank)


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time: the job advances at the pace of its slowest shard."""
    if world <= 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, flops_per_rank_step: float, ms_per_step: float) -> float:
    """Whole-job TFLOP/s: every rank does `flops_per_rank_step` per step, in `ms_per_step`."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


class Layer:
    """Device buffers of one workload plus the calls of one step."""

    KERNELS = ("fwd_append", "bwd_rows", "bwd_seq", "bwd_finish")

    def __init__(self, w: synthetic.Workload, seed: int, device, with_backward: bool = True, e4m3: bool = False):
        import paper_2603_15619_b200 as moda
        self.moda, self.w, self.e4m3 = moda, w, e4m3
        self.q = synthetic.tensor(w, "Q", seed, 0, device)
        self.k = synthetic.tensor(w, "K", seed, 0, device)
        self.v = synthetic.tensor(w, "V", seed, 0, device)
        self.cache = self.dcache = None
        if w.l > 0:
            alloc, append = ((moda.alloc_depth_cache_e4m3, moda.moda_depth_cache_append_e4m3) if e4m3 else
                             (moda.alloc_depth_cache, moda.moda_depth_cache_append))
            self.cache = alloc(w.B, w.T, w.H, w.d, w.l, device)
            for i in range(w.l):
                append(self.cache, i, synthetic.tensor(w, "Kd", seed, i, device), synthetic.tensor(w, "Vd", seed, i, device))
        # slot this layer writes for later layers (same format as the cache it reads)
        self.next_slot = (moda.alloc_depth_cache_e4m3 if e4m3 else moda.alloc_depth_cache)(w.B, w.T, w.H, w.d, 1, device)
        self.O = torch.empty_like(self.q)
        self.LSE = torch.empty((w.B, w.H, w.T), dtype=torch.float32, device=device)
        if with_backward:
            self.dO = synthetic.tensor(w, "dO", seed, 0, device)
            if w.l > 0:
                self.dcache = moda.alloc_depth_cache(w.B, w.T, w.H, w.d, w.l, device)
            self.dQ, self.dK, self.dV = (torch.empty_like(self.q) for _ in range(3))
            self.ws = torch.empty(moda.moda_bwd_workspace_bytes(w.B, w.T, w.H, w.d, w.l), dtype=torch.uint8, device=device)

    def fwd_append(self):
        """Forward with the depth stream's write step fused in: this layer's K, V go to the slot the later layers read."""
        f = self.moda.moda_attn_fwd_append_e4m3 if self.e4m3 else self.moda.moda_attn_fwd_append
        f(self.q, self.k, self.v, self.cache, self.w.l, self.w.scale, self.next_slot, 0, O=self.O, LSE=self.LSE)

    def fwd(self):
        f = self.moda.moda_attn_fwd_e4m3 if self.e4m3 else self.moda.moda_attn_fwd
        f(self.q, self.k, self.v, self.cache, self.w.l, self.w.scale, O=self.O, LSE=self.LSE)

    def bwd(self, stages=None):
        if self.e4m3:
            self.moda.moda_attn_bwd_e4m3(self.q, self.k, self.v, self.cache, self.O, self.dO, self.LSE, self.w.l, self.w.scale,
                                         dQ=self.dQ, dK=self.dK, dV=self.dV, d_depth_kv=self.dcache, workspace=self.ws)
            return
        self.moda.moda_attn_bwd(self.q, self.k, self.v, self.cache, self.O, self.dO, self.LSE, self.w.l, self.w.scale,
                                dQ=self.dQ, dK=self.dK, dV=self.dV, d_depth_kv=self.dcache, workspace=self.ws, stages=stages)

    def step(self, events=None):
        """One pass of the hot path; with `events` (5 CUDA events) records one between launches."""
        calls = (self.fwd_append, lambda: self.bwd(1), lambda: self.bwd(2), lambda: self.bwd(4))
        if events is None:
            self.fwd_append(); self.bwd()
            return
        events[0].record()
        for i, c in enumerate(calls):
            c()
            events[i + 1].record()

    # algorithmic HBM bytes / FLOPs per launch (every tensor moved once)
    def kernel_model(self):
        w = self.w
        E = w.B * w.T * w.H * w.d
        rows = w.B * w.H * w.T
        f_fwd = flops.fwd_flops(w.B, w.T, w.H, w.d, w.l)
        seq = flops.fwd_flops(w.B, w.T, w.H, w.d, 0)
        dep = flops.depth_fwd_flops(w.B, w.T, w.H, w.d, w.l)
        return {
            # the forward's own bytes plus the slot it writes (K and V once more, in cache layout)
            "fwd_append": {"bytes": flops.fwd_bytes(w.B, w.T, w.H, w.d, w.l) + 2.0 * 2 * E, "flops": f_fwd},
            # reads Q O dO (bf16), LSE and the depth cache; writes the row terms, the depth gradients and the fp32 dQ accumulator
            "bwd_rows": {"bytes": 2.0 * (3 * E + 4 * w.l * E) + 4.0 * E + 8.0 * rows, "flops": 2.0 * E + 2.5 * dep},
            # reads Q K V dO + LSE, D; writes dK dV; reads and writes the fp32 dQ accumulator; the five sequence contractions
            "bwd_seq": {"bytes": 2.0 * 6 * E + 2 * 4.0 * E + 8.0 * rows, "flops": 2.5 * seq},
            "bwd_finish": {"bytes": 4.0 * E + 2.0 * E, "flops": 0.0},
        }


def pick_workload(args):
    import dataclasses
    w = synthetic.WORKLOADS[args.workload.split("_")[0]]
    if "_l" in args.workload:
        w = w.with_l(int(args.workload.split("_l")[1]))
    if args.batch > 0:
        w = dataclasses.replace(w, B=args.batch, name=f"{w.name}_B{args.batch}")
    return w


def run_moda(args, rank, world, device):
    import paper_2603_15619_b200 as moda
    peaks = load_peaks()
    w = pick_workload(args)
    layer = Layer(w, seed=shard_seed(rank), device=device)

    def barrier():
        if world > 1:
            torch.distributed.barrier()

    W = max(args.warmup, 3)
    for _ in range(W):
        layer.step()
    torch.cuda.synchronize()
    if moda.moda_last_status() != 0:
        raise RuntimeError(f"device status {moda.moda_last_status()} after warm-up")

    K = args.steps
    evs = [[ev() for _ in range(5)] for _ in range(K)]
    sampler = ClockSampler(device.index)
    sampler.start()
    time.sleep(0.3)
    barrier()
    torch.cuda.synchronize()
    t_begin = time.time()
    for s in range(K):
        layer.step(evs[s])
    torch.cuda.synchronize()
    t_end = time.time()
    barrier()
    clocks = sampler.stop(t_begin, t_end)
    total_ms = evs[0][0].elapsed_time(evs[-1][4])
    ms_per_step = total_ms / K
    ms_per_step = max_over_ranks(ms_per_step, world, device)
    status = moda.moda_last_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")

    per_kernel = {}
    for i, name in enumerate(Layer.KERNELS):
        per_kernel[name] = sum(e[i].elapsed_time(e[i + 1]) for e in evs) / K
    step_flops = flops.fwd_bwd_flops(w.B, w.T, w.H, w.d, w.l)
    value = job_value(world, step_flops, ms_per_step)

    # ---- roofline of the dominant kernel ----
    model = layer.kernel_model()
    dom = max(per_kernel, key=per_kernel.get)
    dur = per_kernel[dom] * 1e-3
    long_region = (t_end - t_begin) > 1.0        # a kernel timed inside a seconds-long step runs under the power cap
    tensor_peak = peaks["bf16_tflops_sustained"] if long_region else peaks["bf16_tflops"]
    t_hbm = model[dom]["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tensor = model[dom]["flops"] / (tensor_peak * 1e12)
    if t_hbm >= t_tensor:
        roof = {"bound": "hbm", "achieved": model[dom]["bytes"] / dur / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": model[dom]["flops"] / dur / 1e12, "peak": tensor_peak, "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get((w.name, dom))
    mhz = clocks.get("sm_mhz")
    roof.update({"kernel": dom, "kernel_ms": round(per_kernel[dom], 4), "peak_source": peaks["source"],
                 "peak_kind": ("sustained" if long_region else "burst") if roof["bound"] == "tensor" else "copy",
                 "algorithmic_bytes": model[dom]["bytes"], "algorithmic_flops": model[dom]["flops"],
                 "kernel_ms_x_sm_mhz": None if mhz is None else round(per_kernel[dom] * mhz, 1)})

    fwd_tflops = flops.fwd_flops(w.B, w.T, w.H, w.d, w.l) / (per_kernel["fwd_append"] * 1e-3) / 1e12
    bwd_ms = per_kernel["bwd_rows"] + per_kernel["bwd_seq"] + per_kernel["bwd_finish"]
    detail = {
        "kernel_ms": {k: round(v, 4) for k, v in per_kernel.items()},
        "fwd_tflops": round(fwd_tflops, 1),
        "bwd_tflops": round(flops.bwd_flops(w.B, w.T, w.H, w.d, w.l) / (bwd_ms * 1e-3) / 1e12, 1),
        "bwd_over_fwd_time": round(bwd_ms / per_kernel["fwd_append"], 3),
        "fwd_frac_of_measured_burst_bf16": round(fwd_tflops / peaks["bf16_tflops"], 4),
        "fwd_frac_of_measured_sustained_bf16": round(fwd_tflops / peaks["bf16_tflops_sustained"], 4),
        "flops": "fwd = 4BHd T^2/2 + 4BHTld; bwd = 2.5 fwd",
    }
    log("detail", {"fwd_depth_read_gbs": round(flops.depth_bytes_fwd(w.B, w.T, w.H, w.d, w.l) / (per_kernel["fwd_append"] * 1e-3) / 1e9, 1),
                   "ms_per_step_x_sm_mhz": None if mhz is None else round(ms_per_step * mhz, 1)})

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: B={w.B} T={w.T} H={w.H} d={w.d} l={w.l} (per GPU), bf16 N(0,1) inputs, fp32 accumulate",
                   "step": "forward (writes the layer's own K, V as the next depth slot) + backward (row-local part incl. "
                           "depth gradients, sequence part dK/dV/dQ tiles, dQ finish)",
                   "l2_policy": "inputs larger than L2 (depth cache %.2f GiB + 4 x %.0f MiB activations per step)"
                                % (flops.depth_bytes_fwd(w.B, w.T, w.H, w.d, w.l) / 2 ** 30, w.B * w.T * w.H * w.d * 2 / 2 ** 20),
                   "parallelism": f"independent batch shards x{world}, no collective"},
        "roofline": roof, "clocks": clocks, "gpu_launches": 4 * K, "detail": detail,
    }

    headline = {"fwd_ms": per_kernel["fwd_append"], "bwd_ms": bwd_ms}
    if not args.no_e2e:
        out["e2e"] = run_e2e(layer, args.e2e_steps, world, step_flops, device)
    del layer
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_sweep:
        roof["targets"] = run_targets(peaks, device, w, headline)
        extra = [x for x in args.sweeps.split(",") if x]
        if "gqa" in extra:
            out["gqa_sweep"] = run_gqa_sweep(device)
        if "decode" in extra:
            out["decode_sweep"] = run_decode_sweep(peaks, device)
        if "prefill" in extra:
            out["prefill_sweep"] = run_prefill_sweep(peaks, device)
        if "kvproj" in extra:
            out["kvproj_sweep"] = run_kvproj_sweep(peaks, device)
        if "mass" in extra:
            out["mass_sweep"] = run_mass_sweep(peaks, device)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w, budget_s=20.0)
    return out


def time_calls(fn, iters, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = ev(), ev()
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / iters


def run_targets(peaks, device, headline_w, headline):
    """The points the throughput targets are stated on, each timed alone (burst clocks) with its l = 0 twin:
    forward % of the measured burst bf16 peak at T = 8192 for the six depths of c3, at c4 (T = 65536) and at c5
    (T = 32768, d = 64); ratio of the MoDA kernels to the same kernels with l = 0 at c4 (forward, and forward +
    backward).  Each row also says what bounds its forward: the slower of the algorithmic HBM bytes at the measured
    copy rate and the credited FLOPs at the measured cuBLAS rate."""
    W = synthetic.WORKLOADS
    plan = [(f"c3_l{l}", W["c3"].with_l(l), 8, True) for l in synthetic.C3_DEPTHS] + \
           [("c4", W["c4"], 3, True), ("c5", W["c5"], 3, True)]
    timed = {}

    def timings(ww, iters, bwd, e4m3=False):
        key = (ww.B, ww.T, ww.H, ww.d, ww.l, e4m3)
        if key not in timed:
            torch.cuda.empty_cache()
            layer = Layer(ww, seed=0, device=device, with_backward=bwd, e4m3=e4m3)
            f_ms = time_calls(layer.fwd, iters)
            b_ms = time_calls(layer.bwd, iters) if bwd else None
            timed[key] = (f_ms, b_ms)
            del layer
        return timed[key]

    rows = {}
    for name, w, iters, bwd in plan:
        f_ms, b_ms = timings(w, iters, bwd)
        f0, b0 = timings(w.with_l(0), iters, bwd)
        ff = flops.fwd_flops(w.B, w.T, w.H, w.d, w.l)
        t_tensor = ff / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_hbm = flops.fwd_bytes(w.B, w.T, w.H, w.d, w.l) / (peaks["hbm_gbs"] * 1e9) * 1e3
        t_tensor_b = 2.5 * ff / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_hbm_b = flops.bwd_bytes(w.B, w.T, w.H, w.d, w.l) / (peaks["hbm_gbs"] * 1e9) * 1e3
        full = {
            "fwd_ms": round(f_ms, 4), "fwd_tflops": round(ff / f_ms / 1e9, 1),
            "fwd_pct_of_burst_peak": round(100.0 * ff / f_ms / 1e9 / peaks["bf16_tflops"], 1),
            "fwd_bound": "hbm" if t_hbm > t_tensor else "tensor",
            "fwd_frac_of_roofline": round(max(t_tensor, t_hbm) / f_ms, 3),
            "roofline_cap_pct_of_burst_peak": round(100.0 * t_tensor / max(t_tensor, t_hbm), 1),
            "bwd_ms": round(b_ms, 4), "bwd_frac_of_roofline": round(max(t_tensor_b, t_hbm_b) / b_ms, 3),
            "bwd_over_fwd_time": round(b_ms / f_ms, 2),
            "fwd_ratio_to_l0": round(f0 / f_ms, 3), "fwd_bwd_ratio_to_l0": round((f0 + b0) / (f_ms + b_ms), 3),
            "l0_fwd_ms": round(f0, 4), "l0_bwd_ms": round(b0, 4),
        }
        log("target", name, full)
        # the line on stdout keeps the figures the targets are stated on (the full row went to stderr)
        rows[name] = {k: full[k] for k in ("fwd_ms", "fwd_pct_of_burst_peak", "fwd_bound", "fwd_frac_of_roofline",
                                            "bwd_ms", "bwd_frac_of_roofline", "fwd_ratio_to_l0", "fwd_bwd_ratio_to_l0")}
    # The same kernels on a depth cache kept in e4m3 with a scale per row (half the depth bytes), at the depth-heavy
    # points: the roofline is recomputed with the smaller cache.
    for name, w, iters in [(f"c3_l{l}_e4m3", W["c3"].with_l(l), 8) for l in (16, 24, 32)] + [("c4_e4m3", W["c4"], 3)]:
        f_ms, b_ms = timings(w, iters, True, e4m3=True)
        f0, b0 = timings(w.with_l(0), iters, True)
        ff = flops.fwd_flops(w.B, w.T, w.H, w.d, w.l)
        cache16 = 2.0 * 2 * w.l * w.B * w.T * w.H * w.d
        cache8 = cache16 / 2 + 2.0 * 4 * w.l * w.B * w.T * w.H
        t_tensor = ff / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_hbm = (flops.fwd_bytes(w.B, w.T, w.H, w.d, w.l) - cache16 + cache8) / (peaks["hbm_gbs"] * 1e9) * 1e3
        full = {"fwd_ms": round(f_ms, 4), "fwd_pct_of_burst_peak": round(100.0 * ff / f_ms / 1e9 / peaks["bf16_tflops"], 1),
                "fwd_frac_of_roofline": round(max(t_tensor, t_hbm) / f_ms, 3), "bwd_ms": round(b_ms, 4)}
        full.update({"fwd_ratio_to_l0": round(f0 / f_ms, 3), "fwd_bwd_ratio_to_l0": round((f0 + b0) / (f_ms + b_ms), 3)})
        log("target", name, full)
        if name in ("c3_l32_e4m3", "c4_e4m3"):              # the other two rows go to stderr only (line length)
            rows[name] = {k: full[k] for k in ("fwd_ms", "fwd_pct_of_burst_peak", "bwd_ms", "fwd_bwd_ratio_to_l0")}
    torch.cuda.empty_cache()
    return rows


# Rows of the paper's kernel table (Table 2: B = 1, d = 64, 8 key/value heads, G query heads per
# key/value head, L depth slots; sweeps over T, over G and over L) as (T, G, L, extra time of MoDA
# over the depth-free kernel that the table prints for an A100 with Triton kernels, in percent --
# context, not a target).
GQA_SHAPES = [(4096, 8, 64, 25.86), (8192, 8, 64, 18.99), (16384, 8, 64, 8.59), (32768, 8, 64, 4.38),
              (65536, 8, 64, 2.73), (16384, 2, 64, 27.07), (16384, 4, 64, 15.76), (16384, 16, 64, 4.57),
              (16384, 32, 64, 2.84), (16384, 8, 128, 15.57), (16384, 8, 256, 30.52)]


def run_gqa_sweep(device, shapes=None):
    """Grouped-query forward + backward at the paper's Table 2 shapes, with the l = 0 twin."""
    import paper_2603_15619_b200 as moda
    rows = []
    B, d, Hk = 1, 64, 8
    base_cache = {}
    for T, G, l_full, paper_pct in (shapes or GQA_SHAPES):
        H = Hk * G
        res = {}
        for l in (0, l_full):
            if l == 0 and (T, G) in base_cache:
                res[0] = base_cache[(T, G)]
                continue
            torch.cuda.empty_cache()
            x = synthetic.make_gqa(B, T, H, Hk, d, 0, seed=0, device=device)
            cache = dcache = None
            if l > 0:
                wk = synthetic.Workload("gqa/kv", B, T, Hk, d, l)
                cache = moda.alloc_depth_cache(B, T, Hk, d, l, device)
                dcache = moda.alloc_depth_cache(B, T, Hk, d, l, device)
                for i in range(l):
                    moda.moda_depth_cache_append(cache, i, synthetic.tensor(wk, "Kd", 0, i, device),
                                                 synthetic.tensor(wk, "Vd", 0, i, device))
            O = torch.empty_like(x["Q"])
            LSE = torch.empty((B, H, T), dtype=torch.float32, device=device)
            dQ, dK, dV = torch.empty_like(x["Q"]), torch.empty_like(x["K"]), torch.empty_like(x["V"])
            ws = torch.empty(moda.moda_bwd_workspace_bytes_gqa(B, T, H, Hk, d, l), dtype=torch.uint8, device=device)
            scale = d ** -0.5
            fwd = lambda: moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], cache, l, scale, O=O, LSE=LSE)
            bwd = lambda: moda.moda_attn_bwd_gqa(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale,
                                                 dQ=dQ, dK=dK, dV=dV, d_depth_kv=dcache, workspace=ws)
            iters = 2 if T >= 32768 else 5
            res[l] = (time_calls(fwd, iters), time_calls(bwd, iters))
            if l == 0:
                base_cache[(T, G)] = res[0]
            elif G > 1:
                # the same call with the depth cache (and the depth gradients) in the position-major layout
                for i in range(l):
                    moda.moda_depth_cache_append_pm(cache, i, synthetic.tensor(wk, "Kd", 0, i, device),
                                                    synthetic.tensor(wk, "Vd", 0, i, device))
                fwd_pm = lambda: moda.moda_attn_fwd_gqa_pm(x["Q"], x["K"], x["V"], cache, l, scale, O=O, LSE=LSE)
                bwd_pm = lambda: moda.moda_attn_bwd_gqa_pm(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale,
                                                           dQ=dQ, dK=dK, dV=dV, d_depth_kv_pm=dcache, workspace=ws)
                res["pm"] = (time_calls(fwd_pm, iters), time_calls(bwd_pm, iters))
            del x, cache, dcache, O, LSE, dQ, dK, dV, ws
        (f0, b0), (f1, b1) = res[0], res[l_full]
        ff = 4.0 * B * H * d * (T * (T + 1) / 2) + 4.0 * B * H * T * l_full * d
        rows.append({"B": B, "T": T, "H": H, "H_kv": Hk, "G": G, "d": d, "l": l_full,
                     "fwd_ms": round(f1, 4), "bwd_ms": round(b1, 4), "fwd_bwd_ms": round(f1 + b1, 4),
                     "l0_fwd_bwd_ms": round(f0 + b0, 4),
                     "extra_time_pct": round(100.0 * ((f1 + b1) / (f0 + b0) - 1.0), 2),
                     "paper_extra_time_pct_a100_triton": paper_pct,
                     "fwd_bwd_ratio_to_l0": round((f0 + b0) / (f1 + b1), 4),
                     "fwd_tflops": round(ff / f1 / 1e9, 1), "fwd_bwd_tflops": round(3.5 * ff / (f1 + b1) / 1e9, 1)})
        if "pm" in res:
            fp, bp = res["pm"]
            cache_bytes = 2.0 * 2 * l_full * B * T * Hk * d
            rows[-1].update({"pm_fwd_ms": round(fp, 4), "pm_bwd_ms": round(bp, 4),
                             "pm_extra_time_pct": round(100.0 * ((fp + bp) / (f0 + b0) - 1.0), 2),
                             # depth part alone (time over the l = 0 twin) against the bytes it must move: the cache once
                             # (forward), the cache and its gradients (backward), plus Q / O (dO, dQ) of all heads once each
                             "pm_depth_fwd_gbs": round((cache_bytes + 3 * 2.0 * B * T * H * d) / max(fp - f0, 1e-6) / 1e6, 0),
                             "pm_depth_bwd_gbs": round((2 * cache_bytes + 4 * 2.0 * B * T * H * d) / max(bp - b0, 1e-6) / 1e6, 0)})
        log("gqa_sweep", rows[-1])
    torch.cuda.empty_cache()
    return rows


# Decode step (T_q = 1): B sequences x T_kv cached positions; the paper's 700M / 1.5B models use G = 2.
# (B, T_kv, H, H_kv, d, l); every KV cache here is larger than L2.
DECODE_SHAPES = [
    (1, 8192, 16, 8, 128, 24), (8, 8192, 16, 8, 128, 24),
    (32, 8192, 16, 16, 128, 24), (32, 8192, 16, 8, 128, 24), (32, 8192, 32, 8, 128, 24), (32, 8192, 64, 8, 128, 24),
    (64, 8192, 16, 8, 64, 32), (128, 2048, 16, 8, 128, 24), (2, 131072, 16, 8, 128, 24),
]


def run_decode_sweep(peaks, device, shapes=None, iters=20):
    """One decode step per shape: time of the two launches and the HBM bytes they must move (K and V of the
    cached positions once, the token's depth pairs, q and O) against the measured copy bandwidth."""
    import paper_2603_15619_b200 as moda
    rows = []
    for B, T, H, Hk, d, l in (shapes or DECODE_SHAPES):
        torch.cuda.empty_cache()
        # Steps are queued back to back (a step is shorter than the host's launch path when timed alone) and
        # rotate over copies of the KV cache that together exceed L2 several times, so every step reads HBM.
        kv_bytes = 2 * B * T * Hk * d * 2
        n_sets = max(2, int(1.0e9 // kv_bytes) + 1) if kv_bytes < 1.0e9 else 1
        sets = [synthetic.make_decode(B, T, H, Hk, d, l, seed=i, device=device) for i in range(n_sets)]
        O = torch.empty_like(sets[0]["q"])
        LSE = torch.empty((B, H), dtype=torch.float32, device=device)
        ws = torch.empty(moda.moda_decode_workspace_bytes(B, H, d), dtype=torch.uint8, device=device)

        def fn(i):
            x = sets[i % n_sets]
            moda.moda_attn_decode(x["q"], x["K"], x["V"], x["depth"] if l else None, T, l, d ** -0.5,
                                  O=O, LSE=LSE, workspace=ws)
        for i in range(max(3, n_sets)):
            fn(i)
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for i in range(iters):
            fn(i)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / iters
        # The same steps replayed from a CUDA graph: device time without the host's launch path, which is
        # longer than a small-batch step (about 20 us per step through the Python binding).
        ms_graph = None
        try:
            per_graph = max(4, n_sets)
            side = torch.cuda.Stream(device=device)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(per_graph):
                        fn(i)
                graph.replay()
                side.synchronize()
                a, b = ev(), ev()
                a.record(side)
                reps = max(1, iters // per_graph)
                for _ in range(reps):
                    graph.replay()
                b.record(side)
                side.synchronize()
                ms_graph = a.elapsed_time(b) / (reps * per_graph)
            del graph
        except Exception as e:          # capture not possible here: keep the eagerly launched number
            log("decode_sweep: graph replay unavailable:", repr(e)[:200])
        if ms_graph is not None and ms_graph < ms:
            ms_eager, ms = ms, ms_graph
        else:
            ms_eager = ms
        # the same cache seen as 64-position pages in a shuffled order (host launches, rotating sets)
        paged_us = None
        if T % 64 == 0:
            blocks = T // 64
            gen = torch.Generator(device=device).manual_seed(7)
            tables = [torch.randperm(B * blocks, generator=gen, device=device).to(torch.int32).view(B, blocks).contiguous()
                      for _ in range(n_sets)]
            lens = torch.full((B,), T, dtype=torch.int32, device=device)

            def fn_paged(i):
                x = sets[i % n_sets]
                moda.moda_attn_decode_paged(x["q"], x["K"].view(B * blocks, 64, Hk, d), x["V"].view(B * blocks, 64, Hk, d),
                                            tables[i % n_sets], lens, x["depth"] if l else None, T, l, d ** -0.5,
                                            O=O, LSE=LSE, workspace=ws)
            paged_us = time_calls(lambda c=[0]: (fn_paged(c[0]), c.__setitem__(0, c[0] + 1)), iters, warm=max(3, n_sets)) * 1e3
        byt = 2 * B * T * Hk * d * 2 + 2 * l * B * Hk * d * 2 + 2 * B * H * d * 2
        gbs = byt / ms / 1e6
        rows.append({"B": B, "T_kv": T, "H": H, "H_kv": Hk, "G": H // Hk, "d": d, "l": l, "us": round(ms * 1e3, 1),
                     "us_launched_from_host": round(ms_eager * 1e3, 1), "timed": "cuda graph replay" if ms is not ms_eager else "host launches",
                     "us_paged_64_host_launches": None if paged_us is None else round(paged_us, 1),
                     "algorithmic_GB": round(byt / 1e9, 3), "GBps": round(gbs, 0),
                     "ratio_to_measured_copy_rate": round(gbs / peaks["hbm_gbs"], 3),   # a read-only stream can beat a read+write copy
                     "tokens_per_s": round(B / ms * 1e3, 0)})
        log("decode_sweep", rows[-1])
        del sets, O, LSE, ws
    torch.cuda.empty_cache()
    return rows


# Prefill with a cache: a chunk of T_q new positions over T_kv cached keys (B, T_q, T_kv, H, H_kv, d, l).
PREFILL_SHAPES = [(4, 2048, 16384, 16, 8, 128, 24), (1, 8192, 65536, 16, 8, 128, 24), (4, 2048, 16384, 32, 8, 64, 32)]


def run_prefill_sweep(peaks, device, shapes=None, iters=5):
    """Forward of a chunk against a long cached prefix; FLOPs = 4 d per (query row, visible key) pair."""
    import paper_2603_15619_b200 as moda
    rows = []
    for B, Tq, Tkv, H, Hk, d, l in (shapes or PREFILL_SHAPES):
        torch.cuda.empty_cache()
        wq = synthetic.Workload("prefill/q", B, Tq, H, d, l)
        wk = synthetic.Workload("prefill/kv", B, Tkv, Hk, d, l)
        wd = synthetic.Workload("prefill/depth", B, Tq, Hk, d, l)
        Q = synthetic.tensor(wq, "Q", 0, 0, device)
        K = synthetic.tensor(wk, "K", 0, 0, device)
        V = synthetic.tensor(wk, "V", 0, 0, device)
        cache = None
        if l > 0:
            cache = moda.alloc_depth_cache(B, Tq, Hk, d, l, device)
            for i in range(l):
                moda.moda_depth_cache_append(cache, i, synthetic.tensor(wd, "Kd", 0, i, device), synthetic.tensor(wd, "Vd", 0, i, device))
        O = torch.empty_like(Q)
        LSE = torch.empty((B, H, Tq), dtype=torch.float32, device=device)
        fn = lambda: moda.moda_attn_fwd_prefill(Q, K, V, cache, l, d ** -0.5, O=O, LSE=LSE)
        ms = time_calls(fn, iters)
        off = Tkv - Tq
        pairs = Tq * (off + 1) + Tq * (Tq - 1) / 2 + Tq * l
        fl = 4.0 * B * H * d * pairs
        rows.append({"B": B, "T_q": Tq, "T_kv": Tkv, "H": H, "H_kv": Hk, "d": d, "l": l, "ms": round(ms, 4),
                     "tflops": round(fl / ms / 1e9, 1), "frac_measured_burst_bf16": round(fl / ms / 1e9 / peaks["bf16_tflops"], 4)})
        log("prefill_sweep", rows[-1])
        del Q, K, V, cache, O, LSE
    torch.cuda.empty_cache()
    return rows


# Key / value projection with the write step in its epilogue (B, T, D_model, H_kv, d).
KVPROJ_SHAPES = [(1, 65536, 2048, 16, 128), (2, 8192, 2048, 16, 128), (2, 32768, 2048, 32, 64), (1, 16384, 4096, 8, 128)]


def run_kvproj_sweep(peaks, device, shapes=None, iters=10):
    """K = X Wk^T, V = X Wv^T plus the depth slot in one launch; FLOPs = 2 * positions * D_model * 2 H_kv d.  The library
    columns (one GEMM on the concatenated weights, then the separate append) are what the fused launch replaces."""
    import paper_2603_15619_b200 as moda
    rows = []
    for B, T, Dm, Hk, d in (shapes or KVPROJ_SHAPES):
        torch.cuda.empty_cache()
        g = torch.Generator(device=device).manual_seed(0)
        X = torch.randn((B, T, Dm), device=device, generator=g).to(torch.bfloat16)
        Wk = (torch.randn((Hk * d, Dm), device=device, generator=g) * Dm ** -0.5).to(torch.bfloat16)
        Wv = (torch.randn((Hk * d, Dm), device=device, generator=g) * Dm ** -0.5).to(torch.bfloat16)
        cache = moda.alloc_depth_cache(B, T, Hk, d, 1, device)
        K = torch.empty((B, T, Hk, d), dtype=torch.bfloat16, device=device)
        V = torch.empty_like(K)
        Wkv = torch.cat([Wk, Wv], 0)
        ms = time_calls(lambda: moda.moda_kv_project_append(X, Wk, Wv, Hk, cache=cache, slot=0, K_out=K, V_out=V), iters)
        ms_slot = time_calls(lambda: moda.moda_kv_project_append(X, Wk, Wv, Hk, cache=cache, slot=0, store_kv=False), iters)
        cache8 = moda.alloc_depth_cache_e4m3(B, T, Hk, d, 1, device)
        ms_e4m3 = time_calls(lambda: moda.moda_kv_project_append_e4m3(X, Wk, Wv, Hk, cache=cache8, slot=0, K_out=K, V_out=V), iters)
        del cache8
        ms_lib = time_calls(lambda: torch.nn.functional.linear(X, Wkv), iters)
        ms_app = time_calls(lambda: moda.moda_depth_cache_append(cache, 0, K, V), iters)
        fl = 2.0 * B * T * Dm * 2 * Hk * d
        rows.append({"B": B, "T": T, "D_model": Dm, "H_kv": Hk, "d": d, "ms": round(ms, 4), "tflops": round(fl / ms / 1e9, 1),
                     "frac_measured_burst_bf16": round(fl / ms / 1e9 / peaks["bf16_tflops"], 4),
                     "slot_only_ms": round(ms_slot, 4), "e4m3_slot_ms": round(ms_e4m3, 4), "library_gemm_ms": round(ms_lib, 4), "separate_append_ms": round(ms_app, 4)})
        log("kvproj_sweep", rows[-1])
        del X, Wk, Wv, Wkv, cache, K, V
    torch.cuda.empty_cache()
    return rows


def run_mass_sweep(peaks, device, names=("c3_l32", "c4", "c5"), batch=0, iters=10):
    """Attention mass of the depth slots (moda_depth_slot_mass): one pass over the depth keys; bytes = l E + E."""
    import dataclasses
    import paper_2603_15619_b200 as moda
    rows = []
    for nm in names:
        w = synthetic.WORKLOADS[nm.split("_")[0]]
        if "_l" in nm:
            w = w.with_l(int(nm.split("_l")[1]))
        if batch:
            w = dataclasses.replace(w, B=batch)
        torch.cuda.empty_cache()
        L = Layer(w, 0, device, with_backward=False)
        L.fwd()
        mass = torch.empty((w.B, w.H, w.l), dtype=torch.float32, device=device)
        ws = torch.empty((max(16, moda.binding.load().moda_depth_slot_mass_workspace_bytes(w.B, w.T, w.H, w.l)),), dtype=torch.uint8, device=device)
        ms = time_calls(lambda: moda.moda_depth_slot_mass(L.q, L.cache, L.LSE, w.l, w.scale, mass=mass, workspace=ws), iters)
        byts = (w.l + 1) * w.B * w.T * w.H * w.d * 2
        rows.append({"workload": nm, "B": w.B, "ms": round(ms, 4), "gbs": round(byts / ms / 1e6, 1),
                     "frac_measured_copy": round(byts / ms / 1e6 / peaks["hbm_gbs"], 4),
                     "depth_share_of_probability": round(float(mass.sum()) / (w.B * w.H * w.T), 5)})
        log("mass_sweep", rows[-1])
        del L, mass, ws
    torch.cuda.empty_cache()
    return rows


def run_e2e(layer, steps, world, step_flops, device):
    """The same step driven from pinned HOST buffers: every step copies its inputs host->device and
    its results device->host inside the timed region.  Two device buffer sets and three streams let
    the upload of step i+1 and the download of step i-1 run beside the kernels of step i, as a caller
    that streams batches through the library would; every step still moves all of its bytes."""
    sets = [layer, Layer(layer.w, seed=1, device=device)]
    tensors_in = lambda L: [L.q, L.k, L.v, L.dO] + ([L.cache] if L.cache is not None else [])
    tensors_out = lambda L: [L.O, L.LSE, L.dQ, L.dK, L.dV] + ([L.dcache] if L.dcache is not None else [])
    ins, outs = [tensors_in(L) for L in sets], [tensors_out(L) for L in sets]
    h_in = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in ins[0]]
    h_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs[0]]
    s_in, s_run, s_out = (torch.cuda.Stream(device=device) for _ in range(3))
    done_in = [torch.cuda.Event() for _ in range(2)]
    done_run = [torch.cuda.Event() for _ in range(2)]
    done_out = [torch.cuda.Event() for _ in range(2)]

    def one(i):
        k = i % 2
        with torch.cuda.stream(s_in):
            s_in.wait_event(done_run[k])            # the kernels of step i-2 have finished with this set's inputs
            for d, h in zip(ins[k], h_in):
                d.copy_(h, non_blocking=True)
            done_in[k].record(s_in)
        with torch.cuda.stream(s_run):
            s_run.wait_event(done_in[k])
            s_run.wait_event(done_out[k])           # the results of step i-2 have left this set's outputs
            sets[k].step()
            done_run[k].record(s_run)
        with torch.cuda.stream(s_out):
            s_out.wait_event(done_run[k])
            for h, d in zip(h_out, outs[k]):
                h.copy_(d, non_blocking=True)
            done_out[k].record(s_out)

    torch.cuda.synchronize()
    for i in range(2):
        one(i)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    a, b = ev(), ev()
    a.record(s_in)
    for i in range(steps):
        one(i)
    b.record(s_out)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    ms = max_over_ranks(ms, world, device)
    nbytes = lambda ts: int(sum(t.numel() * t.element_size() for t in ts))
    return {"value": round(job_value(world, step_flops, ms), 3), "unit": UNIT, "ms_per_step": round(ms, 3),
            "steps": steps, "h2d_bytes_per_step": nbytes(ins[0]), "d2h_bytes_per_step": nbytes(outs[0]),
            "overlap": "copies double-buffered beside the kernels"}


def cpu_sample(w, T_sample, seed=0):
    """One (b, h) slice of workload `w`, cut to its first `T_sample` positions, as float64 numpy arrays.  Heads are
    independent and causal attention over a prefix is the operator on that prefix, so this is a bounded piece of the
    same workload: same head width, depth, value recipe; drawn from the same seeded generators at the reduced shape."""
    import dataclasses
    import numpy as np
    ws = dataclasses.replace(w, B=1, H=1, T=int(T_sample), name=f"{w.name}/cpu-sample")
    f64 = lambda t: t.double().numpy()
    out = {n: f64(synthetic.tensor(ws, n, seed, 0, "cpu")) for n in ("Q", "K", "V", "dO")}
    out["Kd"] = np.stack([f64(synthetic.tensor(ws, "Kd", seed, i, "cpu")) for i in range(w.l)]) if w.l else np.zeros((0,) + out["Q"].shape)
    out["Vd"] = np.stack([f64(synthetic.tensor(ws, "Vd", seed, i, "cpu")) for i in range(w.l)]) if w.l else np.zeros((0,) + out["Q"].shape)
    return out, ws


def time_oracle(sample):
    """Seconds of one oracle forward + backward over the sample, the FLOPs it is credited with (same convention
    as the GPU arm) and the threads it used."""
    from oracle import moda_oracle as orc
    x, ws = sample
    t0 = time.time()
    orc.forward(x["Q"], x["K"], x["V"], x["Kd"], x["Vd"], ws.scale)
    orc.backward(x["Q"], x["K"], x["V"], x["Kd"], x["Vd"], x["dO"], ws.scale)
    dt = time.time() - t0
    return dt, flops.fwd_bwd_flops(1, ws.T, 1, ws.d, ws.l), orc.threads()


def sized_sample(w, seconds):
    """A sample whose oracle run takes about `seconds`: a short probe gives the rate, the cost grows with T^2."""
    T_probe = min(w.T, 2048)
    dt, fl, _ = time_oracle(cpu_sample(w, T_probe))
    rate = fl / max(dt, 1e-4)
    # fl(T) = 3.5 * (2 d T^2 + 4 T l d)  ->  solve for the T that costs seconds * rate
    a, b, c = 3.5 * 2.0 * w.d, 3.5 * 4.0 * w.l * w.d, -seconds * rate
    T_fit = int((-b + (b * b - 4 * a * c) ** 0.5) / (2 * a))
    T_s = max(256, min(w.T, (T_fit // 256) * 256))
    return cpu_sample(w, T_s)


def cpu_baseline(w, budget_s=20.0):
    """The fp64 oracle, as it stands, on a bounded sample of the benchmarked workload."""
    sample = sized_sample(w, budget_s)
    dt, fl, cores = time_oracle(sample)
    T_s = sample[1].T
    return {"value": round(fl / dt / 1e12, 6), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"one (b,h) slice of {w.name} cut to its first {T_s} of {w.T} positions (d={w.d}, l={w.l}), forward + "
                      f"backward, fp64, {dt:.1f} s; same FLOP convention",
            "seconds": round(dt, 2)}


def run_reference(args, rank, world):
    """--impl reference: the oracle timed on the host cores, same metric / config keys."""
    w = pick_workload(args)
    if rank != 0:
        return None
    K, W = max(args.steps, 1), max(args.warmup, 0)
    # bounded: each step is one (b, h) slice cut to a prefix sized so that the whole run stays near three minutes
    budget = 170.0
    sample = sized_sample(w, budget / (K + W))
    cores = 0
    for _ in range(W):
        time_oracle(sample)
    times = []
    for _ in range(K):
        dt, fl, cores = time_oracle(sample)
        times.append(dt)
    dt = sum(times) / K
    val = fl / dt / 1e12
    T_s = sample[1].T
    what = f"one (b,h) slice of {w.name} cut to its first {T_s} of {w.T} positions, forward + backward, fp64"
    return {
        "impl": "reference", "metric": METRIC, "value": round(val, 6), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": round(dt * 1e3, 2), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: B={w.B} T={w.T} H={w.H} d={w.d} l={w.l}; each step = {what} on the host cores"},
        "cpu_baseline": {"value": round(val, 6), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": f"{what}, per step"},
        "e2e": {"value": round(val, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def spawn_local_ranks(n: int) -> int:
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script on the local GPUs (one process per
    GPU, rendezvous on 127.0.0.1) and wait for them; rank 0 prints the line."""
    import socket
    with socket.socket() as sck:
        sck.bind(("127.0.0.1", 0))
        port = sck.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    return max(p.wait() for p in procs)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="moda", choices=["moda", "reference"])
    ap.add_argument("--workload", default="c4", help="c1..c5, optionally with _l<depth> (e.g. c3_l8)")
    ap.add_argument("--e2e-steps", type=int, default=3, help="steps of the host-to-host leg (each moves every input and output over PCIe)")
    ap.add_argument("--sweeps", default="", help="comma list of extra sweeps printed in the line: gqa, decode, prefill, kvproj, mass")
    ap.add_argument("--batch", type=int, default=0, help="override B of the workload (smaller profiling cases)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gqa-shape", default="", help="T,G[,L]: time only this grouped-query shape (B=1, d=64, 8 key/value "
                                                    "heads, L depth slots (default 32) and l=0) and print its row; for profiling")
    ap.add_argument("--prefill-sweep", action="store_true", help="time only the prefill-with-cache shapes and print their rows")
    ap.add_argument("--mass-workload", default="", help="comma list of workloads (c3_l32, c4, ...): time only the depth-slot attention "
                    "mass on them and print its rows; --batch overrides B; for profiling")
    ap.add_argument("--kvproj-shape", default="", help="B,T,D_model,H_kv,d (or 'all'): time only the key/value projection with the "
                    "write step in its epilogue and print its rows; for profiling")
    ap.add_argument("--decode-shape", default="", help="B,T_kv,H,H_kv,d,l: time only this decode step and print its row; for profiling")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        if args.impl == "moda" and torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus} but only {torch.cuda.device_count()} CUDA device(s) are visible")
        return spawn_local_ranks(args.gpus)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        out = run_reference(args, rank, world)
        if out is not None:
            print(json.dumps(out), flush=True)
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the MoDA operator has no CPU path)")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)
    try:
        if args.gqa_shape:
            v = [int(t) for t in args.gqa_shape.split(",")]
            out = {"gqa_sweep": run_gqa_sweep(device, [(v[0], v[1], v[2] if len(v) > 2 else 32, None)])}
        elif args.prefill_sweep:
            out = {"prefill_sweep": run_prefill_sweep(load_peaks(), device)}
        elif args.mass_workload:
            out = {"mass_sweep": run_mass_sweep(load_peaks(), device, tuple(args.mass_workload.split(",")), args.batch,
                                                iters=max(1, min(args.steps, 20)))}
        elif args.kvproj_shape:
            v = args.kvproj_shape
            shapes = None if v == "all" else [tuple(int(t) for t in v.split(","))]
            out = {"kvproj_sweep": run_kvproj_sweep(load_peaks(), device, shapes, iters=max(1, min(args.steps, 20)))}
        elif args.decode_shape:
            v = tuple(int(t) for t in args.decode_shape.split(","))
            out = {"decode_sweep": run_decode_sweep(load_peaks(), device, [v], iters=max(1, min(args.steps, 20)))}
        else:
            out = run_moda(args, rank, world, device)
        if rank == 0:
            print(json.dumps(out), flush=True)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
