#!/usr/bin/env python
"""Benchmark of the FLASH-D attention forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c2|c3|c4]
                    [--impl ours|reference] [--no-extra]

One step = one forward pass over one batch of the workload (default: the
encoder-shaped bf16 configuration, B=8 H=12 N=1024 d=64).  Prints one JSON line.
The attention path does not shard: with N > 1 every rank runs an independent
replica on its own GPU and the value is the sum over replicas divided by the
slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

L2_BYTES = 126e6
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (c4: a batch-4 capture scaled by 16, traffic being
# proportional to the bytes streamed).  Must be set back to None when that kernel changes.
NCU_TRAFFIC_BYTES = {"c1": 38.1e6, "c2": 591.5e6, "c3": None, "c4": 34.51e9, "c2_e4m3": 198.4e6}


def f32(x: float) -> float:
    return float(np.float32(x))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# ----------------------------------------------------------------------------- distributed helpers
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_max(value: float, world: int, device=None) -> float:
    """Max over ranks of a per-rank scalar (identity when not distributed)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank: float, world: int, max_ms: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / (max_ms * 1e-3)


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi every 20 ms; only
    the samples taken between mark_start() and mark_end() are summarised."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None
        self.t0 = self.t1 = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            deadline = time.time() + 5.0
            while time.time() < deadline and os.path.getsize(self.path) == 0:
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    @staticmethod
    def _stamp(text):
        import datetime
        try:
            return datetime.datetime.strptime(text.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    rows.append((self._stamp(f[0]), float(f[1]), float(f[2]), float(f[3]), f[5:9]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if r[0] is not None and self.t0 is not None and self.t0 <= r[0] <= self.t1 + 0.02]
        out["window"] = "timed region" if inside else "whole run (no sample fell inside the timed region)"
        use = inside or rows
        if use:
            reasons = set()
            for r in use:
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            out.update(sm_mhz=statistics.median(r[1] for r in use), sm_max_mhz=max(r[2] for r in use),
                       power_w=statistics.median(r[3] for r in use), samples=len(use), reasons=sorted(reasons))
        return out


# ----------------------------------------------------------------------------- oracle leg (CPU)
def oracle_rate(w):
    """Counted flop/s of the oracle on a small probe shaped like workload ``w``."""
    import oracle
    from paper_2505_14201_b200 import synth
    probe = synth.Workload("probe", 1, 2, min(w.Nq, 256), min(w.Nk, 2048), w.d, w.causal, w.dtype, 99)
    q, k, v = synth.make_inputs(probe)
    oracle.attn_naive(q, k, v, f32(w.scale), probe.causal)          # builds / loads the oracle, warms the threads
    t0 = time.perf_counter()
    oracle.attn_naive(q, k, v, f32(w.scale), probe.causal)
    return probe.flops / max(time.perf_counter() - t0, 1e-4)


def oracle_sample(w, target_s=12.0, rate=None):
    """Time the fp64 oracle, as it stands, on a bounded sample of workload ``w``:
    the leading heads, the last query rows, every key.  Returns (metric value in
    TFLOP/s, seconds, description, threads)."""
    import torch
    import oracle
    from paper_2505_14201_b200 import synth
    threads = oracle.num_threads()
    rate = rate or oracle_rate(w)
    per_head = w.flops / (w.B * w.H)
    if per_head <= rate * target_s:
        heads = max(1, min(w.B * w.H, int(rate * target_s / per_head)))
        rows = w.Nq
    else:
        heads = 1
        rows = max(1, int(w.Nq * rate * target_s / per_head))
    g = torch.Generator().manual_seed(w.seed)
    q = (torch.randn(1, heads, w.Nq, w.d, generator=g) * w.q_gain)
    k = (torch.randn(1, heads, w.Nk, w.d, generator=g) * w.k_gain)
    v = torch.randn(1, heads, w.Nk, w.d, generator=g)
    if w.outlier_every:
        k[:, :, :: w.outlier_every] *= w.outlier_gain
    dt_ = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    q, k, v = q.to(dt_), k.to(dt_), v.to(dt_)
    row_idx = list(range(w.Nq - rows, w.Nq))              # the last rows: the longest ones when causal
    qs = q[:, :, row_idx].contiguous()
    t0 = time.perf_counter()
    oracle.attn_naive(qs, k, v, f32(w.scale), w.causal, q_index=row_idx)
    secs = time.perf_counter() - t0
    if w.causal:
        pairs = sum(min(i + 1, w.Nk) for i in row_idx) * heads
    else:
        pairs = rows * w.Nk * heads
    flops = 4.0 * pairs * w.d
    desc = (f"oracle.attn_naive (fp64, OpenMP) on {heads} of {w.B * w.H} heads, last {rows} of {w.Nq} query rows, "
            f"all {w.Nk} keys, same recipe as the workload; {secs:.2f} s")
    return flops / secs / 1e12, secs, desc, threads


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores (rank 0 only)."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    from paper_2505_14201_b200 import synth
    w = synth.WORKLOADS[args.workload]
    vals, secs_all, desc, threads = [], [], "", 1
    budget = 120.0                                       # seconds for the whole run
    per_step = min(12.0, 0.6 * budget / max(1, args.steps + args.warmup))
    rate = oracle_rate(w)
    for i in range(args.warmup + args.steps):
        val, secs, desc, threads = oracle_sample(w, target_s=per_step, rate=rate)
        if i >= args.warmup:
            vals.append(val); secs_all.append(secs)
    value = statistics.mean(vals) if vals else 0.0
    line = {
        "impl": "reference", "metric": "attn_fwd_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * statistics.mean(secs_all) if secs_all else None,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, extra={"note": "each step is a bounded sample of the workload"}),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, extra=None):
    c = {"workload": w.name, "B": w.B, "H": w.H, "Nq": w.Nq, "Nk": w.Nk, "d": w.d, "causal": w.causal,
         "in_dtype": w.dtype, "scale": "1/sqrt(d)", "seed": w.seed}
    if extra:
        c.update(extra)
    return c


# ----------------------------------------------------------------------------- GPU legs
def time_gpu(fn, steps, warmup, torch):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def make_sets(w, device, min_bytes):
    """Enough distinct input sets that one pass over all of them exceeds L2."""
    import torch
    from paper_2505_14201_b200 import synth
    q, k, v = synth.make_inputs(w, device=device)
    esz = q.element_size()
    set_bytes = (2 * q.numel() + 2 * k.numel()) * esz
    n = max(1, math.ceil(min_bytes / set_bytes))
    sets = [(q, k, v, torch.empty_like(q))]
    for i in range(1, n):
        g = torch.Generator(device=device).manual_seed(1000 + w.seed * 16 + i)
        perm = torch.randperm(w.Nk, device=device, generator=g)
        sets.append((q.roll(i, dims=2).contiguous(), k[:, :, perm].contiguous(), v[:, :, perm].contiguous(),
                     torch.empty_like(q)))
    return sets, set_bytes


def bench_workload(fd, w, steps, warmup, torch, device, e4m3=False):
    """Device-resident timing of one workload; returns a dict of results."""
    sc = f32(w.scale)
    if w.splitk:
        q, k, v = make_c4(w, device)
        S = fd.flashd_splitk_num_splits(w.B, w.H, w.Nq, w.Nk, w.d)
        ws = torch.empty((w.B, w.H, w.Nq, S, w.d + 1), dtype=torch.float32, device=device)
        o = torch.empty_like(q)
        fn = lambda i: fd.flashd_attn_fwd_splitk(q, k, v, sc, S, workspace=ws, o=o)
        n0 = fd.launch_count()
        ms = time_gpu(fn, steps, warmup, torch)
        launches = (fd.launch_count() - n0) * steps // (steps + warmup)
        alg_bytes = w.kv_bytes
        return {"ms_per_step": ms / steps, "tflops": w.flops * steps / (ms * 1e-3) / 1e12,
                "gbs": alg_bytes * steps / (ms * 1e-3) / 1e9, "launches": launches, "num_splits": S,
                "l2": "inputs (34 GB) exceed L2", "tensors": (q, k, v, o)}
    sets, set_bytes = make_sets(w, device, 1.5 * L2_BYTES)
    if e4m3:
        # the same tensors stored as FP8-E4M3 (the paper's second format), bf16 output
        sets = [(q.to(torch.float8_e4m3fn), k.to(torch.float8_e4m3fn), v.to(torch.float8_e4m3fn), o)
                for (q, k, v, o) in sets]
        set_bytes = set_bytes * 5 // 8
        fn = lambda i: fd.flashd_attn_fwd_fp8(*sets[i % len(sets)][:3], sc, w.causal, o=sets[i % len(sets)][3])
    else:
        fn = lambda i: fd.flashd_attn_fwd(*sets[i % len(sets)][:3], sc, w.causal, o=sets[i % len(sets)][3])
    n0 = fd.launch_count()
    ms = time_gpu(fn, steps, warmup, torch)
    launches = (fd.launch_count() - n0) * steps // (steps + warmup)
    return {"ms_per_step": ms / steps, "tflops": w.flops * steps / (ms * 1e-3) / 1e12, "launches": launches,
            "l2": f"rotating {len(sets)} input sets of {set_bytes / 1e6:.0f} MB (> 126 MB L2 in total)",
            "tensors": sets[0]}


def make_c4(w, device):
    from paper_2505_14201_b200 import synth
    return synth.make_inputs(w, device=device)


def bench_e2e(fd, w, steps, warmup, torch):
    """Same metric through the host-buffer C-ABI call: pinned host inputs, H2D,
    kernel(s), D2H of the result, all inside the timed region."""
    from paper_2505_14201_b200 import synth
    if w.splitk:
        # 34 GB of pinned host memory is not a sane benchmark input; time a
        # batch slice (B = 4) and scale the metric by the work it covers
        w = synth.Workload(w.name + " (B=4 slice)", 4, w.H, w.Nq, w.Nk, w.d, w.causal, w.dtype, w.seed,
                           splitk=True, per_batch=True)
    q, k, v = synth.make_inputs(w)
    q, k, v = q.pin_memory(), k.pin_memory(), v.pin_memory()
    o = torch.empty_like(q).pin_memory()
    sc = f32(w.scale)
    path = 2 if w.splitk else 0
    t_steps = max(3, min(steps, 20))
    for _ in range(max(3, min(warmup, 5))):
        fd.flashd_attn_fwd_host(q, k, v, sc, w.causal, path=path, o=o)
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(t_steps):
        fd.flashd_attn_fwd_host(q, k, v, sc, w.causal, path=path, o=o)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / t_steps
    h2d = (q.numel() + k.numel() + v.numel()) * q.element_size()
    d2h = o.numel() * o.element_size()
    return {"tflops": w.flops / (ms * 1e-3) / 1e12, "ms_per_step": ms, "h2d": h2d, "d2h": d2h, "steps": t_steps,
            "workload": w.name}


def run_skip_stats(fd, synth, torch, device):
    """The paper's second experiment in shape: share of output updates that the static range
    rule [-6, 11] on s_i - s_{i-1} (and the adaptive reading on the sigmoid argument, [-6, 6])
    would bypass, on the synthetic workloads (config 4 on its first 4 batch elements)."""
    import dataclasses
    out = {}
    for name in ("c0", "c1", "c2", "c3", "c4"):
        w = synth.WORKLOADS[name]
        if name == "c4":
            w = dataclasses.replace(w, B=4)
        q, k, _ = synth.make_inputs(w, device=device)
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        c = fd.flashd_skip_stats(q, k, f32(w.scale), w.causal)
        e1.record(); torch.cuda.synchronize()
        out[name] = {"steps": c[0], "static_keep_pct": 100.0 * c[1] / c[0], "static_replace_pct": 100.0 * c[2] / c[0],
                     "static_total_pct": 100.0 * (c[1] + c[2]) / c[0], "adaptive_keep_pct": 100.0 * c[3] / c[0],
                     "adaptive_replace_pct": 100.0 * c[4] / c[0], "ms": e0.elapsed_time(e1)}
        del q, k
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "bypassable_output_updates_pct", "static_range": [-6, 11], "adaptive_range": [-6, 6],
                      "data": "synthetic", "workloads": out}), flush=True)


def run_pwl_study(fd, synth, torch, device):
    """Sec. IV-B in numbers: output error of Algorithm 3 when the sigmoid and ln are 8-segment PWL
    fits and the sigmoid argument is confined to [-6, 11], against the exact per-key kernel, on the
    synthetic workloads (config 4 on its first 4 batch elements)."""
    import dataclasses
    from paper_2505_14201_b200 import pwl
    sig, ln = pwl.paper_tables()
    variants = {"exact_saturate": (None, None, 0), "exact_bypass": (None, None, 1),
                "pwl8_saturate": (sig, ln, 0), "pwl8_bypass": (sig, ln, 1)}
    out = {}
    for name in ("c0", "c1", "c2", "c3", "c4"):
        w = synth.WORKLOADS[name]
        if name == "c4":
            w = dataclasses.replace(w, B=4)
        q, k, v = synth.make_inputs(w, device=device)
        sc = f32(w.scale)
        ref = fd.flashd_attn_fwd_perkey(q, k, v, sc, w.causal, out_dtype=torch.float32)
        steps = (w.B * w.H * (w.Nq * (w.Nq + 1) // 2 if w.causal else w.Nq * w.Nk))
        res = {}
        for vn, (st, lt, mode) in variants.items():
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            got, cnt = fd.flashd_attn_fwd_pwl(q, k, v, sc, w.causal, sig=st, ln=lt, lo=-6.0, hi=11.0, range_mode=mode,
                                              out_dtype=torch.float32, return_counts=True)
            e1.record(); torch.cuda.synchronize()
            err = (got - ref).abs()
            res[vn] = {"max_abs_err": float(err.max()), "mean_abs_err": float(err.mean()),
                       "bypassed_pct": 100.0 * cnt[0] / steps, "replaced_pct": 100.0 * cnt[1] / steps,
                       "ms": e0.elapsed_time(e1)}
            del got, err
        out[name] = res
        del q, k, v, ref
        torch.cuda.empty_cache()
    st_, detail = fd.flashd_last_device_status()
    if st_ != 0:
        raise SystemExit(f"device status {st_} {detail}")
    print(json.dumps({"metric": "pwl_output_error_vs_exact", "segments": 8, "range": [-6, 11], "data": "synthetic",
                      "sigmoid_table_max_err": pwl.max_error(sig, pwl.sigmoid, *pwl.SIGMOID_RANGE),
                      "ln_table_max_err": pwl.max_error(ln, __import__("numpy").log, *pwl.ln_range()),
                      "workloads": out}), flush=True)


def run_gqa(fd, synth, torch, device, peaks, steps, batch=0):
    """Grouped-query decode: config 4 with its 32 query heads sharing 32/G K/V heads.  The K/V
    stream (the algorithmic bytes) shrinks by G, the arithmetic per K/V byte grows by G."""
    w4 = synth.WORKLOADS["c4"]
    if batch > 0:
        import dataclasses
        w4 = dataclasses.replace(w4, B=batch)
    out = {}
    for G in (1, 4, 8):
        Hkv = w4.H // G
        g = torch.Generator(device=device).manual_seed(w4.seed + G)
        q = torch.randn(w4.B, w4.H, 1, w4.d, generator=g, device=device).to(torch.bfloat16)
        k = torch.randn(w4.B, Hkv, w4.Nk, w4.d, generator=g, device=device).to(torch.bfloat16)
        v = torch.randn(w4.B, Hkv, w4.Nk, w4.d, generator=g, device=device).to(torch.bfloat16)
        sc = f32(w4.scale)
        S = fd.flashd_gqa_num_splits(w4.B, Hkv, G, w4.Nk, w4.d)
        ws = torch.empty((w4.B, w4.H, 1, S, w4.d + 1), dtype=torch.float32, device=device)
        o = torch.empty_like(q)
        ms = time_gpu(lambda i: fd.flashd_attn_fwd_gqa(q, k, v, sc, S, workspace=ws, o=o), steps, 3, torch) / steps
        alg = (k.numel() + v.numel() + q.numel() + o.numel()) * 2
        flops = 4.0 * w4.B * w4.H * w4.Nk * w4.d
        out[f"G={G}"] = {"B": w4.B, "Hkv": Hkv, "G": G, "Nk": w4.Nk, "d": w4.d, "num_splits": S, "ms_per_step": ms,
                         "gbs": alg / (ms * 1e-3) / 1e9, "frac_hbm_measured": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         "frac_hbm_nominal": alg / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                         "tflops": flops / (ms * 1e-3) / 1e12, "kv_gb": (k.numel() + v.numel()) * 2 / 1e9}
        del q, k, v, ws, o
        torch.cuda.empty_cache()
    # config 4 itself with K and V stored as FP8-E4M3: half the bytes per key
    g = torch.Generator(device=device).manual_seed(w4.seed + 99)
    q = torch.randn(w4.B, w4.H, 1, w4.d, generator=g, device=device).to(torch.bfloat16)
    k = torch.empty(w4.B, w4.H, w4.Nk, w4.d, dtype=torch.float8_e4m3fn, device=device)
    v = torch.empty_like(k)
    for b in range(w4.B):
        k[b] = torch.randn(w4.H, w4.Nk, w4.d, generator=g, device=device).to(torch.float8_e4m3fn)
        v[b] = torch.randn(w4.H, w4.Nk, w4.d, generator=g, device=device).to(torch.float8_e4m3fn)
    sc = f32(w4.scale)
    S = fd.flashd_splitk_num_splits(w4.B, w4.H, 1, w4.Nk, w4.d)
    ws = torch.empty((w4.B, w4.H, 1, S, w4.d + 1), dtype=torch.float32, device=device)
    o = torch.empty_like(q)
    ms = time_gpu(lambda i: fd.flashd_attn_fwd_splitk_fp8kv(q, k, v, sc, S, workspace=ws, o=o), steps, 3, torch) / steps
    alg = k.numel() + v.numel() + (q.numel() + o.numel()) * 2
    out["fp8_kv"] = {"B": w4.B, "H": w4.H, "Nk": w4.Nk, "d": w4.d, "num_splits": S, "ms_per_step": ms,
                     "gbs": alg / (ms * 1e-3) / 1e9, "frac_hbm_measured": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "frac_hbm_nominal": alg / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                     "keys_per_s": w4.B * w4.H * w4.Nk / (ms * 1e-3), "kv_gb": (k.numel() + v.numel()) / 1e9}
    del q, k, v, ws, o
    torch.cuda.empty_cache()
    # config 4 over a paged pool: pages of 256 keys in shuffled order, sequence lengths mixed
    # uniformly between a quarter and the whole of Nk (a serving batch in mid-flight)
    page = 256
    g = torch.Generator(device=device).manual_seed(w4.seed + 7)
    lens = torch.randint(w4.Nk // 4, w4.Nk + 1, (w4.B,), generator=g, device=device, dtype=torch.int32)
    max_pages = w4.Nk // page
    per_seq = (lens + page - 1) // page
    num_pages = int(per_seq.sum().item())
    perm = torch.randperm(num_pages, generator=g, device=device).to(torch.int32)
    table = torch.zeros((w4.B, max_pages), dtype=torch.int32, device=device)
    off = 0
    for b in range(w4.B):
        n = int(per_seq[b].item())
        table[b, :n] = perm[off:off + n]
        off += n
    q = torch.randn(w4.B, w4.H, 1, w4.d, generator=g, device=device).to(torch.bfloat16)
    kp = torch.empty(num_pages, w4.H, page, w4.d, dtype=torch.bfloat16, device=device)
    vp = torch.empty_like(kp)
    step_pages = max(1, num_pages // 64)
    for p0 in range(0, num_pages, step_pages):
        n = min(step_pages, num_pages - p0)
        kp[p0:p0 + n] = torch.randn(n, w4.H, page, w4.d, generator=g, device=device).to(torch.bfloat16)
        vp[p0:p0 + n] = torch.randn(n, w4.H, page, w4.d, generator=g, device=device).to(torch.bfloat16)
    S = fd.flashd_splitk_num_splits(w4.B, w4.H, 1, w4.Nk, w4.d)
    ws = torch.empty((w4.B, w4.H, 1, S, w4.d + 1), dtype=torch.float32, device=device)
    o = torch.empty_like(q)
    ms = time_gpu(lambda i: fd.flashd_attn_fwd_splitk_paged(q, kp, vp, table, lens, sc, S, workspace=ws, o=o),
                  steps, 3, torch) / steps
    keys = int(lens.sum().item()) * w4.H
    alg = keys * w4.d * 2 * 2 + (q.numel() + o.numel()) * 2
    out["paged"] = {"B": w4.B, "H": w4.H, "d": w4.d, "page_size": page, "num_pages": num_pages, "num_splits": S,
                    "seq_lens": f"uniform in [{w4.Nk // 4}, {w4.Nk}], mean {float(lens.float().mean().item()):.0f}",
                    "ms_per_step": ms, "gbs": alg / (ms * 1e-3) / 1e9,
                    "frac_hbm_measured": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "frac_hbm_nominal": alg / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                    "keys_per_s": keys / (ms * 1e-3), "kv_gb": keys * w4.d * 4 / 1e9}
    del q, kp, vp, ws, o
    torch.cuda.empty_cache()
    st, detail = fd.flashd_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} {detail}")
    print(json.dumps({"metric": "gqa_decode_hbm_gbs", "unit": "GB/s", "data": "synthetic", "steps": steps,
                      "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "groups": out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--workload", default="c1", choices=["c1", "c2", "c3", "c4"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations and the CPU baseline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--skip-stats", action="store_true",
                    help="print the bypassable-update statistic (Sec. III-C / V-B) of every workload instead of timing")
    ap.add_argument("--pwl-study", action="store_true",
                    help="print the output error of the PWL / confined-range datapath model (Sec. IV-B) instead of timing")
    ap.add_argument("--gqa", action="store_true",
                    help="time the decode variants (config 4 with shared K/V heads; config 4 with FP8-E4M3 K/V) instead")
    ap.add_argument("--e4m3", action="store_true",
                    help="time the workload (c2 or c3, d = 128) with FP8-E4M3 operands on the tensor path; no "
                         "end-to-end leg (the host entry point takes bf16 / fp32)")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch size B (smaller case for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2505_14201_b200 as fd
    from paper_2505_14201_b200 import synth

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)
    fd.lib()
    peaks = load_peaks()
    w = synth.WORKLOADS[args.workload]
    if args.batch > 0:
        import dataclasses
        w = dataclasses.replace(w, B=args.batch, name=f"{w.name} (B={args.batch})")

    if args.skip_stats:
        run_skip_stats(fd, synth, torch, device)
        return

    if args.pwl_study:
        run_pwl_study(fd, synth, torch, device)
        return
    if args.gqa:
        run_gqa(fd, synth, torch, device, peaks, min(args.steps, 30), args.batch)
        return

    sampler = ClockSampler(local_rank)
    # ---- headline: device-resident inputs
    # build inputs, then barrier + sync, time K steps, sync + barrier, max over ranks
    sc = f32(w.scale)
    if w.splitk:
        q, k, v = make_c4(w, device)
        S = fd.flashd_splitk_num_splits(w.B, w.H, w.Nq, w.Nk, w.d)
        ws = torch.empty((w.B, w.H, w.Nq, S, w.d + 1), dtype=torch.float32, device=device)
        o = torch.empty_like(q)
        step = lambda i: fd.flashd_attn_fwd_splitk(q, k, v, sc, S, workspace=ws, o=o)
        l2_note = "inputs (34 GB) exceed L2"
    else:
        sets, set_bytes = make_sets(w, device, 1.5 * L2_BYTES)
        step = lambda i: fd.flashd_attn_fwd(*sets[i % len(sets)][:3], sc, w.causal, o=sets[i % len(sets)][3])
        if args.e4m3:
            if w.d != 128:
                raise SystemExit("--e4m3 needs a workload with d = 128 (c2, c3)")
            sets = [(q.to(torch.float8_e4m3fn), k.to(torch.float8_e4m3fn), v.to(torch.float8_e4m3fn), o)
                    for (q, k, v, o) in sets]
            set_bytes = set_bytes * 5 // 8
            step = lambda i: fd.flashd_attn_fwd_fp8(*sets[i % len(sets)][:3], sc, w.causal, o=sets[i % len(sets)][3])
            args.no_e2e = True
        l2_note = f"rotating {len(sets)} input sets of {set_bytes / 1e6:.0f} MB each (> 126 MB L2 in total)"
    sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    n0 = fd.launch_count()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.mark_start()
    e0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record()
    torch.cuda.synchronize()
    sampler.mark_end()
    launches = fd.launch_count() - n0
    if world > 1:
        dist.barrier()
    local_ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    st, detail = fd.flashd_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} {detail}")
    max_ms = reduce_max(local_ms, world, device)
    value = aggregate_value(w.flops * args.steps, world, max_ms) / 1e12
    ms_per_step = max_ms / args.steps

    # ---- roofline of the dominant kernel (one launch per step for prefill; partial kernel for decode)
    if w.splitk:
        alg = w.kv_bytes
        achieved = alg / (local_ms / args.steps * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(args.workload) if args.batch == 0 else None,
                "peak_source": peaks["source"],
                "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                "kernel": "splitk_partial_kernel (+combine, timed together)"}
    else:
        achieved = w.flops / (local_ms / args.steps * 1e-3) / 1e12
        # E4M3 products: the peak of that dtype = the measured bf16 figure x the nominal ratio of 2
        pk_scale = 2.0 if args.e4m3 else 1.0
        traffic = NCU_TRAFFIC_BYTES.get(args.workload + ("_e4m3" if args.e4m3 else "")) if args.batch == 0 else None
        roof = {"bound": "tensor", "achieved": achieved, "peak": pk_scale * peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / (pk_scale * peaks["bf16_tflops"]), "traffic": traffic,
                "peak_source": peaks["source"] + (" bf16 x 2 (nominal fp8 : bf16 ratio)" if args.e4m3 else ""),
                "frac_of_nominal": achieved / (pk_scale * NOMINAL_BF16_TFLOPS),
                "kernel": f"prefill_kernel<{w.d}, 1>" if args.e4m3 else f"prefill_kernel<{w.d}>"}

    line = {
        "metric": "attn_fwd_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "e4m3" if args.e4m3 else "bf16", "data": "synthetic",
        "config": workload_config(w, {"l2": l2_note, "parallelism": "replicas only" if world > 1 else "1 gpu"}),
        "roofline": roof, "clocks": clocks, "gpu_launches": int(launches),
    }

    if args.e4m3:
        line["config"]["in_dtype"] = "e4m3"
        line["config"]["workload"] = line["config"]["workload"].replace(" bf16", "") + " (FP8-E4M3 operands)"

    if rank == 0 and world == 1 and not w.splitk:
        # launch gaps: the same launches replayed from a CUDA graph (50 per replay)
        try:
            n_graph = 50
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step(0)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(n_graph):
                        step(i)
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            g0 = torch.cuda.Event(enable_timing=True); g1 = torch.cuda.Event(enable_timing=True)
            reps = max(1, min(args.steps // n_graph, 40))
            g0.record()
            for _ in range(reps):
                graph.replay()
            g1.record()
            torch.cuda.synchronize()
            gms = g0.elapsed_time(g1) / (reps * n_graph)
            line["cuda_graph"] = {"launches_per_replay": n_graph, "replays": reps, "ms_per_step": gms,
                                  "value": w.flops / (gms * 1e-3) / 1e12, "unit": "TFLOP/s"}
            del graph
        except Exception as ex:  # the headline number stands on its own
            line["cuda_graph"] = {"error": repr(ex)}

    if rank == 0 and not args.no_e2e:
        e2e = bench_e2e(fd, w, args.steps, args.warmup, torch)
        line["e2e"] = {"value": e2e["tflops"] * world, "unit": "TFLOP/s", "h2d_bytes_per_step": e2e["h2d"],
                       "d2h_bytes_per_step": e2e["d2h"], "ms_per_step": e2e["ms_per_step"], "workload": e2e["workload"],
                       "note": "flashd_attn_fwd_host: pinned host q,k,v -> device, kernel, o -> host, every step (chunks of heads pipelined on three streams inside the call)"}
    if world > 1:
        # replicas: every rank does the same end-to-end work; report rank 0's rate times the replica count
        dist.barrier()

    if rank == 0 and world == 1 and not args.no_extra:
        # free the headline inputs before the larger configurations
        others = {}
        try:
            del step
            if w.splitk:
                del q, k, v, ws, o
            else:
                del sets
            torch.cuda.empty_cache()
            for name in ("c1", "c2", "c3", "c4"):
                if name == args.workload:
                    continue
                ow = synth.WORKLOADS[name]
                free, _ = torch.cuda.mem_get_info()
                if ow.splitk and free < 50e9:
                    others[name] = {"skipped": "not enough free device memory"}
                    continue
                smp = ClockSampler(local_rank)
                smp.start()
                smp.mark_start()
                r = bench_workload(fd, ow, 30 if name in ("c3", "c4") else 200, 3, torch, device)
                smp.mark_end()
                r["clocks"] = smp.stop()
                r.pop("tensors", None)
                if ow.splitk:
                    r["frac_hbm_measured"] = r["gbs"] / peaks["hbm_gbs"]
                    r["frac_hbm_nominal"] = r["gbs"] / NOMINAL_HBM_GBS
                else:
                    r["frac_tensor_measured"] = r["tflops"] / peaks["bf16_tflops"]
                    r["frac_tensor_nominal"] = r["tflops"] / NOMINAL_BF16_TFLOPS
                others[name] = r
                torch.cuda.empty_cache()
            # configurations 2 and 3 with E4M3 operands on the tensor path; the peak of that
            # dtype is the measured bf16 figure times the nominal ratio of 2
            for name in ("c2", "c3"):
                ow = synth.WORKLOADS[name]
                smp = ClockSampler(local_rank)
                smp.start()
                smp.mark_start()
                r = bench_workload(fd, ow, 30 if name == "c3" else 200, 3, torch, device, e4m3=True)
                smp.mark_end()
                r["clocks"] = smp.stop()
                r.pop("tensors", None)
                r["dtype"] = "e4m3 operands, fp32 accumulate, bf16 output"
                r["frac_tensor_measured"] = r["tflops"] / (2 * peaks["bf16_tflops"])
                r["frac_tensor_nominal"] = r["tflops"] / (2 * NOMINAL_BF16_TFLOPS)
                others[name + "_e4m3"] = r
                torch.cuda.empty_cache()
            # the paper's largest hidden size on the tensor path (not one of the five configurations):
            # config 3's shape with half the heads and d = 256, bf16 and E4M3
            ow = synth.Workload("d256 decoder prefill causal", 1, 16, 16384, 16384, 256, True, "bf16", 5)
            for tag, e4 in (("d256", False), ("d256_e4m3", True)):
                r = bench_workload(fd, ow, 30, 3, torch, device, e4m3=e4)
                r.pop("tensors", None)
                r["shape"] = "B1 H16 N16384 d256 causal"
                scale_pk = 2.0 if e4 else 1.0
                r["frac_tensor_measured"] = r["tflops"] / (scale_pk * peaks["bf16_tflops"])
                r["frac_tensor_nominal"] = r["tflops"] / (scale_pk * NOMINAL_BF16_TFLOPS)
                others[tag] = r
                torch.cuda.empty_cache()
        except Exception as ex:  # the headline number stands on its own
            others["error"] = repr(ex)
        line["other_configs"] = others
        val, secs, desc, threads = oracle_sample(w, target_s=12.0)
        line["cpu_baseline"] = {"value": val, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc}

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
