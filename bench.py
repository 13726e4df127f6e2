#!/usr/bin/env python
"""Benchmark of the fused alpha-entmax / ASEntmax attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--alpha A]

One step = one forward call + one backward call of the C-ABI library on the long-context workload
(batch 1, 16 heads, 32768 tokens, head dim 128, causal, bf16, 8 planted keys per planted query,
per-head ASEntmax scales).  Prints ONE JSON line.  `value` is the useful attention throughput of the
whole step in TFLOP/s: forward 4*d and backward 10*d FLOPs per visible (query, key) pair, i.e. the
dense-equivalent work with causal halving, divided by the device time of the step.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import re
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2506_16640_b200.inputs import WORKLOADS, make_inputs, sample_rows, scaled, seeded_d_o

METRIC = "entmax_attn_fwd_bwd_useful_tflops_n32k"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
BASE_SEED_DENSITY = 20250616 + 808
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# The ncu summary of the forward score sweep on the benchmark workload; its dram__bytes_read.sum and
# dram__bytes_write.sum lines (first column: the forward launch) give `roofline.traffic`.
SWEEP_PROFILE = os.path.join("profiles", "sweep_kernel_d128_cfg4_n32768.md")


def sweep_dram_traffic():
    """DRAM bytes (read + write) of one forward sweep launch as captured under ncu, read from the profile summary;
    None when the summary is missing or says that the kernel has changed since the capture."""
    path = os.path.join(ROOT, SWEEP_PROFILE)
    try:
        text = open(path).read()
    except OSError:
        return None
    if "counters predate the current kernel" in text:
        return None
    total = 0.0
    for name in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        m = re.search(re.escape(name) + r"\s+Mbyte\s+([0-9.]+)", text)
        if not m:
            return None
        total += float(m.group(1)) * 1e6
    return int(total)


def visible_pairs(w) -> int:
    per_head = w.N * (w.N + 1) // 2 if w.causal else w.N * w.N
    return per_head * w.B * w.H


def useful_flops(w):
    pairs = visible_pairs(w)
    return 4 * w.d * pairs, 10 * w.d * pairs


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_setup(n_gpus: int):
    """One process per GPU under torchrun; a single process otherwise."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend="nccl" if torch.cuda.is_available() else "gloo")
    return rank, world, local


def aggregate_over_ranks(step_ms: float, units: float, world: int, device):
    """Whole-job numbers: the slowest rank's time, the sum of all ranks' work.  The data path has no
    collective (every rank owns whole (batch, head) problems); these two reductions are bookkeeping."""
    if world == 1:
        return step_ms, units
    import torch.distributed as dist
    t = torch.tensor([step_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def make_bench_inputs(alpha: float):
    """The long-context workload plus a seeded dO (the workload itself is forward-only)."""
    w = WORKLOADS[4]
    inp = make_inputs(w)
    inp.d_o = seeded_d_o(w)
    return w, inp


def run_ours(args):
    from paper_2506_16640_b200 import binding

    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    binding.load()
    alpha = args.alpha
    w, inp = make_bench_inputs(alpha)
    host = {"q": inp.q, "k": inp.k, "v": inp.v, "d_o": inp.d_o, "beta": inp.beta, "gamma": inp.gamma,
            "delta": inp.delta}
    host = {n: t.pin_memory() for n, t in host.items()}
    d = {n: t.to(dev) for n, t in host.items()}
    params = binding.make_params(d["q"], alpha, w.causal)
    ws = binding.alloc_workspace(params, True, dev)          # the backward size covers the forward one
    status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
    o = torch.empty_like(d["q"])
    tau = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(d["q"]) for _ in range(3))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def fwd():
        binding.entmax_attn_fwd(d["q"], d["k"], d["v"], alpha, w.causal, d["beta"], d["gamma"], d["delta"], o=o,
                                tau=tau, workspace=ws, status=status)

    def bwd():
        binding.entmax_attn_bwd(d["q"], d["k"], d["v"], tau, d["d_o"], alpha, w.causal, d["beta"], d["gamma"],
                                d["delta"], dq=dq, dk=dk, dv=dv, workspace=ws, status=status)

    for _ in range(max(args.warmup, 3)):
        fwd()
        bwd()
    torch.cuda.synchronize()
    assert int(status[binding.STATUS_FLAGS].item()) == 0, "device status flags set during warm-up"
    dense_rows = int(status[binding.STATUS_DENSE_ROWS].item())

    K = args.steps
    ev = lambda: torch.cuda.Event(enable_timing=True)
    e_start, e_mid, e_stop = [ev() for _ in range(K)], [ev() for _ in range(K)], [ev() for _ in range(K)]
    s_start, s_stop = [ev() for _ in range(K)], [ev() for _ in range(K)]
    for e in s_start + s_stop:
        e.record()                                          # creates the CUDA handles the hook needs
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    barrier(world)
    torch.cuda.synchronize()
    sampler.start()
    for i in range(K):
        flush.zero_()                                       # evict L2 between steps (outside the timed events)
        binding.entmax_attn_profile_events(0, s_start[i], s_stop[i])
        e_start[i].record()
        fwd()
        e_mid[i].record()
        bwd()
        e_stop[i].record()
    binding.entmax_attn_profile_events(0, None, None)
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop()
    fwd_all = [a.elapsed_time(b) for a, b in zip(e_start, e_mid)]
    bwd_all = [a.elapsed_time(b) for a, b in zip(e_mid, e_stop)]
    step_all = [a.elapsed_time(b) for a, b in zip(e_start, e_stop)]
    sweep_all = [a.elapsed_time(b) for a, b in zip(s_start, s_stop)]
    fwd_ms, bwd_ms, step_ms, sweep_ms = (sum(x) / K for x in (fwd_all, bwd_all, step_all, sweep_all))
    spread = lambda xs: {"mean": sum(xs) / len(xs), "median": statistics.median(xs), "min": min(xs), "max": max(xs)}
    assert int(status[binding.STATUS_FLAGS].item()) == 0, "device status flags set during the timed region"

    # secondary: the backward pass fed with the forward call's workspace (its supports are reused, no second sweep)
    ws_fwd = binding.alloc_workspace(params, False, dev)
    b_start, b_stop = [ev() for _ in range(K)], [ev() for _ in range(K)]
    for i in range(K + 2):
        binding.entmax_attn_fwd(d["q"], d["k"], d["v"], alpha, w.causal, d["beta"], d["gamma"], d["delta"], o=o, tau=tau,
                                workspace=ws_fwd, status=status)
        j = max(i - 2, 0)
        b_start[j].record()
        binding.entmax_attn_bwd_ex(d["q"], d["k"], d["v"], tau, d["d_o"], alpha, w.causal, d["beta"], d["gamma"],
                                   d["delta"], fwd_workspace=ws_fwd, dq=dq, dk=dk, dv=dv, workspace=ws, status=status)
        b_stop[j].record()
    torch.cuda.synchronize()
    bwd_saved_ms = sum(a.elapsed_time(b) for a, b in zip(b_start, b_stop)) / K
    # the same with the compact copy of the supports (260 bytes per row instead of the whole forward workspace):
    # the copy itself and the backward pass fed with it are timed together
    saved = binding.entmax_attn_save_supports(d["q"], alpha, w.causal, ws_fwd)
    c_start, c_stop = [ev() for _ in range(K)], [ev() for _ in range(K)]
    for i in range(K + 2):
        binding.entmax_attn_fwd(d["q"], d["k"], d["v"], alpha, w.causal, d["beta"], d["gamma"], d["delta"], o=o, tau=tau,
                                workspace=ws_fwd, status=status)
        j = max(i - 2, 0)
        c_start[j].record()
        binding.entmax_attn_save_supports(d["q"], alpha, w.causal, ws_fwd, saved=saved)
        binding.entmax_attn_bwd_ex(d["q"], d["k"], d["v"], tau, d["d_o"], alpha, w.causal, d["beta"], d["gamma"],
                                   d["delta"], saved_supports=saved, dq=dq, dk=dk, dv=dv, workspace=ws, status=status)
        c_stop[j].record()
    torch.cuda.synchronize()
    bwd_compact_ms = sum(a.elapsed_time(b) for a, b in zip(c_start, c_stop)) / K
    compact_recomputed = int(status[binding.STATUS_DENSE_ROWS].item())
    saved_bytes = saved.numel()
    del ws_fwd, saved

    # secondary: the decode shape on the same tensors: the last q_len rows of Q as the new queries, K and V as the cache
    decode = time_decode(d, w, alpha, flush) if world == 1 else None
    # secondary: the temperature axis on this shape, the other alphas and the other workloads
    density = other = nape = None
    if world == 1 and not args.no_secondary:
        density = time_density_axis(d, w, alpha, flush, ws)
        nape = time_nape(d, w, alpha, flush, ws)
        other = [time_workload(4, a2, flush, tensors=d, ws=ws) for a2 in (1.25, 2.0) if a2 != alpha]

    # end to end: pinned host buffers in, results back to pinned host buffers, copies inside the timed region
    names = ("q", "k", "v", "d_o", "beta", "gamma", "delta")
    outs_dev = {"o": o, "tau": tau, "dq": dq, "dk": dk, "dv": dv}
    outs_host = {n: torch.empty(t.shape, dtype=t.dtype).pin_memory() for n, t in outs_dev.items()}
    h2d = sum(host[n].numel() * host[n].element_size() for n in names)
    d2h = sum(t.numel() * t.element_size() for t in outs_dev.values())
    E = max(1, min(K, 10))
    ee_start, ee_stop = [ev() for _ in range(E)], [ev() for _ in range(E)]
    # Three streams (copies in, compute, copies out) and the heads in groups: a group's forward and backward calls run
    # while the next group's inputs arrive and the previous group's results leave (PCIe is full duplex), so a step
    # costs about what its larger copy direction costs.  The entry points take strided tensors, so a group is just
    # a view; one group-sized workspace serves all groups (their calls are ordered on the compute stream).  A step
    # starts when the previous one has delivered everything.
    G = next((g for g in (8, 4, 2) if w.B == 1 and w.H % g == 0), 1)
    hg = w.H // G
    view = lambda t, g: t[:, g * hg:(g + 1) * hg]
    gview = {n: [view(d[n], g) for g in range(G)] for n in ("q", "k", "v", "d_o")}
    hview = {n: [view(host[n], g) for g in range(G)] for n in ("q", "k", "v", "d_o")}
    sview = {n: [d[n][g * hg:(g + 1) * hg] for g in range(G)] for n in ("beta", "gamma", "delta")}
    oview = {n: [view(t, g) for g in range(G)] for n, t in outs_dev.items()}
    ohost = {n: [view(t, g) for g in range(G)] for n, t in outs_host.items()}
    ws_g = binding.alloc_workspace(binding.make_params(gview["q"][0], alpha, w.causal), True, dev)
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    e_in1, e_in2 = [ev() for _ in range(G)], [ev() for _ in range(G)]
    e_f, e_b = [ev() for _ in range(G)], [ev() for _ in range(G)]
    barrier(world)
    torch.cuda.synchronize()
    for i in range(E):
        ee_start[i].record(s_in)
        with torch.cuda.stream(s_in):
            for n in ("beta", "gamma", "delta"):
                d[n].copy_(host[n], non_blocking=True)
            for g in range(G):
                for n in ("q", "k", "v"):
                    gview[n][g].copy_(hview[n][g], non_blocking=True)
                e_in1[g].record(s_in)
                gview["d_o"][g].copy_(hview["d_o"][g], non_blocking=True)
                e_in2[g].record(s_in)
        with torch.cuda.stream(s_cmp):
            for g in range(G):
                s_cmp.wait_event(e_in1[g])
                binding.entmax_attn_fwd(gview["q"][g], gview["k"][g], gview["v"][g], alpha, w.causal, sview["beta"][g],
                                        sview["gamma"][g], sview["delta"][g], o=oview["o"][g], tau=oview["tau"][g],
                                        workspace=ws_g, status=status, stream=s_cmp)
                e_f[g].record(s_cmp)
                s_cmp.wait_event(e_in2[g])
                binding.entmax_attn_bwd(gview["q"][g], gview["k"][g], gview["v"][g], oview["tau"][g], gview["d_o"][g], alpha,
                                        w.causal, sview["beta"][g], sview["gamma"][g], sview["delta"][g],
                                        dq=oview["dq"][g], dk=oview["dk"][g], dv=oview["dv"][g], workspace=ws_g,
                                        status=status, stream=s_cmp)
                e_b[g].record(s_cmp)
        with torch.cuda.stream(s_out):
            for g in range(G):
                s_out.wait_event(e_f[g])
                ohost["o"][g].copy_(oview["o"][g], non_blocking=True)
                ohost["tau"][g].copy_(oview["tau"][g], non_blocking=True)
                s_out.wait_event(e_b[g])
                for n in ("dq", "dk", "dv"):
                    ohost[n][g].copy_(oview[n][g], non_blocking=True)
            ee_stop[i].record(s_out)
        # the next step's input copies must not overwrite tensors this step still reads
        s_in.wait_event(ee_stop[i])
    torch.cuda.synchronize()
    barrier(world)
    assert int(status[binding.STATUS_FLAGS].item()) == 0, "device status flags set during the end-to-end steps"
    # the grouped calls give what the whole-tensor calls gave (O and tau bit for bit)
    ref_o, ref_tau = o.clone(), tau.clone()
    fwd()
    torch.cuda.synchronize()
    assert torch.equal(ref_o, o) and torch.equal(ref_tau, tau), "grouped end-to-end calls disagree with the full call"
    del ws_g
    e2e_ms = sum(a.elapsed_time(b) for a, b in zip(ee_start, ee_stop)) / E

    if other is not None:
        del ws, o, dq, dk, dv
        torch.cuda.empty_cache()
        other += [time_workload(idx, 1.5, flush) for idx in (2, 3, 5)]
    f_fwd, f_bwd = useful_flops(w)
    step_ms_all, flops_all = aggregate_over_ranks(step_ms, float(f_fwd + f_bwd), world, dev)
    e2e_ms_all, _ = aggregate_over_ranks(e2e_ms, 0.0, world, dev)
    if rank != 0:
        return
    peaks, peak_kind = load_peaks()
    burst = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    sustained = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    sweep_flops = 2 * w.d * visible_pairs(w)                # algorithmic: one QK^T contraction per visible pair
    sample_extra = 1.0 / 8.0 * (1.0 - (4096.0 / w.N) ** 2) if w.N >= 4096 else 0.0   # share of pairs scored twice
    sweep_tflops = sweep_flops / (sweep_ms * 1e-3) / 1e12
    fwd_tflops = f_fwd / (fwd_ms * 1e-3) / 1e12
    bwd_tflops = f_bwd / (bwd_ms * 1e-3) / 1e12
    # Two ways of counting.  "Dense-equivalent" FLOPs (the metric: forward 4 d, backward 10 d per visible pair) are what
    # a dense schedule would spend; the method skips almost all of it, so those rates are speed-ups over a dense
    # schedule and may exceed the tensor peak.  "Method" FLOPs are what the calls really contract on the tensor cores:
    # one Q K^T per visible pair in the forward sweep, one more in the tau-only backward (gathers over supports of a
    # few keys are noise beside them).
    method_fwd, method_bwd = sweep_flops, sweep_flops
    ws_bytes = {"forward": binding.entmax_attn_workspace_bytes(params, False),
                "backward": binding.entmax_attn_workspace_bytes(params, True)}
    line = {
        "metric": METRIC, "value": flops_all / (step_ms_all * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": step_ms_all, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.B, "heads": w.H, "seq": w.N, "head_dim": w.d, "causal": w.causal,
                   "alpha": alpha, "step": "entmax_attn_fwd + entmax_attn_bwd", "l2": "256 MiB memset between steps; "
                   "inputs (134 MB per tensor) and workspace (>1 GB) larger than L2",
                   "parallelism": "independent replicas, no collective" if world > 1 else "single GPU",
                   "value_counts": "dense-equivalent FLOPs: fwd 4*d, bwd 10*d per visible (query,key) pair",
                   "workspace_bytes": ws_bytes},
        "ms_per_step_stats": spread(step_all),
        "fwd": {"ms": fwd_ms, "ms_stats": spread(fwd_all),
                "dense_equivalent_tflops": fwd_tflops, "dense_equivalent_speedup_vs_burst_peak": fwd_tflops / burst,
                "method_tflops": method_fwd / (fwd_ms * 1e-3) / 1e12,
                "method_frac_of_burst_peak": method_fwd / (fwd_ms * 1e-3) / 1e12 / burst,
                "note": "method = the one Q K^T contraction the call performs; dense-equivalent = the metric's 4*d count "
                        "(a speed-up over a dense schedule, not a fraction of peak)"},
        "bwd": {"ms": bwd_ms, "ms_stats": spread(bwd_all),
                "dense_equivalent_tflops": bwd_tflops, "dense_equivalent_speedup_vs_burst_peak": bwd_tflops / burst,
                "method_tflops": method_bwd / (bwd_ms * 1e-3) / 1e12,
                "method_frac_of_burst_peak": method_bwd / (bwd_ms * 1e-3) / 1e12 / burst},
        "bwd_with_saved_forward_workspace": {"ms": bwd_saved_ms, "dense_equivalent_tflops": f_bwd / (bwd_saved_ms * 1e-3) / 1e12,
                                             "note": "not part of `value`: entmax_attn_bwd_ex given the forward call's "
                                                     "workspace reuses its support lists instead of sweeping QK^T again"},
        "bwd_with_compact_saved_supports": {"ms": bwd_compact_ms, "dense_equivalent_tflops": f_bwd / (bwd_compact_ms * 1e-3) / 1e12,
                                            "saved_bytes": saved_bytes, "rows_recomputed": compact_recomputed,
                                            "note": "not part of `value`: entmax_attn_save_supports after the forward call "
                                                    "+ entmax_attn_bwd_ex fed with the compact copy"},
        "tau_search_extra": {"tensor_flops": int(sweep_flops * sample_extra), "note": "single score sweep: the threshold is "
                             "solved on the per-row candidate lists, no extra QK^T pass; the figure is the sampled pre-pass "
                             "of the forward sweep (every 8th key scored once more, for rows that see 4096 keys or more)",
                             "dense_fallback_rows": dense_rows},
        # the timed loop lasts a fraction of a second at boost clocks (see `clocks`): the burst cuBLAS figure is the
        # denominator; the sustained one is given beside it
        "roofline": {"bound": "tensor", "kernel": "sweep_kernel<128> (forward score sweep)", "achieved": sweep_tflops,
                     "peak": burst, "unit": "TFLOP/s", "frac": sweep_tflops / burst,
                     "peak_source": peak_kind + " burst (timed region %.2f s)" % (step_ms * K * 1e-3),
                     "frac_of_sustained": sweep_tflops / sustained, "sustained_peak": sustained,
                     "ms_per_launch": sweep_ms, "ms_per_launch_stats": spread(sweep_all),
                     "algorithmic_flops_per_launch": sweep_flops, "traffic": sweep_dram_traffic(),
                     "traffic_source": SWEEP_PROFILE},
        "e2e": {"value": flops_all / (e2e_ms_all * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms_all,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        # forward: scale table, score sweep, row solve, its long-list rows, tile order, dense tiles; backward: scale
        # table, score sweep, row gradients, their long-list rows, tile marking, tile order, dense tiles (query-major
        # and key-major kernels), two gradient stores
        "gpu_launches": 16 * K,
        "clocks": clocks,
    }
    if density is not None:
        line["density_axis"] = {"note": "not part of `value`: the same shape and tensors with the temperature swept -- the "
                                "paper's regime (delta = 1, gamma = -0.5, Sec. 4.1) and fixed scales c; "
                                "supports grow as c falls", "runs": density}
    if nape is not None:
        line["nape_alibi"] = {"note": "not part of `value`: ALiBi slopes as in the paper's NAPE scheme (App. B); the hard "
                              "cutoff of entmax + ALiBi lets the sweep start each 256-row item at the first K tile that can "
                              "still hold a candidate", "runs": nape}
    if other is not None:
        line["other_workloads"] = {"note": "not part of `value`: forward / backward of the other workloads and alphas, median "
                                   "of 5 calls, L2 flushed before each", "runs": other}
    if decode is not None:
        hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
        for entry in decode:
            entry["frac_of_measured_hbm"] = entry["k_stream_gbs"] / hbm
        line["decode"] = {"note": "not part of `value`: entmax_attn_decode_fwd, q_len new rows against the workload's K, V "
                                  "as a cache of 32768 keys; bound by reading K once (algorithmic bytes = K bytes: 2*d per cached key "
                                  "and head); L2 flushed before every call", "hbm_peak_gbs": hbm, "runs": decode}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(inp, w, alpha, budget_s=args.cpu_seconds)
    print(json.dumps(line), flush=True)


def support_stats(params, ws, status):
    """Realised sparsity of a finished forward call: support sizes from the workspace (list rows and dense-path rows)."""
    from paper_2506_16640_b200 import binding
    lay = binding.entmax_attn_workspace_layout(params)
    total = params.batch * params.heads * params.seq
    cnt = ws[lay.row_count_offset: lay.row_count_offset + 4 * total].view(torch.int32)
    dn = ws[lay.dense_count_offset: lay.dense_count_offset + 8 * total].view(torch.int32).view(total, 2).sum(1)
    supp = torch.where(cnt == -2, dn, cnt).float()
    sample = supp[:: max(1, total // 200000)]
    st = status.tolist()
    return {"mean_support": float(supp.mean().item()), "p99_support": float(torch.quantile(sample, 0.99).item()),
            "max_support": int(supp.max().item()), "dense_path_rows": st[1], "dense_path_row_frac": st[1] / total,
            "dense_tiles": st[3], "sweeps_per_dense_tile": (st[2] / st[3]) if st[3] else 0.0}


def time_fwd_bwd(t, alpha, causal, beta, gamma, delta, flush, ws=None, iters=5):
    """Median forward / backward / forward-sweep times of one problem (L2 flushed before every call) and the
    realised sparsity of the forward pass."""
    from paper_2506_16640_b200 import binding
    dev = t["q"].device
    B, H, N, D = t["q"].shape
    params = binding.make_params(t["q"], alpha, causal)
    if ws is None:
        ws = binding.alloc_workspace(params, True, dev)
    st_f = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
    st_b = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
    o = torch.empty_like(t["q"])
    tau = torch.empty((B, H, N), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(t["q"]) for _ in range(3))
    ev = lambda: torch.cuda.Event(enable_timing=True)
    s0, s1 = ev(), ev()
    s0.record(); s1.record()
    torch.cuda.synchronize()
    binding.entmax_attn_profile_events(0, s0, s1)
    tf, tb, tsw, stats = [], [], [], None
    for it in range(iters + 2):
        flush.zero_()
        e0, e1, e2, e3 = ev(), ev(), ev(), ev()
        e0.record()
        binding.entmax_attn_fwd(t["q"], t["k"], t["v"], alpha, causal, beta, gamma, delta, o=o, tau=tau, workspace=ws,
                                status=st_f)
        e1.record()
        torch.cuda.synchronize()
        if stats is None:
            stats = support_stats(params, ws, st_f)     # before the backward call reuses the workspace
        flush.zero_()
        e2.record()
        binding.entmax_attn_bwd(t["q"], t["k"], t["v"], tau, t["d_o"], alpha, causal, beta, gamma, delta, dq=dq, dk=dk,
                                dv=dv, workspace=ws, status=st_b)
        e3.record()
        torch.cuda.synchronize()
        if it >= 2:
            tf.append(e0.elapsed_time(e1)); tb.append(e2.elapsed_time(e3)); tsw.append(s0.elapsed_time(s1))
    binding.entmax_attn_profile_events(0, None, None)
    assert int(st_f[0].item()) == 0 and int(st_b[0].item()) == 0, "device status flags set"
    pairs = (N * (N + 1) // 2 if causal else N * N) * B * H
    fwd_ms, bwd_ms, sweep_ms = statistics.median(tf), statistics.median(tb), statistics.median(tsw)
    out = {"fwd_ms": fwd_ms, "bwd_ms": bwd_ms, "fwd_sweep_ms": sweep_ms,
           "fwd_method_tflops": 2 * D * pairs / (fwd_ms * 1e-3) / 1e12,
           "fwd_sweep_method_tflops": 2 * D * pairs / (sweep_ms * 1e-3) / 1e12,
           "fwd_dense_equivalent_tflops": 4 * D * pairs / (fwd_ms * 1e-3) / 1e12,
           "bwd_dense_equivalent_tflops": 10 * D * pairs / (bwd_ms * 1e-3) / 1e12,
           "bwd_dense_path_rows": int(st_b[1].item())}
    out.update(stats)
    return out


def time_workload(index, alpha, flush, tensors=None, ws=None):
    """One of the seeded workloads (its own tensors unless given), forward + backward."""
    w = WORKLOADS[index]
    if tensors is None:
        inp = make_inputs(w)
        if inp.d_o is None:
            inp.d_o = seeded_d_o(w)
        dev = flush.device
        tensors = {n: getattr(inp, n).to(dev) for n in ("q", "k", "v", "d_o", "beta", "gamma", "delta")}
    res = time_fwd_bwd(tensors, alpha, w.causal, tensors["beta"], tensors["gamma"], tensors["delta"], flush, ws=ws)
    res.update({"workload": w.name, "alpha": alpha, "batch": w.B, "heads": w.H, "seq": w.N, "head_dim": w.d, "causal": w.causal})
    return res


def time_density_axis(d, w, alpha, flush, ws):
    """The benchmark's shape with the temperature swept: the paper's regime (delta = 1, gamma = -0.5, beta in
    {0.5, 1, 2}) and fixed scales c, on the workload's planted tensors and on plain seeded N(0,1) tensors."""
    dev = d["q"].device
    gen = torch.Generator(device=dev).manual_seed(BASE_SEED_DENSITY)
    plain = {n: torch.randn(d["q"].shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
             for n in ("q", "k", "v")}
    plain["d_o"] = d["d_o"]
    runs = []
    for label, t in (("planted", d), ("plain", plain)):
        cases = [("paper: delta=1, gamma=-0.5, beta=%g" % b, b, -0.5, 1.0) for b in (0.5, 1.0, 2.0)]
        cases += [("fixed c=%g" % c, 0.0, 1.0, c) for c in (1.0, 2.0, 4.0, 8.0)]
        for name, b, g, dl in cases:
            full = lambda x: torch.full((w.H,), x, dtype=torch.float32, device=dev)
            res = time_fwd_bwd(t, alpha, w.causal, full(b), full(g), full(dl), flush, ws=ws, iters=3)
            res.update({"tensors": label, "scale": name, "c_at_last_row": dl + b * float(np.log(w.N)) ** g})
            runs.append(res)
    return runs


def time_nape(d, w, alpha, flush, ws, iters=3):
    """The paper's NAPE scheme on the benchmark's tensors: ALiBi slopes on half of the heads (the original
    geometric sequence 2^(-8 j / n), j = 1..n), none on the other half; beside it all heads without and all heads
    with a slope.  The score sweep leaves out the K tiles beyond each item's hard-cutoff window."""
    from paper_2506_16640_b200 import binding
    dev = d["q"].device
    H = w.H
    geo = lambda n: [2.0 ** (-8.0 * (j + 1) / n) for j in range(n)]
    cases = [("no slopes (every head NoPE, same kernels)", [0.0] * H),
             ("NAPE: slopes on the first half of the heads", geo(H // 2) + [0.0] * (H - H // 2)),
             ("slopes on every head", geo(H))]
    o = torch.empty_like(d["q"])
    tau = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(d["q"]) for _ in range(3))
    ev = lambda: torch.cuda.Event(enable_timing=True)
    runs = []
    for label, slopes in cases:
        sl = torch.tensor(slopes, dtype=torch.float32, device=dev)
        st_f = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
        st_b = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
        tf, tb = [], []
        for it in range(iters + 2):
            flush.zero_()
            e0, e1, e2, e3 = ev(), ev(), ev(), ev()
            e0.record()
            binding.entmax_attn_fwd_ex(d["q"], d["k"], d["v"], alpha, w.causal, d["beta"], d["gamma"], d["delta"],
                                       alibi_slopes=sl, o=o, tau=tau, workspace=ws, status=st_f)
            e1.record()
            flush.zero_()
            e2.record()
            binding.entmax_attn_bwd_ex(d["q"], d["k"], d["v"], tau, d["d_o"], alpha, w.causal, d["beta"], d["gamma"],
                                       d["delta"], alibi_slopes=sl, dq=dq, dk=dk, dv=dv, workspace=ws, status=st_b)
            e3.record()
            torch.cuda.synchronize()
            if it >= 2:
                tf.append(e0.elapsed_time(e1)); tb.append(e2.elapsed_time(e3))
        f, b = st_f.tolist(), st_b.tolist()
        assert f[0] == 0 and b[0] == 0, "device status flags set"
        runs.append({"heads": label, "slopes": slopes, "fwd_ms": statistics.median(tf), "bwd_ms": statistics.median(tb),
                     "fwd_sweep_steps_skipped": f[4], "fwd_sweep_steps_scored": f[5],
                     "fwd_skipped_frac": f[4] / max(f[4] + f[5], 1), "bwd_skipped_frac": b[4] / max(b[4] + b[5], 1),
                     "dense_path_rows": f[1]})
    return runs


def time_decode(d, w, alpha, flush, iters=20):
    """Times entmax_attn_decode_fwd (two kernels per call) for 1 and 8 new query rows, on the workload's own
    tensors (one sequence) and on a batch of 8 seeded N(0,1) caches of the same shape; returns a list of dicts."""
    from paper_2506_16640_b200 import binding
    out = []
    ev = lambda: torch.cuda.Event(enable_timing=True)
    gen = torch.Generator(device=d["q"].device).manual_seed(20250616)
    big = [torch.randn((8, w.H, w.N, w.d), generator=gen, device=d["q"].device, dtype=torch.float32).to(torch.bfloat16)
           for _ in range(3)]
    cases = [("workload tensors, 1 sequence", d["q"], d["k"], d["v"]), ("seeded N(0,1), 8 sequences", *big)]
    for label, qf, kf, vf in cases:
        B = qf.shape[0]
        for q_len in (1, 8):
            q = qf[:, :, w.N - q_len:, :].contiguous()
            o, tau, supp = binding.entmax_attn_decode_fwd(q, kf, vf, alpha, None, d["beta"], d["gamma"], d["delta"])
            params = binding.DecodeParams(B, w.H, q_len, w.N, w.d, float(alpha), 0.0, 0, 0, 0)
            ws = torch.empty(binding.load().entmax_attn_decode_workspace_bytes(ctypes.byref(params)), dtype=torch.uint8,
                             device=q.device)
            starts, stops = [ev() for _ in range(iters)], [ev() for _ in range(iters)]
            for i in range(iters + 3):
                flush.zero_()
                j = max(i - 3, 0)
                starts[j].record()
                binding.entmax_attn_decode_fwd(q, kf, vf, alpha, None, d["beta"], d["gamma"], d["delta"], o=o, tau=tau,
                                               support_size=supp, workspace=ws)
                stops[j].record()
            torch.cuda.synchronize()
            ms = sorted(a.elapsed_time(b) for a, b in zip(starts, stops))[iters // 2]
            k_bytes = B * w.H * w.N * w.d * 2
            out.append({"inputs": label, "batch": B, "q_len": q_len, "ms": ms, "k_bytes": k_bytes,
                        "k_stream_gbs": k_bytes / (ms * 1e-3) / 1e9, "mean_support": float(supp.float().mean().item())})
    return out


def _oracle_heads(inp, w):
    """Per (batch, head) float32 numpy views of the inputs, prepared once outside any timed region."""
    out = []
    for bh in range(w.B * w.H):
        b, h = divmod(bh, w.H)
        out.append(tuple(t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o)))
    return out


def _oracle_pass(inp, w, alpha, heads, rows_per_head: int, seed: int):
    """Oracle forward rows + row-local backward (dQ) rows on `rows_per_head` sampled rows of every head.
    Returns (seconds, useful FLOPs of those rows, number of rows)."""
    import oracle
    flops = 0
    nrows = 0
    t0 = time.perf_counter()
    for bh in range(w.B * w.H):
        h = bh % w.H
        rows = sample_rows(inp, bh, rows_per_head, seed=seed)
        q, k, v, g = heads[bh]
        oracle.attn_fwd_rows(q, k, v, rows, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h))
        oracle.attn_bwd_rows(q, k, v, g, rows, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h))
        vis = (rows + 1) if w.causal else np.full_like(rows, w.N)
        flops += int(vis.sum()) * 14 * w.d
        nrows += len(rows)
    return time.perf_counter() - t0, flops, nrows


def _sized_rows_per_head(inp, w, alpha, heads, budget_s: float):
    """Rows per head that make one oracle pass last about `budget_s` seconds (two pilots, the second
    large enough that fixed per-call costs no longer dominate the estimate)."""
    rows = 16
    for _ in range(2):
        secs, _, n = _oracle_pass(inp, w, alpha, heads, rows, seed=1)
        per_row = max(secs / n, 1e-7)
        rows = int(max(8, min(w.N, budget_s / per_row / (w.B * w.H))))
        if secs > 0.2 * budget_s:
            break
    return rows


def cpu_baseline(inp, w, alpha, budget_s: float = 15.0):
    """The fp64 oracle, as it stands, on the host cores of this machine, on a bounded row sample of the same
    workload (pilots size the sample for about `budget_s` seconds)."""
    import oracle
    heads = _oracle_heads(inp, w)
    rows_per_head = _sized_rows_per_head(inp, w, alpha, heads, budget_s)
    secs, flops, nrows = _oracle_pass(inp, w, alpha, heads, rows_per_head, seed=2)
    cores = oracle.num_threads()
    # the same oracle on one thread, on a sample sized for a few seconds
    one_rows = max(4, int(rows_per_head * 4.0 / max(secs, 1e-3) / max(cores, 1)))
    oracle.set_num_threads(1)
    try:
        secs1, flops1, nrows1 = _oracle_pass(inp, w, alpha, heads, min(one_rows, rows_per_head), seed=3)
    finally:
        oracle.set_num_threads(cores)
    return {"value": flops / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d sampled query rows (%d per head) of the same workload: oracle forward rows plus the "
                      "row-local backward (dQ) rows, %.1f s; useful FLOPs of those rows / time" % (nrows, rows_per_head, secs),
            "rows_per_s": nrows / secs, "extrapolated_full_step_s": (w.B * w.H * w.N) * secs / nrows,
            "one_thread": {"value": flops1 / secs1 / 1e12, "unit": UNIT, "rows_per_s": nrows1 / secs1,
                           "sample": "%d rows, %.1f s" % (nrows1, secs1)}}


def run_reference(args):
    """The reference arm: the CPU oracle itself, timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w, inp = make_bench_inputs(args.alpha)
    heads = _oracle_heads(inp, w)
    total_budget = 90.0
    steps = args.steps + max(args.warmup, 1)
    rows_per_head = _sized_rows_per_head(inp, w, args.alpha, heads, total_budget / steps)
    for i in range(max(args.warmup, 1)):
        _oracle_pass(inp, w, args.alpha, heads, rows_per_head, seed=10 + i)
    secs = flops = nrows = 0
    for i in range(args.steps):
        s, f, n = _oracle_pass(inp, w, args.alpha, heads, rows_per_head, seed=100 + i)
        secs, flops, nrows = secs + s, flops + f, nrows + n
    value = flops / secs / 1e12
    sample = "each step = %d sampled query rows per head (oracle forward + row-local backward)" % rows_per_head
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": secs / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.B, "heads": w.H, "seq": w.N, "head_dim": w.d, "causal": w.causal,
                       "alpha": args.alpha, "step": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--alpha", type=float, default=1.5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the temperature axis and the other workloads")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
