#!/usr/bin/env python
"""Benchmark of the d2Cache decode step (d2c_step) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole hot path (selection, gather, layers on the selected rows,
LM head on the masked rows, rollout) over one batch of seeded synthetic input.  The default
workload is one LLaDA-8B-shaped layer at sequence length 1024 (prefill, then the timed partial
step with k=32, p=0.9).  Prints one JSON line.

The path does not shard (one model replica per GPU, no exchange step): with --gpus N every rank
runs an independent replica and the line reports the aggregate.  Started without a launcher,
`--gpus N` (N > 1) re-executes itself under `python -m torch.distributed.run` with N ranks on
127.0.0.1; started by a launcher (WORLD_SIZE set) it takes its rank from the environment.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_23094_b200 import inputs  # noqa: E402

METRIC = "d2c_step selected tokens/s"
UNIT = "selected_tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only queries) from a thread while the
    timed region runs; nvidia-smi's own sampling period is longer than a whole timed pass of the small
    workloads.  Falls back to one nvidia-smi query if NVML cannot be loaded."""

    def __init__(self, index: int):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop, self._thread, self._nvml = False, None, None

    def _loop(self):
        nv, h = self._nvml, self._handle
        bits = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown, "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown, "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        while not self._stop:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                for name, bit in bits.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.0005)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            # NVML counts physical devices; honour CUDA_VISIBLE_DEVICES when it lists ordinals
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            ids = [v for v in vis.split(",") if v.strip().isdigit()]
            phys = int(ids[self.index]) if self.index < len(ids) else self.index
            self._handle = nv.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(self._handle, nv.NVML_CLOCK_SM))
            self._nvml = nv
            import threading
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        except Exception:
            self._nvml = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self._nvml is not None:
            self._stop = True
            self._thread.join(timeout=2)
            if self.samples:
                out.update(sm_mhz=float(statistics.median(self.samples)), sm_max_mhz=self.max_mhz,
                           reasons=sorted(self.reasons), samples=len(self.samples))
            return out
        try:
            q = "clocks.sm,clocks.max.sm"
            txt = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}", "--format=csv,noheader,nounits"],
                                 capture_output=True, text=True, timeout=10).stdout.strip().split(",")
            out.update(sm_mhz=float(txt[0]), sm_max_mhz=float(txt[1]), samples=1)
        except Exception:
            pass
        return out


def algorithmic_work(shape, batch, L, n_b, n_m, rollout_layers):
    """FLOPs and HBM bytes one step has to do (selected rows only; each weight read once)."""
    n = sum(n_b)
    P_l = shape.params_per_layer
    N, d, Hq, Hkv, Dh, V = shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.vocab
    flops = N * (2 * n * P_l + 4 * Hq * Dh * sum(nb * L for nb in n_b)) + 2 * n_m * d * V
    byts = 2 * N * P_l + 2 * d * V
    byts += N * sum(2 * L * Hkv * Dh * 2 + 2 * nb * Hkv * Dh * 2 for nb in n_b)
    byts += 2 * n * d * 2
    byts += rollout_layers * sum(2 * nb * L * 4 for nb in n_b)
    return flops, byts


def profiled_traffic(kernel_tag, path=None):
    """DRAM bytes (read + write) of one launch of a kernel, from the committed ncu summary of this workload:
    the first block of profiles/gemm_tc2_kernel_llada1l_1024.txt whose header names `kernel_tag`.
    Returns (bytes, source) or (None, reason)."""
    path = path or os.path.join(ROOT, "profiles", "gemm_tc2_kernel_llada1l_1024.txt")
    unit = {"Gbyte": 1e9, "Mbyte": 1e6, "Kbyte": 1e3, "byte": 1.0}
    try:
        lines = open(path).read().splitlines()
    except OSError:
        return None, "no committed ncu summary"
    rd = wr = None
    inside = False
    for ln in lines:
        if not ln.startswith(" "):
            if inside and rd is not None and wr is not None:
                break
            inside = kernel_tag in ln
            continue
        if inside:
            f = ln.split()
            if len(f) >= 3 and f[0] == "dram__bytes_read.sum":
                rd = float(f[1]) * unit.get(f[2], 1.0)
            if len(f) >= 3 and f[0] == "dram__bytes_write.sum":
                wr = float(f[1]) * unit.get(f[2], 1.0)
    if rd is None or wr is None:
        return None, "kernel not found in " + os.path.relpath(path, ROOT)
    return rd + wr, os.path.relpath(path, ROOT) + " (ncu, committed capture of this workload)"


def aggregate_replicas(total_ms, e2e_s, rows, world, device):
    """Whole-job numbers of `world` independent replicas: the slowest rank's times, the sum of the rows."""
    if world <= 1:
        return total_ms, e2e_s, rows
    t = torch.tensor([total_ms, e2e_s, rows], dtype=torch.float64, device=device)
    tmax = t.clone(); torch.distributed.all_reduce(tmax, op=torch.distributed.ReduceOp.MAX)
    tsum = t.clone(); torch.distributed.all_reduce(tsum, op=torch.distributed.ReduceOp.SUM)
    return float(tmax[0]), float(tmax[1]), float(tsum[2])


def build_pair(wl, device, rollout_layers=0, flags=0):
    from paper_2509_23094_b200 import binding
    w_cpu = inputs.make_weights(wl.shape, seed=wl.seed, device=device if wl.shape.n_layers > 4 else "cpu")
    w_dev = {"layers": [{k: (None if v is None else v.to(device)) for k, v in lyr.items()} for lyr in w_cpu["layers"]],
             "g_final": w_cpu["g_final"].to(device), "w_lm": w_cpu["w_lm"].to(device), "embed": w_cpu["embed"].to(device)}
    cfg = binding.make_config(wl.shape, wl.batch, wl.seq_len, sigma=wl.sigma, rollout_layers=rollout_layers, flags=flags)
    ctx = binding.Context(cfg, w_dev, device=device)
    mask = inputs.make_mask(wl)
    tokens = inputs.make_tokens(wl, mask)
    h0 = w_dev["embed"][tokens.to(device)].contiguous()
    return w_cpu, w_dev, ctx, mask, tokens, h0


def run_ours(args, rank, world, device):
    wl = inputs.WORKLOADS[args.workload]
    if args.p is not None or args.k is not None:
        from dataclasses import replace as _replace
        wl = _replace(wl, p=wl.p if args.p is None else args.p, k=wl.k if args.k is None else args.k)
    shape, B, L, d = wl.shape, wl.batch, wl.seq_len, wl.shape.d_model
    w_cpu, w_dev, ctx, mask, tokens, h0 = build_pair(wl, device, args.rollout_layers, args.flags)
    mask_dev = mask.to(device)
    stream = torch.cuda.current_stream()

    # prefill: every row, fills the cache, the confidences and the rollout scores
    ctx.step(h0, mask_dev, 10 ** 6, 1.0)
    ctx.sync_status()
    snap = {n: ctx.view(n, B, L).clone() for n in ("conf", "pred", "c")}
    if args.scores == "zipf":
        # paper-like peaked stage-2 scores instead of the nearly flat ones random weights give: seeded Zipf(1.0)
        # over the positions of every sequence; top-p then keeps few rows for the same p
        for b in range(B):
            snap["c"][b] = inputs.make_scores(L, seed=wl.seed + 1000 + b, kind="zipf").to(device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)       # > L2 (126 MB)
    hid = torch.zeros(B * L, d, dtype=torch.bfloat16, device=device)

    def restore():
        for n, t in snap.items():
            ctx.view(n, B, L).copy_(t)
        flush.fill_(1)

    sampler = ClockSampler(torch.cuda.current_device())
    for _ in range(args.warmup):
        restore()
        ctx.step(h0, mask_dev, wl.k, wl.p, hidden_out=hid)
        torch.cuda.synchronize()         # lets the library's row-count hint settle before the timed passes
    ctx.sync_status()
    row_off = ctx.view("row_off", B, L).cpu().numpy()
    lm_off = ctx.view("lm_off", B, L).cpu().numpy()
    n_b = [int(row_off[b + 1] - row_off[b]) for b in range(B)]
    n, n_m = int(row_off[B]), int(lm_off[B])

    def timed_pass(profile, steps, p=None):
        """`steps` steps, each bracketed by CUDA events on the step's stream; state restored and L2 flushed between steps."""
        p = wl.p if p is None else p
        e0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        e1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        if profile:
            ctx.profile(True)
            ctx.profile_read(reset=True)
        for i in range(steps):
            restore()
            e0[i].record(stream)
            ctx.step(h0, mask_dev, wl.k, p, hidden_out=hid)
            e1[i].record(stream)
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        ph = None
        if profile:
            ph = ctx.profile_read(reset=True)
            ctx.profile(False)
        return [a.elapsed_time(b) for a, b in zip(e0, e1)], ph

    # Pass 1 gives the headline: exactly K steps with no events inside the step, so the kernels' programmatic
    # dependent launches overlap as they do for a user.  Pass 2 repeats the step with one event at every phase
    # boundary (which serialises the launches) and gives the per-phase and per-kernel times; it runs long enough
    # (at least 100 steps of the short workloads) for the clock sampler to collect a usable number of readings.
    prof_steps = args.profile_steps if args.profile_steps > 0 else (args.steps if shape.n_layers > 4 else max(args.steps, 100))
    sampler.start()
    per_step_ms, _ = timed_pass(False, args.steps)
    per_step_ms_profiled, phases = timed_pass(True, prof_steps)
    clocks = sampler.stop()
    ctx.sync_status()
    total_ms = sum(per_step_ms)
    # SM clock inside the last profiled gate/up launch: clock64 against the global timer, stamped by CTA 0
    gc = ctx.view("gemm_clocks").cpu().tolist()
    mhz_in_gemm = round((gc[2] - gc[0]) / (gc[3] - gc[1]) * 1e3, 1) if gc[3] > gc[1] else None

    # end to end: host buffers in, host results out, through d2c_step_host
    h0_host = h0.cpu().pin_memory(); mask_host = mask.pin_memory()
    sel_h = torch.empty(B * L, dtype=torch.int32).pin_memory(); ro_h = torch.empty(B + 1, dtype=torch.int32).pin_memory()
    hid_h = torch.empty(B * L, d, dtype=torch.bfloat16).pin_memory()
    conf_h = torch.empty(B, L).pin_memory(); pred_h = torch.empty(B, L, dtype=torch.int32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    e2e_s = 0.0
    for i in range(2 + e2e_steps):
        restore()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ctx.step_host(h0_host, mask_host, wl.k, wl.p, sel_idx=sel_h, row_off=ro_h, hidden_out=hid_h, conf=conf_h, pred=pred_h)
        if i >= 2:
            e2e_s += time.perf_counter() - t0
    h2d = B * L * d * 2 + B * L
    d2h = (B + 1) * 4 + B * L * 4 + B * L * d * 2 + 2 * B * L * 4       # worst-case sizes: the row count is not known when the copies start

    total_ms, e2e_s, n_all = aggregate_replicas(total_ms, e2e_s, float(n), world, device)
    ms_per_step = total_ms / args.steps
    value = n_all / (ms_per_step * 1e-3)
    e2e_value = n_all / (e2e_s / e2e_steps)

    peaks = measured_peaks()
    depth = args.rollout_layers if 0 < args.rollout_layers < shape.n_layers else shape.n_layers
    flops, byts = algorithmic_work(shape, B, L, n_b, n_m, depth)
    t_roof = max(flops / (peaks["bf16_tflops"] * 1e12), byts / (peaks["hbm_gbs"] * 1e9))
    # The same bound taken stage by stage: the LM head needs the last layer's output, so the layers (tensor-bound at
    # many rows, weight-stream-bound at few) and the LM head (always bound by its weight stream) cannot overlap and
    # their bounds add.  Reported beside the single max(), which lets the two resources overlap freely.
    lm_flops, lm_byts = 2 * n_m * shape.d_model * shape.vocab, 2 * shape.d_model * shape.vocab
    bound = lambda f, b: max(f / (peaks["bf16_tflops"] * 1e12), b / (peaks["hbm_gbs"] * 1e9))
    t_roof_serial = bound(flops - lm_flops, byts - lm_byts) + bound(lm_flops, lm_byts)
    # Denominator: the burst cuBLAS figure for a kernel inside a short step; the sustained one when the clock
    # record of the timed region shows the power cap holding the SM clock below 90 % of its maximum.
    capped = "sw_power_cap" in clocks.get("reasons", []) and clocks.get("sm_mhz", 0) < 0.9 * (clocks.get("sm_max_mhz") or 0)
    tensor_peak = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
    peak_kind = " sustained (power-capped step)" if capped else " burst"
    # Per-kernel figures come from the events of the second (profiled) pass.  The four projection GEMMs of a
    # layer are tensor-bound at this row count, the LM head streams its weights once and is HBM-bound.
    Hq, Hkv, Dh, F = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn
    gemm_shapes = {"gemm_qkv": (d, (Hq + 2 * Hkv) * Dh), "gemm_o": (Hq * Dh, d), "gemm_gate_up": (d, 2 * F), "gemm_down": (F, d)}
    gemms = {}
    for name, (kk, nn) in gemm_shapes.items():
        ms = phases[name]["ms"] / prof_steps / shape.n_layers
        tf = 2.0 * n * kk * nn / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
        gemms[name] = {"launch_ms": round(ms, 4), "achieved": round(tf, 1), "frac": round(tf / tensor_peak, 4)}
    gu_ms = gemms["gemm_gate_up"]["launch_ms"]
    achieved = gemms["gemm_gate_up"]["achieved"]
    gemm_ms = sum(phases[k]["ms"] for k in gemm_shapes) / prof_steps
    gemm_flops = shape.n_layers * 2 * n * shape.params_per_layer
    # DRAM bytes of one gate/up launch: read from the committed ncu summary of this workload, null elsewhere
    traffic, traffic_source = (profiled_traffic("gate/up") if wl.name == "llada1l_1024" and args.p is None and args.scores == "rollout"
                               else (None, "no capture of this workload"))
    roofline = {"bound": "tensor", "kernel": "gemm_tc2_kernel<SWIGLU> (gate/up projection, 1 launch per layer; the GEMM with the most FLOPs)",
                "achieved": round(achieved, 2), "peak": tensor_peak, "peak_source": peaks["source"] + peak_kind,
                "unit": "TFLOP/s", "frac": round(achieved / tensor_peak, 4),
                "frac_of_burst": round(achieved / peaks["bf16_tflops"], 4), "traffic": traffic, "traffic_source": traffic_source,
                "algorithmic_bytes": 2 * d * 2 * shape.d_ffn + n * d * 2 + n * shape.d_ffn * 2,
                "launch_ms": round(gu_ms, 4),
                # what the launch took in SM clocks: by the NVML samples of the timed region, and by the clock the
                # kernel itself saw (clock64 against the global timer inside CTA 0)
                "launch_cycles_at_sampled_clock": round(gu_ms * 1e-3 * (clocks.get("sm_mhz") or 0) * 1e6),
                "sm_mhz_inside_launch": mhz_in_gemm,
                "launch_cycles_at_kernel_clock": round(gu_ms * 1e-3 * mhz_in_gemm * 1e6) if mhz_in_gemm else None,
                "gemms": gemms,
                "all_gemms": {"achieved": round(gemm_flops / (gemm_ms * 1e-3) / 1e12, 2) if gemm_ms > 0 else 0.0,
                              "ms_per_step": round(gemm_ms, 4)},
                "step_roofline_ms": round(t_roof * 1e3, 4), "step_frac": round(t_roof * 1e3 / ms_per_step, 4),
                "step_roofline_layers_then_lm_head_ms": round(t_roof_serial * 1e3, 4),
                "step_frac_layers_then_lm_head": round(t_roof_serial * 1e3 / ms_per_step, 4),
                "step_flops": flops, "step_bytes": byts}
    lm_ms = phases["lm_head"]["ms"] / prof_steps
    lm_bytes = 2 * d * shape.vocab
    roofline["lm_head"] = {"bound": "hbm", "kernel": "gemm_tc_kernel<LMSTATS> (the longest single launch of the step)",
                           "achieved": round(lm_bytes / (lm_ms * 1e-3) / 1e9, 1) if lm_ms > 0 else 0.0,
                           "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": round(lm_bytes / (lm_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4) if lm_ms > 0 else 0.0,
                           "ms_per_step": round(lm_ms, 4)}
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "shape": shape.name, "batch": B, "seq_len": L, "k": wl.k, "p": wl.p,
                   "selected_rows": n_b, "lm_rows": n_m, "l2": "flushed between steps; weights (%.2f GB) exceed L2" %
                   ((2 * shape.n_layers * shape.params_per_layer + 2 * d * shape.vocab) / 1e9),
                   "replicas": world, "scores": args.scores, "rollout_layers": depth},
        "clocks": clocks,
        "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_s / e2e_steps * 1e3, 4)},
        "gpu_launches": int(round(sum(p["launches"] for p in phases.values()) * args.steps / prof_steps)),
        "roofline": roofline,
        "phases_ms_per_step": {k: round(v["ms"] / prof_steps, 4) for k, v in phases.items()},
        "step_ms_min": round(min(per_step_ms), 4), "step_ms_median": round(statistics.median(per_step_ms), 4),
        "ms_per_step_with_phase_events": round(sum(per_step_ms_profiled) / prof_steps, 4), "profiled_steps": prof_steps,
    }
    # The same workload at the paper's default threshold (Section 5.1: p = 0.1, about a hundred selected rows:
    # the weight-streaming regime), as a labelled extra; the library picks its few-row kernels from the previous
    # step's row count, so two untimed steps come first.
    if rank == 0 and world == 1 and shape.n_layers <= 4 and args.p is None and args.scores == "rollout" and not args.no_extras:
        for _ in range(3):
            restore()
            ctx.step(h0, mask_dev, wl.k, 0.1, hidden_out=hid)
            torch.cuda.synchronize()
        ro01 = ctx.view("row_off", B, L).cpu().numpy(); lo01 = ctx.view("lm_off", B, L).cpu().numpy()
        nb01 = [int(ro01[b + 1] - ro01[b]) for b in range(B)]
        ms01, _ = timed_pass(False, args.steps, p=0.1)
        _, ph01 = timed_pass(True, prof_steps, p=0.1)
        fl01, by01 = algorithmic_work(shape, B, L, nb01, int(lo01[B]), depth)
        roof01 = max(fl01 / (peaks["bf16_tflops"] * 1e12), by01 / (peaks["hbm_gbs"] * 1e9))
        g01 = sum(ph01[k]["ms"] for k in gemm_shapes) / prof_steps
        wbytes = 2 * shape.n_layers * shape.params_per_layer
        line["paper_default_p0.1"] = {
            "selected_rows": nb01, "lm_rows": int(lo01[B]), "ms_per_step": round(sum(ms01) / args.steps, 4),
            "step_roofline_ms": round(roof01 * 1e3, 4), "step_frac": round(roof01 * 1e3 / (sum(ms01) / args.steps), 4),
            "all_gemms": {"ms_per_step": round(g01, 4), "weight_gbs": round(wbytes / (g01 * 1e-3) / 1e9, 1) if g01 > 0 else 0.0,
                          "frac_of_hbm": round(wbytes / (g01 * 1e-3) / 1e9 / peaks["hbm_gbs"], 4) if g01 > 0 else 0.0},
            "phases_ms_per_step": {k: round(v["ms"] / prof_steps, 4) for k, v in ph01.items()}}
        for _ in range(2):                                    # back to the workload's own regime
            restore()
            ctx.step(h0, mask_dev, wl.k, wl.p, hidden_out=hid)
            torch.cuda.synchronize()
    if args.decode:
        line["decode"] = decode_loop(ctx, wl, w_dev, mask, tokens, device)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, w_cpu, mask, tokens, ctx, B, L)
    return line


def decode_loop(ctx, wl, w_dev, mask, tokens, device):
    """The whole decoding loop of the workload (Eq. 2): prefill, then until no [MASK] is left: commit
    the most confident refreshed position of every sequence, run one d2c_step with that position forced.
    Everything stays on the device; the host synchronises once at the end."""
    B, L = wl.batch, wl.seq_len
    gen = int(mask[0].sum())
    mask_dev = mask.to(device).contiguous()
    tok = tokens.to(torch.int32).to(device).contiguous()
    h0 = w_dev["embed"][tokens.to(device)].contiguous()
    committed = torch.full((B,), -1, dtype=torch.int32, device=device)
    forced_off = torch.arange(B + 1, dtype=torch.int32, device=device)
    torch.cuda.synchronize()
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    stream = torch.cuda.current_stream()
    e0.record(stream)
    ctx.step(h0, mask_dev, 10 ** 6, 1.0)
    e1.record(stream)
    for _ in range(gen):
        ctx.commit(w_dev["embed"], h0, mask_dev, tok, committed, rule=0)
        ctx.step(h0, mask_dev, wl.k, wl.p, forced=committed, forced_off=forced_off)
    e2.record(stream)
    torch.cuda.synchronize()
    ctx.sync_status()
    left = int(mask_dev.sum())
    prefill_ms, loop_ms = e0.elapsed_time(e1), e1.elapsed_time(e2)
    return {"generated_tokens": B * gen - left, "masks_left": left, "steps": gen, "prefill_ms": round(prefill_ms, 3),
            "ms_per_step": round(loop_ms / gen, 4), "tokens_per_s": round((B * gen - left) / ((prefill_ms + loop_ms) * 1e-3), 2),
            "total_s": round((prefill_ms + loop_ms) * 1e-3, 4)}


def oracle_setup(wl, w_cpu, mask, tokens):
    from oracle import step as ostep
    wf = ostep.weights_to_f64(w_cpu)
    h0 = inputs.make_h0(w_cpu["embed"].cpu(), tokens).double().numpy()
    st = ostep.OracleState(wl.shape.n_layers, wl.batch, wl.seq_len, wl.shape.n_kv_heads, wl.shape.head_dim)
    return ostep, wf, h0, st


def blas_threads():
    """Threads the oracle's numpy matmuls run on (the BLAS pool's size), else the host's core count."""
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n and max(n) > 0:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count()


def cpu_baseline(wl, w_cpu, mask, tokens, ctx, B, L, max_rows=1024):
    """The oracle, as it stands, on the host cores: one partial step on a bounded sample of the rows."""
    if wl.shape.n_layers > 4:
        return {"value": None, "unit": UNIT, "kind": "oracle", "cores": blas_threads(),
                "sample": "skipped: the full-depth model does not fit the CPU time budget"}
    ostep, wf, h0, st = oracle_setup(wl, w_cpu, mask, tokens)
    row_off = ctx.view("row_off", B, L).cpu().numpy()
    sel = ctx.view("sel_idx").cpu().numpy()
    # the cache the sampled rows attend to: taken from a full oracle forward of layer inputs would cost
    # a prefill; the timing only needs a cache of the right shape, so it is filled with random values
    rng = np.random.default_rng(0)
    st.Kc[:] = rng.standard_normal(st.Kc.shape) * 0.1
    st.Vc[:] = rng.standard_normal(st.Vc.shape) * 0.1
    sample = []
    for b in range(B):
        S = sel[row_off[b]: row_off[b + 1]].astype(np.int64)
        take = max(1, max_rows // B)
        sample.append(S[:: max(1, len(S) // take)][:take])
    rows = sum(len(s) for s in sample)
    # the same step is repeated until about 10 s of CPU work have been timed (at most 30 times)
    reps, dt = 0, 0.0
    while reps < 30 and dt < 10.0:
        t0 = time.perf_counter()
        ostep.oracle_step(st, wf, wl.shape, h0, mask.numpy(), k=0, p=0.0, sigma=wl.sigma, sel_override=sample)
        dt += time.perf_counter() - t0
        reps += 1
    return {"value": round(rows * reps / dt, 2), "unit": UNIT, "kind": "oracle (fp64 numpy, as it stands)", "cores": blas_threads(),
            "sample": f"{reps} oracle steps, each on {rows} of the selected rows (fp64 numpy), {dt:.1f} s in all"}


def run_reference(args):
    """Times the oracle on the host cores; each step is one partial step on a bounded sample of rows."""
    wl = inputs.WORKLOADS[args.workload]
    if wl.shape.n_layers > 4:
        print(json.dumps({"impl": "reference", "unavailable": "the full-depth workload does not fit the CPU time budget"}))
        return
    B, L = wl.batch, wl.seq_len
    w_cpu = inputs.make_weights(wl.shape, seed=wl.seed)
    mask = inputs.make_mask(wl)
    tokens = inputs.make_tokens(wl, mask)
    ostep, wf, h0, st = oracle_setup(wl, w_cpu, mask, tokens)
    rng = np.random.default_rng(0)
    st.Kc[:] = rng.standard_normal(st.Kc.shape) * 0.1
    st.Vc[:] = rng.standard_normal(st.Vc.shape) * 0.1
    st.conf[:] = rng.random(st.conf.shape).astype(np.float32)
    st.c[:] = (1.0 + 0.05 * rng.standard_normal(st.c.shape)).astype(np.float32)
    from oracle import selection as osel
    rows_per_step = 256
    sample = []
    for b in range(B):
        S, _, _ = osel.select_rows(mask[b].numpy(), st.conf[b], st.c[b], wl.k, wl.p, wl.sigma)
        take = max(1, rows_per_step // B)
        sample.append(S[:: max(1, len(S) // take)][:take])
    rows = sum(len(s) for s in sample)
    snap_conf, snap_c = st.conf.copy(), st.c.copy()
    times = []
    for i in range(args.warmup + args.steps):
        st.conf[:] = snap_conf; st.c[:] = snap_c
        t0 = time.perf_counter()
        ostep.oracle_step(st, wf, wl.shape, h0, mask.numpy(), k=0, p=0.0, sigma=wl.sigma, sel_override=sample)
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * sum(times) / len(times)
    value = rows / (ms * 1e-3)
    desc = f"each step: one oracle step on {rows} of the selected rows (fp64 numpy)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 2), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "shape": wl.shape.name, "batch": B, "seq_len": L, "k": wl.k, "p": wl.p},
        "cpu_baseline": {"value": round(value, 2), "unit": UNIT, "kind": "oracle (fp64 numpy, as it stands)", "cores": blas_threads(), "sample": desc},
        "e2e": {"value": round(value, 2), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="llada1l_1024", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode", action="store_true", help="also run the workload's whole decoding loop")
    ap.add_argument("--p", type=float, default=None, help="override the workload's top-p threshold (e.g. the paper's default 0.1)")
    ap.add_argument("--k", type=int, default=None, help="override the workload's k")
    ap.add_argument("--rollout-layers", type=int, default=0,
                    help="roll the attention out over the first n layers only (the paper's Rollout-5 variant); 0 = all layers")
    ap.add_argument("--flags", type=int, default=0, help="D2C_FLAG_* bits for the context (kernel variants kept as cross-checks)")
    ap.add_argument("--profile-steps", type=int, default=0, help="steps of the second, phase-timed pass (default: max(steps, 100) for the short workloads)")
    ap.add_argument("--no-extras", action="store_true", help="skip the labelled extra run at the paper's default p = 0.1")
    ap.add_argument("--scores", default="rollout", choices=["rollout", "zipf"],
                    help="stage-2 scores before each timed step: the prefill's rollout (default) or a seeded Zipf(1.0)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher: start the N ranks ourselves (one process per GPU, rendezvous on the loopback address)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=torch.device(device))
    line = run_ours(args, rank, world, device)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
