#!/usr/bin/env python
"""Benchmark of the beam-shared GDN decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4]

One STEP is one whole generation of the workload through the C ABI: reset, store every shared state
(a1), then for every decode call: reorder_beams (a2) and, per layer, append_records (a3) and the fused
decode_step (a4-a6); by default the last two are the one-launch append_decode_step.  The default workload is the 16-layer beam-512 decode stack (benchmark config 4:
4 requests x 16 layers x 32 heads, dk = dv = 128, depth 8, Zipf(1.5) parents, bf16 records, fp32 S_0),
whose per-step inputs (4.6 GiB) are far larger than L2.

Printed JSON line: `value` = beam-head decodes/s with inputs resident in HBM (CUDA-graph replay of the
step, timed with CUDA events, max over ranks); `e2e` = the same metric with every input copied from
pinned host memory and every output copied back inside the timed region; `roofline` = algorithmic bytes
of the decode launches / their CUDA-event durations against the measured HBM peak; `cpu_baseline` = the
fp64 oracle timed on the host cores on a bounded sample of the same workload.

`--impl reference` times the CPU oracle alone (there is no other reference implementation).
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
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2609_12399_b200 import accounting, inputs, replicas  # noqa: E402

METRIC = "beam-head GDN decodes/s per layer at beam 512"
UNIT = "decodes/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of ONE fused append + decode launch of the default workload at its
# deepest call, as the latest ncu capture found it: read from the summary that the capture's notes keep under
# profiles/ (key = value lines, with the commit the capture was taken on), never a constant in this file.
TRAFFIC_SUMMARY = ROOT / "profiles" / "decode_ws_kernel_cfg4_traffic.txt"


def ncu_traffic() -> dict:
    if not TRAFFIC_SUMMARY.exists():
        return {"bytes": None, "source": "no capture summary under profiles/"}
    kv = {}
    for ln in TRAFFIC_SUMMARY.read_text().splitlines():
        if "=" in ln and not ln.lstrip().startswith("#"):
            k, v = ln.split("=", 1)
            kv[k.strip()] = v.strip()
    try:
        total = float(kv["dram_bytes_read"]) + float(kv["dram_bytes_write"])
    except (KeyError, ValueError):
        return {"bytes": None, "source": f"{TRAFFIC_SUMMARY.name} is incomplete"}
    return {"bytes": total, "source": f"profiles/{TRAFFIC_SUMMARY.name}: ncu capture of one launch at depth {kv.get('depth', '?')}, "
                                      f"kernel source at commit {kv.get('commit', '?')}"}


def workload_by_name(name: str) -> inputs.Workload:
    for i, wl in enumerate(inputs.WORKLOADS):
        if name in (wl.name, f"cfg{i}"):
            return wl
    raise SystemExit(f"unknown workload {name!r}")


def describe(wl: inputs.Workload) -> str:
    idx = inputs.WORKLOADS.index(wl) if wl in inputs.WORKLOADS else -1
    dims = f"dk=dv={wl.dk}" if wl.dk == wl.dv else f"dk={wl.dk}, dv={wl.dv}"
    return (f"configs[{idx}] {wl.name}: {wl.R} requests x {wl.L} layers x {wl.H} heads, {dims}, "
            f"{wl.prompt_len}-token prompts, beam {wl.W}, depth {wl.D}, {wl.parents} parents"
            + (f"(s={wl.zipf_s})" if wl.parents == "zipf" else "") + f", {wl.dtype} records, fp32 S_0")


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=5)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def launch_bytes(wl: inputs.Workload, out_bytes: int, fused: bool) -> list:
    """Algorithmic / un-deduplicated bytes of one decode launch (all requests, one layer) per call depth.
    A fused append + decode launch also writes the call's records to the arena (it reads them from the
    caller's tensors instead of the arena: same read bytes)."""
    res = []
    par = {r: [None] + [inputs.parents(wl, r, t).numpy() for t in range(1, wl.D)] for r in range(wl.R)}
    for t in range(wl.D):
        distinct = [sum(accounting.distinct_records(par[r][:t + 1], [wl.W] * (t + 1))) for r in range(wl.R)]
        d = accounting.decode_bytes(R=wl.R, H=wl.H, dk=wl.dk, dv=wl.dv, W=wl.W, depth=t + 1,
                                    elem_bytes=wl.elem_bytes, out_bytes=out_bytes, distinct_per_request=distinct)
        if fused:
            extra = wl.R * wl.W * wl.H * wl.record_bytes
            d["algorithmic"] += extra
            d["undeduplicated"] += extra
        res.append(d)
    return res


def run_ours(args, rank: int, world: int, local_rank: int) -> dict:
    from paper_2609_12399_b200.runner import WorkloadRun

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    wl = workload_by_name(args.workload)
    if args.layers:
        wl = wl.scaled(L=args.layers)
    # the other shapes of the operator suite (Section 4.1), on a named workload's beams, depths and parents
    shape = {k: v for k, v in (("dk", args.dk), ("dv", args.dv), ("dtype", args.rec_dtype)) if v}
    if shape:
        wl = wl.scaled(name=wl.name + "_shape", **shape)
    out_dtype = args.out_dtype or wl.dtype
    out_bytes = 4 if out_dtype == "fp32" else 2
    run = WorkloadRun(wl, dev, out_dtype, flags=(2 if args.force_generic else 0) | (4 if args.delta_records else 0) | (8 if args.shared_chains else 0))
    ctx = run.ctx
    if wl.dk == wl.dv and wl.dk in (32, 64, 128):
        run.prefill_states()
    else:    # no prefill kernel for this shape: seeded random states of a prefilled state's magnitude
        gen = torch.Generator(device=dev).manual_seed(wl.seed)
        run.prefill_states({(r, l): 0.05 * torch.randn((wl.H, wl.dv, wl.dk), generator=gen, device=dev)
                            for r in range(wl.R) for l in range(wl.L)})
    S0 = {(r, l): ctx.onela_export_shared_state(r, l) for r in range(wl.R) for l in range(wl.L)}
    S0_all = torch.stack([torch.stack([S0[(r, l)] for l in range(wl.L)]) for r in range(wl.R)])   # [R][L][H][dv][dk]
    calls = [run.generate_call(t) for t in range(wl.D)]
    outs = run.alloc_outputs()
    torch.cuda.synchronize()
    units_per_step = wl.R * wl.W * wl.H * wl.L * wl.D
    fused = not args.unfused
    per_depth = launch_bytes(wl, out_bytes, fused)

    def generation(decode_events=None, stream=None):
        ctx.onela_reset(stream)
        ctx.onela_init_shared_states(0, wl.R, S0_all, stream)     # all layers of all requests: one copy
        for call in calls:
            run.run_call(call, outs, stream, decode_events, fused=fused, group_events=True)

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()

    if args.profile:   # plain eager generations for a profiler to attach to: no graph, no timing legs
        for _ in range(args.steps):
            generation()
        torch.cuda.synchronize()
        return {"profile": True, "workload": describe(wl), "generations": args.steps,
                "launches": int(ctx.onela_launch_count()), "decode_bytes_per_depth": per_depth}

    # ---- A. whole-step throughput, inputs resident: CUDA-graph replay of one generation -----------
    side = torch.cuda.Stream()
    launches_before = ctx.onela_launch_count()
    with torch.cuda.stream(side):
        generation()                      # eager once: primes lazy kernel attributes outside capture
    torch.cuda.synchronize()
    launches_per_step = ctx.onela_launch_count() - launches_before
    graph, mode = None, "eager"
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                generation()
            mode = "cuda_graph"
        except Exception as e:  # capture unavailable: fall back to plain launches, and say so
            graph, mode = None, f"eager (graph capture failed: {type(e).__name__})"
            torch.cuda.synchronize()

    def step():
        if graph is not None:
            graph.replay()
        else:
            generation()

    with ClockSampler(local_rank) as clocks:
        for _ in range(args.warmup):
            step()
        t_warm = time.perf_counter()          # keep the GPU busy a little longer so clocks settle under load
        while time.perf_counter() - t_warm < args.settle_seconds:
            step()
            torch.cuda.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        ms_total = e0.elapsed_time(e1)

        # ---- B. per-launch decode durations for the roofline (eager, GPU kept ahead of the CPU) ------
        pairs = []
        torch.cuda._sleep(int(2.0e7))      # ~10 ms of spin so event timestamps are paced by the GPU, not by Python
        n_b = max(1, min(args.steps, 5))
        for _ in range(n_b):
            generation(decode_events=pairs)
        torch.cuda.synchronize()

        # ---- B'. the same kernel with a WARM L2 (labelled; not the bench value): the deepest call's decode-only
        # launch repeated on one layer, so S_0, the records, the queries and the outputs stay L2-resident
        warm = None
        if wl.R <= 8 and not args.delta_records:
            lay = calls[-1]["layers"][0]
            reps = 20
            for _ in range(3):
                ctx.onela_decode_step(0, wl.R, 0, lay["q"], outs[0])
            w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            w0.record()
            for _ in range(reps):
                ctx.onela_decode_step(0, wl.R, 0, lay["q"], outs[0])
            w1.record()
            torch.cuda.synchronize()
            warm_us = w0.elapsed_time(w1) * 1e3 / reps
            warm_alg = launch_bytes(wl, out_bytes, False)[-1]["algorithmic"]
            warm = {"us_per_launch": warm_us, "depth": wl.D, "algorithmic_MB": warm_alg / 1e6,
                    "gbs": warm_alg / (warm_us * 1e-6) / 1e9,
                    "note": "decode_step (no append) of the deepest call repeated %d times on one layer: its working set "
                            "stays in L2, so this is NOT an HBM figure" % reps}
    # event pairs: one per decode launch, or (fused launches: nothing else runs between the layers of a call)
    # one around the L back-to-back launches of a call; either way [step, call, pairs] with `per` launches each
    per = pairs[0][2]
    dur_ms = np.array([a.elapsed_time(b) for a, b, _ in pairs]).reshape(n_b, wl.D, -1)
    ms_depth = dur_ms.mean(axis=(0, 2)) / per                                               # mean per launch at each depth
    n_per_depth = dur_ms.shape[2] * per
    alg_total = sum(per_depth[t]["algorithmic"] for t in range(wl.D)) * n_per_depth * n_b
    und_total = sum(per_depth[t]["undeduplicated"] for t in range(wl.D)) * n_per_depth * n_b
    achieved_gbs = alg_total / (dur_ms.sum() * 1e-3) / 1e9

    # ---- C. end to end: host buffers in, host buffers out, copies inside the timed region ----------
    if args.no_e2e:
        e2e = {"value": None, "ms_per_step": 0.0, "h2d": 0, "d2h": 0}
    else:
        e2e = run_e2e(args, run, S0, calls, outs, units_per_step, barrier)

    ms_total, e2e["ms_per_step"] = replicas.max_over_ranks([ms_total, e2e["ms_per_step"]], device=dev)
    if not args.no_e2e:
        e2e["value"] = replicas.aggregate_throughput(units_per_step, e2e["ms_per_step"], world)

    peaks_file = ROOT / "MEASURED_PEAKS.json"
    if peaks_file.exists():
        peak, peak_src = float(json.loads(peaks_file.read_text())["hbm_gbs"]), "of measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "of fallback"
    ms_per_step = ms_total / args.steps
    traffic = ncu_traffic()
    default_path = not (args.unfused or args.delta_records or args.force_generic or args.shared_chains) and wl.name.startswith("cfg4")
    clk = clocks.summary()
    mhz = clk["sm_mhz"] or 0.0
    line = {
        "metric": METRIC, "value": replicas.aggregate_throughput(units_per_step, ms_per_step, world), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 fold and corrections; the S_0 contraction on the tensor cores with fp16 operands (11-bit significand, "
                 "exact power-of-two scales) and f32 accumulation",
        "data": "synthetic",
        "config": {"workload": describe(wl), "step": "one whole generation: reset, store S_0, then per decode call "
                   "reorder + per layer append + decode (one fused launch per layer unless --unfused)", "units_per_step": units_per_step,
                   "l2": "inputs larger than L2 (%.1f GiB of records, queries and states per step)" %
                         ((wl.R * wl.W * wl.H * wl.L * wl.D * (wl.record_bytes + wl.dk * wl.elem_bytes)
                           + wl.R * wl.L * wl.H * wl.dk * wl.dv * 4) / 2 ** 30),
                   "out_dtype": out_dtype, "launch": mode,
                   "per_layer_calls": "append_records + decode_step" if args.unfused else "append_decode_step (one launch)", "parallelism": f"replicas x{world} (requests are independent)",
                   "tensor_core_path": bool(ctx.onela_uses_tensor_core_path()),
                   "record_format": "(alpha, delta, k), forward projection replay" if args.delta_records
                                    else "(k, v, alpha, beta), backward query fold"},
        "clocks": {**clk, "window": "sampled from the warm-up to the end of the timed legs"},
        "e2e": {"value": e2e["value"], "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "ms_per_step": e2e["ms_per_step"]},
        "gpu_launches": int(launches_per_step * args.steps),
        "roofline": {"bound": "hbm", "achieved": achieved_gbs, "peak": peak, "unit": "GB/s",
                     "frac": achieved_gbs / peak,
                     "traffic": traffic["bytes"] if default_path else None,
                     "traffic_note": "ncu DRAM read+write bytes of one launch at the deepest call (depth %d), whose algorithmic "
                                     "bytes are %.1f MB (writes still in L2 when the kernel ends are not in it); %s"
                                     % (wl.D, per_depth[-1]["algorithmic"] / 1e6, traffic["source"]),
                     "headline": {"deepest_call_frac": per_depth[-1]["algorithmic"] / (ms_depth[-1] * 1e-3) / 1e9 / peak,
                                  "mean_over_calls_frac": achieved_gbs / peak},
                     "warm_l2": warm,
                     "peak_source": peak_src,
                     "frac_of_nominal_8_tbs": achieved_gbs / 8000.0,   # context: the paper-independent nominal HBM3e figure
                     "timing": "CUDA events around every decode launch" if per == 1 else
                               "CUDA events around the %d back-to-back decode launches (one per layer) of each decode call" % per,
                     "kernel": ("decode_step" if args.unfused else "append_decode_step") + " (all requests of one layer per launch)",
                     "bytes": "algorithmic: S_0 once + each distinct record once + q + o + ancestry rows"
                              + ("" if args.unfused else " + the call's records written to the arena"),
                     "undeduplicated_gbs": und_total / (dur_ms.sum() * 1e-3) / 1e9,
                     "per_depth": [{"depth": t + 1, "us": float(ms_depth[t] * 1e3),
                                    "sm_cycles": float(ms_depth[t] * 1e3 * mhz),     # us x the sampled median SM MHz
                                    "algorithmic_MB": per_depth[t]["algorithmic"] / 1e6,
                                    "frac": per_depth[t]["algorithmic"] / (ms_depth[t] * 1e-3) / 1e9 / peak}
                                   for t in range(wl.D)]},
    }
    if rank == 0 and world == 1 and default_path and not args.no_secondary:
        del graph
        # the other beam-512 config and the large-batch config, in the same run (context, not the bench value)
        # configs 2 and 3 as they are (one layer: every launch alone after a flushed L2), and config 2's launch as a
        # decoder's layer loop issues it (16 layers back to back)
        line["secondary"] = [secondary_roofline("cfg2", dev, peak, mhz), secondary_roofline("cfg2", dev, peak, mhz, layers=16),
                             secondary_roofline("cfg3", dev, peak, mhz)]
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, reps=1, gen_device=dev)
    return line


def secondary_roofline(name: str, dev, peak: float, mhz: float, reps: int = 5, layers: int = 0) -> dict:
    """The same roofline block for another benchmark config, timed in this run: whole generations launched eagerly
    with the fused call, one CUDA-event pair around each decode call's launches.  These workloads are smaller than
    L2, so a buffer larger than L2 is overwritten before every decode call's launches (outside the event pairs)."""
    from paper_2609_12399_b200.runner import WorkloadRun

    wl = workload_by_name(name)
    if layers:     # the same launch over a decoder's layers, back to back: each starts under its predecessor's tail
        wl = wl.scaled(name=f"{wl.name}_x{layers}layers", L=layers, prompt_len=min(wl.prompt_len, 1024))
    run = WorkloadRun(wl, dev, wl.dtype)
    ctx = run.ctx
    run.prefill_states()
    S0_all = torch.stack([torch.stack([ctx.onela_export_shared_state(r, l) for l in range(wl.L)]) for r in range(wl.R)])
    calls = [run.generate_call(t) for t in range(wl.D)]
    outs = run.alloc_outputs()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    per_depth = launch_bytes(wl, 2 if wl.dtype == "bf16" else 4, True)
    pairs = []

    def generation(record):
        ctx.onela_reset()
        ctx.onela_init_shared_states(0, wl.R, S0_all)
        for call in calls:
            flush.zero_()
            if wl.L > 1:
                torch.cuda._sleep(int(1.0e6))     # ~0.5 ms of spin: the call's launches queue up behind it, so the event
                                                  # pair times them back to back, not the host's launch rate
            run.run_call(call, outs, None, pairs if record else None, fused=True, group_events=True)

    for _ in range(3):
        generation(False)
    torch.cuda.synchronize()
    for _ in range(reps):
        generation(True)
    torch.cuda.synchronize()
    per = pairs[0][2]
    dur_ms = np.array([a.elapsed_time(b) for a, b, _ in pairs]).reshape(reps, wl.D, -1)
    ms_depth = dur_ms.mean(axis=(0, 2)) / per
    alg = sum(d["algorithmic"] for d in per_depth) * dur_ms.shape[2] * per * reps
    achieved = alg / (dur_ms.sum() * 1e-3) / 1e9
    units = wl.R * wl.W * wl.H
    del run, calls, outs, flush
    return {"workload": describe(wl), "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": None, "l2": "a 256 MiB buffer is overwritten before every decode call's launches (one layer of these workloads is smaller than L2)",
            "decodes_per_s": units * wl.L * wl.D / (float(ms_depth.sum()) * 1e-3 * wl.L),
            "per_depth": [{"depth": t + 1, "us": float(ms_depth[t] * 1e3), "sm_cycles": float(ms_depth[t] * 1e3 * mhz),
                           "algorithmic_MB": per_depth[t]["algorithmic"] / 1e6,
                           "frac": per_depth[t]["algorithmic"] / (ms_depth[t] * 1e-3) / 1e9 / peak} for t in range(wl.D)]}


def run_e2e(args, run, S0, calls, outs, units_per_step, barrier) -> dict:
    """The same generation with every input starting in pinned host memory and every output read back."""
    ctx, wl = run.ctx, run.wl
    pin = lambda t: t.cpu().pin_memory()
    hS0 = {k: pin(v) for k, v in S0.items()}
    hcalls = [{"parents": None if c["parents"] is None else pin(c["parents"]),
               "layers": [{n: pin(x) for n, x in lay.items()} for lay in c["layers"]]} for c in calls]
    houts = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs]
    # Double-buffered device staging and three streams (copies in, library calls, copies out): the upload of call
    # t+1 and the read-back of call t-1 run under the kernels of call t.  Everything stays inside the timed region.
    dS0 = [next(iter(S0.values())).clone() for _ in range(2)]
    dcalls = [{"parents": torch.empty_like(calls[-1]["parents"]) if wl.D > 1 else None,
               "layers": [{n: torch.empty_like(x) for n, x in lay.items()} for lay in calls[0]["layers"]]} for _ in range(2)]
    douts = [outs, [torch.empty_like(o) for o in outs]]
    h2d = sum(v.numel() * v.element_size() for v in hS0.values())
    for c in hcalls:
        h2d += 0 if c["parents"] is None else c["parents"].numel() * 4
        h2d += sum(x.numel() * x.element_size() for lay in c["layers"] for x in lay.values())
    d2h = sum(o.numel() * o.element_size() for o in houts) * wl.D
    comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def generation():
        start = torch.cuda.Event()
        start.record(comp)
        s_in.wait_event(start)
        s_out.wait_event(start)
        ctx.onela_reset()
        state_used = [None, None]
        for i, (key, hS) in enumerate(hS0.items()):
            with torch.cuda.stream(s_in):
                if state_used[i % 2] is not None:
                    s_in.wait_event(state_used[i % 2])          # the store call has read this staging buffer
                dS0[i % 2].copy_(hS, non_blocking=True)
                up = torch.cuda.Event()
                up.record(s_in)
            comp.wait_event(up)
            ctx.onela_init_shared_state(key[0], key[1], dS0[i % 2])
            state_used[i % 2] = torch.cuda.Event()
            state_used[i % 2].record(comp)
        computed, read_back = [None, None], [None, None]
        for t, hc in enumerate(hcalls):
            b = t % 2
            dc = dcalls[b]
            with torch.cuda.stream(s_in):
                if computed[b] is not None:
                    s_in.wait_event(computed[b])                # call t-2 has consumed this staging buffer
                stage = {"parents": None, "layers": dc["layers"]}
                if hc["parents"] is not None:
                    dc["parents"].copy_(hc["parents"], non_blocking=True)
                    stage["parents"] = dc["parents"]
                for dl, hl in zip(dc["layers"], hc["layers"]):
                    for n in dl:
                        dl[n].copy_(hl[n], non_blocking=True)
                up = torch.cuda.Event()
                up.record(s_in)
            comp.wait_event(up)
            if read_back[b] is not None:
                comp.wait_event(read_back[b])                   # call t-2's outputs have left this buffer
            run.run_call(stage, douts[b], fused=not args.unfused)
            computed[b] = torch.cuda.Event()
            computed[b].record(comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(computed[b])
                for ho, o in zip(houts, douts[b]):
                    ho.copy_(o, non_blocking=True)
                read_back[b] = torch.cuda.Event()
                read_back[b].record(s_out)
        comp.wait_stream(s_in)
        comp.wait_stream(s_out)

    for _ in range(max(1, min(args.warmup, 2))):
        generation()
    barrier()
    n = max(1, min(args.steps, 3))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        generation()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1) / n
    return {"value": units_per_step / (ms * 1e-3), "ms_per_step": ms, "h2d": int(h2d), "d2h": int(d2h)}


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (the reported baseline, and the whole of --impl reference)
# ------------------------------------------------------------------------------------------------
def cpu_sample(wl: inputs.Workload, gen_device) -> dict:
    """Inputs of the bounded sample: every (beam, head) unit of every decode call of up to EIGHT (request,
    layer) pairs of the workload - every request at its first and its last layer - with their true S_0 (oracle
    prefill): about ten seconds of oracle time per pass at the default workload."""
    import oracle
    pairs = sorted({(r, l) for r in range(wl.R) for l in (0, wl.L - 1)})[:8]
    sample = []
    for (r, l) in pairs:
        parts = [inputs.prompt_tokens(wl, r, l, a, min(a + 2048, wl.prompt_len), device=gen_device)
                 for a in range(0, wl.prompt_len, 2048)]
        p = {n: torch.cat([x[n] for x in parts]).cpu() for n in ("k", "v", "alpha", "beta")}
        S0 = oracle.prefill(p["k"], p["v"], p["alpha"], p["beta"]).astype(np.float32)
        steps = [{n: x.cpu().float().numpy() for n, x in inputs.decode_token(wl, r, l, t, device=gen_device).items()}
                 for t in range(wl.D)]
        qs = [inputs.decode_query(wl, r, l, t, device=gen_device).cpu().float().numpy() for t in range(wl.D)]
        par = [None] + [inputs.parents(wl, r, t).numpy() for t in range(1, wl.D)]
        sample.append((S0, steps, par, qs))
    return {"pairs": pairs, "data": sample, "units": len(pairs) * wl.D * wl.W * wl.H}


def time_cpu_sample(sample) -> float:
    import oracle
    t0 = time.perf_counter()
    for (S0, steps, par, qs) in sample["data"]:
        for t in range(len(steps)):
            oracle.decode(S0, steps[:t + 1], par[:t + 1], qs[t])
    return time.perf_counter() - t0


def cpu_baseline(wl: inputs.Workload, reps: int, gen_device) -> dict:
    import oracle
    sample = cpu_sample(wl, gen_device)
    secs = min(time_cpu_sample(sample) for _ in range(max(1, reps)))
    return {"value": sample["units"] / secs, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "seconds": secs,
            "sample": f"all {wl.W}x{wl.H} (beam, head) units of all {wl.D} decode calls of (request, layer) pairs "
                      f"{sample['pairs']} = {sample['units']} decodes, fp64 full-state replay (OpenMP)"}


def run_reference(args) -> dict:
    import oracle
    wl = workload_by_name(args.workload)
    gen_device = torch.device("cuda", 0) if torch.cuda.is_available() else torch.device("cpu")
    sample = cpu_sample(wl, gen_device)
    for _ in range(args.warmup):
        time_cpu_sample(sample)
    secs = [time_cpu_sample(sample) for _ in range(args.steps)]
    per = sum(secs) / len(secs)
    value = sample["units"] / per
    desc = {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"each step = all {wl.W}x{wl.H} units of all {wl.D} decode calls of (request, layer) pairs "
                      f"{sample['pairs']} = {sample['units']} decodes"}
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(wl), "note": "CPU fp64 oracle (full-state replay) on the host cores; "
                       "the paper ships no code, so the oracle is the reference arm"},
            "cpu_baseline": desc,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--out-dtype", default=None, choices=[None, "fp32", "bf16"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--unfused", action="store_true", help="separate append_records and decode_step launches per layer")
    ap.add_argument("--settle-seconds", type=float, default=1.0, help="extra untimed warm-up after the W steps")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling)")
    ap.add_argument("--force-generic", action="store_true", help="run the CUDA-core decode kernel")
    ap.add_argument("--dk", type=int, default=0, help="override the workload's key width (64, 128, 256)")
    ap.add_argument("--dv", type=int, default=0, help="override the workload's value width (64 ... 512)")
    ap.add_argument("--rec-dtype", default=None, choices=[None, "bf16", "fp32"], help="override the record dtype")
    ap.add_argument("--delta-records", action="store_true",
                    help="(alpha, delta, k) records with forward projection replay (Section 3.2) instead of raw records "
                         "with the backward fold: the CUDA-core comparison kernel")
    ap.add_argument("--shared-chains", action="store_true", help="run the shared-ancestor tensor-core kernel (ONELA_FLAG_SHARED_CHAINS)")
    ap.add_argument("--profile", action="store_true", help="eager generations only, for ncu")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (kernel experiments)")
    ap.add_argument("--no-secondary", action="store_true", help="skip the roofline blocks of configs 2 and 3")
    ap.add_argument("--rank-plumbing-only", action="store_true",
                    help="no GPU work: every rank reports a made-up time (rank + 1 ms) through the timing protocol over gloo; "
                         "checks the launch, barrier, max-over-ranks and aggregation logic on a CPU box")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" and not args.profile else args.warmup

    # `--gpus N` on its own starts the N replicas itself: one process per GPU under torch.distributed.run on this
    # node (a launcher that already set RANK / WORLD_SIZE is left alone).
    if args.gpus > 1 and "RANK" not in os.environ and args.impl == "ours":
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
                                  "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *sys.argv[1:]])
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "ours" and world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s)")

    if args.rank_plumbing_only:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if world > 1:
            torch.distributed.init_process_group("gloo")
        replicas.barrier()
        units = 1000
        (ms,) = replicas.max_over_ranks([float(rank + 1)])
        replicas.barrier()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": replicas.aggregate_throughput(units, ms, world), "unit": UNIT,
                              "n_gpus": world, "ms_per_step": ms, "scaling": "weak", "rank_plumbing_only": True}), flush=True)
        if world > 1:
            torch.distributed.destroy_process_group()
        return

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    line = run_ours(args, rank, world, local_rank)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
