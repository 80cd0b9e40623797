#!/usr/bin/env python
"""Benchmark of the separate-rejection-sampling hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input: draft-side sparse
compression (picospec_compress, with the draft-token draw) followed by target-side verification
with the fused residual / bonus sample (picospec_verify).  The headline metric is verified
draft positions per second (B * gamma per step); the roofline entry is the achieved HBM
bandwidth of the dominant kernel (the one with the longest average launch of the step: the
compress filter pass or the verify streaming pass; the other one is listed under "kernels").

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config4] [--impl ours|reference]

With N > 1 and no torchrun environment the script starts N ranks of itself (torch.distributed.run,
one rank per GPU); every rank runs its own batch (the path shards by sequence, no collective on the
data path), so scaling is weak.

Three loops per workload, all over the same rotating input sets:
  1. the timed loop (the headline): K steps back to back, no per-kernel events;
  2. the roofline loop: at least 64 more steps with every kernel group bracketed by its own pair
     of CUDA events on the launching stream (mean, median and minimum per kernel, and per call);
  3. if the two together kept the GPU busy for less than 0.6 s, more back-to-back steps so that
     the clock sampler sees the SM clock under this load.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "verified_draft_positions_per_sec"
UNIT = "positions/s"
NOMINAL_GBPS = 8000.0

# kernel kinds of picospec_profile_* (include/picospec.h)
K_COMPRESS_STREAM, K_VERIFY_STREAM, K_VERIFY_FINISH, K_VERIFY_PRECISE = 0, 1, 2, 3
K_COMPRESS_PRECISE, K_COMPRESS_REDO, K_COMPRESS_FINISH = 4, 5, 6
KIND_NAMES = {K_COMPRESS_STREAM: "compress_stream", K_VERIFY_STREAM: "verify_stream", K_VERIFY_FINISH: "verify_finish",
              K_VERIFY_PRECISE: "verify_precise", K_COMPRESS_PRECISE: "compress_precise",
              K_COMPRESS_REDO: "compress_redo", K_COMPRESS_FINISH: "compress_finish"}

CSRC = os.path.join(ROOT, "paper_2603_19133_b200", "csrc")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def source_hash(files):
    """Short hash of kernel source files: ties an ncu capture to the code it was taken from."""
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def ncu_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of `kernel` on `workload` (dram__bytes_read.sum + dram__bytes_write.sum,
    scaled to the full batch), read from the ncu summaries under profiles/.  A summary carries a line
        bench-traffic: kernel=<name> workload=<name> bytes=<int> sources=<a.cuh,b.cuh> hash=<12 hex>
    and the figure is used only while the named source files still hash to the recorded value:
    once the kernel has changed the counters no longer describe it and the entry is null."""
    pdir = os.path.join(ROOT, "profiles")
    if not os.path.isdir(pdir):
        return None
    pat = re.compile(r"bench-traffic:\s*kernel=(\S+)\s+workload=(\S+)\s+bytes=(\d+)\s+sources=(\S+)\s+hash=([0-9a-f]+)")
    for fn in sorted(os.listdir(pdir)):
        if not fn.endswith((".md", ".txt")):
            continue
        with open(os.path.join(pdir, fn)) as f:
            for m in pat.finditer(f.read()):
                if m.group(1) == kernel and m.group(2) == workload:
                    try:
                        current = source_hash(m.group(4).split(","))
                    except OSError:
                        return None
                    return int(m.group(3)) if current == m.group(5) else None
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the GPU works; every sample is
    stamped with the host time it arrived at, so that only samples taken under load are used."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "25",
                 "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return

        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.perf_counter(), line.strip()))

        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self, t_begin=None, t_end=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        for t, r in self.rows:
            if t_begin is not None and not (t_begin <= t <= t_end):
                continue
            f = [x.strip() for x in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "sm_mhz_min": min(sm) if sm else None,
                "power_w_max": max(power) if power else None,
                "window_s": None if t_begin is None else round(t_end - t_begin, 3)}


def _dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def _np(t):
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def input_sets(w) -> int:
    """Distinct input sets a workload rotates through, so that consecutive steps never find their
    logits in the 126 MB L2: enough sets for 320 MB (at most 288 of them), one when a single set is
    larger than that already."""
    per_set = (w.B * (2 * w.G + 1)) * w.V * w.bytes_per_logit
    return max(1, min(288, -(-(320 << 20) // per_set))) if per_set < (320 << 20) else 1


def config_of(w, world):
    """The `config` object of the JSON line; the same for both arms."""
    nsets = input_sets(w)
    return {"workload": w.name, "V": w.V, "B_per_gpu": w.B, "gamma": w.G, "logits": w.dtype,
            "top_k": w.top_k, "top_p": w.top_p, "k_max": w.k_max,
            "accumulate": "f32 streaming sums, f64 per-row arithmetic",
            "step": "picospec_compress + picospec_verify (fused residual/bonus sample)",
            "l2": f"inputs larger than L2: {nsets} input set(s) of "
                  f"{(w.B * (2 * w.G + 1)) * w.V * w.bytes_per_logit / 1e6:.0f} MB rotated",
            "parallelism": f"dp{world} (sequences sharded, no collective)"}


# -------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# -------------------------------------------------------------------------------------------------

def oracle_step_time(w, inputs_cpu, nthreads):
    """One pass of the whole path (compress + verify with fused sample) by the oracle; seconds."""
    import oracle
    t0 = time.perf_counter()
    qi, qp, qc, tok = oracle.compress(inputs_cpu["draft_logits"], inputs_cpu["temperature"], w.top_k, w.top_p,
                                      w.k_max, inputs_cpu["u_draft"], nthreads=nthreads)
    oracle.verify(inputs_cpu["target_logits"], inputs_cpu["temperature"], tok, qi, qp, qc, inputs_cpu["u_accept"],
                  inputs_cpu["u_resample"], nthreads=nthreads)
    return time.perf_counter() - t0


def oracle_sample(w, seed, sample_B):
    ws = gen.scaled(w, B=sample_B)
    inp = gen.make_inputs(ws, seed=seed, device="cpu")
    return ws, {k: _np(v) for k, v in inp.items()}


def run_reference(args):
    rank, _, world = _dist_env()
    if rank != 0:
        return
    import oracle
    w = gen.WORKLOADS[args.workload]
    cores = oracle.cores()
    # size the per-step sample so that steps + warm-up end within about two minutes: calibrate on
    # a few sequences first (sequences are independent, so the cost is linear in their number)
    cal_B = min(w.B, 4)
    wc, ic = oracle_sample(w, 4241, cal_B)
    per_seq = oracle_step_time(wc, ic, cores) / cal_B
    budget_s = 100.0
    sample_B = int(budget_s / (max(args.steps + args.warmup, 1) * per_seq))
    sample_B = max(1, min(w.B, args.ref_sample, sample_B))
    ws, inp = oracle_sample(w, 4242, sample_B)
    for _ in range(args.warmup):
        oracle_step_time(ws, inp, cores)
    times = [oracle_step_time(ws, inp, cores) for _ in range(args.steps)]
    t = sum(times)
    value = ws.B * ws.G * args.steps / t
    sample = f"{sample_B} of {w.B} sequences of {w.name} per step, all {cores} host threads (OpenMP over rows)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": max(args.gpus, world),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, max(args.gpus, world)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "ranks_launched": world,
    }
    print(json.dumps(line), flush=True)


# -------------------------------------------------------------------------------------------------
# our arm
# -------------------------------------------------------------------------------------------------

class Step:
    """Pre-allocated outputs and the two calls of one step on device-resident inputs."""

    def __init__(self, ps, ctx, w, inputs):
        self.ctx, self.w, self.inp = ctx, w, inputs
        dev = inputs["draft_logits"].device
        B, G, K = w.B, w.G, w.k_max
        i32, f32 = torch.int32, torch.float32
        self.c_out = (torch.empty((B, G, K), dtype=i32, device=dev), torch.empty((B, G, K), dtype=f32, device=dev),
                      torch.empty((B, G), dtype=i32, device=dev), torch.empty((B, G), dtype=i32, device=dev))
        self.v_out = {"accept_len": torch.empty((B,), dtype=i32, device=dev),
                      "p_draft": torch.empty((B, G), dtype=f32, device=dev),
                      "resid_mass": torch.empty((B, G), dtype=f32, device=dev),
                      "borderline_count": torch.empty((1,), dtype=i32, device=dev),
                      "token": torch.empty((B,), dtype=i32, device=dev)}
        # kernels per step: compress = filter, finish, redo list (+ the double-precision cut with top-p);
        # verify = statistics, finish, exact sums, double-precision finish
        self.launches_per_step = (4 if w.top_p < 1.0 else 3) + 4

    def compress(self, inp=None):
        inp = inp or self.inp
        w = self.w
        return self.ctx.compress(inp["draft_logits"], inp["temperature"], w.top_k, w.top_p, w.k_max, inp["u_draft"],
                                 out=self.c_out)

    def verify(self, inp=None):
        inp = inp or self.inp
        qi, qp, qc, tok = self.c_out
        return self.ctx.verify(inp["target_logits"], inp["temperature"], tok, qi, qp, qc, inp["u_accept"],
                               inp["u_resample"], out=self.v_out)

    def __call__(self, inp=None):
        self.compress(inp)
        self.verify(inp)


def timed_loop(fn, steps, warmup, sync):
    for _ in range(warmup):
        fn()
    sync()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    sync()
    return e0.elapsed_time(e1) * 1e-3


def algorithmic_bytes(w):
    """Bytes the method itself has to move: per launch of each streaming kernel, and per call."""
    nch = (w.V + 1023) // 1024
    rows_t, rows_d = w.B * (w.G + 1), w.B * w.G
    verify_stream = rows_t * w.V * w.bytes_per_logit + rows_t * nch * 8
    compress_stream = rows_d * w.V * w.bytes_per_logit + rows_d * (w.k_max * 8 + 8)
    # whole calls: compress also writes the sparse rows, counts and draft tokens; verify reads the
    # chunk statistics back, the sparse rows (id + prob per slot, count, token, uniform), one chunk
    # per sequence again for the draw, and writes its per-position and per-sequence results
    compress_call = rows_d * w.V * w.bytes_per_logit + rows_d * (w.k_max * 8 + 4 + 4 + 4)
    verify_call = (verify_stream + rows_t * nch * 8 + rows_d * (w.k_max * 8 + 12) + w.B * 1024 * w.bytes_per_logit
                   + rows_d * 8 + w.B * 8)
    return {"verify_stream": verify_stream, "compress_stream": compress_stream,
            "compress_call": compress_call, "verify_call": verify_call}


def _stats_us(samples_ms):
    if not samples_ms:
        return {"launches": 0, "avg_us": None, "median_us": None, "min_us": None}
    us = [1e3 * x for x in samples_ms]
    return {"launches": len(us), "avg_us": sum(us) / len(us), "median_us": statistics.median(us), "min_us": min(us)}


def bench_workload(ps, w, steps, warmup, rank, world, device, with_e2e, with_clocks, roofline_launches=64,
                   min_busy_s=0.6):
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    nsets = input_sets(w)
    sets = [gen.make_inputs(w, seed=1000 * (rank + 1) + 17 * i + sum(map(ord, w.name)), device=device)
            for i in range(nsets)]
    step = Step(ps, ctx, w, sets[0])
    state = {"i": 0}

    def one():
        step(sets[state["i"] % nsets])
        state["i"] += 1

    def sync():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    ctx.status(clear=True)
    ctx.counters(clear=True)
    ctx.profile_enable(0)
    sampler = ClockSampler(torch.cuda.current_device()) if with_clocks else None
    if sampler:
        sampler.start()
        time.sleep(0.1)
    # ---- 1. the timed loop ------------------------------------------------------------------
    for _ in range(warmup):
        one()
    sync()
    t_busy0 = time.perf_counter()
    t = timed_loop(one, steps, 0, sync)
    if world > 1:
        tt = torch.tensor([t], device=device, dtype=torch.float64)
        torch.distributed.all_reduce(tt, op=torch.distributed.ReduceOp.MAX)
        t = float(tt.item())
    _, redo = ctx.counters()
    st, slow = ctx.status(clear=True)
    steps_counted = steps + warmup

    # ---- 2. the roofline loop: every kernel group and both calls bracketed -------------------
    ctx.profile_enable(2, every=1)
    n_roof = max(roofline_launches, 1)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_roof)]
    torch.cuda.synchronize()
    for i in range(n_roof):
        inp = sets[state["i"] % nsets]
        state["i"] += 1
        ev[i][0].record()
        step.compress(inp)
        ev[i][1].record()
        step.verify(inp)
        ev[i][2].record()
    torch.cuda.synchronize()
    kinds = {name: _stats_us(ctx.profile_samples(k)) for k, name in KIND_NAMES.items()}
    calls = {"compress_call": _stats_us([e[0].elapsed_time(e[1]) for e in ev]),
             "verify_call": _stats_us([e[1].elapsed_time(e[2]) for e in ev])}
    ctx.profile_enable(0)
    ctx.status(clear=True)

    # ---- 3. keep the GPU busy long enough for the clock sampler -------------------------------
    if sampler:
        while time.perf_counter() - t_busy0 < min_busy_s:
            for _ in range(32):
                one()
            torch.cuda.synchronize()
    t_busy1 = time.perf_counter()
    clocks = sampler.stop(t_busy0 + 0.03, t_busy1) if sampler else None
    ctx.status(clear=True)
    ctx.counters(clear=True)

    alg = algorithmic_bytes(w)
    peak, peak_kind = _peaks()

    def with_bw(stats, nbytes):
        out = dict(stats)
        out["alg_bytes"] = nbytes
        for key in ("avg", "median", "min"):
            us = stats.get(f"{key}_us")
            out[f"GBps_{key}"] = nbytes / us / 1e3 if us else None
        out["GBps"] = out["GBps_avg"]
        out["frac_of_peak"] = (out["GBps"] or 0) / peak
        out["frac_of_8TBps_nominal"] = (out["GBps"] or 0) / NOMINAL_GBPS
        return out

    res = {
        "seconds": t, "status": st,
        "slow_rows_per_step": slow / float(steps_counted),
        "redo_rows_per_step": redo / float(steps_counted),
        "value": world * w.B * w.G * steps / t,
        "rows_streamed_per_sec": world * w.B * (2 * w.G + 1) * steps / t,
        "verify_stream": with_bw(kinds["verify_stream"], alg["verify_stream"]),
        "compress_stream": with_bw(kinds["compress_stream"], alg["compress_stream"]),
        "verify_call": with_bw(calls["verify_call"], alg["verify_call"]),
        "compress_call": with_bw(calls["compress_call"], alg["compress_call"]),
        "other_kernels_us": {k: v["avg_us"] for k, v in kinds.items() if k not in ("verify_stream", "compress_stream")},
        "peak": peak, "peak_kind": peak_kind, "clocks": clocks, "nsets": nsets,
        "launches_per_step": step.launches_per_step,
    }

    if with_e2e:
        # end to end: host-resident inputs (pinned), copied in every step; results read back
        host = {k: v.cpu().pin_memory() for k, v in sets[0].items()}
        dev = {k: torch.empty_like(v) for k, v in sets[0].items()}
        h_out = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in step.v_out.items()}
        h2d = sum(v.numel() * v.element_size() for v in host.values())
        d2h = sum(v.numel() * v.element_size() for v in h_out.values())

        def one_e2e():
            for k in host:
                dev[k].copy_(host[k], non_blocking=True)
            step(dev)
            for k in h_out:
                h_out[k].copy_(step.v_out[k], non_blocking=True)
            torch.cuda.current_stream().synchronize()      # the caller reads the result

        k_e2e = max(2, min(steps, 10))
        t0 = time.perf_counter()
        te = timed_loop(one_e2e, k_e2e, 1, sync)
        if world > 1:
            tt = torch.tensor([te], device=device, dtype=torch.float64)
            torch.distributed.all_reduce(tt, op=torch.distributed.ReduceOp.MAX)
            te = float(tt.item())
        res["e2e"] = {"value": world * w.B * w.G * k_e2e / te, "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": k_e2e, "wall_s": time.perf_counter() - t0}
        del host, dev, h_out
    ctx.close()
    del sets, step
    torch.cuda.empty_cache()
    return res


def summary_of(r, steps):
    """The per-workload entry of `other_configs`."""
    vs, cs = r["verify_stream"], r["compress_stream"]
    return {"positions_per_sec": r["value"], "ms_per_step": 1e3 * r["seconds"] / steps,
            "verify_stream_us": vs["avg_us"], "verify_stream_median_us": vs["median_us"],
            "verify_stream_GBps": vs["GBps"], "verify_stream_frac_of_peak": vs["frac_of_peak"],
            "verify_stream_frac_of_8TBps": vs["frac_of_8TBps_nominal"],
            "compress_stream_us": cs["avg_us"], "compress_stream_median_us": cs["median_us"],
            "compress_stream_GBps": cs["GBps"], "compress_stream_frac_of_peak": cs["frac_of_peak"],
            "compress_stream_frac_of_8TBps": cs["frac_of_8TBps_nominal"],
            "verify_call_us": r["verify_call"]["avg_us"], "verify_call_GBps": r["verify_call"]["GBps"],
            "verify_call_frac_of_peak": r["verify_call"]["frac_of_peak"],
            "compress_call_us": r["compress_call"]["avg_us"], "compress_call_GBps": r["compress_call"]["GBps"],
            "sparse_row_bytes_share_of_verify_call": (r["verify_call"]["alg_bytes"] - vs["alg_bytes"]) / r["verify_call"]["alg_bytes"],
            "bracketed_launches": vs["launches"], "input_sets_rotated": r["nsets"],
            "slow_rows_per_step": r["slow_rows_per_step"], "redo_rows_per_step": r["redo_rows_per_step"],
            "device_status": r["status"]}


def bench_pipelined(ps, w, device, n_streams, iters):
    """Many calls in flight (the latency-bound configurations): one CUDA graph per input set, each
    holding one whole step, replayed over `n_streams` streams with a context each.  Reported next
    to the single-call latency of the same workload; not the headline."""
    nsets = max(n_streams, input_sets(w))
    nsets = (nsets + n_streams - 1) // n_streams * n_streams
    sets = [gen.make_inputs(w, seed=9000 + i, device=device) for i in range(nsets)]
    streams = [torch.cuda.Stream() for _ in range(n_streams)]
    ctxs = [ps.Context(w.B, w.G, w.V, w.k_max) for _ in range(n_streams)]
    steps = [Step(ps, ctxs[i % n_streams], w, sets[i]) for i in range(nsets)]
    graphs = []
    torch.cuda.synchronize()
    for i, stp in enumerate(steps):
        s = streams[i % n_streams]
        with torch.cuda.stream(s):
            stp()                       # warm-up outside capture (function attributes are set on first use)
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            stp()
        graphs.append(g)
    torch.cuda.synchronize()

    def sweep():
        for i, g in enumerate(graphs):
            with torch.cuda.stream(streams[i % n_streams]):
                g.replay()

    for _ in range(3):
        sweep()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    e0.record()
    for s in streams:
        s.wait_event(e0)
    for _ in range(iters):
        sweep()
    for s in streams:
        done = torch.cuda.Event()
        done.record(s)
        cur.wait_event(done)
    e1.record()
    torch.cuda.synchronize()
    sec = e0.elapsed_time(e1) * 1e-3
    nsteps = iters * len(graphs)
    alg = algorithmic_bytes(w)
    peak, _ = _peaks()
    status = 0
    for c in ctxs:
        status |= c.status(clear=True)[0]
        c.close()
    step_bytes = alg["verify_call"] + alg["compress_call"]
    how = (f"replayed round-robin on {n_streams} streams, {iters} sweeps; throughput of many calls in flight, not a latency"
           if n_streams > 1 else
           f"replayed back to back on one stream, {iters} sweeps: a step whose eight launches come from one graph launch")
    return {"what": f"{len(graphs)} CUDA graphs (one step each) {how}",
            "positions_per_sec": w.B * w.G * nsteps / sec, "us_per_step": 1e6 * sec / nsteps,
            "step_GBps": step_bytes * nsteps / sec / 1e9, "step_frac_of_peak": step_bytes * nsteps / sec / 1e9 / peak,
            "verify_stream_bytes_GBps": alg["verify_stream"] * nsteps / sec / 1e9, "device_status": status}


def bench_vocab_parallel(ps, w, device, ranks, iters):
    """Vocabulary-parallel verification (Sec. 4.1: the verifier spans several GPUs) with the slices of
    all ranks in this one GPU's memory and the exchanges done as copies: every kernel of the path runs
    as it would on `ranks` devices, one rank after the other, so the time of a call divided by `ranks`
    approximates one rank's compute; the NCCL transport itself is not measured here."""
    from paper_2603_19133_b200 import vocab_parallel as vp
    inp = gen.make_inputs(w, seed=7300, device=device)
    ctx0 = ps.Context(w.B, w.G, w.V, w.k_max)
    qi, qp, qc, tok = ctx0.compress(inp["draft_logits"], inp["temperature"], w.top_k, w.top_p, w.k_max, inp["u_draft"])
    ctx0.close()
    ctxs = [ps.Context(w.B, w.G, w.V, w.k_max) for _ in range(ranks)]
    states = []
    for r in range(ranks):
        v0, v1 = vp.slice_bounds(w.V, ranks, r)
        states.append(vp.RankState(ctxs[r], r, ranks, w.V, inp["target_logits"][:, :, v0:v1].contiguous()))
    rep = lambda t: [t] * ranks
    exch = vp.LocalExchange(ranks)

    def call():
        return vp.verify_sharded(states, exch, rep(inp["temperature"]), rep(tok), rep(qi), rep(qp), rep(qc),
                                 rep(inp["u_accept"]), rep(inp["u_resample"]))

    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / iters
    status = 0
    for c in ctxs:
        status |= c.status(clear=True)[0]
        c.close()
    slice_bytes = w.B * (w.G + 1) * (vp.slice_bounds(w.V, ranks, 0)[1]) * w.bytes_per_logit
    return {"ranks": ranks, "us_per_call_all_ranks_on_one_gpu": us, "us_per_rank": us / ranks,
            "slice_bytes_per_rank": slice_bytes, "kernels_per_rank_per_call": 12,
            "exchanges_per_call": "2 all-gathers (chunk records, exact sums), 4 element-wise maxima",
            "transport": "not measured: one GPU per run, the exchanges are copies", "device_status": status}


def bench_paper_direction(ps, w, device, k, iters):
    """The paper's own data flow (Sec. 3.3) on the same shape, timed per call with CUDA events:
    picospec_target_topk (Top-K of the target row at one position per sequence, K = 10 as in the
    paper's payload example) and picospec_edge_resample (against the dense draft row)."""
    ctx = ps.Context(w.B, w.G, w.V, max(k, 1))
    nsets = 3
    sets = [gen.make_inputs(w, seed=7000 + i, device=device) for i in range(nsets)]
    gpos = torch.Generator(device="cpu").manual_seed(7)
    pos = torch.randint(0, w.G, (w.B,), generator=gpos, dtype=torch.int32).to(device)
    out = {}

    def timed(fn):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / iters

    payload = [ctx.target_topk(s["target_logits"], s["temperature"], pos, k) for s in sets]
    # outputs are preallocated: at a few tens of microseconds per call the host side of the binding counts
    topk_out = tuple(torch.empty_like(t) for t in payload[0])
    out["target_topk_us"] = timed(lambda i: ctx.target_topk(sets[i % nsets]["target_logits"], sets[i % nsets]["temperature"],
                                                            pos, k, out=topk_out))
    u = [s["u_resample"][:, 0].contiguous() for s in sets]
    tok_out = (torch.empty((w.B,), dtype=torch.int32, device=device), None)
    out["edge_resample_us"] = timed(lambda i: ctx.edge_resample(sets[i % nsets]["draft_logits"], sets[i % nsets]["temperature"],
                                                                pos, *payload[i % nsets], u[i % nsets], want_mass=False,
                                                                out=tok_out))
    row_bytes = w.B * w.V * w.bytes_per_logit
    out.update({"k": k, "rows_per_call": w.B, "row_bytes_per_call": row_bytes,
                "target_topk_GBps": row_bytes / out["target_topk_us"] / 1e3,
                "edge_resample_GBps": row_bytes / out["edge_resample_us"] / 1e3,
                "status": ctx.status(clear=True)[0]})
    ctx.close()
    return out


def bench_wire(ps, w, device, iters):
    """The wire codec of the sparse rows (Sec. 3.3) on the rows picospec_compress leaves for this
    shape, timed per call with CUDA events, and the size of the paper's K = 10 example message."""
    ctx = ps.Context(w.B, w.G, w.V, w.k_max)
    inp = gen.make_inputs(w, seed=7100, device=device)
    qi, qp, qc, _ = ctx.compress(inp["draft_logits"], inp["temperature"], w.top_k, w.top_p, w.k_max, inp["u_draft"])
    R = qc.numel()
    out = {"rows": R, "k_max": w.k_max, "dense_bytes": R * w.k_max * 8}
    for fp16 in (False, True):
        buf, nbytes = ctx.wire_pack(qi, qp, qc, fp16=fp16)
        n = int(nbytes.item())
        dense = ctx.wire_unpack(buf, n, R, w.k_max)

        def timed(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / iters

        tag = "fp16" if fp16 else "fp32"
        out[f"message_bytes_{tag}"] = n
        out[f"pack_us_{tag}"] = timed(lambda: ctx.wire_pack(qi, qp, qc, fp16=fp16, buf=buf, bytes_out=nbytes))
        out[f"unpack_us_{tag}"] = timed(lambda: ctx.wire_unpack(buf, n, R, w.k_max, out=dense))
    out["k10_message_bytes_fp32"] = ps.wire_bytes(1, 10, 0)
    out["k10_message_bytes_fp16"] = ps.wire_bytes(1, 10, 1)
    out["status"] = ctx.status(clear=True)[0]
    ctx.close()
    return out


def run_ours(args):
    rank, local_rank, world = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    import paper_2603_19133_b200 as ps
    ps.lib()
    w = gen.WORKLOADS[args.workload]
    if args.batch > 0:
        w = gen.scaled(w, B=args.batch)
    main = bench_workload(ps, w, args.steps, args.warmup, rank, world, device, with_e2e=True,
                          with_clocks=(rank == 0), roofline_launches=args.roofline_launches)

    others = {}
    if args.all_configs and world == 1:
        k_other = min(args.steps, 200)
        for name in ("config1", "config2", "config3"):
            if name == args.workload:
                continue
            r = bench_workload(ps, gen.WORKLOADS[name], k_other, args.warmup, rank, world, device, with_e2e=False,
                               with_clocks=False, roofline_launches=64)
            others[name] = summary_of(r, k_other)
        # configuration 5: the bandwidth sweep, every point at its full batch
        k_sweep = min(args.steps, 20)
        for V in gen.SWEEP_V:
            for k in gen.SWEEP_K:
                ws = gen.sweep_workload(V, k)
                r = bench_workload(ps, ws, k_sweep, 3, rank, world, device, with_e2e=False, with_clocks=False,
                                   roofline_launches=16)
                others[ws.name] = summary_of(r, k_sweep)

    paper_direction = wire_codec = vocab_parallel = None
    pipelined = {}
    if args.all_configs and world == 1:
        paper_direction = bench_paper_direction(ps, w, device, k=10, iters=min(args.steps, 200))
        wire_codec = bench_wire(ps, w, device, iters=min(args.steps, 200))
        vocab_parallel = {f"ranks{r}": bench_vocab_parallel(ps, w, device, r, iters=min(args.steps, 20)) for r in (2, 4)}
        for name in ("config1", "config2"):
            try:
                pipelined[name] = bench_pipelined(ps, gen.WORKLOADS[name], device, n_streams=4,
                                                  iters=max(4, min(args.steps, 50)))
                pipelined[name + "_one_stream"] = bench_pipelined(ps, gen.WORKLOADS[name], device, n_streams=1,
                                                                  iters=max(4, min(args.steps, 50)))
            except Exception as e:      # noqa: BLE001  (reported, not fatal: the headline does not depend on it)
                pipelined[name] = {"error": f"{type(e).__name__}: {e}"[:300]}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        cores = oracle.cores()
        sample_B = min(w.B, args.ref_sample)
        ws, inp = oracle_sample(w, 4242, sample_B)
        tcpu = oracle_step_time(ws, inp, cores)
        cpu_baseline = {"value": ws.B * ws.G / tcpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"{sample_B} of {w.B} sequences of {w.name}, one pass, {tcpu:.2f} s, "
                                  f"all {cores} host threads (OpenMP over rows)"}

    if rank == 0:
        peak = main["peak"]
        kern = {
            "compress_filter_kernel (picospec_compress streaming pass)": main["compress_stream"],
            "chunk_stats_bulk_kernel (picospec_verify streaming pass)": main["verify_stream"],
        }
        dom_name = max(kern, key=lambda k: kern[k]["avg_us"] or 0)
        dom = kern[dom_name]
        line = {
            "metric": METRIC, "value": main["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * main["seconds"] / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": config_of(w, world),
            "roofline": {"bound": "hbm", "kernel": dom_name,
                         "achieved": dom["GBps"], "peak": peak, "unit": "GB/s",
                         "frac": (dom["GBps"] or 0) / peak, "peak_kind": f"of {main['peak_kind']}",
                         "frac_of_8TBps_nominal": (dom["GBps"] or 0) / NOMINAL_GBPS,
                         "avg_launch_us": dom["avg_us"], "median_launch_us": dom["median_us"],
                         "min_launch_us": dom["min_us"], "launches_timed": dom["launches"],
                         "frac_at_median": (dom["GBps_median"] or 0) / peak,
                         "algorithmic_bytes_per_launch": dom["alg_bytes"],
                         "traffic": None if args.batch > 0 else ncu_traffic(w.name, dom_name.split(" ")[0])},
            "kernels": kern,
            "calls": {"picospec_compress": main["compress_call"], "picospec_verify": main["verify_call"]},
            "other_kernels_avg_us": main["other_kernels_us"],
            "e2e": {k: main["e2e"][k] for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step")},
            "gpu_launches": main["launches_per_step"] * args.steps,
            "cpu_baseline": cpu_baseline,
            "clocks": main["clocks"],
            "rows_streamed_per_sec": main["rows_streamed_per_sec"],
            "slow_path_rows_per_step": main["slow_rows_per_step"],
            "compress_redo_rows_per_step": main["redo_rows_per_step"],
            "device_status": main["status"],
            "other_configs": others,
            "pipelined": pipelined,
            "paper_direction": paper_direction,
            "wire_codec": wire_codec,
            "vocab_parallel": vocab_parallel,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()


def launch_ranks(n: int) -> int:
    """Start `n` ranks of this script under torch.distributed.run on this node, one per GPU, and
    return its exit code.  Used when --gpus N > 1 is given without a torchrun environment."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    # keep NCCL's communicator line (rank / nranks) in the log of a multi-GPU run
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config4", choices=sorted(gen.WORKLOADS))
    ap.add_argument("--ref-sample", type=int, default=256,
                    help="most sequences per step of the CPU oracle legs (256 of config 4: about 20 core-seconds)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override B of the workload (profiling on a small case)")
    ap.add_argument("--roofline-launches", type=int, default=64,
                    help="bracketed launches per kernel behind the roofline entry (at most 128 are kept)")
    ap.add_argument("--all-configs", action="store_true", default=True)
    ap.add_argument("--only-main", dest="all_configs", action="store_false")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(launch_ranks(args.gpus))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
