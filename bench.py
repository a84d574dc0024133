#!/usr/bin/env python
"""Benchmark of the SMTM semantic-memory hot path on B200.

One step = one pass of the whole path over one batch: 512 concurrent streams,
one bf16 frame each, looked up at the ResNet-50 stage-3 exit (1024x14x14) and,
for frames that did not exit, at the stage-4 exit (2048x7x7), followed by the
table / centre update and the adaptive resize of every stream's fast memory.
Inputs are synthetic, seeded, resident in HBM and distinct per step (308 MB per
step, larger than L2).  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import smtm_inputs as si  # noqa: E402

WORKLOAD = si.C5   # the default and the benchmark line of record; --workload picks another for profiling
METRIC = "frames/sec through encode+lookup+exit per exit layer (whole path incl. update+resize)"


# DRAM bytes (read + write) of one launch of the dominant kernel from an ncu capture, per workload,
# with the digest of the kernel's sources at the time: a changed kernel reports no traffic until recaptured.
NCU_TRAFFIC = {"c5_streaming_bf16": (211_305_728, "753063d277df5b74")}
_KERNEL_SOURCES = ("encode.cu", "common.cuh", "lookup_common.cuh")


def ncu_traffic(workload_name: str, frames: int, full_frames: int):
    import hashlib

    if workload_name not in NCU_TRAFFIC or frames != full_frames:
        return None
    h = hashlib.sha256()
    for f in _KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2112_02644_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    traffic, digest = NCU_TRAFFIC[workload_name]
    return traffic if h.hexdigest()[:16] == digest else None


# --------------------------------------------------------------------------- helpers

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy read+write)"
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# --------------------------------------------------------------------------- sharding across ranks

def shard_for_rank(base, rank: int):
    """Every rank serves its own streams: the same workload recipe under a rank-specific seed."""
    return base.scaled(seed=base.seed + rank, T=max(base.T, 8))


def job_throughput(frames_per_rank: int, ms_local: float, world: int, device="cuda"):
    """Whole-job frames/s: all ranks' frames over the slowest rank's time (max over ranks)."""
    ms = ms_local
    if world > 1:
        import torch.distributed as dist

        t = torch.tensor([ms_local], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return frames_per_rank * world / (ms * 1e-3), ms


# --------------------------------------------------------------------------- the CUDA arm

def make_cache(smtm, w, cents, counts):
    return smtm.smtm_cache_create(w.n, w.dims, [w.tau] * w.L, cents, counts, n_streams=w.S, k_init=w.k_init,
                                  k_min=w.k_min, k_max=w.k_max, window_W=w.window_W, max_batch=w.B,
                                  flags=(smtm.FLAG_FORGET_FT if w.forgetting else 0) | smtm.FLAG_MAPS_READY)


def run_ours(args):
    import paper_2112_02644_b200 as smtm

    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    # every rank serves its own 512 streams (weak scaling by stream); no data-path collective
    base = si.WORKLOADS[[k for k in si.WORKLOADS if k.startswith(args.workload)][0]]
    w = shard_for_rank(base, rank)
    K, W = args.steps, args.warmup
    G = math.gcd(K, 32)         # steps captured into one CUDA graph
    while G > 1 and G > w.T:    # not more than the workload has
        G //= 2
    m = G if G % 2 == 0 else 2 * G   # resident steps: a whole number of graphs, and even (two carries alternate)
    T = min(w.T, max(K, W, m))
    T = max(m, T - T % m)
    labs = si.labels(w)
    cents, counts = si.initial_centers(w)
    sid = si.stream_ids(w)
    maps, fmaps, fbs = [], [], []
    for t in range(T):
        m = [si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)]
        maps.append(m)
        fmaps.append([smtm.Fmap(m[l], w.dtype, w.layout, *si.shape4(w, l)) for l in range(w.L)])
        fbs.append(torch.from_numpy(si.fallback_labels(w, labs[t])).cuda())
    torch.cuda.synchronize()
    # All launches go to one side stream so that every step can be captured into a CUDA graph.
    stream = torch.cuda.Stream()
    sh = stream.cuda_stream
    PROFILE_EVERY = 16  # every 16th step carries timing events and device-clock stamps (they cost a few us and break the chain of launches)

    def step(cache, gbs, t):
        gb = gbs[t % 2]   # two carries alternate: the cache was created with FLAG_MAPS_READY (maps are resident)
        smtm.smtm_lookup_exit_begin(cache, 0, fmaps[t % T][0], gb, sh)     # starts the batch: no separate reset
        for l in range(1, w.L):
            smtm.smtm_lookup_exit(cache, l, fmaps[t % T][l], gb, sh)
        smtm.smtm_cache_update_resize(cache, gb, fbs[t % T], sh)

    cache = make_cache(smtm, w, cents, counts)
    gb = [smtm.Batch(cache, w.B, stream_id=sid, with_diagnostics=False) for _ in range(2)]
    with torch.cuda.stream(stream):
        for t in range(W):          # eager warm-up: kernels, clocks, one-time function attributes
            step(cache, gb, t)
        stream.synchronize()
        # One graph per G resident steps (their feature maps are baked in); the cache state lives in
        # device memory the graphs point to, so replaying them in order advances it as eager calls
        # would.  Inside a graph the kernels of consecutive steps are chained like those of one step.
        smtm.smtm_cache_profile(cache, (T // PROFILE_EVERY + 1) * w.L, PROFILE_EVERY)
        launches0 = smtm.smtm_cache_get_launches(cache)
        graphs = []
        for g0 in range(0, T, G):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for t in range(g0, g0 + G):
                    step(cache, gb, t)
            graphs.append(g)
        launches_per_cycle = smtm.smtm_cache_get_launches(cache) - launches0
        for g in graphs:   # every graph once, untimed: its first launch uploads it to the device
            g.replay()
        stream.synchronize()
        ctr0 = smtm.smtm_cache_get_counters(cache)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler = ClockSampler(local_rank)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler.start()
        start.record(stream)
        for i in range(K // G):
            graphs[i % len(graphs)].replay()
        stop.record(stream)
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ms = start.elapsed_time(stop)
    launches = launches_per_cycle * K // T
    ctr = smtm.smtm_cache_get_counters(cache) - ctr0
    status = smtm.smtm_cache_status(cache)
    value, ms = job_throughput(K * w.B, ms, world)

    # roofline of the dominant launch (stage-3 lookup: every frame active)
    dom_total_ms, dom_n = smtm.smtm_cache_get_profile(cache, 0)
    dom_ms = dom_total_ms / max(dom_n, 1)
    dev_total, dev_cnt = smtm.smtm_cache_get_profile_device(cache)
    dev_n = int(dev_cnt[0])
    dev_ms = float(dev_total[0]) / dev_n if dev_n else None
    dev_names = ["lookup_layer%d" % l for l in range(w.L)] + ["update_plan", "update_centers", "update_tables"]
    dev_idx = list(range(w.L)) + [smtm.PROF_PLAN, smtm.PROF_CENTERS, smtm.PROF_TABLES]
    dev_us = {nm: (float(dev_total[i]) / int(dev_cnt[i]) * 1e3 if dev_cnt[i] else None) for nm, i in zip(dev_names, dev_idx)}
    l1_total_ms, l1_n = smtm.smtm_cache_get_profile(cache, 1) if w.L > 1 else (0.0, 0)
    C0 = w.stages[0][0]
    dom_bytes = w.B * (w.frame_bytes(0) + 4 * C0)
    peak, peak_src = measured_peaks()
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    exits = [int(v) for v in ctr[: w.L]]
    sid = sid if w.S > 1 else None

    e2e = None
    if rank == 0 or world > 1:
        e2e = run_e2e(smtm, w, cents, counts, labs, maps, sid if w.S > 1 else None, min(K, 16), world, sh)
    out = None
    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": "frames/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "streams_per_gpu": w.S, "frames_per_step_per_gpu": w.B,
                       "exit_layers": [list(s) for s in w.stages],
                       "map_dtype": {si.F32: "f32", si.F16: "f16", si.BF16: "bf16"}[w.dtype],
                       "layout": "NCHW" if w.layout == si.NCHW else "NHWC",
                       "classes": w.n, "fast_memory": [w.k_min, w.k_max], "tau": w.tau, "window_W": w.window_W,
                       "distinct_steps_resident": T, "l2_policy": "distinct maps per step, %.0f MB per step (L2 is 126 MB)" % (sum(w.B * w.frame_bytes(l) for l in range(w.L)) / 1e6),
                       "sharding": "streams across GPUs, no collective",
                       "launch": "CUDA graphs of %d steps (per step: %d lookups, update+refresh), chained launches, SMTM_FLAG_MAPS_READY with two alternating carries" % (G, w.L)},
            "e2e": e2e,
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "streaming kernel of the first exit layer (fused encode + similarity scoring where the fast memory has <= 64 entries), %d frames per launch" % w.B, "achieved": achieved,
                         "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                         "traffic": ncu_traffic(base.name, w.B, base.B), "bytes_per_launch": dom_bytes, "us_per_launch": dom_ms * 1e3,
                         "frac_of_nominal_8TBs": achieved / 8000.0, "launches_timed": int(dom_n),
                         "stage4_kernel_us_per_launch": l1_total_ms / max(l1_n, 1) * 1e3,
                         "device_clock": None if dev_ms is None else {
                             "us_per_launch": dev_ms * 1e3, "achieved": dom_bytes / (dev_ms * 1e-3) / 1e9,
                             "frac": dom_bytes / (dev_ms * 1e-3) / 1e9 / peak, "launches_timed": int(dev_n),
                             "note": "first CTA's start to last CTA's end by %globaltimer; the CUDA-event figure above also holds the two event nodes around the kernel"}},
            "step_kernels_device_clock_us": dev_us,
            "exit_histogram": {"per_layer": exits, "none": K * w.B - sum(exits)},
            "near_threshold_lookups": int(ctr[smtm.CTR_NEAR]),
            "device_status": status,
        }
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(w, budget_s=12.0)
    smtm.smtm_cache_destroy(cache)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out


def run_e2e(smtm, w, cents, counts, labs, maps, sid, K, world, sh):
    """Same metric through smtm_step_host: host buffers in, decisions out, copies inside the timed region."""
    cache = make_cache(smtm, w, cents, counts)
    hm = [[m.cpu().pin_memory() for m in maps[t]] for t in range(min(K, len(maps)))]
    fm = [smtm.Fmap(None, w.dtype, w.layout, *si.shape4(w, l)) for l in range(w.L)]
    done = torch.zeros(w.B, dtype=torch.uint8).pin_memory().numpy()
    el = torch.zeros(w.B, dtype=torch.int32).pin_memory().numpy()
    pred = torch.zeros(w.B, dtype=torch.int32).pin_memory().numpy()
    fbs = [si.fallback_labels(w, labs[t]) for t in range(len(hm))]
    smtm.smtm_step_host(cache, fm, hm[0], sid, fbs[0], True, done, el, pred, sh)   # allocates staging
    smtm.smtm_cache_destroy(cache)
    cache = make_cache(smtm, w, cents, counts)
    smtm.smtm_step_host(cache, fm, hm[0], sid, fbs[0], True, done, el, pred, sh)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    h2d_total = 0   # bytes of feature maps that crossed the bus: every frame at layer 0, then the frames still in
    for t in range(K):
        smtm.smtm_step_host(cache, fm, hm[t % len(hm)], sid, fbs[t % len(hm)], True, done, el, pred, sh)
        h2d_total += sum(int(((el == 0) | (el > l)).sum()) * w.frame_bytes(l) for l in range(w.L))
    dt = time.perf_counter() - t0
    if world > 1:
        import torch.distributed as dist

        tt = torch.tensor([dt], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        dt = float(tt.item())
    smtm.smtm_cache_destroy(cache)
    h2d = h2d_total / K + 2 * 4 * w.B
    return {"value": K * w.B * world / dt, "unit": "frames/s", "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": w.B * 9 + (w.L - 1) * w.B, "steps": K,
            "api": "smtm_step_host (pinned host buffers; later layers' maps are copied only for frames still in)"}


# --------------------------------------------------------------------------- the oracle arm

def oracle_steps(w, n_steps, budget_s=None, device="cpu"):
    """Runs the CPU oracle over the first steps of the workload; returns (frames, seconds in the oracle)."""
    import oracle

    labs = si.labels(w)
    cents, counts = si.initial_centers(w)
    mem = oracle.OracleMemory(w.n, w.dims, [w.tau] * w.L, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W,
                              forgetting=w.forgetting)
    sid = si.stream_ids(w)
    spent, frames = 0.0, 0
    for t in range(n_steps):
        maps = [si.frames(w, l, labs[t % w.T], t % w.T, device=device).cpu() for l in range(w.L)]
        fb = si.fallback_labels(w, labs[t % w.T])
        t0 = time.perf_counter()
        ob = mem.new_batch(w.B, sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps[l], w.dtype, w.layout, si.shape4(w, l), ob)
        mem.update(ob, fb)
        mem.resize()
        spent += time.perf_counter() - t0
        frames += w.B
        if budget_s is not None and spent >= budget_s:
            break
    return frames, spent


def cpu_baseline(w, budget_s):
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    frames, spent = oracle_steps(w, 32, budget_s=budget_s, device=dev)
    return {"value": frames / spent, "unit": "frames/s", "cores": 1, "kind": "oracle",
            "sample": f"first {frames // w.B} steps of {w.name} at full width ({w.B} streams), oracle time only",
            "host_cores_available": os.cpu_count()}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return None
    w = WORKLOAD.scaled(B=128, S=128)   # a bounded sample: 128 of the 512 streams per step
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    if args.warmup:
        oracle_steps(w, min(args.warmup, 2), device=dev)
    frames, spent = oracle_steps(w, args.steps, device=dev)
    value = frames / spent
    sample = f"{args.steps} steps of {WORKLOAD.name} restricted to 128 of its 512 streams, oracle time only"
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": "frames/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": spent / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "frames/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=640)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", help="c1..c5 (prefix of a workload name); c5 is the benchmark of record")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
