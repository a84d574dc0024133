#!/usr/bin/env python
"""Benchmark of the SMTM semantic-memory hot path on B200.

One step = one pass of the whole path over one batch: 512 concurrent streams,
one bf16 frame each, looked up at the ResNet-50 stage-3 exit (1024x14x14) and,
for frames that did not exit, at the stage-4 exit (2048x7x7), followed by the
table / centre update and the adaptive resize of every stream's fast memory.
Inputs are synthetic, seeded, resident in HBM and distinct per step (308 MB per
step, larger than L2).  The timed steps are steps W .. W+K-1 of the workload:
the memory is put back into the state it had after the W warm-up steps right
before the clock starts, and the exit histogram of the timed steps is checked
against the CPU oracle run over the same steps.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import concurrent.futures
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
L2_BYTES = 126e6


# DRAM bytes (read + write) of one launch of the dominant kernel from an ncu capture, per workload,
# with the digest of the kernel's sources at the time: a changed kernel reports no traffic until recaptured.
NCU_TRAFFIC = {"c5_streaming_bf16": (209_888_000, "95ec4214b44589b1")}
def kernel_digest() -> str:
    """Digest of the pooling kernel's source: its body in encode.cu (from the pipeline's heading to the next
    one), the parameter block it takes, and the copy / barrier helpers of common.cuh."""
    import hashlib

    csrc = os.path.join(ROOT, "paper_2112_02644_b200", "csrc")
    with open(os.path.join(csrc, "encode.cu")) as fh:
        enc = fh.read()
    body = enc[enc.index("// ---- persistent bulk-copy pipeline"):enc.index("// ---- fused lookup")]
    params = enc[enc.index("struct NchwParams {"):enc.index("};", enc.index("struct NchwParams {"))]
    h = hashlib.sha256((params + body).encode())
    with open(os.path.join(csrc, "common.cuh"), "rb") as fh:
        h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload_name: str, frames: int, full_frames: int):
    if workload_name not in NCU_TRAFFIC or frames != full_frames:
        return None
    traffic, digest = NCU_TRAFFIC[workload_name]
    return traffic if kernel_digest() == digest else None


# --------------------------------------------------------------------------- helpers

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops", 1590.0)), "measured (MEASURED_PEAKS.json, copy read+write)"
    return 6650.0, 1590.0, "fallback (earlier measurement on this pool)"


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


def launch_ranks(n: int, argv, port=None) -> int:
    """Starts `n` ranks of this script on this node (one per GPU) under torch's launcher and returns its exit
    code; used when --gpus N is given and no launcher has set WORLD_SIZE."""
    port = port or 29500 + os.getpid() % 1000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def rank_check(args):
    """The multi-rank plumbing alone, on the host (gloo): rendezvous, one shard of streams per rank, the
    job's time as the maximum over ranks.  No GPU work; rank 0 prints one JSON line."""
    import torch.distributed as dist

    rank, _, world = dist_env()
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
    w = shard_for_rank(WORKLOAD.scaled(B=16, S=16), rank)
    value, ms = job_throughput(1000, 10.0 * (rank + 1), world, device="cpu")
    seeds = [None] * world
    if world > 1:
        dist.all_gather_object(seeds, w.seed)
        dist.barrier()
        dist.destroy_process_group()
    else:
        seeds = [w.seed]
    return {"rank_check": True, "n_gpus": world, "value": value, "ms": ms, "seeds": seeds} if rank == 0 else None


# --------------------------------------------------------------------------- the oracle on the host cores

class OracleRun:
    """The CPU oracle stepped over a workload from a fresh memory, either on one thread or with the frames of a
    step split over a pool of threads (the C functions release the interpreter lock).  Lookups of a step are
    independent per frame; tables and fast memories per stream; Eq. 7 per class."""

    def __init__(self, w, threads: int = 1):
        import oracle

        self.o = oracle
        self.w = w
        cents, counts = si.initial_centers(w)
        self.mem = oracle.OracleMemory(w.n, w.dims, [w.tau] * w.L, cents, counts, w.S, w.k_init, w.k_min, w.k_max,
                                       w.window_W, forgetting=w.forgetting)
        self.sid = si.stream_ids(w)
        self.threads = threads
        self.pool = concurrent.futures.ThreadPoolExecutor(threads) if threads > 1 else None
        self.seconds = 0.0
        self.frames = 0
        self.exits_after = []   # cumulative exits per layer after each step

    def close(self):
        if self.pool:
            self.pool.shutdown()

    def step(self, maps_cpu, fallback):
        t0 = time.perf_counter()
        (self._step_threaded if self.pool else self._step_serial)(maps_cpu, fallback)
        self.seconds += time.perf_counter() - t0
        self.frames += self.w.B
        self.exits_after.append(self.mem.exits_per_layer.copy())

    def _step_serial(self, maps_cpu, fallback):
        w, mem = self.w, self.mem
        ob = mem.new_batch(w.B, self.sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps_cpu[l], w.dtype, w.layout, si.shape4(w, l), ob)
        mem.update(ob, fallback)
        mem.resize()

    def _step_threaded(self, maps_cpu, fallback):
        # Frames are cut into one contiguous slice per thread.  Every slice is looked up against the memory as
        # it stood when the step began; then tables and fast memories are updated per slice of streams (this
        # split needs each stream's frames inside one slice: one frame per stream, or a single stream), and
        # Eq. 7 per range of classes (each range sees every frame, in ascending order, with the labels outside
        # the range blanked).  The arithmetic is the oracle's own functions, untouched.
        o, w, mem = self.o, self.w, self.mem
        B, n_thr = w.B, self.threads
        cuts = [B * i // n_thr for i in range(n_thr + 1)]
        slices = [(a, b) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]
        ob = mem.new_batch(B, self.sid)
        exits = np.zeros(w.L, np.int64)
        for l in range(w.L):
            B_, C, H, W = si.shape4(w, l)
            raw = o._raw(maps_cpu[l]).reshape(B, -1)

            def look(ab, l=l, C=C, H=H, W=W, raw=raw):
                a, b = ab
                todo = ob["done"][a:b] == 0
                o.gap(raw[a:b], w.dtype, w.layout, b - a, C, H, W, skip=ob["done"][a:b], out=ob["sv"][l][a:b])
                ac, sep, top, near = o.lookup_layer(l + 1, ob["sv"][l][a:b], mem.centers[l], ob["stream_id"][a:b],
                                                    mem.members, mem.k, mem.tau[l], ob["sa"][a:b], ob["done"][a:b],
                                                    ob["exit_layer"][a:b], ob["pred"][a:b])
                return int(np.count_nonzero(todo & (ob["done"][a:b] == 1))), int(near[todo].sum())

            for ex, near in self.pool.map(look, slices):
                exits[l] += ex
                mem.near_count += near
        mem.exits_per_layer += exits
        fb = np.where(fallback >= mem.n, -1, fallback).astype(np.int32)
        exited = ob["done"] == 1
        final = np.ascontiguousarray(np.where(exited, ob["pred"], fb), np.int32)
        stop = np.ascontiguousarray(np.where(exited, ob["exit_layer"], mem.L), np.int32)
        per_stream = w.S > 1      # one frame per stream: slice b0..b1 of the frames is streams b0..b1

        def tables(ab):
            a, b = ab
            if per_stream:
                o.tables_update(np.ascontiguousarray(ob["stream_id"][a:b] - a), final[a:b], mem.ft[a:b], mem.ts[a:b],
                                mem.W if mem.forgetting else 0)
                o.resize(mem.ft[a:b], mem.ts[a:b], mem.W, mem.k_min, mem.k_max, mem.cl_num, mem.cl_den,
                         mem.members[a:b], mem.k[a:b], forgetting=mem.forgetting)

        def centres(job):
            l0, lo, hi = job
            mine = np.ascontiguousarray(np.where((final >= lo) & (final < hi), final, -1), np.int32)
            o.centers_update(l0, ob["sv"][l0 - 1], mine, stop, mem.centers[l0 - 1], mem.m[l0 - 1])

        ccuts = [mem.n * i // n_thr for i in range(n_thr + 1)]
        jobs = [(l0, a, b) for l0 in range(1, mem.L + 1) for a, b in zip(ccuts[:-1], ccuts[1:]) if b > a]
        if per_stream:
            futs = [self.pool.submit(tables, ab) for ab in slices] + [self.pool.submit(centres, j) for j in jobs]
        else:       # a single stream: its tables are one sequential replay
            o.tables_update(ob["stream_id"], final, mem.ft, mem.ts, mem.W if mem.forgetting else 0)
            futs = [self.pool.submit(centres, j) for j in jobs]
        for f in futs:
            f.result()
        if not per_stream:
            mem.resize()


# --------------------------------------------------------------------------- the CUDA arm

def make_cache(smtm, w, cents, counts):
    # every workload here keeps its maps resident and alternates two carries: the library may pipeline its steps
    # (for NHWC maps only the first layer of a step; its later layers keep their one kernel per layer)
    flags = (smtm.FLAG_FORGET_FT if w.forgetting else 0) | smtm.FLAG_MAPS_READY
    return smtm.smtm_cache_create(w.n, w.dims, [w.tau] * w.L, cents, counts, n_streams=w.S, k_init=w.k_init,
                                  k_min=w.k_min, k_max=w.k_max, window_W=w.window_W, max_batch=w.B, flags=flags)


PROFILE_EVERY = 20  # every 20th step carries timing events and device-clock stamps (they cost a few us and break the chain of launches)


class Resident:
    """A workload's inputs resident in HBM: distinct maps for enough steps that consecutive steps never find
    their maps in L2 (and, for the streaming workload, every step of the timed region its own maps)."""

    def __init__(self, smtm, w, steps_needed: int):
        self.w = w
        step_bytes = sum(w.B * w.frame_bytes(l) for l in range(w.L))
        if w.T > 1:
            self.R = min(w.T, steps_needed)
        else:   # a single-batch workload: the same labels under fresh noise, enough copies to defeat L2
            self.R = max(2, int(math.ceil(2.2 * L2_BYTES / step_bytes)))
            self.R += self.R % 2
        self.step_bytes = step_bytes
        self.labs = si.labels(w)
        self.maps, self.fmaps, self.fbs = [], [], []
        for r in range(self.R):
            lab = self.labs[r % w.T]
            m = [si.frames(w, l, lab, r, device="cuda") for l in range(w.L)]
            self.maps.append(m)
            self.fmaps.append([smtm.Fmap(m[l], w.dtype, w.layout, *si.shape4(w, l)) for l in range(w.L)])
            self.fbs.append(torch.from_numpy(si.fallback_labels(w, lab)).cuda())
        torch.cuda.synchronize()

    def fallback_host(self, t):
        return si.fallback_labels(self.w, self.labs[(t % self.R) % self.w.T])


def measure(smtm, w, K, W, local_rank, world, verify_steps=0, graph_steps=64):
    """Times steps W .. W+K-1 of workload `w` through CUDA graphs and returns the figures of the run.
    verify_steps > 0: the CPU oracle is run over steps 0 .. W+verify_steps-1 of the same maps and the exits it
    takes in steps W .. W+verify_steps-1 are compared with the library's."""
    if world > 1:
        import torch.distributed as dist
    res = Resident(smtm, w, W + K)
    R = res.R
    G = max(d for d in range(1, graph_steps + 1) if K % d == 0)   # steps captured into one CUDA graph
    cents, counts = si.initial_centers(w)
    sid = si.stream_ids(w) if w.S > 1 else None
    # All launches go to one side stream so that every step can be captured into a CUDA graph.
    stream = torch.cuda.Stream()
    sh = stream.cuda_stream

    def step(cache, gbs, t):
        gb = gbs[t % 2]   # two carries alternate: the cache was created with FLAG_MAPS_READY (maps are resident)
        smtm.smtm_lookup_exit_begin(cache, 0, res.fmaps[t % R][0], gb, sh)     # starts the batch: no separate reset
        for l in range(1, w.L):
            smtm.smtm_lookup_exit(cache, l, res.fmaps[t % R][l], gb, sh)
        smtm.smtm_cache_update_resize(cache, gb, res.fbs[t % R], sh)

    cache = make_cache(smtm, w, cents, counts)
    gb = [smtm.Batch(cache, w.B, stream_id=sid, with_diagnostics=False) for _ in range(2)]
    with torch.cuda.stream(stream):
        for t in range(W):          # eager warm-up: kernels, clocks; these are steps 0 .. W-1 of the workload
            step(cache, gb, t)
        stream.synchronize()
        snapshot = smtm.smtm_cache_export(cache)   # the memory after the warm-up steps: where the timed region starts
        # One graph per G consecutive steps (their feature maps are baked in); the cache state lives in
        # device memory the graphs point to, so replaying them in order advances it as eager calls
        # would.  Inside a graph the kernels of consecutive steps are chained like those of one step.
        n_prof = (K // PROFILE_EVERY + 2) * w.L
        smtm.smtm_cache_profile(cache, n_prof, PROFILE_EVERY)
        launches0 = smtm.smtm_cache_get_launches(cache)
        graphs, order = {}, []
        for t0 in range(W, W + K, G):
            key = (t0 % R, t0 % 2) if R % G == 0 else t0     # steps t0 and t0 + R read the same maps
            if key not in graphs:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    for t in range(t0, t0 + G):
                        step(cache, gb, t)
                graphs[key] = g
            order.append(graphs[key])
        launches_per_graph = (smtm.smtm_cache_get_launches(cache) - launches0) // max(len(graphs), 1)
        for g in graphs.values():   # every graph once, untimed: its first launch uploads it to the device
            g.replay()
        stream.synchronize()

        def restart():
            smtm.smtm_cache_import(cache, snapshot)      # back to the state after step W-1 (synchronises)

        check = None
        V = min(verify_steps, K) // G * G
        if V > 0:
            check = {"steps": [W, W + V]}
            if V < K:   # the timed region is longer than what the oracle covers: a separate, untimed pass
                restart()
                for g in order[: V // G]:
                    g.replay()
                stream.synchronize()
                ctr = smtm.smtm_cache_get_counters(cache)
                check["gpu_exits"] = [int(v) for v in ctr[: w.L]]
                check["near_threshold_lookups"] = int(ctr[smtm.CTR_NEAR])
        restart()
        ctr0 = smtm.smtm_cache_get_counters(cache)
        if check is not None and "gpu_exits" in check:
            check["gpu_exits"] = [a - int(b) for a, b in zip(check["gpu_exits"], ctr0[: w.L])]
            check["near_threshold_lookups"] -= int(ctr0[smtm.CTR_NEAR])
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler = ClockSampler(local_rank)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler.start()
        start.record(stream)
        for g in order:
            g.replay()
        stop.record(stream)
        torch.cuda.synchronize()
        ctr = smtm.smtm_cache_get_counters(cache) - ctr0
        # The timed region lasts milliseconds, less than one sampling period of nvidia-smi: the same graphs
        # are replayed for a quarter of a second more (untimed) so that the clocks are read under this load.
        t_end = time.perf_counter() + 0.25
        while time.perf_counter() < t_end:
            for g in order:
                g.replay()
            stream.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    clocks["sampled"] = "timed region plus 0.25 s more of the same graphs, untimed"
    ms_local = start.elapsed_time(stop)
    out = {
        "w": w, "res": res, "cents": cents, "counts": counts, "sid": sid, "sh": sh, "G": G, "R": R,
        "ms_local": ms_local, "clocks": clocks, "launches": int(launches_per_graph * len(order)),
        "exits": [int(v) for v in ctr[: w.L]], "near": int(ctr[smtm.CTR_NEAR]),
        "status": smtm.smtm_cache_status(cache), "routes": [int(v) for v in smtm.smtm_cache_get_routes(cache)],
    }
    if check is not None and "gpu_exits" not in check:
        check["gpu_exits"], check["near_threshold_lookups"] = out["exits"], out["near"]
    # per-kernel figures of the profiled steps
    ev = [smtm.smtm_cache_get_profile(cache, l) for l in range(w.L)]
    out["event_us"] = [tot / max(n, 1) * 1e3 for tot, n in ev]
    out["event_n"] = [int(n) for _, n in ev]
    dev_total, dev_cnt = smtm.smtm_cache_get_profile_device(cache)
    names = ["lookup_layer%d" % l for l in range(w.L)] + ["score_layer%d" % l for l in range(w.L)] + \
        ["update_plan", "update_centers", "update_tables", "score_tc", "finish_dense", "refresh"]
    idx = list(range(w.L)) + [smtm.PROF_SCORE + l for l in range(w.L)] + \
        [smtm.PROF_PLAN, smtm.PROF_CENTERS, smtm.PROF_TABLES, smtm.PROF_SCORE_TC, smtm.PROF_FINISH_DENSE,
         smtm.PROF_REFRESH]
    out["device_us"] = {nm: (float(dev_total[i]) / int(dev_cnt[i]) * 1e3 if dev_cnt[i] else None) for nm, i in zip(names, idx)}
    out["device_n"] = int(dev_cnt[0])
    # the first layer's pooling kernel alone on the device (smtm_encode over the resident maps, back to back):
    # what the streaming kernel does when nothing shares the machine with it
    sv_tmp = torch.empty((w.B, w.stages[0][0]), dtype=torch.float32, device="cuda")
    n_alone = min(R, 16)
    with torch.cuda.stream(stream):
        for t in range(min(R, 3)):
            smtm.smtm_encode(cache, 0, res.fmaps[t][0], sv_tmp, stream=sh)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for t in range(n_alone):
            smtm.smtm_encode(cache, 0, res.fmaps[(t + 3) % R][0], sv_tmp, stream=sh)
        e1.record(stream)
        stream.synchronize()
    out["pool_alone_us"] = e0.elapsed_time(e1) / n_alone * 1e3
    smtm.smtm_cache_destroy(cache)

    if check is not None:   # the oracle over the same steps, from a fresh memory
        run = OracleRun(w, threads=1)
        for t in range(W + V):
            run.step([m.cpu() for m in res.maps[t % R]], res.fallback_host(t))
        before = run.exits_after[W - 1] if W > 0 else np.zeros(w.L, np.int64)
        check["oracle_exits"] = [int(a - b) for a, b in zip(run.exits_after[-1], before)]
        diff = sum(abs(a - b) for a, b in zip(check["gpu_exits"], check["oracle_exits"]))
        # a decision within 1e-4 of the threshold may fall either way; anything beyond that is an error
        check["match"] = diff <= 2 * (check["near_threshold_lookups"] + run.mem.near_count)
        check["frames"] = V * w.B
        out["oracle_check"] = check
        out["oracle_run"] = run
    return out


def roofline_of(w, m, peak, layer=0):
    """Roofline figures of the streaming kernel of `layer`: algorithmic bytes of one launch over its duration.
    Layer 0 sees every frame of the batch (the batch starts there)."""
    C = w.stages[layer][0]
    nbytes = w.B * (w.frame_bytes(layer) + 4 * C)
    us_ev, us_dev = m["event_us"][layer], m["device_us"]["lookup_layer%d" % layer]
    ach = nbytes / (us_ev * 1e-6) / 1e9 if us_ev else None
    ach_dev = nbytes / (us_dev * 1e-6) / 1e9 if us_dev else None
    return nbytes, us_ev, ach, us_dev, ach_dev


def run_ours(args):
    import paper_2112_02644_b200 as smtm

    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    # every rank serves its own 512 streams (weak scaling by stream); no data-path collective
    base = si.WORKLOADS[[k for k in si.WORKLOADS if k.startswith(args.workload)][0]]
    w = shard_for_rank(base, rank) if base.T > 1 else base
    K, W = args.steps, args.warmup
    peak, tc_peak, peak_src = measured_peaks()
    with_oracle = rank == 0 and world == 1 and not args.no_cpu_baseline
    verify = min(K, max(w.T - W, 0) if w.T > 1 else 4) if with_oracle else 0
    m = measure(smtm, w, K, W, local_rank, world, verify_steps=verify)
    value, ms = job_throughput(K * w.B, m["ms_local"], world)
    dom_bytes, dom_us, achieved, dev_us, dev_ach = roofline_of(w, m, peak)

    e2e = run_e2e(smtm, w, m, min(K, 16), world)
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
                       "timed_steps": [W, W + K], "workload_steps": w.T, "distinct_steps_resident": m["R"],
                       "l2_policy": "distinct maps per step, %.0f MB per step (L2 is 126 MB)" % (m["res"].step_bytes / 1e6),
                       "state": "the memory is put back to its state after step W-1 (smtm_cache_import) right before the timed region",
                       "sharding": "streams across GPUs, no collective",
                       "launch": "CUDA graphs of %d steps (per step: %d lookups, update+refresh), chained launches, SMTM_FLAG_MAPS_READY with two alternating carries" % (m["G"], w.L)},
            "e2e": e2e,
            "gpu_launches": m["launches"],
            "clocks": m["clocks"],
            "roofline": {"bound": "hbm", "kernel": "streaming kernel of the first exit layer, %d frames per launch (pipelined route: the pooling kernel, timed while the previous step's later layers and update share the device with it; otherwise the fused encode + scoring kernel)" % w.B,
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak if achieved else None,
                         "peak_source": peak_src, "traffic": ncu_traffic(base.name, w.B, base.B),
                         "bytes_per_launch": dom_bytes, "us_per_launch": dom_us,
                         "frac_of_nominal_8TBs": achieved / 8000.0 if achieved else None, "launches_timed": m["event_n"][0],
                         "later_layers_kernel_us_per_launch": m["event_us"][1:],
                         "device_clock": None if dev_us is None else {
                             "us_per_launch": dev_us, "achieved": dev_ach, "frac": dev_ach / peak, "launches_timed": m["device_n"],
                             "note": "first CTA's start to last CTA's end by %globaltimer; the CUDA-event figure above also holds the two event nodes around the kernel"},
                         "alone": {"us_per_launch": m["pool_alone_us"], "achieved": dom_bytes / (m["pool_alone_us"] * 1e-6) / 1e9,
                                   "frac": dom_bytes / (m["pool_alone_us"] * 1e-6) / 1e9 / peak,
                                   "note": "the pooling kernel of the same layer back to back with nothing beside it (smtm_encode, CUDA events around 16 launches)"},
                         "whole_step": {"bytes": None, "achieved": None, "frac": None}},
            "step_kernels_device_clock_us": m["device_us"],
            "exit_histogram": {"per_layer": m["exits"], "none": K * w.B - sum(m["exits"])},
            "near_threshold_lookups": m["near"],
            "routes": dict(zip(("fused", "dense", "plain", "pipelined", "pipelined_dense"), m["routes"])),
            "device_status": m["status"],
        }
        # bytes the whole step had to move (maps of the frames still in at each layer + their SV rows) over the step time
        step_bytes = w.B * (w.frame_bytes(0) + 4 * w.stages[0][0])
        left = K * w.B
        for l in range(1, w.L):
            left -= m["exits"][l - 1]
            step_bytes += left / K * (w.frame_bytes(l) + 4 * w.stages[l][0])
        ws = step_bytes / (ms / K * 1e-3) / 1e9
        out["roofline"]["whole_step"] = {"bytes": int(step_bytes), "achieved": ws, "frac": ws / peak}
        if "oracle_check" in m:
            out["oracle_check"] = m["oracle_check"]
            run = m["oracle_run"]
            out["cpu_baseline"] = {"value": run.frames / run.seconds, "unit": "frames/s", "cores": 1, "kind": "oracle",
                                   "sample": f"steps 0..{len(run.exits_after) - 1} of {w.name} at full width ({w.B} frames per step), oracle time only",
                                   "host_cores_available": os.cpu_count()}
            out["cpu_baseline_all_cores"] = cpu_all_cores(w, m, run, budget_s=10.0)
    del m["res"]
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_other_workloads and base.name == WORKLOAD.name:
        out["other_workloads"] = [other_workload(smtm, si.WORKLOADS[k], peak, tc_peak, with_oracle)
                                  for k in si.WORKLOADS if k[:2] in ("c1", "c2", "c3", "c4")]
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if out is not None and "oracle_check" in out and not out["oracle_check"]["match"]:
        print(json.dumps(out))
        sys.exit("exit histogram of the timed steps differs from the oracle's: %r" % (out["oracle_check"],))
    return out


def cpu_all_cores(w, m, serial_run, budget_s):
    """The oracle with the frames of a step split over all host cores, from a fresh memory; its exits must be
    the single-thread run's."""
    cores = os.cpu_count() or 1
    run = OracleRun(w, threads=cores)
    res = m["res"]
    t = 0
    while t < len(serial_run.exits_after) and run.seconds < budget_s:
        run.step([mm.cpu() for mm in res.maps[t % res.R]], res.fallback_host(t))
        t += 1
    run.close()
    same = all(np.array_equal(a, b) for a, b in zip(run.exits_after, serial_run.exits_after))
    return {"value": run.frames / run.seconds, "unit": "frames/s", "cores": cores, "kind": "oracle",
            "sample": f"steps 0..{t - 1} of {w.name}, frames of a step split over {cores} threads, oracle time only",
            "same_exits_as_one_thread": bool(same)}


def other_workload(smtm, w, peak, tc_peak, with_oracle):
    """A short pass of one of the single-batch workloads: the same machinery, fewer steps."""
    K, W = 16, 3
    m = measure(smtm, w, K, W, 0, 1, verify_steps=8 if with_oracle else 0, graph_steps=8)
    nbytes, us_ev, ach, us_dev, ach_dev = roofline_of(w, m, peak)
    ms = m["ms_local"] / K
    out = {"workload": w.name, "steps": K, "warmup": W, "ms_per_step": ms, "frames_per_s": w.B / (ms * 1e-3),
           "dominant_kernel_us": us_dev if us_dev else us_ev, "dominant_kernel_us_cuda_events": us_ev,
           "frac": (ach_dev if ach_dev else ach) / peak if (ach_dev or ach) else None,
           "bytes_per_launch": nbytes, "routes": dict(zip(("fused", "dense", "plain", "pipelined", "pipelined_dense"), m["routes"])),
           "exit_histogram": {"per_layer": m["exits"], "none": K * w.B - sum(m["exits"])},
           "near_threshold_lookups": m["near"], "step_kernels_device_clock_us": m["device_us"],
           "distinct_steps_resident": m["R"], "device_status": m["status"]}
    step_bytes = sum(w.B * w.frame_bytes(l) for l in range(w.L))
    out["hbm_floor_us_all_frames_active"] = step_bytes / (peak * 1e9) * 1e6
    if m["device_us"].get("score_tc"):   # Eq. 1 as a dense contraction: three bf16 products of B x n x D
        flops = 3 * 2.0 * w.B * w.n * w.stages[0][0]
        out["score_tc"] = {"us": m["device_us"]["score_tc"], "tflops_split_bf16": flops / (m["device_us"]["score_tc"] * 1e-6) / 1e12,
                           "frac_of_bf16_peak": flops / (m["device_us"]["score_tc"] * 1e-6) / 1e12 / tc_peak}
    if "oracle_check" in m:
        out["oracle_check"] = m["oracle_check"]
    del m["res"]
    torch.cuda.empty_cache()
    return out


def run_e2e(smtm, w, m, K, world):
    """Same metric through smtm_step_host: host buffers in, decisions out, copies inside the timed region."""
    res, sid, sh = m["res"], m["sid"], m["sh"]
    cache = make_cache(smtm, w, m["cents"], m["counts"])
    hm = [[x.cpu().pin_memory() for x in res.maps[t]] for t in range(min(K, res.R))]
    fm = [smtm.Fmap(None, w.dtype, w.layout, *si.shape4(w, l)) for l in range(w.L)]
    done = torch.zeros(w.B, dtype=torch.uint8).pin_memory().numpy()
    el = torch.zeros(w.B, dtype=torch.int32).pin_memory().numpy()
    pred = torch.zeros(w.B, dtype=torch.int32).pin_memory().numpy()
    fbs = [res.fallback_host(t) for t in range(len(hm))]
    smtm.smtm_step_host(cache, fm, hm[0], sid, fbs[0], True, done, el, pred, sh)   # allocates staging
    smtm.smtm_cache_destroy(cache)
    cache = make_cache(smtm, w, m["cents"], m["counts"])
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
    run = OracleRun(w, threads=1)
    labs = si.labels(w)
    for t in range(n_steps):
        maps = [si.frames(w, l, labs[t % w.T], t % w.T, device=device).cpu() for l in range(w.L)]
        run.step(maps, si.fallback_labels(w, labs[t % w.T]))
        if budget_s is not None and run.seconds >= budget_s:
            break
    return run.frames, run.seconds


def run_timeline(args):
    """Where the kernels of consecutive steps sit in time: one CUDA graph of N steps in which every kernel stamps
    the device clock (no events; a memset per step and stream clears the stamps, which costs each step about a
    microsecond), replayed three times from the same memory; the last replay is printed, in microseconds from the
    begin of the first step's first kernel."""
    import paper_2112_02644_b200 as smtm

    torch.cuda.set_device(0)
    w = si.WORKLOADS[[k for k in si.WORKLOADS if k.startswith(args.workload)][0]]
    N, W = args.timeline, max(args.warmup, 3)
    res = Resident(smtm, w, W + N)
    cents, counts = si.initial_centers(w)
    cache = make_cache(smtm, w, cents, counts)
    gbs = [smtm.Batch(cache, w.B, stream_id=si.stream_ids(w) if w.S > 1 else None, with_diagnostics=False) for _ in range(2)]
    stream = torch.cuda.Stream()
    sh = stream.cuda_stream
    R = len(res.fmaps)

    def step(t):
        gb = gbs[t % 2]
        smtm.smtm_lookup_exit_begin(cache, 0, res.fmaps[t % R][0], gb, sh)
        for l in range(1, w.L):
            smtm.smtm_lookup_exit(cache, l, res.fmaps[t % R][l], gb, sh)
        smtm.smtm_cache_update_resize(cache, gb, res.fbs[t % R], sh)

    with torch.cuda.stream(stream):
        for t in range(W):
            step(t)
        stream.synchronize()
        blob = smtm.smtm_cache_export(cache)
        smtm.smtm_cache_profile(cache, (N + 1) * w.L, -1)   # every step, device-clock stamps alone
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for t in range(W, W + N):
                step(t)
        for _ in range(3):
            smtm.smtm_cache_import(cache, blob)
            g.replay()
            stream.synchronize()
    names = {}
    for l in range(w.L):
        names[l] = "stream_layer%d" % l
        names[smtm.PROF_SCORE + l] = "score_layer%d" % l
    names.update({smtm.PROF_SCORE_TC: "score_tc", smtm.PROF_FINISH_DENSE: "finish_dense", smtm.PROF_PLAN: "update_plan",
                  smtm.PROF_CENTERS: "update_centers", smtm.PROF_TABLES: "update_tables", smtm.PROF_REFRESH: "refresh"})
    t0, steps = None, []
    for i in range(N):
        b, e = smtm.smtm_cache_get_profile_timeline(cache, i)
        if t0 is None:
            t0 = min(int(b[k]) for k in names if int(b[k]))
        steps.append({nm: [round((int(b[k]) - t0) / 1e3, 2), round((int(e[k]) - t0) / 1e3, 2)] for k, nm in names.items() if int(b[k])})
    out = {"timeline_us": steps, "workload": w.name, "steps": N, "warmup": W,
           "routes": [int(v) for v in smtm.smtm_cache_get_routes(cache)], "device_status": smtm.smtm_cache_status(cache)}
    smtm.smtm_cache_destroy(cache)
    return out


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
    global PROFILE_EVERY
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60, help="timed steps; warm-up + steps = 64 walks the streaming workload once")
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", help="c1..c5 (prefix of a workload name); c5 is the benchmark of record")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle legs (profiling runs)")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the short passes of c1..c4")
    ap.add_argument("--profile-every", type=int, default=PROFILE_EVERY,
                    help="every N-th step of the timed region carries timing events and device-clock stamps")
    ap.add_argument("--timeline", type=int, default=0, metavar="N",
                    help="print where the kernels of N consecutive steps sit in time (device clock) instead of the benchmark line")
    ap.add_argument("--rank-check", action="store_true", help="multi-rank plumbing only, on the host (gloo)")
    args = ap.parse_args()
    PROFILE_EVERY = max(1, args.profile_every)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:   # no launcher above us: start the ranks ourselves
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.rank_check:
        out = rank_check(args)
    elif args.timeline > 0:
        out = run_timeline(args)
    else:
        out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
