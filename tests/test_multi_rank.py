"""The multi-rank logic of bench.py on CPU with two gloo ranks: streams are sharded across
ranks (no data-path collective), the job's time is the maximum over ranks, and the reference
arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    import smtm_inputs as si

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.shard_for_rank(si.C5.scaled(B=16, S=16), rank)
    lab = si.labels(w)
    mine = torch.from_numpy(lab[:4].astype(np.int64))
    both = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(both, mine)
    value, ms = bench.job_throughput(1000, 10.0 * (rank + 1), world, device="cpu")   # rank 1 is the slow one
    ref = bench.run_reference.__code__.co_name   # the function exists; its rank filter is checked below
    assert bench.dist_env() == (rank, rank, world)
    json.dump({"labels_differ": bool((both[0] != both[1]).any()), "value": value, "ms": ms, "seed": w.seed,
               "ref": ref}, open(os.path.join(out_dir, f"r{rank}.json"), "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_streams_and_take_the_slowest_time(tmp_path):
    port = 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0["labels_differ"] and r1["labels_differ"]          # different streams on different ranks
    assert r0["seed"] != r1["seed"]
    assert r0["ms"] == r1["ms"] == 20.0                          # max over ranks
    assert r0["value"] == r1["value"] == 2 * 1000 / 20e-3        # all ranks' frames over that time


def test_reference_arm_runs_the_oracle_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and out.stdout.strip() == ""     # other ranks exit 0 without work
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "frames/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_that_many_ranks_itself():
    # without a launcher above it, `bench.py --gpus 2` starts two ranks on this node; --rank-check runs only the
    # multi-rank plumbing (gloo rendezvous, one shard of streams per rank, time = max over ranks) on the host
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check"], env=env,
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["ms"] == 20.0 and line["value"] == 2 * 1000 / 20e-3
    assert len(set(line["seeds"])) == 2                      # every rank serves its own streams


def test_oracle_split_over_threads_equals_the_oracle_on_one_thread():
    # the all-cores leg of the CPU baseline splits the frames of a step over threads; it must leave exactly the
    # state the plain frame-by-frame run leaves (one frame per stream, a single stream, the forgetting tables)
    sys.path.insert(0, ROOT)
    import bench
    import smtm_inputs as si

    for w in (si.C5.scaled(B=24, S=24, T=5), si.C2.scaled(B=16), si.C6.scaled(B=16, S=16, T=3)):
        a, b = bench.OracleRun(w, 1), bench.OracleRun(w, 3)
        labs = si.labels(w)
        for t in range(4):
            lab = labs[t % w.T]
            maps = [si.frames(w, l, lab, t) for l in range(w.L)]
            fb = si.fallback_labels(w, lab)
            a.step(maps, fb)
            b.step(maps, fb)
        b.close()
        assert all(np.array_equal(x, y) for x, y in zip(a.exits_after, b.exits_after))
        for name in ("ft", "ts", "members", "k"):
            assert np.array_equal(getattr(a.mem, name), getattr(b.mem, name)), (w.name, name)
        for x, y in zip(a.mem.centers + a.mem.m, b.mem.centers + b.mem.m):
            assert np.array_equal(x, y)
