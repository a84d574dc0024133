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
