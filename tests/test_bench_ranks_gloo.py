"""Host logic of the multi-GPU benchmark, on CPU: two gloo ranks, world size 2.

The path shards by sequence: every rank verifies its own sequences and there is no collective on the
data path; only the timing is reduced (max over ranks) and only rank 0 reports."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    from paper_2603_03383_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.WORKLOADS["batched"]
    mine = 10.0 + 5.0 * rank                       # this rank's "time"
    slowest = bench.max_over_ranks(mine, world)
    seeds = [None] * world
    dist.all_gather_object(seeds, bench.rank_seed(w, rank))
    lens = synth.seq_lens(w, seed=bench.rank_seed(w, rank)).tolist()
    all_lens = [None] * world
    dist.all_gather_object(all_lens, lens)
    dist.barrier()
    out[rank] = dict(slowest=slowest, seeds=seeds, lens=all_lens)
    dist.destroy_process_group()


def test_two_ranks_reduce_timing_and_work_on_different_sequences():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29517, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["slowest"] == res[1]["slowest"] == 15.0          # max over ranks, seen by every rank
    assert len(set(res[0]["seeds"])) == world                      # independent sequences per rank
    assert res[0]["lens"][0] != res[0]["lens"][1]
    assert res[0]["lens"] == res[1]["lens"]                        # deterministic: a rank's data depends on its rank only


def test_max_over_ranks_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, 1) == 3.25


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True,
                       timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_one_json_line_on_rank_zero():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny", "--layers", "2"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "steps/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
