"""The N > 1 path of the benchmark on CPU: two gloo ranks check the whole-job aggregation
(max of times, sum of counts), the per-rank inputs of a weak-scaling run (shared weights,
different sequences), and that the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e_s, tokens, e2e_tokens, launches = bench.aggregate(dist, torch.device("cpu"), 10.0 + rank, 2.0 - rank, 100 + rank, 7, 50)
    _, _, _, ph, pr, prefix = bench._setup_inputs(rank)
    dist.barrier()
    if rank == 0:
        json.dump({"ms": ms, "e2e_s": e2e_s, "tokens": tokens, "e2e_tokens": e2e_tokens, "launches": launches}, open(out, "w"))
    json.dump({"prefix": prefix[:32].tolist(), "n": int(len(prefix))}, open(out + f".{rank}", "w"))
    dist.destroy_process_group()


def test_two_rank_aggregation_and_inputs(tmp_path):
    out = str(tmp_path / "agg.json")
    port = 29500 + os.getpid() % 1000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["ms"] == 11.0 and r["e2e_s"] == 2.0             # slowest rank
    assert r["tokens"] == 201 and r["e2e_tokens"] == 14 and r["launches"] == 100
    p0, p1 = json.load(open(out + ".0")), json.load(open(out + ".1"))
    assert p0["n"] == p1["n"] == 325 and p0["prefix"] != p1["prefix"]     # same shape, different sequences


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_both_arms_describe_the_same_workload():
    import bench
    a, b = bench.workload_config(), bench.workload_config({"x": 1})
    assert a["workload"] == b["workload"] and "C2" in a["workload"]
