"""The N > 1 plumbing of bench.py (replicas only: barrier + max-over-ranks), on 2 gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), RANK=str(rank),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    from paper_2603_17803_b200 import replicas
    assert replicas.env_world() == (world, rank, rank)
    replicas.init("gloo")
    replicas.barrier()
    ms = [10.0 + 5 * rank, 3.0 - rank]                     # rank 1 is slower on the first, faster on the second
    got = replicas.max_over_ranks(ms)
    value = replicas.aggregate_steps_per_s(world, 100, got[0])
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"max": got, "value": value, "seeds": [replicas.replica_seed(rank, r) for r in range(3)]}, f)
    replicas.barrier()
    replicas.shutdown()


def test_two_ranks_agree_on_the_slowest_time(tmp_path):
    mp.spawn(_worker, args=(2, 29000 + os.getpid() % 2000, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0["max"] == r1["max"] == [15.0, 3.0]
    assert r0["value"] == 2 * 100 / 0.015
    assert not set(r0["seeds"]) & set(r1["seeds"])         # ranks draw different data


def test_reference_arm_runs_only_on_rank_zero():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
