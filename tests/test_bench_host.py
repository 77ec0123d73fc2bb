"""Host-side logic of bench.py: the algorithmic work model, and the multi-GPU plan (replicas only: the max over
ranks of the elapsed time is the only cross-rank exchange), exercised with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench
from paper_2511_12934_b200 import synth

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["AIF_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
plan = bench.replica_plan(world, rank)
elapsed = 10.0 + 5.0 * rank                    # rank 1 is the slow one
total = bench.reduce_max(elapsed, dist)
dist.barrier()
with open(os.path.join(os.environ["AIF_OUT"], f"rank{rank}.json"), "w") as fh:   # one file per rank: stdout of two ranks can interleave
    json.dump({"rank": rank, "total": total, "plan": plan}, fh)
dist.destroy_process_group()
"""


def test_flop_model_matches_the_scope_table():
    # per-candidate flops of the base blocks: 0.21 M / 1.15 M / 1.56 M / 6.17 M / 7.07 M
    want = {"c1": 0.21e6, "c2": 1.15e6, "c3": 1.56e6, "c4": 6.17e6, "c5": 7.07e6}
    for k, v in want.items():
        got = bench.flops_per_candidate(synth.SHORT[k])["total"]
        assert abs(got - v) / v < 0.01, (k, got)
    f = bench.flops_per_candidate(synth.C2)
    assert f["layer1"] == 2 * 768 * 512 and f["layer2"] == 2 * 512 * 256 + 2 * 256 and f["attention"] == 4 * 200 * 128
    assert bench.kernel_flops("layer1", synth.C2, 10) == 10 * f["layer1"]


def test_replica_plan_and_max_over_ranks_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, AIF_ROOT=ROOT, AIF_OUT=str(tmp_path))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29617", str(script)]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads((tmp_path / f"rank{k}.json").read_text()) for k in range(2)]
    assert sorted(x["rank"] for x in lines) == [0, 1]
    for x in lines:
        assert x["total"] == 15.0                     # max over ranks, seen by every rank
        assert x["plan"]["replica"] is True and x["plan"]["world"] == 2 and x["plan"]["share_of_work"] == 1.0


def test_single_process_reduce_is_identity():
    assert bench.reduce_max(3.5, None) == 3.5
