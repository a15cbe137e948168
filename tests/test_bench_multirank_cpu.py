"""Host logic of the N > 1 benchmark path, run as two gloo ranks on the CPU: every rank times its
own replica, the job's time is the maximum over ranks, the value counts all ranks' states; the
reference arm prints on rank 0 only and the other ranks leave without work."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(1.0 + rank, dist, "cpu")      # rank 1 is the slower one
dist.barrier()
print(json.dumps({"rank": rank, "world": world, "ms": ms, "value": bench.job_value(100, world, ms)}))
dist.destroy_process_group()
"""


def _run_ranks(code_or_args, port):
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable] + code_or_args, env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    return [o for o, _ in outs]


def test_max_over_ranks_and_job_value_with_two_gloo_ranks():
    outs = _run_ranks(["-c", WORKER % ROOT], 29731)
    recs = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    for r in recs:
        assert r["world"] == 2
        assert r["ms"] == 2.0                 # the maximum, on every rank
        assert r["value"] == 100 * 2 / 2.0e-3  # both ranks' states over the slowest time


def test_reference_arm_prints_on_rank_zero_only():
    outs = _run_ranks(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "3",
                       "--workload", "cartpole_mlp", "--ref-sample", "64"], 29732)
    assert outs[1].strip() == ""
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
