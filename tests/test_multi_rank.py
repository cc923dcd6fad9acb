"""Host-side multi-rank logic of the benchmark on CPU ranks (gloo, world size 2): the operator shards
by independent frames with no data-path collective, so what there is to test is the aggregation
(whole-job value = all ranks' units / slowest rank's time) and the reference arm's rank handling."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["FB_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + os.environ["FB_PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
def reduce_max(x):
    t = torch.tensor([x], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
local_ms = 10.0 if rank == 0 else 25.0          # rank 1 is the slow one
value, total_ms = bench.whole_job_value(local_ms, 1000.0, world, reduce_max)
dist.barrier()
print(json.dumps({"rank": rank, "value": value, "total_ms": total_ms}), flush=True)
dist.destroy_process_group()
"""


def test_whole_job_value_takes_the_slowest_rank(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(29500 + os.getpid() % 2000)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", FB_ROOT=ROOT, FB_PORT=port, MASTER_ADDR="127.0.0.1")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = [json.loads(p.communicate(timeout=120)[0].strip().splitlines()[-1]) for p in procs]
    assert all(p.returncode == 0 for p in procs)
    for o in outs:
        assert o["total_ms"] == 25.0                      # max over ranks, not the local time
        assert o["value"] == pytest.approx(2 * 1000.0 / 25e-3)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == ""       # other ranks exit 0 without work
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
