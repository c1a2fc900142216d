"""The benchmark's multi-rank plumbing on CPU: two `gloo` ranks on 127.0.0.1 run the same helper calls
`bench.py --gpus N` makes under torch.distributed.run (barrier, slowest-rank time, whole-job value, per-rank
seeds), and the reference arm does no work on ranks other than 0.  No GPU and no kernels involved."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, os, sys
sys.path.insert(0, os.environ["LPDT_ROOT"])
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
bench.barrier(world, device="cpu")
ms = bench.max_over_ranks(world, 100.0 * (rank + 1), device="cpu")          # rank 1 is the slow one
value = bench.job_value(world, 512, ms, 10)
from paper_2111_09389_b200 import workloads
wl = workloads.make_workload("conv16", seed=bench.rank_seed(rank))
print(json.dumps({"rank": rank, "ms": ms, "value": value, "x0": float(wl["x"].ravel()[0])}))
dist.destroy_process_group()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_job_value():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), LPDT_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["ms"] == outs[1]["ms"] == 200.0                      # the maximum over ranks, on every rank
    assert outs[0]["value"] == outs[1]["value"] == 2 * 512 / (200.0 / 10 * 1e-3)
    assert outs[0]["x0"] != outs[1]["x0"]                               # replicas draw different inputs


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
