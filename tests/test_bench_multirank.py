"""The N > 1 path of bench.py on CPU: two gloo ranks, no GPU.  The workload shards as independent replicas (every
output element is independent and there is no exchange step), so the only cross-rank logic is the barrier and the
max-over-ranks of the device-timed milliseconds; the reference arm runs on rank 0 alone."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
dist.barrier()
ms = bench.max_over_ranks(10.0 * (rank + 1), dist)           # rank r "took" 10 (r + 1) ms
value = bench.whole_job_value(1e9, steps=2, world=world, slowest_ms=ms)
dist.barrier()
if rank == 0:
    print(json.dumps({{"ms": ms, "value": value, "world": world}}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_take_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29617", str(script)],
                         capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["world"] == 2 and res["ms"] == 20.0                 # the slower rank decides
    assert res["value"] == pytest.approx(1e9 * 2 * 2 / 20e-3)      # both replicas' MACs over that time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == ""        # non-zero ranks exit without work
