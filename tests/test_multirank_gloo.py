"""The N > 1 benchmark path on CPU: two gloo ranks, replicas only (no collective on the data path)."""
import json
import os
import subprocess
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["OOCO_ROOT"])
import torch, torch.distributed as dist
import bench
from paper_2511_21862_b200 import inputs
rank, local, world = bench.dist_env()
dist.init_process_group("gloo")
cfg = inputs.replace(inputs.CONFIGS["cfg0"], seed=inputs.CONFIGS["cfg0"].seed + 100 * rank)
batch = inputs.make_batch(cfg, "cpu")
ms, units = bench.aggregate(world, 1.0 + rank, float(batch.total_tokens))      # rank 1 is the slow one
vals = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
dist.all_gather(vals, torch.tensor([int(batch.q.view(torch.int16).sum())]))
if rank == 0:
    print(json.dumps({"ms": ms, "units": units, "world": world, "checksums": [int(v) for v in vals]}))
dist.barrier()
dist.destroy_process_group()
"""


def test_two_ranks_aggregate_max_time_and_sum_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, OOCO_ROOT=ROOT, OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29571", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    got = json.loads(line)
    assert got["world"] == 2
    assert got["ms"] == 2.0                                   # max over ranks
    assert got["units"] == 2 * 467                            # both replicas' tokens (cfg0 has 467)
    assert got["checksums"][0] != got["checksums"][1]         # replicas draw different data (seed + 100 * rank)


def test_replica_count_keeps_working_set_above_l2():
    import bench
    assert bench.replica_count(600 << 20, 170 << 30) * (600 << 20) >= 4 << 30
    assert bench.replica_count(20 << 30, 170 << 30) == 2
    assert bench.replica_count(20 << 30, 30 << 30) == 1
