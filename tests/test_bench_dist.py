"""Host logic of the multi-process benchmark path, on CPU with gloo (world size 2): every rank
runs an independent replica, the step time is the maximum over ranks and the value is the sum
of the replicas' tokens over that time."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
sys.path.insert(0, os.environ["GSD_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = [1.0, 3.0][rank]                      # rank 1 is the slow replica
agg = bench.aggregate_over_ranks(ms, tokens_per_step=2048, world=world, dist=dist, device="cpu")
if rank == 0:
    print(json.dumps(agg))
dist.barrier()
dist.destroy_process_group()
'''


def test_max_over_ranks_and_aggregate_value(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, GSD_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29611")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                          "--nproc-per-node=2", "--master-addr", "127.0.0.1", "--master-port",
                          "29611", str(script)], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    import json
    agg = json.loads(line)
    assert agg["ms_per_step"] == 3.0                      # the slowest rank sets the step time
    assert abs(agg["value"] - 2 * 2048 / 3.0e-3) < 1e-6   # both replicas' tokens over that time


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    agg = bench.aggregate_over_ranks(2.0, tokens_per_step=100, world=1, dist=None, device="cpu")
    assert agg == {"ms_per_step": 2.0, "value": 100 / 2.0e-3}
