"""bench.py on N GPUs runs N independent replicas; this checks its aggregation over ranks with two gloo
processes on the CPU (the job is as slow as its slowest rank, and throughput sums over ranks)."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
# rank 0 is the fast one, rank 1 the slow one
dec_ms, tot_ms, wall = (100.0, 150.0, 0.2) if rank == 0 else (125.0, 160.0, 0.3)
out = bench.aggregate_replicas(250, dec_ms, tot_ms, wall, dist.get_world_size())
dist.barrier()
if rank == 0:
    print("RESULT " + json.dumps(out))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_aggregate_like_the_benchmark(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29731", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("RESULT ")][0]
    import json
    value, dec_ms, tot_ms, wall = json.loads(line[7:])
    assert (dec_ms, tot_ms, wall) == (125.0, 160.0, 0.3)           # max over ranks
    assert abs(value - 2 * 250 / 0.125) < 1e-9                     # both ranks' tokens over the slowest rank's time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_replicas(100, 50.0, 60.0, 0.1, 1) == (2000.0, 50.0, 60.0, 0.1)
