"""The path has no exchange step: with N > 1 ranks bench.py runs independent replicas and only the
timing crosses ranks (maximum over ranks).  Two gloo ranks on the CPU cover that host logic."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
assert world == 2
slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world)
assert slowest == 15.0, slowest
seeds = [None] * world
dist.all_gather_object(seeds, bench.replica_seed(rank))
assert len(set(seeds)) == world, seeds
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_two_replicas_share_only_the_timing(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, REPO_ROOT=ROOT, OMP_NUM_THREADS="1")
    res = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr",
         "127.0.0.1", "--master-port", "29631", str(script)],
        capture_output=True, text=True, timeout=240, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok") == 2
