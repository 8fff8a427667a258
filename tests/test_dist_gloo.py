"""The multi-GPU path of the benchmark is N independent replicas plus a max-over-ranks
reduction of the timings; that reduction is exercised here with two gloo ranks on CPU."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
from paper_2408_15562_b200 import dist_util
rank, world, local = dist_util.rank_info()
dist.init_process_group("gloo")
vals = dist_util.max_over_ranks([10.0 + rank, 5.0 - rank, 7.0])
assert vals == [11.0, 5.0, 7.0], vals
assert abs(dist_util.aggregate_replicas(vals[0], world) - 2e6 / 11.0) < 1e-6
dist.barrier()
if rank == 0:
    print("GLOO_OK", world)
dist.destroy_process_group()
"""


def test_max_over_ranks_two_gloo_processes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "GLOO_OK 2" in out.stdout


def test_single_process_is_identity():
    from paper_2408_15562_b200 import dist_util
    assert dist_util.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert dist_util.rank_info()[1] >= 1


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--workload", "tiny_greedy", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0 and out.stdout.strip() == ""
