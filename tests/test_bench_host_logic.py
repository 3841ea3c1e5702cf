"""The N > 1 path of bench.py without GPUs: two gloo ranks aggregate replica results
(units summed over ranks, time = max over ranks), as the benchmark's JSON line requires."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
r = dist.get_rank()
units, ms = bench.aggregate(100.0 * (r + 1), 10.0 + 5.0 * r, True, "cpu")
assert units == 300.0 and ms == 15.0, (units, ms)
# a single process is its own aggregate
assert bench.aggregate(7.0, 3.0, False, "cpu") == (7.0, 3.0)
dist.barrier()
dist.destroy_process_group()
sys.stdout.write("rank%dok\n" % r)  # one write per rank: the ranks share a pipe
sys.stdout.flush()
"""


def test_two_rank_aggregation():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    import tempfile
    with tempfile.TemporaryDirectory() as d:
        path = os.path.join(d, "worker.py")
        with open(path, "w") as f:
            f.write(_WORKER.format(root=ROOT))
        p = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                            "--master-addr", "127.0.0.1", "--master-port", "29533", path], env=env,
                           capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stdout[-2000:] + p.stderr[-2000:]
    assert p.stdout.count("rank0ok") == 1 and p.stdout.count("rank1ok") == 1, p.stdout


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
