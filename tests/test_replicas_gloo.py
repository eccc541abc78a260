"""The N > 1 path of the benchmark on CPU: two gloo ranks stand in for two GPUs.  Videos are
independent, so the only exchange between replicas is the max-reduce of the step time; the reference
arm runs on rank 0 alone."""

import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["METOK_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))    # rank 1 is the slow one
assert ms == 15.0, ms
val = bench.replica_throughput(18432, world, ms)
assert abs(val - 2 * 18432 / 15e-3) < 1e-6, val
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_their_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, METOK_ROOT=ROOT)
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                        "--master-addr", "127.0.0.1", "--master-port", "29517", str(script)],
                       capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.count("ok") == 2


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stderr
    assert r.stdout.strip() == ""


def test_single_gpu_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.replica_throughput(1000, 4, 2.0) == 4 * 1000 / 2e-3
    line = json.dumps({"value": bench.replica_throughput(18432, 1, 0.5)})
    assert json.loads(line)["value"] == 18432 / 0.5e-3
