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


SHARD_WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["METOK_ROOT"])
import numpy as np, torch, torch.distributed as dist
from oracle import metok_oracle as O
from paper_2506_02850_b200 import binding as B
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
rng = np.random.default_rng(3)                                  # the same tensors on every rank
Hq, Hkv, Lt, dh, n_vis, vis_start = 8, 4, 3, 16, 40, 2
S = vis_start + n_vis + 1 + Lt
Q = rng.standard_normal((Hq, Lt, dh)); K = rng.standard_normal((Hkv, S, dh))
(h0, h1), (g0, g1) = B.head_shard(Hq, Hkv, rank, world)
assert (h1 - h0) * world == Hq and (g1 - g0) * world == Hkv and h0 == g0 * (Hq // Hkv)
# what a rank computes: the mean over ITS heads, rescaled to the normaliser of all heads
local = O.attention_scores(Q[h0:h1], K[g0:g1], vis_start, n_vis, 0.25) * ((h1 - h0) * Lt) / (Hq * Lt)
t = torch.from_numpy(local.copy())
dist.all_reduce(t, op=dist.ReduceOp.SUM)
full = O.attention_scores(Q, K, vis_start, n_vis, 0.25)
assert np.allclose(t.numpy(), full, rtol=1e-12, atol=1e-15), np.abs(t.numpy() - full).max()
others = [torch.zeros_like(t) for _ in range(world)]
dist.all_gather(others, t)
assert all(torch.equal(o, t) for o in others)                   # every rank selects on the same scores
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_head_sharded_scores_add_up_over_two_ranks(tmp_path):
    """KV-head sharding of the attention scores: each rank's partial (its own heads, the global
    normaliser) summed by one all-reduce is the unsharded score, identical on every rank.  The oracle
    stands in for the per-rank kernels here; the GPU suite checks the kernels' partials themselves."""
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER)
    env = dict(os.environ, METOK_ROOT=ROOT)
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                        "--master-addr", "127.0.0.1", "--master-port", "29519", str(script)],
                       capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.count("ok") == 2
