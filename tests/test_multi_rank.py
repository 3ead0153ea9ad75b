"""The N>1 plumbing of bench.py on CPU: two gloo ranks, barrier, max-over-ranks timing and
whole-job aggregation (the data path itself has no collective)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import bench
ranks = bench.Ranks(2, backend="gloo")
ranks.barrier()
units, seconds = (100.0, 2.0) if ranks.rank == 0 else (300.0, 4.0)     # rank 1 is the slow one
value, job_seconds = bench.aggregate(ranks, units, seconds)
total = ranks.sum(float(ranks.rank + 1))
# the head-sharded section's aggregation: rank 0 owns 3 of 5 heads, rank 1 the other 2
heads = 3 if ranks.rank == 0 else 2
sharded = bench.head_sharded_result(ranks, 10.0 * heads, 1.0 + ranks.rank, heads, 5, 0.0 if ranks.rank == 0 else None)
if ranks.rank == 0:
    print(json.dumps({"value": value, "seconds": job_seconds, "world": ranks.world, "sum": total,
                      "sharded": sharded}))
ranks.close()
"""


def test_two_gloo_ranks_aggregate_to_whole_job_throughput(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    env = dict(os.environ, REPO_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)]
    done = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240)
    assert done.returncode == 0, done.stderr[-2000:]
    line = [x for x in done.stdout.splitlines() if x.startswith("{")][-1]
    got = json.loads(line)
    assert got["world"] == 2 and got["sum"] == 3.0
    assert got["seconds"] == 4.0                       # the slowest rank sets the time
    assert got["value"] == (100.0 + 300.0) / 4.0       # all ranks' units over that time
    sharded = got["sharded"]                           # one instance: all heads' bytes over the slowest rank
    assert sharded["heads_covered"] == sharded["total_heads"] == 5 and sharded["scaling"] == "strong"
    assert sharded["value"] == 50.0 / 2.0 and sharded["seconds"] == 2.0


def test_reference_arm_only_rank_zero_prints(tmp_path):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29532", os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "0"]
    done = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert done.returncode == 0, done.stderr[-2000:]
    lines = [x for x in done.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    got = json.loads(lines[0])
    assert got["impl"] == "reference" and got["cpu_baseline"]["kind"] == "oracle"
    assert got["e2e"]["h2d_bytes_per_step"] == 0 and got["value"] > 0
