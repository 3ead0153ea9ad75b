"""Host logic of the head-sharded path on CPU: the shard arithmetic, and two gloo ranks
that each compute their heads with the oracle and assemble the full output through
`sharding.gather_heads` (heads are independent, Sec. IV-D, so the assembled tensor must be
the whole-problem oracle output exactly)."""
import json
import os
import subprocess
import sys

import pytest

from paper_2409_04992_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("heads", [1, 5, 16, 40, 41])
@pytest.mark.parametrize("world", [1, 2, 3, 8, 16])
def test_shards_partition_the_heads_evenly(heads, world):
    shards = sharding.all_shards(heads, world)
    covered = [h for off, cnt in shards for h in range(off, off + cnt)]
    assert covered == list(range(heads))                      # in rank order, each head once
    sizes = [cnt for _, cnt in shards]
    assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)


def test_bad_shard_requests_raise():
    for args in [(0, 1, 0), (8, 0, 0), (8, 2, 2), (8, 2, -1)]:
        with pytest.raises(ValueError):
            sharding.head_shard(*args)


CHILD = r"""
import json, os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import numpy as np, torch, torch.distributed as dist
from oracle import capi
from paper_2409_04992_b200 import sharding, workloads as wl

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
H = 5                                                    # uneven: 3 + 2
lens = [1, 17, 0, 130]
w = wl.Workload("gloo", 1, batch=len(lens), len_lo=0, len_hi=130, layout="paged", s_max=0,
                block_tokens=16, heads=H)
case = wl.generate(w, seq_lens=lens)                     # same seed on both ranks
lens_np = np.array(lens, dtype=np.int32)
table = case.block_table.numpy()
capi.kv_append(case.k_cache.numpy(), case.v_cache.numpy(), case.k_new.numpy(), case.v_new.numpy(),
               lens_np, block_table=table)               # the step's append, before sharding

def attend(q, k, v):
    out, lse, _ = capi.decode_attention(q.numpy(), k.numpy(), v.numpy(), lens_np, case.scale,
                                        block_table=table)
    return out

full = attend(case.q, case.k_cache, case.v_cache)
off, cnt = sharding.head_shard(H, world, rank)
mine = attend(sharding.take_heads(case.q, off, cnt), sharding.take_heads(case.k_cache, off, cnt),
              sharding.take_heads(case.v_cache, off, cnt))
gathered = sharding.gather_heads(torch.from_numpy(np.ascontiguousarray(mine)), H)
same = bool(np.array_equal(gathered.numpy(), full))
flag = torch.tensor([1.0 if same else 0.0])
dist.all_reduce(flag, op=dist.ReduceOp.MIN)
if rank == 0:
    print(json.dumps({"world": world, "same_on_all_ranks": bool(flag.item() == 1.0),
                      "shape": list(gathered.shape), "nonzero": bool(np.isfinite(full).all() and np.abs(full).sum() > 0)}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_assemble_the_whole_output(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    env = dict(os.environ, REPO_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)]
    done = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240)
    assert done.returncode == 0, done.stderr[-2000:]
    got = json.loads([x for x in done.stdout.splitlines() if x.startswith("{")][-1])
    assert got == {"world": 2, "same_on_all_ranks": True, "shape": [4, 5, 128], "nonzero": True}
