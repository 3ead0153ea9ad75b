"""Head-sharded decode attention across a process boundary: two processes share one GPU, each
owns half of the heads of the same case and its own [B, H, 128] output buffer, and each maps
the other's buffer through CUDA IPC (torch's sharing of CUDA tensors between processes).
Every process calls the head-sharded entry point on its shard with both buffers as targets,
so half of every buffer is written by the other process through a peer mapping -- the path a
multi-GPU deployment takes, with one device standing in for two.  No kernel waits for
another process: each call completes by itself, the processes meet on the host afterwards,
and then both buffers must equal the oracle's output."""
import os
import sys
import traceback

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

LENS = [1, 9, 64, 100, 0, 257, 640, 1500]
HEADS = 6
WORLD = 2


def _rank_main(rank, layout, tokens, chunk, to_peer, from_peer, barrier, results):
    """Child process: build the (seeded, identical) case, run this rank's shard, check."""
    try:
        if ROOT not in sys.path:
            sys.path.insert(0, ROOT)
        from paper_2409_04992_b200 import binding, sharding, workloads as wl
        from tests import gpu_util as gu

        torch.cuda.set_device(0)
        w = wl.Workload("sharded_ipc", 2, batch=len(LENS), len_lo=min(LENS), len_hi=max(LENS),
                        layout=layout, s_max=max(LENS) if layout == "contiguous" else 0,
                        block_tokens=tokens, heads=HEADS)
        cpu = wl.generate(w, seq_lens=LENS)
        dev = gu.to_device(cpu)
        gu.gpu_step(dev)                                         # the step's append (all heads)
        B, H, D = dev.q.shape
        mine = torch.full((B, H, D), float("nan"), dtype=torch.float16, device="cuda")
        to_peer.put(mine)                                        # exported through CUDA IPC
        theirs = from_peer.get(timeout=120)                      # the other process's buffer, mapped here
        assert theirs.data_ptr() != mine.data_ptr() and theirs.shape == mine.shape
        buffers = [mine, theirs] if rank == 0 else [theirs, mine]      # indexed by rank
        off, cnt = sharding.head_shard(H, WORLD, rank)
        max_len = max(dev.max_seq_len, 1)
        flags = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.set_chunk_tokens(chunk)
        ws = torch.empty(binding.allgather_workspace_bytes(B, cnt, D, max_len), dtype=torch.uint8, device="cuda")
        binding.decode_attention_allgather(buffers, None, sharding.take_heads(dev.q, off, cnt),
                                           sharding.take_heads(dev.k_cache, off, cnt),
                                           sharding.take_heads(dev.v_cache, off, cnt), dev.block_table,
                                           dev.seq_lens, off, H, max_len, dev.scale, ws, flags)
        torch.cuda.synchronize()                                 # this rank's stores have landed
        barrier.wait(timeout=120)                                # ... and so have the other rank's
        assert int(flags.item()) == 0
        got = mine.cpu()
        want, _ = gu.oracle_step(cpu)
        gu.assert_close(got, want, what=f"rank {rank} buffer")
        # this rank's own rows, bit for bit, against the single-GPU entry point on the shard
        shard = wl.Case(**{**dev.__dict__, "q": sharding.take_heads(dev.q, off, cnt),
                           "k_cache": sharding.take_heads(dev.k_cache, off, cnt),
                           "v_cache": sharding.take_heads(dev.v_cache, off, cnt)})
        alone, _, _ = gu.gpu_step(shard, do_append=False, chunk_tokens=chunk)
        assert np.array_equal(gu.bits(got[:, off:off + cnt]), gu.bits(alone))
        results.put((rank, "ok", gu.bits(got).tobytes()))
        barrier.wait(timeout=120)                                # keep the exported buffer alive until both are done
    except Exception:
        results.put((rank, traceback.format_exc(), b""))
        try:
            barrier.abort()
        except Exception:
            pass


@pytest.mark.parametrize("layout,tokens,chunk", [("paged", 16, 0), ("contiguous", 0, 64), ("paged", 32, 2048)])
def test_two_processes_store_into_each_others_buffers(layout, tokens, chunk):
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q01, q10, results = ctx.Queue(), ctx.Queue(), ctx.Queue()
    barrier = ctx.Barrier(WORLD)
    procs = [ctx.Process(target=_rank_main, args=(0, layout, tokens, chunk, q01, q10, barrier, results)),
             ctx.Process(target=_rank_main, args=(1, layout, tokens, chunk, q10, q01, barrier, results))]
    for p in procs:
        p.start()
    got = {}
    try:
        for _ in range(WORLD):
            rank, status, bits = results.get(timeout=300)
            got[rank] = (status, bits)
    finally:
        for p in procs:
            p.join(timeout=60)
            if p.is_alive():
                p.kill()                                         # the exact child this test started
    for rank in range(WORLD):
        assert got[rank][0] == "ok", f"rank {rank}:\n{got[rank][0]}"
    assert got[0][1] == got[1][1], "the two processes' buffers differ"
    assert all(p.exitcode == 0 for p in procs)
