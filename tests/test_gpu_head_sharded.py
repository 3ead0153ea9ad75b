"""Head-sharded decode attention with the fused all-gather, on one GPU: the ranks' calls run
one after another on the same device, each on its own head shard of the same case, each
storing into all ranks' output buffers (here ordinary buffers of this GPU).  No call waits
for another.  Afterwards all buffers must be identical, each shard's rows must be, bit for
bit, what the single-GPU entry point gives on that shard (same number of (sequence, head)
pairs, hence the same chunking), and the whole must agree with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, sharding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

LENS = [1, 9, 64, 100, 0, 257, 640, 1500]


def make_case(layout, tokens, heads, lens=LENS, index=2):
    w = wl.Workload("sharded", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout=layout, s_max=max(lens) if layout == "contiguous" else 0,
                    block_tokens=tokens, heads=heads)
    return wl.generate(w, seq_lens=lens)


def run_sharded(dev: wl.Case, world: int, chunk_tokens=0):
    """All ranks' calls on this GPU.  Returns (list of output buffers on cpu, lse [B,H] cpu)."""
    B, H, D = dev.q.shape
    max_len = max(dev.max_seq_len, 1)
    outs = [gu.Guarded((B, H, D), torch.float16) for _ in range(world)]
    lse_full = torch.empty((B, H), dtype=torch.float32)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.set_chunk_tokens(chunk_tokens)
    try:
        for rank in range(world):
            off, cnt = sharding.head_shard(H, world, rank)
            q = sharding.take_heads(dev.q, off, cnt)
            k = sharding.take_heads(dev.k_cache, off, cnt)
            v = sharding.take_heads(dev.v_cache, off, cnt)
            lse = gu.Guarded((B, cnt), torch.float32)
            ws = gu.Guarded((binding.allgather_workspace_bytes(B, cnt, D, max_len),), torch.uint8)
            binding.decode_attention_allgather([o.view for o in outs], lse.view, q, k, v,
                                               dev.block_table, dev.seq_lens, off, H, max_len,
                                               dev.scale, ws.view, flags)
            torch.cuda.synchronize()
            assert lse.intact() and ws.intact()
            lse_full[:, off:off + cnt] = lse.view.cpu()
    finally:
        binding.set_chunk_tokens(0)
    assert all(o.intact() for o in outs), "a kernel wrote outside an output buffer"
    assert int(flags.item()) == 0
    return [o.view.cpu() for o in outs], lse_full


@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 16), ("paged", 64)])
@pytest.mark.parametrize("world,heads", [(1, 3), (2, 4), (3, 8), (4, 40), (16, 16)])
def test_every_rank_ends_with_all_heads(layout, tokens, world, heads):
    cpu = make_case(layout, tokens, heads)
    dev = gu.to_device(cpu)
    gu.gpu_step(dev)                                            # the step's append
    outs, lse = run_sharded(dev, world)
    for r, out in enumerate(outs):
        assert np.array_equal(gu.bits(out), gu.bits(outs[0])), f"rank {r}'s buffer differs"
    for rank in range(world):
        off, cnt = sharding.head_shard(heads, world, rank)
        shard = wl.Case(**{**dev.__dict__, "q": sharding.take_heads(dev.q, off, cnt),
                           "k_cache": sharding.take_heads(dev.k_cache, off, cnt),
                           "v_cache": sharding.take_heads(dev.v_cache, off, cnt)})
        alone, alone_lse, _ = gu.gpu_step(shard, do_append=False)
        assert np.array_equal(gu.bits(outs[0][:, off:off + cnt]), gu.bits(alone)), f"shard {rank}"
        assert np.array_equal(lse[:, off:off + cnt].numpy(), alone_lse.numpy())
    want, want_lse = gu.oracle_step(cpu)
    gu.assert_close(outs[0], want, lse, want_lse, f"{layout} world={world}")


@pytest.mark.parametrize("chunk", [64, 2048])
def test_one_chunk_and_many_chunks(chunk):
    # chunk 2048 > longest sequence: one chunk, the split kernel finishes the rows itself and
    # the last kernel only fans them out; chunk 64: up to 24 partials merged per row.
    cpu = make_case("paged", 32, 6)
    dev = gu.to_device(cpu)
    gu.gpu_step(dev)
    outs, lse = run_sharded(dev, 2, chunk_tokens=chunk)
    want, want_lse = gu.oracle_step(cpu)
    for out in outs:
        gu.assert_close(out, want, lse, want_lse, f"chunk={chunk}")
    assert np.array_equal(gu.bits(outs[0]), gu.bits(outs[1]))


def test_other_shards_rows_are_left_alone():
    cpu = make_case("paged", 16, 4, lens=[33, 200])
    dev = gu.to_device(cpu)
    gu.gpu_step(dev)
    B, H, D = dev.q.shape
    out = torch.full((B, H, D), 7.0, dtype=torch.float16, device="cuda")
    off, cnt = sharding.head_shard(H, 2, 1)
    ws = torch.empty(binding.allgather_workspace_bytes(B, cnt, D, 200), dtype=torch.uint8, device="cuda")
    binding.decode_attention_allgather([out], None, sharding.take_heads(dev.q, off, cnt),
                                       sharding.take_heads(dev.k_cache, off, cnt),
                                       sharding.take_heads(dev.v_cache, off, cnt), dev.block_table,
                                       dev.seq_lens, off, H, 200, dev.scale, ws)
    torch.cuda.synchronize()
    assert torch.all(out[:, :off] == 7.0)
    assert not torch.any(out[:, off:] == 7.0)


def test_bad_arguments_are_refused_before_any_launch():
    cpu = make_case("contiguous", 0, 2, lens=[40, 50])
    dev = gu.to_device(cpu)
    B, H, D = dev.q.shape
    out = torch.zeros((B, 4, D), dtype=torch.float16, device="cuda")
    ws = torch.empty(binding.allgather_workspace_bytes(B, H, D, 50), dtype=torch.uint8, device="cuda")

    def call(outs, offset, total, workspace=ws):
        binding.decode_attention_allgather(outs, None, dev.q, dev.k_cache, dev.v_cache, None,
                                           dev.seq_lens, offset, total, 50, dev.scale, workspace)

    for outs, offset, total in [([out], 3, 4), ([out], -1, 4), ([out] * 17, 0, 4), ([], 0, 4),
                                ([out, 0], 0, 4), ([out.view(-1)[1:]], 0, 4)]:
        with pytest.raises(binding.InstInferError) as err:
            call(outs, offset, total)
        assert err.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.InstInferError) as err:
        call([out], 0, 4, ws[:binding.workspace_bytes(B, H, D, 50)])
    assert err.value.status == binding.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.all(out == 0)
