"""GPU parity of the grouped-head / multi-token entry point at the full shapes the benchmark
times (automatic split plan, device-generated inputs, NaN-poisoned padding): the oracle
recomputes sampled (sequence, KV head) pairs, all their query rows, from rows gathered off
the device."""
import numpy as np
import pytest
import torch

import bench
from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", bench.GROUPED_SHAPES, ids=[s[0] for s in bench.GROUPED_SHAPES])
def test_sampled_pairs_at_benchmark_shapes(shape):
    name, batch, ctx, tokens, kv_heads, q_heads, q_tokens, dim = shape
    free, _ = torch.cuda.mem_get_info()
    if free < 8 * 2 ** 30:
        pytest.skip("needs 8 GiB of free device memory")
    w = wl.Workload(name, 7, batch=batch, len_lo=ctx, len_hi=ctx, layout="paged",
                    block_tokens=tokens, heads=kv_heads, head_dim=dim)
    g = wl.generate_grouped(w, q_tokens, q_heads, device="cuda")
    c = g.base
    group = q_heads // kv_heads
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty_like(g.q)
    lse = torch.empty(g.q.shape[:3], dtype=torch.float32, device="cuda")
    ws = torch.empty(binding.grouped_workspace_bytes(batch, q_tokens, q_heads, kv_heads, dim, ctx),
                     dtype=torch.uint8, device="cuda")
    binding.kv_append_bulk(c.k_cache, c.v_cache, g.k_new, g.v_new, c.seq_lens, g.new_lens,
                           c.block_table, flags)
    binding.decode_attention_grouped(out, lse, g.q, c.k_cache, c.v_cache, c.block_table,
                                     c.seq_lens, ctx, c.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    assert torch.isfinite(out.float()).all(), "poison leaked into an output"

    rng = np.random.default_rng(len(name))
    pairs = {(0, 0), (batch - 1, kv_heads - 1)}
    while len(pairs) < 4:
        pairs.add((int(rng.integers(batch)), int(rng.integers(kv_heads))))
    pairs = sorted(pairs)
    n = len(pairs)
    k = np.zeros((n, 1, ctx, dim), dtype=np.float16)
    v = np.zeros((n, 1, ctx, dim), dtype=np.float16)
    q = np.zeros((n, q_tokens, group, dim), dtype=np.float16)
    for i, (b, hk) in enumerate(pairs):
        kr, vr = wl.gather_rows(c, b, hk)
        k[i, 0], v[i, 0] = kr.cpu().numpy(), vr.cpu().numpy()
        q[i] = g.q[b, :, hk * group:(hk + 1) * group].cpu().numpy()
        # the bulk append put the new tokens at the end of the sequence, bit for bit
        assert np.array_equal(gu.bits(kr[ctx - q_tokens:]), gu.bits(g.k_new[b, :, hk]))
        assert np.array_equal(gu.bits(vr[ctx - q_tokens:]), gu.bits(g.v_new[b, :, hk]))
    want, want_lse = capi.decode_attention_grouped(q, k, v, np.full(n, ctx, dtype=np.int32), c.scale)
    got = torch.stack([out[b, :, hk * group:(hk + 1) * group] for b, hk in pairs]).cpu()
    got_lse = torch.stack([lse[b, :, hk * group:(hk + 1) * group] for b, hk in pairs]).cpu()
    rows = q_tokens * group
    gu.assert_close(got.reshape(n, rows, dim), want.reshape(n, rows, dim),
                    got_lse.reshape(n, rows), want_lse.reshape(n, rows), name)
