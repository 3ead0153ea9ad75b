"""GPU parity of the grouped-head / multi-token / other-head-size variant: the CUDA path
through the C ABI (bulk append, then `decode_attention_grouped`) against the CPU oracle on
the same seeded bits, element by element.  Shapes span several tiles, several chunks,
ragged tails, sequences shorter than the step's token count, and NaN-poisoned padding."""
import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

RAGGED = [1, 2, 15, 16, 17, 31, 33, 64, 65, 100, 257, 0, 511, 640, 3, 1100]


@pytest.fixture(autouse=True, params=[1, 2], ids=["warp-mma", "tcgen05"])
def grouped_path(request):
    """Every test runs on both implementations (shapes the tcgen05 form does not take fall back
    to the warp-level one inside the library)."""
    binding.set_grouped_path(request.param)
    yield request.param
    binding.set_grouped_path(0)


def make(layout, tokens, kv_heads, q_tokens, q_heads, dim=128, lens=RAGGED, index=5):
    w = wl.Workload("grouped", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout=layout, s_max=max(lens) if layout == "contiguous" else 0,
                    block_tokens=tokens, heads=kv_heads, head_dim=dim)
    return wl.generate_grouped(w, q_tokens, q_heads, seq_lens=lens)


def to_device(g: wl.GroupedCase) -> wl.GroupedCase:
    return wl.GroupedCase(base=gu.to_device(g.base), q=g.q.cuda(), k_new=g.k_new.cuda(),
                          v_new=g.v_new.cuda(), new_lens=g.new_lens.cuda())


def gpu_step(g: wl.GroupedCase, chunk_tokens=0, do_append=True):
    c = g.base
    B, Tq, Hq, D = g.q.shape
    Hkv = c.k_cache.shape[1]
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = gu.Guarded((B, Tq, Hq, D), torch.float16)
    lse = gu.Guarded((B, Tq, Hq), torch.float32)
    max_len = max(c.max_seq_len, 1)
    binding.set_chunk_tokens(chunk_tokens)
    try:
        ws = gu.Guarded((binding.grouped_workspace_bytes(B, Tq, Hq, Hkv, D, max_len),), torch.uint8)
        if do_append:
            binding.kv_append_bulk(c.k_cache, c.v_cache, g.k_new, g.v_new, c.seq_lens, g.new_lens,
                                   c.block_table, flags)
        binding.decode_attention_grouped(out.view, lse.view, g.q, c.k_cache, c.v_cache, c.block_table,
                                         c.seq_lens, max_len, c.scale, ws.view, flags)
    finally:
        binding.set_chunk_tokens(0)
    torch.cuda.synchronize()
    assert out.intact() and lse.intact() and ws.intact(), "a kernel wrote outside its buffers"
    return out.view.cpu(), lse.view.cpu(), int(flags.item())


def oracle_step(g: wl.GroupedCase, do_append=True):
    c = g.base
    k, v = c.k_cache.numpy(), c.v_cache.numpy()
    table = None if c.block_table is None else c.block_table.numpy()
    lens = np.array(c.seq_lens_host, dtype=np.int32)
    if do_append:
        capi.kv_append_bulk(k, v, g.k_new.numpy(), g.v_new.numpy(), lens, g.new_lens.numpy(), block_table=table)
    return capi.decode_attention_grouped(g.q.numpy(), k, v, lens, c.scale, block_table=table)


def check(g_cpu, chunk, what):
    dev = to_device(g_cpu)
    out, lse, flags = gpu_step(dev, chunk_tokens=chunk)
    want, want_lse = oracle_step(g_cpu)
    assert flags == 0
    # the appended caches must be the oracle's bit for bit (any head size)
    assert np.array_equal(gu.bits(dev.base.k_cache), gu.bits(g_cpu.base.k_cache)), what
    assert np.array_equal(gu.bits(dev.base.v_cache), gu.bits(g_cpu.base.v_cache)), what
    B, Tq, Hq, D = out.shape
    return gu.assert_close(out.reshape(B, Tq * Hq, D), want.reshape(B, Tq * Hq, D),
                           lse.reshape(B, Tq * Hq), want_lse.reshape(B, Tq * Hq), what)


# (rows per KV head: 1, 4, 8, 16, 4, 8, 16, 15, and 5 and 9: just above the row counts the tcgen05 form is compiled for)
SHAPES = [(1, 3, 3), (1, 8, 2), (1, 16, 2), (1, 16, 1), (4, 4, 4), (2, 8, 2), (16, 1, 1), (3, 10, 2), (5, 1, 1), (3, 3, 1)]


@pytest.mark.parametrize("q_tokens,q_heads,kv_heads", SHAPES)
@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 16), ("paged", 64)])
def test_shapes_and_layouts(layout, tokens, q_tokens, q_heads, kv_heads):
    check(make(layout, tokens, kv_heads, q_tokens, q_heads), 0,
          f"{layout} T={tokens} Tq={q_tokens} Hq={q_heads} Hkv={kv_heads}")


@pytest.mark.parametrize("chunk", [64, 128, 2048])
@pytest.mark.parametrize("q_tokens,q_heads,kv_heads", [(1, 8, 2), (5, 3, 1)])
def test_chunkings(chunk, q_tokens, q_heads, kv_heads):
    # chunk 2048: one chunk, the split kernel writes the result itself; chunk 64: the causal
    # limit of an older new token can fall before the last chunk's first position
    check(make("paged", 32, kv_heads, q_tokens, q_heads), chunk, f"chunk={chunk} Tq={q_tokens}")


@pytest.mark.parametrize("dim", [64, 256])
@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 16), ("paged", 64), ("paged", 128)])
@pytest.mark.parametrize("q_tokens,q_heads,kv_heads", [(1, 2, 2), (1, 8, 2), (2, 8, 1), (3, 3, 1), (1, 5, 1)])
def test_other_head_sizes(dim, layout, tokens, q_tokens, q_heads, kv_heads):
    for chunk in (0, 64, 128):
        check(make(layout, tokens, kv_heads, q_tokens, q_heads, dim=dim), chunk,
              f"D={dim} {layout} Tq={q_tokens} Hq={q_heads} Hkv={kv_heads} chunk={chunk}")


def test_the_tcgen05_form_is_the_one_that_runs(grouped_path):
    """On a GPU machine the driver has the tensor-map encoder, so head size 128 with a contiguous
    cache or 16/32/64-token blocks takes the tcgen05 kernel unless the warp-level one is forced."""
    want = 2 if grouped_path == 2 else 1
    for dim in (128, 256):
        for tokens in (0, 16, 32, 64, 128, 256):
            assert binding.grouped_path_for(dim, tokens) == want
    binding.set_grouped_path(0)
    assert binding.grouped_path_for(128, 16) == 2                                 # the default
    assert binding.grouped_path_for(128, 48) == 1 and binding.grouped_path_for(128, 192) == 1
    binding.set_chunk_tokens(192)                                                # tiles would straddle 128-token blocks
    try:
        assert binding.grouped_path_for(128, 128) == 1 and binding.grouped_path_for(128, 64) == 2
    finally:
        binding.set_chunk_tokens(0)
    assert binding.grouped_path_for(64, 16) == 1 and binding.grouped_path_for(256, 48) == 1
    assert binding.grouped_path_for(96, 16) == 0 and binding.grouped_path_for(128, 8) == 0


@pytest.mark.parametrize("tokens", [128, 256])
@pytest.mark.parametrize("q_tokens,q_heads,kv_heads", [(1, 8, 2), (3, 4, 1)])
def test_blocks_of_128_tokens_and_more(tokens, q_tokens, q_heads, kv_heads):
    for chunk in (0, 128, 64):          # chunk 64: tiles would straddle blocks, the warp-level form takes over
        check(make("paged", tokens, kv_heads, q_tokens, q_heads), chunk, f"T={tokens} chunk={chunk}")


def test_tiny_contiguous_cache_smaller_than_one_tile():
    # fewer rows in the whole cache than one 128-token copy box
    g = make("contiguous", 0, 1, 2, 4, lens=[20])
    check(g, 0, "one sequence of 20 tokens, contiguous")
    g = make("contiguous", 0, 2, 1, 2, lens=[1, 3])
    check(g, 0, "two sequences of 1 and 3 tokens, contiguous")


@pytest.mark.parametrize("dim", [128, 256])
def test_peaked_logits(dim):
    for chunk in (0, 64):
        g = make("paged", 32, 2, 2, 8, dim=dim, lens=[700, 1500, 40])
        g.q.mul_(3.0)                               # logits of a few tens
        check(g, chunk, f"peaked chunk={chunk} D={dim}")


@pytest.mark.parametrize("dim", [128, 256, 64])
@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 16), ("paged", 64)])
def test_reference_moves_in_the_middle_of_a_chunk(layout, tokens, dim):
    """Keys aligned with the query at a few late positions, each with a logit far above all
    earlier ones: the softmax reference moves (and the accumulator is rescaled) several times
    inside one chunk, not only at its first tile."""
    lens = [1700, 900]
    g = make(layout, tokens, 1, 1, 4, dim=dim, lens=lens)
    c = g.base
    T = tokens
    for b, n in enumerate(lens):
        # (|q|^2 * scale grows like sqrt(D): the gains keep the logits tens of units apart for every D)
        for pos, gain in ((n // 3, 2.0 * (128 / dim) ** 0.5), (n // 2 + 5, 4.0 * (128 / dim) ** 0.5),
                          (n - 140, 7.0 * (128 / dim) ** 0.5)):
            row = (g.q[b, 0, 0].float() * gain).half()          # logit = gain * |q|^2 * scale: tens of units apart
            if c.block_table is None:
                c.k_cache[b, 0, pos] = row
            else:
                c.k_cache[int(c.block_table[b, pos // T]), 0, pos % T] = row
    for chunk in (0, 2048, 256):
        check(g, chunk, f"moving reference, {layout} T={tokens} D={dim} chunk={chunk}")


@pytest.mark.parametrize("dim", [128, 256])
def test_a_block_that_cannot_be_read_counts_as_zeros(dim):
    """A block id outside the pool is flagged, and the result is the oracle's on the same cache
    with that block's keys and values zeroed (every form of the kernel)."""
    lens = [200, 330]
    g = make("paged", 16, 2, 2, 4, dim=dim, lens=lens)
    dev = to_device(g)
    c = dev.base
    # append first with the good table, then break one entry for the attention call only
    out_ok, _, _ = gpu_step(dev)
    table = c.block_table.clone()
    victim_block = 3
    phys = int(table[1, victim_block])
    table[1, victim_block] = c.k_cache.shape[0] + 7
    B, Tq, Hq, D = g.q.shape
    out = torch.zeros_like(dev.q)
    lse = torch.zeros((B, Tq, Hq), dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(binding.grouped_workspace_bytes(B, Tq, Hq, 2, D, max(lens)), dtype=torch.uint8, device="cuda")
    binding.decode_attention_grouped(out, lse, dev.q, c.k_cache, c.v_cache, table, c.seq_lens, max(lens),
                                     c.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_BLOCK_RANGE
    k = c.k_cache.cpu().numpy().copy()
    v = c.v_cache.cpu().numpy().copy()
    k[phys] = 0
    v[phys] = 0
    want, want_lse = capi.decode_attention_grouped(g.q.numpy(), k, v, np.array(lens, dtype=np.int32), g.base.scale,
                                                   block_table=g.base.block_table.numpy())
    gu.assert_close(out.cpu().reshape(B, Tq * Hq, D), want.reshape(B, Tq * Hq, D),
                    lse.cpu().reshape(B, Tq * Hq), want_lse.reshape(B, Tq * Hq), "zeroed block")
    assert torch.equal(out[0], out_ok.cuda()[0])            # the other sequence is untouched


def test_one_row_case_agrees_with_the_one_row_entry_point():
    g = make("paged", 16, 3, 1, 3)
    dev = to_device(g)
    out, lse, _ = gpu_step(dev)
    c = dev.base
    plain = wl.Case(**{**c.__dict__, "q": dev.q[:, 0].contiguous()})
    ref, ref_lse, _ = gu.gpu_step(plain, do_append=False)
    assert torch.allclose(out[:, 0].float(), ref.float(), atol=gu.MAX_ABS, rtol=gu.MAX_REL)
    fin = torch.isfinite(ref_lse)
    assert torch.equal(torch.isfinite(lse[:, 0]), fin)
    assert torch.allclose(lse[:, 0][fin], ref_lse[fin], atol=1e-4, rtol=1e-5)


def test_inactive_and_short_sequences():
    g = make("contiguous", 0, 1, 4, 2, lens=[0, 2, 4, 130, 0])
    out, lse, flags = gpu_step(to_device(g))
    want, want_lse = oracle_step(g)
    assert flags == 0
    assert torch.all(out[0] == 0) and torch.all(torch.isneginf(lse[0]))
    assert torch.all(out[1, :2] == 0) and torch.all(torch.isneginf(lse[1, :2]))     # 2 tokens, 4 queries
    B, Tq, Hq, D = out.shape
    gu.assert_close(out.reshape(B, Tq * Hq, D), want.reshape(B, Tq * Hq, D),
                    lse.reshape(B, Tq * Hq), want_lse.reshape(B, Tq * Hq))


def test_flags_and_unsupported_shapes():
    g = to_device(make("paged", 16, 2, 1, 4, lens=[40, 50]))
    c = g.base
    B, Tq, Hq, D = g.q.shape
    out = torch.zeros_like(g.q)
    ws = torch.empty(binding.grouped_workspace_bytes(B, Tq, Hq, 2, D, 50), dtype=torch.uint8, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad = c.seq_lens.clone()
    bad[0] = 51                                      # beyond max_seq_len: inactive and flagged
    binding.decode_attention_grouped(out, None, g.q, c.k_cache, c.v_cache, c.block_table, bad, 50,
                                     c.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_SEQ_LEN_RANGE and torch.all(out[0] == 0)
    flags.zero_()
    table = c.block_table.clone()
    table[1, 0] = c.k_cache.shape[0]                 # out of range: not dereferenced, flagged
    binding.decode_attention_grouped(out, None, g.q, c.k_cache, c.v_cache, table, c.seq_lens, 50,
                                     c.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_BLOCK_RANGE and torch.isfinite(out.float()).all()

    def status(q, k, v, table, max_len=50):
        with pytest.raises(binding.InstInferError) as err:
            binding.decode_attention_grouped(torch.zeros_like(q), None, q, k, v, table, c.seq_lens,
                                             max_len, c.scale, ws)
        return err.value.status

    q17 = torch.zeros((B, 17, 2, D), dtype=torch.float16, device="cuda")           # 17 rows per KV head
    assert status(q17, c.k_cache, c.v_cache, c.block_table) == binding.ERR_UNSUPPORTED
    q3 = torch.zeros((B, 1, 3, D), dtype=torch.float16, device="cuda")             # 3 heads over 2
    assert status(q3, c.k_cache, c.v_cache, c.block_table) == binding.ERR_INVALID_ARG
    k8 = c.k_cache.view(-1, 2, 8, D)                                                # 8-token blocks
    assert status(g.q, k8, k8, c.block_table, 8) == binding.ERR_UNSUPPORTED
    q96 = torch.zeros((B, 1, 4, 96), dtype=torch.float16, device="cuda")
    k96 = torch.zeros((4, 2, 16, 96), dtype=torch.float16, device="cuda")
    assert status(q96, k96, k96, c.block_table) == binding.ERR_UNSUPPORTED
    assert binding.grouped_workspace_bytes(B, 17, 2, 2, D, 50) == 0
