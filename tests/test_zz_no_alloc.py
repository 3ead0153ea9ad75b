"""The allocation-free attention entry point (collected last on purpose).

Some users of this library cannot give it a workspace: their process handed all device
memory to the KV pool when it started, or they run under an allocator they do not own, or
they sit in a loop where an allocation's hidden device synchronisation is not allowed.
`instinfer_decode_attention_static` serves them from a 16 MiB array inside the library.
This test drives it through the C ABI and holds it against the ordinary entry points and
against the CPU oracle, several calls in a row, because the array is shared by all calls and
keeps the previous call's contents.
"""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def make(layout, tokens, lens, index, device=True):
    w = wl.Workload("no_alloc", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout=layout, s_max=max(lens) if layout == "contiguous" else 0,
                    block_tokens=tokens, heads=6)
    cpu = wl.generate(w, seq_lens=lens)
    return gu.to_device(cpu) if device else cpu


def static_step(case, chunk):
    B, H, D = case.q.shape
    out = torch.full((B, H, D), float("nan"), dtype=torch.float16, device="cuda")
    lse = torch.full((B, H), float("nan"), dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.set_chunk_tokens(chunk)
    try:
        binding.decode_attention_static(out, lse, case.q, case.k_cache, case.v_cache,
                                        case.block_table, case.seq_lens, case.max_seq_len,
                                        case.scale, flags)
    finally:
        binding.set_chunk_tokens(0)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    return out.cpu(), lse.cpu()


def test_static_scratch_matches_the_workspace_entry_points_twice_in_a_row():
    # Two different problems back to back: the second runs on whatever the first left in
    # the shared array (more chunks first, then fewer, so stale partials lie beyond its own).
    first = make("paged", 16, [900, 64, 0, 513, 1], 2)
    second = make("contiguous", 0, [130, 257, 31], 1)
    for case, chunk in ((first, 64), (second, 128), (first, 0)):
        want, want_lse, _ = gu.gpu_step(case, do_append=True, chunk_tokens=chunk)
        got, got_lse = static_step(case, chunk)
        fin = torch.isfinite(want_lse)
        assert torch.equal(torch.isneginf(got_lse), torch.isneginf(want_lse))
        diff = (got.double() - want.double()).abs()
        assert float(diff.max()) <= gu.MAX_ABS
        big = want.double().abs() >= gu.REL_FLOOR
        assert float((diff[big] / want.double().abs()[big]).max()) <= gu.MAX_REL
        assert torch.allclose(got_lse[fin], want_lse[fin], rtol=gu.LSE_RTOL, atol=gu.LSE_ATOL)
        assert np.array_equal(gu.bits(got), gu.bits(want))       # same kernels, same plan
    # and against the oracle, on the same bits (the appends above have run on the device copies;
    # the oracle appends into its own)
    for (layout, tokens, lens, index), chunk in (((("paged", 16, [900, 64, 0, 513, 1], 2)), 64),
                                                 (("contiguous", 0, [130, 257, 31], 1), 128)):
        cpu = make(layout, tokens, lens, index, device=False)
        dev = gu.to_device(cpu)
        gu.gpu_step(dev, do_append=True, chunk_tokens=chunk)     # append on the device copy
        got, got_lse = static_step(dev, chunk)
        want, want_lse = gu.oracle_step(cpu)
        gu.assert_close(got, want, got_lse, want_lse, f"static scratch vs oracle, {layout}")


def test_sizes_beyond_the_built_in_array_are_refused():
    # 8 x 32 pairs x 8192 tokens in 64-token chunks: 32768 partials of 516 bytes, just over the
    # 16 MiB array.  Every buffer has its true size (1 GiB of cache), so that even a library
    # that failed to refuse the call would touch only memory it was given.
    B, H, L = 8, 32, 8192
    q = torch.zeros((B, H, 128), dtype=torch.float16, device="cuda")
    out = torch.full_like(q, 7.0)
    k = torch.zeros((B, H, L, 128), dtype=torch.float16, device="cuda")
    v = torch.zeros_like(k)
    lens = torch.full((B,), 5, dtype=torch.int32, device="cuda")
    binding.set_chunk_tokens(64)
    try:
        assert binding.workspace_bytes(B, H, 128, L) > binding.STATIC_WORKSPACE_BYTES
        status = binding.load().instinfer_decode_attention_static(
            out.data_ptr(), None, q.data_ptr(), k.data_ptr(), v.data_ptr(), None, lens.data_ptr(),
            B, H, 128, L, 0, 0, 0, L, 0.1, None, None)
    finally:
        binding.set_chunk_tokens(0)
    torch.cuda.synchronize()
    assert status == binding.ERR_WORKSPACE
    assert "workspace" in binding.status_string(status)
    assert bool((out == 7.0).all())                              # nothing was enqueued
