"""The allocation-free attention entry point (collected last on purpose).

Some users of this library cannot give it a workspace: their process handed all device
memory to the KV pool when it started, or they run under an allocator they do not own, or
they sit in a loop where an allocation's hidden device synchronisation is not allowed.
`instinfer_decode_attention_static` serves them from a 16 MiB array inside the library.
This test drives it through the C ABI and holds it against the ordinary entry points, twice
in a row, because the array is shared by all calls and keeps the previous call's contents.
"""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def make(layout, tokens, lens, index):
    w = wl.Workload("no_alloc", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout=layout, s_max=max(lens) if layout == "contiguous" else 0,
                    block_tokens=tokens, heads=6)
    return gu.to_device(wl.generate(w, seq_lens=lens))


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


def test_sizes_beyond_the_built_in_array_are_refused():
    case = make("contiguous", 0, [64], 1)
    binding.set_chunk_tokens(64)
    try:
        assert binding.workspace_bytes(64, 40, 128, 131072) > binding.STATIC_WORKSPACE_BYTES
        status = binding.load().instinfer_decode_attention_static(
            case.q.data_ptr(), None, case.q.data_ptr(), case.k_cache.data_ptr(),
            case.v_cache.data_ptr(), None, case.seq_lens.data_ptr(), 64, 40, 128, 131072, 0, 0, 0,
            131072, 0.1, None, None)
    finally:
        binding.set_chunk_tokens(0)
    assert status == binding.ERR_WORKSPACE
    assert "workspace" in binding.status_string(status)
