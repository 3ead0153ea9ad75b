"""GPU parity, small shapes: the CUDA path (through the C ABI) against the CPU oracle,
element by element, on the same seeded bits.  Sizes span several tiles, several chunks
and ragged tails; padding is NaN-poisoned."""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

RAGGED = [1, 2, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 129, 257, 0, 511, 640]


def ragged_case(layout, tokens=0, heads=3, lens=RAGGED, index=1, peaked=0.0):
    w = wl.Workload("ragged", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout=layout, s_max=max(lens) if layout == "contiguous" else 0,
                    block_tokens=tokens, heads=heads, peaked_fraction=peaked)
    return wl.generate(w, seq_lens=lens)


def check(case_cpu, chunk, what):
    out, lse, flags = gu.gpu_step(gu.to_device(case_cpu), chunk_tokens=chunk)
    want, want_lse = gu.oracle_step(case_cpu)
    assert flags == 0
    return gu.assert_close(out, want, lse, want_lse, what)


@pytest.mark.parametrize("chunk", [0, 64, 128, 512])
def test_contiguous_ragged(chunk):
    check(ragged_case("contiguous"), chunk, f"contiguous chunk={chunk}")


@pytest.mark.parametrize("tokens", [8, 16, 32, 64, 24])
@pytest.mark.parametrize("chunk", [0, 64, 192])
def test_paged_ragged(tokens, chunk):
    check(ragged_case("paged", tokens), chunk, f"paged T={tokens} chunk={chunk}")


def test_append_is_bit_exact_and_touches_nothing_else():
    for layout, tokens in [("contiguous", 0), ("paged", 16), ("paged", 64)]:
        cpu = ragged_case(layout, tokens)
        dev = gu.to_device(cpu)
        flags = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.kv_append(dev.k_cache, dev.v_cache, dev.k_new, dev.v_new, dev.seq_lens,
                          dev.block_table, flags)
        torch.cuda.synchronize()
        before_k = gu.bits(cpu.k_cache).copy()
        gu.oracle_step(cpu)                       # appends into the CPU copy
        assert np.array_equal(gu.bits(dev.k_cache), gu.bits(cpu.k_cache)), layout
        assert np.array_equal(gu.bits(dev.v_cache), gu.bits(cpu.v_cache)), layout
        assert (gu.bits(cpu.k_cache) != before_k).sum() <= (len(RAGGED) - 1) * 3 * 128
        assert int(flags.item()) == 0


def test_single_token_returns_v_new_bit_for_bit():
    cpu = ragged_case("paged", 16, lens=[1, 1, 1])
    out, lse, _ = gu.gpu_step(gu.to_device(cpu))
    assert np.array_equal(gu.bits(out), gu.bits(cpu.v_new))


def test_inactive_sequences_give_zero_and_minus_infinity():
    for chunk in (0, 64):
        cpu = ragged_case("contiguous", lens=[0, 130, 0])
        out, lse, flags = gu.gpu_step(gu.to_device(cpu), chunk_tokens=chunk)
        assert flags == 0
        assert torch.all(out[0] == 0) and torch.all(out[2] == 0)
        assert torch.all(torch.isneginf(lse[0])) and torch.all(torch.isneginf(lse[2]))
        want, want_lse = gu.oracle_step(cpu)
        gu.assert_close(out, want, lse, want_lse)
    cpu = ragged_case("paged", 16, lens=[0, 0])
    out, lse, _ = gu.gpu_step(gu.to_device(cpu))
    assert torch.all(out == 0) and torch.all(torch.isneginf(lse))


def test_peaked_softmax_and_large_logits():
    cpu = ragged_case("paged", 32, lens=[700, 1500], heads=4, index=3, peaked=0.05)
    cpu.q.mul_(3.0)                                # logits of a few tens
    for chunk in (0, 64, 256):
        out, lse, _ = gu.gpu_step(gu.to_device(cpu), do_append=(chunk == 0), chunk_tokens=chunk)
        want, want_lse = gu.oracle_step(cpu, do_append=(chunk == 0))
        gu.assert_close(out, want, lse, want_lse, f"peaked chunk={chunk}")


def test_forty_heads_head_independence_and_no_lse():
    cpu = ragged_case("contiguous", heads=40, lens=[300, 77])
    dev = gu.to_device(cpu)
    out, lse, _ = gu.gpu_step(dev, chunk_tokens=64)
    out2, _, _ = gu.gpu_step(dev, do_append=False, chunk_tokens=64, want_lse=False)
    assert np.array_equal(gu.bits(out), gu.bits(out2))
    want, want_lse = gu.oracle_step(cpu)
    gu.assert_close(out, want, lse, want_lse)
    dev.q[1, 7] = 0
    dev.k_cache[1, 7] = 1
    out3, _, _ = gu.gpu_step(dev, do_append=False, chunk_tokens=64)
    keep = torch.ones(2, 40, dtype=torch.bool)
    keep[1, 7] = False
    assert np.array_equal(gu.bits(out3[keep]), gu.bits(out[keep]))


def test_runs_on_a_side_stream_and_is_deterministic():
    cpu = ragged_case("paged", 16, lens=[513, 64, 1000])
    dev = gu.to_device(cpu)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        a, lse_a, _ = gu.gpu_step(dev, chunk_tokens=128, stream=side)
    b, lse_b, _ = gu.gpu_step(dev, do_append=False, chunk_tokens=128)
    assert np.array_equal(gu.bits(a), gu.bits(b)) and torch.equal(lse_a, lse_b)
    want, want_lse = gu.oracle_step(cpu)
    gu.assert_close(a, want, lse_a, want_lse)
