"""GPU properties that hold at any size: layout and permutation invariance (bitwise),
data-dependent error flags that never fault the device."""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def paged_from_contiguous(cpu: wl.Case, tokens: int, seed: int) -> wl.Case:
    """The same logical caches, re-laid into pools under a fresh random block table."""
    B, H, S, D = cpu.k_cache.shape
    need = [-(-n // tokens) for n in cpu.seq_lens_host]
    P = sum(need) + 2
    g = torch.Generator().manual_seed(seed)
    perm = torch.randperm(P, generator=g).to(torch.int32)
    table = torch.full((B, max(max(need), 1)), -1, dtype=torch.int32)
    pools = []
    for cache in (cpu.k_cache, cpu.v_cache):
        pool = torch.empty((P, H, tokens, D), dtype=torch.float16)
        pool.view(torch.int16).fill_(wl.NAN_BITS)
        at = 0
        for b, n in enumerate(need):
            table[b, :n] = perm[at:at + n]
            at += n
            for j in range(n):
                rows = cache[b, :, j * tokens:(j + 1) * tokens]
                pool[int(table[b, j]), :, :rows.shape[1]] = rows
        pools.append(pool)
    w = cpu.workload.replace(layout="paged", block_tokens=tokens, s_max=0)
    return wl.Case(w, 0, cpu.q, cpu.k_new, cpu.v_new, pools[0], pools[1], cpu.seq_lens, table,
                   cpu.seq_lens_host, cpu.scale)


def base_case(lens=(200, 64, 333, 1, 90)):
    lens = list(lens)
    w = wl.Workload("inv", 2, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout="contiguous", s_max=max(lens) + 3, heads=4)
    return wl.generate(w, seq_lens=lens)


@pytest.mark.parametrize("chunk", [0, 64, 128])
def test_paged_equals_contiguous_and_ignores_block_placement_bitwise(chunk):
    cpu = base_case()
    flat, lse_flat, _ = gu.gpu_step(gu.to_device(cpu), chunk_tokens=chunk)
    gu.oracle_step(cpu)                                   # append into the CPU copy
    for tokens, seed in [(16, 1), (16, 2), (64, 3), (8, 4)]:
        paged = paged_from_contiguous(cpu, tokens, seed)
        out, lse, flags = gu.gpu_step(gu.to_device(paged), do_append=False, chunk_tokens=chunk)
        assert flags == 0
        assert np.array_equal(gu.bits(out), gu.bits(flat)), (tokens, seed)
        assert torch.equal(lse, lse_flat)


def test_sequence_longer_than_the_bound_is_flagged_and_skipped():
    cpu = base_case()
    for chunk in (0, 64):
        dev = gu.to_device(cpu)
        good, _, _ = gu.gpu_step(dev, chunk_tokens=chunk)
        out, lse, flags = gu.gpu_step(dev, do_append=False, chunk_tokens=chunk, max_seq_len=300)
        assert flags & binding.FLAG_SEQ_LEN_RANGE
        assert torch.all(out[2] == 0) and torch.all(torch.isneginf(lse[2]))      # 333 > 300
        keep = [0, 1, 3, 4]
        if chunk:                       # same chunking => the other sequences are untouched bitwise
            assert np.array_equal(gu.bits(out[keep]), gu.bits(good[keep]))
    dev = gu.to_device(cpu)
    dev.seq_lens[1] = -5
    out, lse, flags = gu.gpu_step(dev, do_append=False)
    assert flags & binding.FLAG_SEQ_LEN_RANGE and torch.all(out[1] == 0)


def test_append_beyond_capacity_is_flagged_and_writes_nothing():
    cpu = base_case()
    dev = gu.to_device(cpu)
    dev.seq_lens[0] = dev.k_cache.shape[2] + 1
    before = dev.k_cache.clone()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kv_append(dev.k_cache, dev.v_cache, dev.k_new, dev.v_new, dev.seq_lens, None, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_SEQ_LEN_RANGE
    assert np.array_equal(gu.bits(dev.k_cache[0]), gu.bits(before[0]))
    assert not np.array_equal(gu.bits(dev.k_cache[1]), gu.bits(before[1]))


def test_bad_block_ids_are_flagged_never_dereferenced():
    cpu = base_case()
    gu.oracle_step(cpu)
    paged = paged_from_contiguous(cpu, 16, 5)
    dev = gu.to_device(paged)
    good, _, _ = gu.gpu_step(dev, do_append=False, chunk_tokens=64)
    dev.block_table[2, 3] = 10 ** 6
    dev.block_table[0, 0] = -1
    out, lse, flags = gu.gpu_step(dev, do_append=False, chunk_tokens=64)
    assert flags == binding.FLAG_BLOCK_RANGE
    assert torch.isfinite(out.float()).all()
    assert np.array_equal(gu.bits(out[[1, 3, 4]]), gu.bits(good[[1, 3, 4]]))
    # append into a bad block: flagged, nothing written
    dev.block_table[4, (90 - 1) // 16] = -7
    before = dev.k_cache.clone()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    lens = dev.seq_lens.clone()
    lens[:4] = 0
    binding.kv_append(dev.k_cache, dev.v_cache, dev.k_new, dev.v_new, lens, dev.block_table, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_BLOCK_RANGE
    assert np.array_equal(gu.bits(dev.k_cache), gu.bits(before))
