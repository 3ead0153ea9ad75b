"""GPU parity of the bulk (prefill) append: bit-exact against the oracle, both layouts,
nothing else touched, bad lengths flagged and skipped."""
import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def case_for(layout, tokens, lens):
    w = wl.Workload("bulk", 1, batch=len(lens), len_lo=min(lens), len_hi=max(lens), layout=layout,
                    s_max=max(lens) + 5 if layout == "contiguous" else 0, block_tokens=tokens, heads=5)
    return wl.generate(w, seq_lens=list(lens))


@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 8), ("paged", 16), ("paged", 64)])
def test_bulk_append_is_bit_exact(layout, tokens):
    lens = [300, 17, 64, 0, 129]
    news = [300, 5, 64, 0, 1]
    cpu = case_for(layout, tokens, lens)
    g = torch.Generator().manual_seed(7)
    kn = torch.randn(5, 300, 5, 128, generator=g).half()
    vn = torch.randn(5, 300, 5, 128, generator=g).half()
    dev = gu.to_device(cpu)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kv_append_bulk(dev.k_cache, dev.v_cache, kn.cuda(), vn.cuda(), dev.seq_lens,
                           torch.tensor(news, dtype=torch.int32, device="cuda"), dev.block_table, flags)
    torch.cuda.synchronize()
    k, v = cpu.k_cache.numpy(), cpu.v_cache.numpy()
    table = None if cpu.block_table is None else cpu.block_table.numpy()
    capi.kv_append_bulk(k, v, kn.numpy(), vn.numpy(), np.array(lens), np.array(news), block_table=table)
    assert int(flags.item()) == 0
    assert np.array_equal(gu.bits(dev.k_cache), k.view(np.uint16))
    assert np.array_equal(gu.bits(dev.v_cache), v.view(np.uint16))
    # a decode step on top of the prefilled cache still matches the oracle
    out, lse, _ = gu.gpu_step(dev, do_append=False)
    want, want_lse = gu.oracle_step(cpu, do_append=False)
    live = np.array(lens) > 0
    full = np.array(news) == np.array(lens)                       # fully rewritten: no poison left
    ok = live & full
    gu.assert_close(out[ok], want[ok], lse[ok], want_lse[ok], "decode after prefill")


def test_bad_lengths_are_flagged_and_skipped():
    lens = [40, 40]
    cpu = case_for("paged", 16, lens)
    dev = gu.to_device(cpu)
    before = dev.k_cache.clone()
    kn = torch.zeros(2, 8, 5, 128, dtype=torch.float16, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kv_append_bulk(dev.k_cache, dev.v_cache, kn, kn, dev.seq_lens,
                           torch.tensor([9, 4], dtype=torch.int32, device="cuda"), dev.block_table, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_SEQ_LEN_RANGE
    table = cpu.block_table.numpy()
    first = table[0, :3]
    assert np.array_equal(gu.bits(dev.k_cache[first]), gu.bits(before[first]))          # sequence 0 untouched
    blk = int(table[1, 2])
    assert torch.all(dev.k_cache[blk, :, 4:8] == 0)                                     # sequence 1 written (positions 36..39)


@pytest.mark.parametrize("tokens,kt_tokens", [(8, 8), (16, 64), (32, 256)])
def test_sparse_bulk_append_is_bit_exact(tokens, kt_tokens):
    lens = [300, 17, 64, 0, 129]
    news = [300, 5, 61, 0, 1]
    cpu = case_for("paged", tokens, lens)
    state = wl.make_sparf_state(cpu, 0.125, kt_tokens)
    g = torch.Generator().manual_seed(8)
    kn = torch.randn(5, 300, 5, 128, generator=g).half()
    vn = torch.randn(5, 300, 5, 128, generator=g).half()
    dev = gu.to_device(cpu)
    kt_dev, sum_dev, kt_table_dev = state.kt_pool.cuda(), state.v_sum.cuda(), state.kt_block_table.cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.sparf_append_bulk(dev.k_cache, dev.v_cache, kt_dev, sum_dev, kn.cuda(), vn.cuda(), dev.seq_lens,
                              torch.tensor(news, dtype=torch.int32, device="cuda"), dev.block_table,
                              kt_table_dev, flags)
    torch.cuda.synchronize()
    k, v, kt, v_sum = cpu.k_cache.numpy(), cpu.v_cache.numpy(), state.kt_pool.numpy(), state.v_sum.numpy()
    capi.sparf_append_bulk(k, v, kt, v_sum, kn.numpy(), vn.numpy(), np.array(lens), np.array(news),
                           cpu.block_table.numpy(), kt_block_table=state.kt_block_table.numpy())
    assert int(flags.item()) == 0
    assert np.array_equal(gu.bits(dev.k_cache), k.view(np.uint16))
    assert np.array_equal(gu.bits(dev.v_cache), v.view(np.uint16))
    assert np.array_equal(gu.bits(kt_dev), kt.view(np.uint16))
    assert np.array_equal(sum_dev.cpu().numpy().view(np.uint32), v_sum.view(np.uint32))
