"""The host-vector decode step (one C call: upload q,k,v, append, attend, download) against
the oracle and against the separate device-resident calls."""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 32)])
def test_decode_step_from_host_vectors(layout, tokens):
    lens = [257, 1, 0, 900, 64]
    w = wl.Workload("host_step", 4, batch=len(lens), len_lo=0, len_hi=max(lens), layout=layout,
                    s_max=max(lens) if layout == "contiguous" else 0, block_tokens=tokens, heads=6)
    cpu = wl.generate(w, seq_lens=lens)
    dev = gu.to_device(cpu)
    B, H, D = cpu.q.shape
    qkv_host = torch.stack([cpu.q, cpu.k_new, cpu.v_new]).contiguous().pin_memory()
    out_host = torch.full((B, H, D), float("nan"), dtype=torch.float16).pin_memory()
    qkv_dev = torch.empty((3, B, H, D), dtype=torch.float16, device="cuda")
    out_dev = torch.empty((B, H, D), dtype=torch.float16, device="cuda")
    lse = torch.empty((B, H), dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = binding.alloc_workspace(B, H, D, max(lens))
    binding.decode_step_host(out_host, qkv_host, qkv_dev, out_dev, lse, dev.k_cache, dev.v_cache,
                             dev.seq_lens, dev.block_table, max(lens), cpu.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    want, want_lse = gu.oracle_step(cpu)                      # appends into the CPU copy
    gu.assert_close(out_host.clone(), want, lse.cpu(), want_lse, f"host step {layout}")
    assert np.array_equal(gu.bits(dev.k_cache), gu.bits(cpu.k_cache))
    assert np.array_equal(gu.bits(dev.v_cache), gu.bits(cpu.v_cache))
    # identical to the separate device-resident calls on the already appended cache
    again, _, _ = gu.gpu_step(dev, do_append=False)
    assert np.array_equal(gu.bits(again), gu.bits(out_host))
