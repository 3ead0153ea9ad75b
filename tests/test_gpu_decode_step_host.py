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


def test_overlapped_step_gives_the_same_bits_on_three_streams():
    """Upload, kernels and download on three streams, two layers in flight: each result equals
    the single-stream call's bit for bit, and the oracle's within tolerance."""
    lens = [300, 77, 0, 1024]
    w = wl.Workload("host_step", 4, batch=len(lens), len_lo=0, len_hi=max(lens), layout="paged",
                    block_tokens=32, heads=5)
    compute, up, down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    layers = []
    for layer in range(3):
        cpu = wl.generate(w, layer=layer, seq_lens=lens)
        dev = gu.to_device(cpu)
        B, H, D = cpu.q.shape
        item = dict(cpu=cpu, dev=dev,
                    qkv_host=torch.stack([cpu.q, cpu.k_new, cpu.v_new]).contiguous().pin_memory(),
                    out_host=torch.full((B, H, D), float("nan"), dtype=torch.float16).pin_memory(),
                    qkv_dev=torch.empty((3, B, H, D), dtype=torch.float16, device="cuda"),
                    out_dev=torch.empty((B, H, D), dtype=torch.float16, device="cuda"),
                    lse=torch.empty((B, H), dtype=torch.float32, device="cuda"),
                    ws=binding.alloc_workspace(B, H, D, max(lens)),
                    uploaded=torch.cuda.Event(), attended=torch.cuda.Event())
        item["uploaded"].record(up)
        item["attended"].record(compute)
        layers.append(item)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    for it in layers:
        d = it["dev"]
        binding.decode_step_host_overlapped(it["out_host"], it["qkv_host"], it["qkv_dev"], it["out_dev"],
                                            it["lse"], d.k_cache, d.v_cache, d.seq_lens, d.block_table,
                                            max(lens), it["cpu"].scale, it["ws"], flags, compute, up, down,
                                            it["uploaded"], it["attended"])
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    for n, it in enumerate(layers):
        want, want_lse = gu.oracle_step(it["cpu"])
        gu.assert_close(it["out_host"].clone(), want, it["lse"].cpu(), want_lse, f"overlapped layer {n}")
        again, _, _ = gu.gpu_step(it["dev"], do_append=False)
        assert np.array_equal(gu.bits(again), gu.bits(it["out_host"]))
    # a copy stream other than the compute stream needs its event
    it = layers[0]
    d = it["dev"]
    lib = binding.load()
    ptr = lambda t: t.data_ptr()
    rc = lib.instinfer_decode_step_host_overlapped(
        ptr(it["out_host"]), ptr(it["qkv_host"]), ptr(it["qkv_dev"]), ptr(it["out_dev"]), None, ptr(d.k_cache),
        ptr(d.v_cache), ptr(d.seq_lens), ptr(d.block_table), d.block_table.shape[1], 32, d.k_cache.shape[0],
        len(lens), 5, 128, 0, max(lens), 0.1, ptr(it["ws"]), it["ws"].numel(), None, compute.cuda_stream,
        up.cuda_stream, compute.cuda_stream, None, None)
    assert rc == binding.ERR_INVALID_ARG
