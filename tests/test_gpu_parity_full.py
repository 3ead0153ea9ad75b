"""GPU parity at the full standard sizes, in the launch configuration the benchmark times
(automatic split plan, device-generated inputs, NaN-poisoned padding).  Workloads 0 and 1 are
compared element by element; for the 20 GiB ones the oracle recomputes sampled (sequence,
head) pairs one by one from rows gathered off the device."""
import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def need_memory(gib):
    free, _ = torch.cuda.mem_get_info()
    if free < gib * 2 ** 30:
        pytest.skip(f"needs {gib} GiB of free device memory")


def device_step(case):
    B, H, D = case.q.shape
    out = torch.empty((B, H, D), dtype=torch.float16, device="cuda")
    lse = torch.empty((B, H), dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = binding.alloc_workspace(B, H, D, case.max_seq_len)
    binding.kv_append(case.k_cache, case.v_cache, case.k_new, case.v_new, case.seq_lens,
                      case.block_table, flags)
    if case.block_table is None:
        binding.decode_attention(out, lse, case.q, case.k_cache, case.v_cache, case.seq_lens,
                                 case.max_seq_len, case.scale, ws, flags)
    else:
        binding.decode_attention_paged(out, lse, case.q, case.k_cache, case.v_cache,
                                       case.block_table, case.seq_lens, case.max_seq_len,
                                       case.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    return out.cpu(), lse.cpu()


def sampled_pairs(case, count, seed):
    lens = case.seq_lens_host
    rng = np.random.default_rng(seed)
    picks = {(int(np.argmin(lens)), 0), (int(np.argmax(lens)), case.workload.heads - 1)}
    while len(picks) < count:
        picks.add((int(rng.integers(len(lens))), int(rng.integers(case.workload.heads))))
    return sorted(picks)


def check_sampled(case, count=6, seed=0, what=""):
    pairs = sampled_pairs(case, count, seed)
    before = {p: wl.gather_rows(case, *p)[0].cpu() for p in pairs}        # K rows before the append
    out, lse = device_step(case)
    assert torch.isfinite(out.float()).all(), "poison leaked into an output"
    longest = max(case.seq_lens_host[b] for b, _ in pairs)
    n = len(pairs)
    k = np.zeros((n, 1, longest, 128), dtype=np.float16)
    v = np.zeros((n, 1, longest, 128), dtype=np.float16)
    q = np.zeros((n, 1, 128), dtype=np.float16)
    lens = np.zeros(n, dtype=np.int32)
    for i, (b, h) in enumerate(pairs):
        kr, vr = wl.gather_rows(case, b, h)
        L = case.seq_lens_host[b]
        k[i, 0, :L], v[i, 0, :L] = kr.cpu().numpy(), vr.cpu().numpy()
        q[i, 0], lens[i] = case.q[b, h].cpu().numpy(), L
        # the append filled exactly the last row with k_new / v_new, bit for bit
        assert np.array_equal(gu.bits(kr[L - 1]), gu.bits(case.k_new[b, h]))
        assert np.array_equal(gu.bits(vr[L - 1]), gu.bits(case.v_new[b, h]))
        assert np.array_equal(gu.bits(kr[:L - 1]), gu.bits(before[(b, h)][:L - 1]))
        assert np.all(gu.bits(before[(b, h)][L - 1]) == wl.NAN_BITS)
    want, want_lse, _ = capi.decode_attention(q, k, v, lens, case.scale)
    got = torch.stack([out[b, h] for b, h in pairs])[:, None, :]
    got_lse = torch.stack([lse[b, h] for b, h in pairs])[:, None]
    return gu.assert_close(got, want, got_lse, want_lse, what)


def test_workload_0_every_element():
    cpu = wl.generate(wl.STANDARD[0])
    out, lse = device_step(gu.to_device(cpu))
    want, want_lse = gu.oracle_step(cpu)
    gu.assert_close(out, want, lse, want_lse, "workload 0")


def test_workload_1_every_element():
    cpu = wl.generate(wl.STANDARD[1])
    dev = gu.to_device(cpu)
    out, lse = device_step(dev)
    want, want_lse = gu.oracle_step(cpu)
    gu.assert_close(out, want, lse, want_lse, "workload 1")
    assert np.array_equal(gu.bits(dev.k_cache), gu.bits(cpu.k_cache))     # appended cache, whole
    assert np.array_equal(gu.bits(dev.v_cache), gu.bits(cpu.v_cache))


def test_workload_2_sampled():
    need_memory(30)
    check_sampled(wl.generate(wl.STANDARD[2], device="cuda"), what="workload 2")


def test_workload_3_sampled_peaked_long_context():
    need_memory(30)
    check_sampled(wl.generate(wl.STANDARD[3], device="cuda"), what="workload 3")


@pytest.mark.parametrize("layer", [0, 17, 39])
def test_workload_4_sampled_layers(layer):
    need_memory(6)
    check_sampled(wl.generate(wl.STANDARD[4], layer=layer, device="cuda"), seed=layer,
                  what=f"workload 4 layer {layer}")
