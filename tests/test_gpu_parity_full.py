"""GPU parity at the full standard sizes, in the launch configuration the benchmark times
(automatic split plan, device-generated inputs, NaN-poisoned padding).  Workloads 0 and 1 are
compared element by element; for the larger ones the oracle recomputes sampled (sequence,
head) pairs one by one from rows gathered off the device: 64 pairs of each 20 GiB workload,
8 pairs of every one of the 40 layers of the 13B-class step, and a batch of that step's shape
whose lengths are placed on the edges of the split plan (last token in the first tile of a
chunk, in a ragged last tile, on a chunk boundary)."""
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
    """The shortest and the longest sequence (first and last head), then random pairs."""
    lens = case.seq_lens_host
    heads = case.workload.heads
    rng = np.random.default_rng(seed)
    lo, hi = int(np.argmin(lens)), int(np.argmax(lens))
    picks = {(lo, 0), (lo, heads - 1), (hi, 0), (hi, heads - 1)}
    while len(picks) < min(count, len(lens) * heads):
        picks.add((int(rng.integers(len(lens))), int(rng.integers(heads))))
    return sorted(picks)


def check_pairs(case, pairs, out, lse, before, what):
    """Oracle on the given pairs, 16 at a time (bounds the host copy of the gathered rows)."""
    worst = (0.0, 0.0)
    for at in range(0, len(pairs), 16):
        part = pairs[at:at + 16]
        longest = max(case.seq_lens_host[b] for b, _ in part)
        n = len(part)
        k = np.zeros((n, 1, longest, 128), dtype=np.float16)
        v = np.zeros((n, 1, longest, 128), dtype=np.float16)
        q = np.zeros((n, 1, 128), dtype=np.float16)
        lens = np.zeros(n, dtype=np.int32)
        for i, (b, h) in enumerate(part):
            kr, vr = wl.gather_rows(case, b, h)
            L = case.seq_lens_host[b]
            k[i, 0, :L], v[i, 0, :L] = kr.cpu().numpy(), vr.cpu().numpy()
            q[i, 0], lens[i] = case.q[b, h].cpu().numpy(), L
            # the append filled exactly the last row with k_new / v_new, bit for bit
            assert np.array_equal(gu.bits(kr[L - 1]), gu.bits(case.k_new[b, h]))
            assert np.array_equal(gu.bits(vr[L - 1]), gu.bits(case.v_new[b, h]))
            if (b, h) in before:
                assert np.array_equal(gu.bits(kr[:L - 1]), gu.bits(before[(b, h)][:L - 1]))
                assert np.all(gu.bits(before[(b, h)][L - 1]) == wl.NAN_BITS)
        want, want_lse, _ = capi.decode_attention(q, k, v, lens, case.scale)
        got = torch.stack([out[b, h] for b, h in part])[:, None, :]
        got_lse = torch.stack([lse[b, h] for b, h in part])[:, None]
        errs = gu.assert_close(got, want, got_lse, want_lse, what)
        worst = (max(worst[0], errs[0]), max(worst[1], errs[1]))
    return worst


def check_sampled(case, count=64, seed=0, what=""):
    pairs = sampled_pairs(case, count, seed)
    before = {p: wl.gather_rows(case, *p)[0].cpu() for p in pairs[:8]}    # K rows before the append
    out, lse = device_step(case)
    assert torch.isfinite(out.float()).all(), "poison leaked into an output"
    return check_pairs(case, pairs, out, lse, before, what)


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


def test_workload_4_every_layer_sampled():
    need_memory(6)
    for layer in range(wl.STANDARD[4].layers):
        case = wl.generate(wl.STANDARD[4], layer=layer, device="cuda")
        check_sampled(case, count=8, seed=layer, what=f"workload 4 layer {layer}")
        del case


def test_workload_4_shape_with_lengths_on_the_edges_of_the_plan():
    """The 13B-class step's shape (16 sequences x 40 heads, 32-token pages, lengths in
    4096..8192) with lengths placed where the split plan has its seams."""
    need_memory(6)
    w = wl.STANDARD[4]
    chunk = binding.plan_chunk_tokens(w.batch, w.heads, w.len_hi)
    splits = binding.plan_num_splits(w.batch, w.heads, w.len_hi)
    # the plan: n_short chunks of 256 tokens, then long chunks; recover n_short from the counts
    n_short = next(n for n in range(0, 64) if n + -(-(w.len_hi - 256 * n) // chunk) == splits)
    first_long = 256 * n_short
    seam = lambda j: first_long + j * chunk                      # start of long chunk j
    mid = [j for j in range(1, splits) if w.len_lo < seam(j) < w.len_hi - 8]
    assert len(mid) >= 3, (chunk, splits, n_short)
    edges = [w.len_hi, w.len_lo,
             seam(mid[0]) + 1, seam(mid[0]) + 8, seam(mid[1]) + 3, seam(mid[-1]) + 8,   # first tile of a chunk
             seam(mid[0]), seam(mid[0]) - 1, seam(mid[1]), seam(mid[-1]) - 5,         # on a seam, just before one
             seam(mid[1]) + 9, seam(mid[-1]) + 17,                                    # second and third tiles
             w.len_hi - 1, w.len_hi - 3, w.len_lo + 5, 6001]                           # ragged last tiles
    lens = [int(min(max(n, w.len_lo), w.len_hi)) for n in edges][:w.batch]
    assert len(lens) == w.batch
    case = wl.generate(w, layer=3, device="cuda", seq_lens=lens)
    pairs = [(b, h) for b in range(w.batch) for h in (0, 13, 26, 39)]
    out, lse = device_step(case)
    assert torch.isfinite(out.float()).all()
    check_pairs(case, pairs, out, lse, {}, "workload 4 shape, lengths on plan edges")
