"""GPU parity of the sparse (SparF, Algorithm 1) path against its CPU oracle.

Floating point decides two integer sets here (the kept query dims and the kept tokens).  The
dims are ranked on fp16 magnitudes, which is exact on both sides.  The tokens are ranked in
fp64 by the oracle, as Algorithm 1 prints step 6, and in fp32 by the CUDA path: the GPU's
kept set must be a valid top-k of the oracle's fp64 scores up to the fp32 rounding band
derived in tests/sparf_check.py (complete check: size, order, range, padding, window, every
token above the band kept, every token below it dropped; exact ties cut by position).  The
oracle then recomputes alpha and the output for the GPU's set, and those are compared with
the usual tolerances."""
import math

import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu, sparf_check

pytestmark = pytest.mark.gpu

ALPHA_ATOL = 2e-5


@pytest.fixture(autouse=True, params=[1, 2], ids=["chunk-parallel", "block-per-row"])
def sparse_path(request):
    """Every test runs on both implementations of steps 1-7 (rows longer than 16384 tokens
    always take the chunk-parallel one)."""
    binding.set_sparse_path(request.param)
    yield request.param
    binding.set_sparse_path(0)


def make(lens, tokens=16, heads=3, index=2, peaked=0.0, keep=0.125, kt_tokens=None):
    w = wl.Workload("sparf", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout="paged", block_tokens=tokens, heads=heads, peaked_fraction=peaked)
    cpu = wl.generate(w, seq_lens=list(lens))
    return cpu, wl.make_sparf_state(cpu, keep, kt_tokens)


def dev_state(state):
    return wl.SparfState(state.kt_pool.cuda(), state.kt_block_table.cuda(), state.v_sum.cuda(),
                         state.k_tokens.cuda(), state.k_tokens_host)


def gpu_sparf(case, state, r, l, do_append=True, max_k=None):
    B, H, D = case.q.shape
    max_len = max(case.max_seq_len, 1)
    max_k = max_k or max(max(state.k_tokens_host), 1)
    out = gu.Guarded((B, H, D), torch.float16)
    alpha = gu.Guarded((B, H), torch.float32)
    sel = gu.Guarded((B, H, max_k), torch.int32)
    ws = gu.Guarded((binding.sparf_workspace_bytes(B, H, D, max_len, max_k),), torch.uint8)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    if do_append:
        binding.sparf_append(case.k_cache, case.v_cache, state.kt_pool, state.v_sum, case.k_new,
                             case.v_new, case.seq_lens, case.block_table, state.kt_block_table, flags)
    binding.sparf_decode_attention(out.view, alpha.view, sel.view, case.q, case.k_cache, case.v_cache,
                                   state.kt_pool, state.v_sum, case.block_table, state.kt_block_table,
                                   case.seq_lens, state.k_tokens, max_len, max_k, r, l, case.scale,
                                   ws.view, flags)
    torch.cuda.synchronize()
    assert out.intact() and alpha.intact() and sel.intact() and ws.intact()
    return out.view.cpu(), alpha.view.cpu().numpy(), sel.view.cpu().numpy(), int(flags.item())


def oracle_sparf(cpu, state, r, l, do_append=True, want_weights=False, given=None):
    k, v, kt = cpu.k_cache.numpy(), cpu.v_cache.numpy(), state.kt_pool.numpy()
    v_sum = state.v_sum.numpy()
    lens = np.array(cpu.seq_lens_host, dtype=np.int32)
    table, kt_table = cpu.block_table.numpy(), state.kt_block_table.numpy()
    if do_append:
        capi.sparf_append(k, v, kt, v_sum, cpu.k_new.numpy(), cpu.v_new.numpy(), lens, table,
                          kt_block_table=kt_table)
    return capi.sparf_attention(cpu.q.numpy(), k, v, kt, v_sum, lens, np.array(state.k_tokens_host),
                                table, r, l, cpu.scale, want_weights=want_weights, given=given,
                                kt_block_table=kt_table)


def check_kept_sets(cpu, sel_gpu, weights, ks, r, l, what):
    """The GPU's kept sets against the oracle's fp64 scores (cpu holds the appended caches).
    Returns the number of (token, row) decisions that fell inside the rounding band."""
    in_band = 0
    for b, S in enumerate(cpu.seq_lens_host):
        for h in range(sel_gpu.shape[1]):
            k_rows, _ = wl.gather_rows(cpu, b, h)
            k_abs_max = float(k_rows.float().abs().max()) if S else 0.0
            delta = sparf_check.logit_band(cpu.q[b, h].numpy(), k_abs_max, r, cpu.scale)
            in_band += sparf_check.check_kept_set(sel_gpu[b, h], weights[b, h], S, ks[b], l, delta,
                                                  f"{what} pair {(b, h)}")
    return in_band


def run_and_check(cpu, state, r, l, what, generic=True):
    """generic: random data without planted ties, where only a handful of decisions may fall
    inside the rounding band (guards against a band so wide that it checks nothing)."""
    dev, dstate = gu.to_device(cpu), dev_state(state)
    out, alpha, sel, flags = gpu_sparf(dev, dstate, r, l)
    assert flags == 0
    # the oracle's own selection and its fp64 scores (this call appends into the CPU copies)
    _, _, own_sel, weights = oracle_sparf(cpu, state, r, l, want_weights=True)
    # the append: both K layouts, V and the running sum, bit for bit
    assert np.array_equal(gu.bits(dev.k_cache), gu.bits(cpu.k_cache))
    assert np.array_equal(gu.bits(dev.v_cache), gu.bits(cpu.v_cache))
    assert np.array_equal(gu.bits(dstate.kt_pool), gu.bits(state.kt_pool))
    assert np.array_equal(dstate.v_sum.cpu().numpy().view(np.uint32), state.v_sum.numpy().view(np.uint32))
    lens, ks = cpu.seq_lens_host, state.k_tokens_host
    in_band = check_kept_sets(cpu, sel, weights, ks, r, l, what)
    decisions = sum(lens) * sel.shape[1]
    if generic:
        assert in_band <= max(16, decisions // 200), f"{what}: the band holds {in_band} of {decisions} decisions"
    # alpha and the output for the GPU's set, in the oracle's fp64 arithmetic
    want, want_alpha, _, _ = oracle_sparf(cpu, state, r, l, do_append=False, given=sel)
    gu.assert_close(out, want, what=what)
    assert np.abs(alpha - want_alpha).max() <= ALPHA_ATOL
    return out, alpha, sel, (want, want_alpha, own_sel, weights)


@pytest.mark.parametrize("tokens", [8, 16, 64])
@pytest.mark.parametrize("r,l", [(16, 0), (32, 8), (1, 3)])
def test_sparse_attention_matches_the_oracle(tokens, r, l):
    cpu, state = make([1, 2, 9, 100, 257, 0, 640, 1500], tokens)
    run_and_check(cpu, state, r, l, f"T={tokens} r={r} l={l}")


@pytest.mark.parametrize("tokens,kt_tokens", [(8, 64), (16, 256), (32, 32), (16, 48)])
def test_transposed_copy_with_its_own_block_size(tokens, kt_tokens):
    cpu, state = make([1, 2, 9, 100, 257, 0, 640, 1500], tokens, kt_tokens=kt_tokens)
    assert state.kt_block_tokens == kt_tokens
    run_and_check(cpu, state, 16, 4, f"T={tokens} Tk={kt_tokens}")


@pytest.mark.parametrize("tokens,kt_tokens", [(16, 1024), (64, 2048)])
def test_transposed_copy_in_blocks_of_1024_tokens_and_more(tokens, kt_tokens):
    """Large blocks of the transposed copy (the paper gives its embedding-indexed mapping groups
    of up to 1K tokens): rows that end inside a block, on a 1024-token edge, rows of a few
    tokens, and rows of more than one 8192-token score block."""
    cpu, state = make([1, 9, 1023, 1024, 1025, 3000, 0, 9000, 2048 + 255], tokens, kt_tokens=kt_tokens)
    assert state.kt_block_tokens == kt_tokens
    run_and_check(cpu, state, 16, 4, f"T={tokens} Tk={kt_tokens}")
    run_and_check(cpu, state, 5, 0, f"T={tokens} Tk={kt_tokens} r=5")


def test_long_peaked_sequences_and_forty_heads():
    cpu, state = make([5000, 3000], tokens=32, heads=40, index=3, peaked=0.02)
    out, alpha, sel, own = run_and_check(cpu, state, 16, 16, "long peaked")
    assert np.all(alpha > 0.05) and np.all(alpha <= 1.0 + 1e-6)


def test_keeping_everything_reduces_to_dense_attention_on_the_gpu():
    cpu, state = make([33, 700, 1, 0], 16, keep=1.0)
    assert state.k_tokens_host == cpu.seq_lens_host
    dev, dstate = gu.to_device(cpu), dev_state(state)
    out, alpha, sel, _ = gpu_sparf(dev, dstate, 128, 0)
    dense, _, _ = gu.gpu_step(dev, do_append=False)
    want, _ = gu.oracle_step(cpu)
    gu.assert_close(out, want, what="sparse with everything kept")
    assert (out.float() - dense.float()).abs().max() <= 2e-3
    live = np.array(cpu.seq_lens_host) > 0
    assert np.allclose(alpha[live], 1.0, atol=1e-5) and np.all(alpha[~live] == 0)
    for b, S in enumerate(cpu.seq_lens_host):
        assert np.array_equal(sel[b, :, :S], np.tile(np.arange(S), (3, 1)))


def test_window_only_and_nothing_kept():
    cpu, state = make([90, 40], 8)
    state.k_tokens_host[:] = [10, 0]
    state.k_tokens = torch.tensor(state.k_tokens_host, dtype=torch.int32)
    dev, dstate = gu.to_device(cpu), dev_state(state)
    out, alpha, sel, _ = gpu_sparf(dev, dstate, 16, 10, max_k=12)
    assert np.array_equal(sel[0, :, :10], np.tile(np.arange(80, 90), (3, 1))) and np.all(sel[0, :, 10:] == -1)
    assert np.all(sel[1] == -1) and np.all(alpha[1] == 0)
    want, want_alpha, _, _ = oracle_sparf(cpu, state, 16, 10)
    gu.assert_close(out, want, what="window only / k = 0")
    # k = 0: the output is the mean value vector
    vbar = state.v_sum.numpy()[1] / 40.0
    assert np.abs(out[1].numpy().astype(np.float64) - vbar).max() <= 2e-3


def test_true_mean_makes_sparse_close_to_dense():
    # With v_sum the real sum of V and an eighth of the tokens kept, the sparse output tracks
    # the dense one (the algorithm's purpose); this guards against a path that is
    # self-consistent with its oracle but wrong as an approximation of attention.
    cpu, state = make([2048], tokens=32, heads=8, index=3, peaked=0.02)
    gu.oracle_step(cpu)                                              # append on the CPU copy
    k_rows = cpu.k_cache.numpy()
    table, S = cpu.block_table.numpy(), 2048
    v_rows = cpu.v_cache.numpy()[table[0, :S // 32]].transpose(1, 0, 2, 3).reshape(8, S, 128)
    state.v_sum = torch.from_numpy(v_rows.astype(np.float64).sum(axis=1).astype(np.float32))[None]
    state.kt_pool, state.kt_block_table = cpu.k_cache.transpose(2, 3).contiguous(), cpu.block_table
    dev, dstate = gu.to_device(cpu), dev_state(state)
    out, alpha, _, _ = gpu_sparf(dev, dstate, 32, 32, do_append=False)
    dense, _ = gu.oracle_step(cpu, do_append=False)
    err = np.abs(out.numpy().astype(np.float64) - dense)
    assert err.mean() < 0.05 and np.all(alpha > 0.3)


def test_heavy_ties_are_cut_by_position():
    # q = 0 makes every approximate score equal: the kept set must be the first positions
    # plus the local window; duplicated key rows give large groups of equal scores.
    cpu, state = make([3000, 500, 40000], tokens=16, heads=2, kt_tokens=64)
    cpu.q[0].zero_()
    cpu.q[2, 1].zero_()
    table = cpu.block_table
    first = cpu.k_cache[int(table[1, 0]), :, 0].clone()
    for j in range(500 // 16):                                       # sequence 1: every key row the same
        cpu.k_cache[int(table[1, j])] = first[:, None, :]
    state.kt_pool, state.kt_block_table = wl.make_sparf_state(cpu, 0.125, 64).kt_pool, \
        wl.make_sparf_state(cpu, 0.125, 64).kt_block_table
    out, alpha, sel, own = run_and_check(cpu, state, 16, 8, "heavy ties", generic=False)
    k0 = state.k_tokens_host[0]
    want = np.concatenate([np.arange(k0 - 8), np.arange(3000 - 8, 3000)])
    assert np.array_equal(sel[0, 0, :k0], want) and np.array_equal(sel[0, 1, :k0], want)
    ours, theirs = sel, own[2][:, :, :sel.shape[2]]                      # ties cut exactly as the oracle cuts them
    assert np.array_equal(ours[0], theirs[0]) and np.array_equal(ours[1], theirs[1])
    assert np.array_equal(ours[2, 1], theirs[2, 1])


def test_length_beyond_the_transposed_copys_table_is_flagged_and_nothing_is_touched():
    # The K/V table has room for 64 tokens per sequence (4 blocks of 16) but the transposed
    # copy's table only for 32 (1 block of 32): a sequence of 40 tokens fits the first and not
    # the second.  The append must flag it before reading either table and leave K, V, the
    # transposed copy and the running sum exactly as they were; the other sequence proceeds.
    cpu, state = make([40, 20], tokens=16, heads=3, kt_tokens=32)
    dev, dstate = gu.to_device(cpu), dev_state(state)
    assert dstate.kt_block_table.shape[1] == 2
    short_table = dstate.kt_block_table[:, :1].contiguous()        # Mk = 1: capacity 32 tokens
    before = [t.clone() for t in (dev.k_cache, dev.v_cache, dstate.kt_pool, dstate.v_sum)]
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.sparf_append(dev.k_cache, dev.v_cache, dstate.kt_pool, dstate.v_sum, dev.k_new, dev.v_new,
                         dev.seq_lens, dev.block_table, short_table, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == binding.FLAG_SEQ_LEN_RANGE
    # sequence 0: untouched everywhere
    for b_table, pool, old, tokens in ((dev.block_table, dev.k_cache, before[0], 16),
                                       (dev.block_table, dev.v_cache, before[1], 16)):
        blk = int(b_table[0, 39 // tokens])
        assert torch.equal(pool[blk].view(torch.int16), old[blk].view(torch.int16))
    assert torch.equal(dstate.v_sum[0], before[3][0])
    for blk in dstate.kt_block_table[0].tolist():
        assert torch.equal(dstate.kt_pool[blk].view(torch.int16), before[2][blk].view(torch.int16))
    # sequence 1 (20 tokens, fits both): appended as usual
    blk, slot = int(dev.block_table[1, 19 // 16]), 19 % 16
    assert torch.equal(dev.k_cache[blk, :, slot].view(torch.int16), dev.k_new[1].view(torch.int16))
    kt_blk = int(short_table[1, 0])
    assert torch.equal(dstate.kt_pool[kt_blk, :, :, 19].view(torch.int16), dev.k_new[1].view(torch.int16))
    assert torch.equal(dstate.v_sum[1], before[3][1] + dev.v_new[1].float())
