"""GPU parity of the sparse (SparF, Algorithm 1) path against its CPU oracle.

Floating point decides two integer sets here (the kept query dims and the kept tokens).  Both
sides take each decision in the same precision: the dims on exact fp16 magnitudes, the tokens
on binary32 logits computed by the rule stated in the oracle's header (ties to the lower
position).  The kept sets must therefore agree exactly; outputs and alpha are then compared
with the usual tolerances against the oracle's fp64 arithmetic."""
import math

import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

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


def oracle_sparf(cpu, state, r, l, do_append=True, want_weights=False):
    k, v, kt = cpu.k_cache.numpy(), cpu.v_cache.numpy(), state.kt_pool.numpy()
    v_sum = state.v_sum.numpy()
    lens = np.array(cpu.seq_lens_host, dtype=np.int32)
    table, kt_table = cpu.block_table.numpy(), state.kt_block_table.numpy()
    if do_append:
        capi.sparf_append(k, v, kt, v_sum, cpu.k_new.numpy(), cpu.v_new.numpy(), lens, table,
                          kt_block_table=kt_table)
    return capi.sparf_attention(cpu.q.numpy(), k, v, kt, v_sum, lens, np.array(state.k_tokens_host),
                                table, r, l, cpu.scale, want_weights=want_weights,
                                kt_block_table=kt_table)


def check_structure(sel_gpu, lens, ks, l):
    """Shape of the kept sets: size, order, range, window membership, -1 padding."""
    for b, S in enumerate(lens):
        k = min(ks[b], S)
        window = min(l, k)
        for h in range(sel_gpu.shape[1]):
            J = sel_gpu[b, h, :k]
            assert np.all(sel_gpu[b, h, k:] == -1)
            assert np.all(np.diff(J) > 0) and (k == 0 or (J[0] >= 0 and J[-1] < S))
            assert np.all(np.isin(np.arange(S - window, S), J))


def run_and_check(cpu, state, r, l, what):
    dev, dstate = gu.to_device(cpu), dev_state(state)
    out, alpha, sel, flags = gpu_sparf(dev, dstate, r, l)
    assert flags == 0
    want, want_alpha, want_sel, weights = oracle_sparf(cpu, state, r, l, want_weights=True)   # appends into the CPU copies
    # the append: both K layouts, V and the running sum, bit for bit
    assert np.array_equal(gu.bits(dev.k_cache), gu.bits(cpu.k_cache))
    assert np.array_equal(gu.bits(dev.v_cache), gu.bits(cpu.v_cache))
    assert np.array_equal(gu.bits(dstate.kt_pool), gu.bits(state.kt_pool))
    assert np.array_equal(dstate.v_sum.cpu().numpy().view(np.uint32), state.v_sum.numpy().view(np.uint32))
    lens, ks = cpu.seq_lens_host, state.k_tokens_host
    check_structure(sel, lens, ks, l)
    width = want_sel.shape[2]
    assert np.array_equal(sel[:, :, :width], want_sel), f"{what}: kept sets differ"
    assert np.all(sel[:, :, width:] == -1)
    gu.assert_close(out, want, what=what)
    assert np.abs(alpha - want_alpha).max() <= ALPHA_ATOL
    return out, alpha, sel, (want, want_alpha, want_sel, weights)


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
    out, alpha, sel, own = run_and_check(cpu, state, 16, 8, "heavy ties")
    k0 = state.k_tokens_host[0]
    want = np.concatenate([np.arange(k0 - 8), np.arange(3000 - 8, 3000)])
    assert np.array_equal(sel[0, 0, :k0], want) and np.array_equal(sel[0, 1, :k0], want)
    ours, theirs = sel, own[2][:, :, :sel.shape[2]]                      # ties cut exactly as the oracle cuts them
    assert np.array_equal(ours[0], theirs[0]) and np.array_equal(ours[1], theirs[1])
    assert np.array_equal(ours[2, 1], theirs[2, 1])
