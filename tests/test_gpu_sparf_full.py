"""Sparse path at the full size of the two long-context workloads, in the configurations the
benchmark times: 8 x 40 heads x 131072 tokens (K/V pages of 64 tokens; chunk-parallel
selection) and 64 x 40 heads x 16384 tokens (pages of 16 tokens; both forms of the selection),
transposed copy in 256-token blocks.  The oracle recomputes sampled (sequence, head) pairs one
by one from rows gathered off the device into single-pair pools: the GPU's kept set must be a
valid top-k of the oracle's fp64 scores (tests/sparf_check.py), and alpha and the output must
match the oracle's fp64 arithmetic on that set."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu, sparf_check

pytestmark = pytest.mark.gpu

R, WINDOW = 16, 16


def single_pair_problem(case, state, b, h):
    """Pools holding just (b, h): identity block tables, same block sizes (memory movement only)."""
    w = case.workload
    T, Tk, D = w.block_tokens, state.kt_block_tokens, w.head_dim
    L = case.seq_lens_host[b]
    k_rows, v_rows = wl.gather_rows(case, b, h)                              # [L, D]
    blocks, kt_blocks = -(-L // T), -(-L // Tk)

    def pool(rows):
        padded = torch.zeros((blocks * T, D), dtype=torch.float16, device=rows.device)
        padded[:L] = rows
        return padded.view(blocks, 1, T, D).cpu().numpy()

    kt_ids = state.kt_block_table[b, :kt_blocks].long()
    kt = state.kt_pool[kt_ids, h].unsqueeze(1).cpu().numpy()                 # [Pk', 1, D, Tk]
    kt = np.ascontiguousarray(kt)
    kt[-1, :, :, L - (kt_blocks - 1) * Tk:] = 0                              # slots past the end: any finite value
    return dict(q=case.q[b:b + 1, h:h + 1].cpu().numpy(), k=pool(k_rows), v=pool(v_rows), kt=kt,
                v_sum=state.v_sum[b:b + 1, h:h + 1].cpu().numpy(), lens=np.array([L]),
                table=np.arange(blocks, dtype=np.int32)[None], kt_table=np.arange(kt_blocks, dtype=np.int32)[None],
                k_abs_max=float(k_rows.float().abs().max()))


def check_pair(pb, k_tokens, scale, sel_row, out_row, alpha_value, what):
    """One (sequence, head): kept set valid against the fp64 scores, then alpha and the output
    against the oracle run on the GPU's set.  Returns the number of decisions inside the band."""
    args = (pb["q"], pb["k"], pb["v"], pb["kt"], pb["v_sum"], pb["lens"], np.array([k_tokens]), pb["table"],
            R, WINDOW, scale)
    _, _, _, weights = capi.sparf_attention(*args, want_weights=True, kt_block_table=pb["kt_table"])
    delta = sparf_check.logit_band(pb["q"][0, 0], pb["k_abs_max"], R, scale)
    in_band = sparf_check.check_kept_set(sel_row, weights[0, 0], int(pb["lens"][0]), k_tokens, WINDOW, delta, what)
    want, want_alpha, _, _ = capi.sparf_attention(*args, given=sel_row[None, None, :], kt_block_table=pb["kt_table"])
    gu.assert_close(out_row, want, what=what)
    assert abs(alpha_value - want_alpha[0, 0]) <= 2e-5, what
    return in_band


def run_workload(index, pairs, path, kt_tokens=256):
    case = wl.generate(wl.STANDARD[index], device="cuda", poison=False)
    state = wl.make_sparf_state(case, 0.125, kt_tokens)
    B, H, D = case.q.shape
    max_len, max_k = case.max_seq_len, max(state.k_tokens_host)
    out = torch.empty((B, H, D), dtype=torch.float16, device="cuda")
    alpha = torch.empty((B, H), dtype=torch.float32, device="cuda")
    sel = torch.empty((B, H, max_k), dtype=torch.int32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(binding.sparf_workspace_bytes(B, H, D, max_len, max_k), dtype=torch.uint8, device="cuda")
    binding.set_sparse_path(path)
    try:
        binding.sparf_append(case.k_cache, case.v_cache, state.kt_pool, state.v_sum, case.k_new, case.v_new,
                             case.seq_lens, case.block_table, state.kt_block_table, flags)
        binding.sparf_decode_attention(out, alpha, sel, case.q, case.k_cache, case.v_cache, state.kt_pool,
                                       state.v_sum, case.block_table, state.kt_block_table, case.seq_lens,
                                       state.k_tokens, max_len, max_k, R, WINDOW, case.scale, ws, flags)
        torch.cuda.synchronize()
    finally:
        binding.set_sparse_path(0)
    assert int(flags.item()) == 0 and torch.isfinite(out.float()).all()
    problems = [(b, h, single_pair_problem(case, state, b, h)) for b, h in pairs]
    sel_host, out_host, alpha_host = sel.cpu().numpy(), out.cpu(), alpha.cpu().numpy()

    def one(item):
        b, h, pb = item
        return check_pair(pb, state.k_tokens_host[b], case.scale, sel_host[b, h], out_host[b:b + 1, h:h + 1],
                          float(alpha_host[b, h]), f"workload {index} pair {(b, h)}")

    with ThreadPoolExecutor(max_workers=8) as pool:          # the oracle releases the GIL inside its C call
        in_band = sum(pool.map(one, problems))
    decisions = sum(case.seq_lens_host[b] for b, _ in pairs)
    assert in_band <= max(8, decisions // 2000), f"the band holds {in_band} of {decisions} decisions"


def spread_pairs(batch, heads, count, seed):
    rng = np.random.default_rng(seed)
    flat = rng.choice(batch * heads, size=count, replace=False)
    must = [(0, 0), (batch - 1, heads - 1)]
    return must + [(int(i) // heads, int(i) % heads) for i in flat if (int(i) // heads, int(i) % heads) not in must][:count - 2]


def test_long_context_workload_sampled_pairs():
    free, _ = torch.cuda.mem_get_info()
    if free < 45 * 2 ** 30:
        pytest.skip("needs 45 GiB of free device memory")
    run_workload(3, spread_pairs(8, 40, 32, 3), 0)


def test_long_context_workload_with_1024_token_transposed_blocks():
    """The same workload with the transposed copy in 1024-token blocks."""
    run_workload(3, spread_pairs(8, 40, 16, 5), 0, kt_tokens=1024)


@pytest.mark.parametrize("path", [1, 2], ids=["chunk-parallel", "block-per-row"])
def test_16k_context_workload_sampled_pairs(path):
    free, _ = torch.cuda.mem_get_info()
    if free < 45 * 2 ** 30:
        pytest.skip("needs 45 GiB of free device memory")
    run_workload(2, spread_pairs(64, 40, 32, 2), path)
