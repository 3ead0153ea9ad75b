"""Sparse path at the full size of the long-context workload (8 x 40 heads x 131072 tokens,
K/V pages of 64 tokens, transposed copy in 256-token blocks), in the configuration the
benchmark times.  The oracle recomputes sampled (sequence, head) pairs one by one from rows
gathered off the device into single-pair pools; kept sets must match exactly."""
import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


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
                table=np.arange(blocks, dtype=np.int32)[None], kt_table=np.arange(kt_blocks, dtype=np.int32)[None])


def test_long_context_workload_sampled_pairs():
    free, _ = torch.cuda.mem_get_info()
    if free < 45 * 2 ** 30:
        pytest.skip("needs 45 GiB of free device memory")
    case = wl.generate(wl.STANDARD[3], device="cuda", poison=False)
    state = wl.make_sparf_state(case, 0.125, 256)
    B, H, D = case.q.shape
    max_len, max_k = case.max_seq_len, max(state.k_tokens_host)
    out = torch.empty((B, H, D), dtype=torch.float16, device="cuda")
    alpha = torch.empty((B, H), dtype=torch.float32, device="cuda")
    sel = torch.empty((B, H, max_k), dtype=torch.int32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(binding.sparf_workspace_bytes(B, H, D, max_len, max_k), dtype=torch.uint8, device="cuda")
    binding.sparf_append(case.k_cache, case.v_cache, state.kt_pool, state.v_sum, case.k_new, case.v_new,
                         case.seq_lens, case.block_table, state.kt_block_table, flags)
    binding.sparf_decode_attention(out, alpha, sel, case.q, case.k_cache, case.v_cache, state.kt_pool,
                                   state.v_sum, case.block_table, state.kt_block_table, case.seq_lens,
                                   state.k_tokens, max_len, max_k, 16, 16, case.scale, ws, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0 and torch.isfinite(out.float()).all()
    for b, h in [(0, 0), (3, 17), (7, 39)]:
        pb = single_pair_problem(case, state, b, h)
        want, want_alpha, want_sel, _ = capi.sparf_attention(
            pb["q"], pb["k"], pb["v"], pb["kt"], pb["v_sum"], pb["lens"], np.array([state.k_tokens_host[b]]),
            pb["table"], 16, 16, case.scale, kt_block_table=pb["kt_table"])
        assert np.array_equal(sel[b, h].cpu().numpy()[:want_sel.shape[2]], want_sel[0, 0]), (b, h)
        gu.assert_close(out[b:b + 1, h:h + 1].cpu(), want, what=f"pair {(b, h)}")
        assert abs(float(alpha[b, h]) - want_alpha[0, 0]) <= 2e-5
