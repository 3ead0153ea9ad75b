"""Runs the sparse (Algorithm 1) attention entry point on two small paged cases, for profiling:
(B=2, L=131072, T=64) and (B=16, L=16384, T=16), each with the transposed K copy in blocks of
T and of 256 tokens; r = 16, an eighth of the tokens kept.

    python -m paper_2409_04992_b200.examples.sparse_small_cases
"""
import torch

from paper_2409_04992_b200 import binding, workloads as wl


def run(w: wl.Workload, kt_block_tokens=None, r: int = 16, keep: float = 0.125, window: int = 16,
        reps: int = 2) -> None:
    case = wl.generate(w, device="cuda", poison=False)
    state = wl.make_sparf_state(case, keep, kt_block_tokens)
    B, H, D = case.q.shape
    max_len, max_k = case.max_seq_len, max(state.k_tokens_host)
    out = torch.empty((B, H, D), dtype=torch.float16, device="cuda")
    ws = torch.empty(binding.sparf_workspace_bytes(B, H, D, max_len, max_k), dtype=torch.uint8, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(reps):
        binding.sparf_decode_attention(out, None, None, case.q, case.k_cache, case.v_cache, state.kt_pool,
                                       state.v_sum, case.block_table, state.kt_block_table,
                                       case.seq_lens, state.k_tokens, max_len, max_k, r, window,
                                       case.scale, ws, flags)
    torch.cuda.synchronize()
    print(w.name, "kt block", state.kt_block_tokens, "status flags", int(flags.item()))


if __name__ == "__main__":
    for kt in (None, 256):
        run(wl.STANDARD[3].replace(batch=2, name="b2_ctx128k_paged64"), kt)
        torch.cuda.empty_cache()
        run(wl.STANDARD[2].replace(batch=16, name="b16_ctx16k_paged16"), kt)
        torch.cuda.empty_cache()
