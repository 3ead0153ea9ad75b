"""Runs the grouped-head / multi-token attention entry point on long-context paged cases,
for timing and profiling.  Each case holds about 1 GB of K and V (far beyond L2).

    python -m paper_2409_04992_b200.examples.grouped_cases            # all cases, timed
    python -m paper_2409_04992_b200.examples.grouped_cases gqa8 2     # one case, 2 launches
"""
import sys

import torch

from paper_2409_04992_b200 import binding, workloads as wl

CASES = {
    # name: batch, context, block_tokens, kv_heads, q_heads, q_tokens, head_dim
    "mha": (4, 16384, 16, 32, 32, 1, 128),
    "gqa8": (16, 16384, 16, 8, 64, 1, 128),
    "gqa4_4new": (16, 16384, 16, 8, 32, 4, 128),
    "d64": (8, 16384, 16, 32, 32, 1, 64),
    "d256": (4, 16384, 16, 16, 16, 1, 256),
}


def run(name: str, reps: int) -> None:
    batch, ctx, tokens, kv_heads, q_heads, q_tokens, dim = CASES[name]
    w = wl.Workload(name, 7, batch=batch, len_lo=ctx, len_hi=ctx, layout="paged",
                    block_tokens=tokens, heads=kv_heads, head_dim=dim)
    g = wl.generate_grouped(w, q_tokens, q_heads, device="cuda")
    c = g.base
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty_like(g.q)
    ws = torch.empty(binding.grouped_workspace_bytes(batch, q_tokens, q_heads, kv_heads, dim, ctx),
                     dtype=torch.uint8, device="cuda")
    binding.kv_append_bulk(c.k_cache, c.v_cache, g.k_new, g.v_new, c.seq_lens, g.new_lens,
                           c.block_table, flags)
    a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        binding.decode_attention_grouped(out, None, g.q, c.k_cache, c.v_cache, c.block_table,
                                         c.seq_lens, ctx, c.scale, ws, flags)
    z.record()
    torch.cuda.synchronize()
    kv_bytes = batch * ctx * kv_heads * dim * 4
    ms = a.elapsed_time(z) / reps
    print(f"{name}: {kv_bytes / 1e9:.2f} GB of K+V, {ms:.3f} ms per call (first calls included), "
          f"{kv_bytes / ms / 1e6:.0f} GB/s, status flags {int(flags.item())}")


if __name__ == "__main__":
    names = [sys.argv[1]] if len(sys.argv) > 1 else list(CASES)
    reps = int(sys.argv[2]) if len(sys.argv) > 2 else 20
    for n in names:
        run(n, reps)
        torch.cuda.empty_cache()
