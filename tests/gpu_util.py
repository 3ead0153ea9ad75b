"""Shared helpers of the GPU parity tests: run the CUDA path through the binding, run the
CPU oracle on the same bits, and compare under the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

from oracle import capi
from paper_2409_04992_b200 import binding, workloads as wl

MAX_ABS = 2e-3            # on fp16 outputs, every element
MAX_REL = 1e-2            # on elements whose exact value is a normal fp16 (|r| >= 2^-14)
REL_FLOOR = 2.0 ** -14
LSE_ATOL, LSE_RTOL = 1e-4, 1e-5
SENTINEL = 0x5A


def to_device(case: wl.Case, device="cuda") -> wl.Case:
    moved = {k: (v.to(device) if isinstance(v, torch.Tensor) else v) for k, v in case.__dict__.items()}
    return wl.Case(**moved)


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


class Guarded:
    """A device buffer with sentinel bytes on both sides, to catch writes outside it."""

    def __init__(self, shape, dtype, pad_bytes=4096):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.pad, self.n = pad_bytes, n
        self.raw = torch.full((n + 2 * pad_bytes,), SENTINEL, dtype=torch.uint8, device="cuda")
        self.view = self.raw[pad_bytes:pad_bytes + n].view(dtype).view(shape)

    def intact(self) -> bool:
        return bool((self.raw[:self.pad] == SENTINEL).all() and
                    (self.raw[self.pad + self.n:] == SENTINEL).all())


def gpu_step(case: wl.Case, do_append=True, chunk_tokens=0, max_seq_len=None, stream=None,
             want_lse=True):
    """append + attention on the GPU.  Returns (out fp16 [B,H,D] cpu, lse fp32 cpu, flags int)."""
    w = case.workload
    B, H, D = case.q.shape
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = Guarded((B, H, D), torch.float16)
    lse = Guarded((B, H), torch.float32)
    max_len = max_seq_len if max_seq_len is not None else max(case.max_seq_len, 1)
    binding.set_chunk_tokens(chunk_tokens)
    try:
        need = binding.workspace_bytes(B, H, D, max_len)
        ws = Guarded((need,), torch.uint8)
        if do_append:
            binding.kv_append(case.k_cache, case.v_cache, case.k_new, case.v_new, case.seq_lens,
                              case.block_table, flags, stream)
        if case.block_table is None:
            binding.decode_attention(out.view, lse.view if want_lse else None, case.q, case.k_cache,
                                     case.v_cache, case.seq_lens, max_len, case.scale, ws.view,
                                     flags, stream)
        else:
            binding.decode_attention_paged(out.view, lse.view if want_lse else None, case.q,
                                           case.k_cache, case.v_cache, case.block_table,
                                           case.seq_lens, max_len, case.scale, ws.view, flags, stream)
    finally:
        binding.set_chunk_tokens(0)
    torch.cuda.synchronize()
    assert out.intact() and lse.intact() and ws.intact(), "a kernel wrote outside its buffers"
    return out.view.cpu(), lse.view.cpu(), int(flags.item())


def oracle_step(case_cpu: wl.Case, do_append=True):
    """The same step on the CPU oracle; mutates case_cpu's caches like the GPU does."""
    k, v = case_cpu.k_cache.numpy(), case_cpu.v_cache.numpy()
    table = None if case_cpu.block_table is None else case_cpu.block_table.numpy()
    lens = np.array(case_cpu.seq_lens_host, dtype=np.int32)
    if do_append:
        capi.kv_append(k, v, case_cpu.k_new.numpy(), case_cpu.v_new.numpy(), lens, block_table=table)
    out, lse, _ = capi.decode_attention(case_cpu.q.numpy(), k, v, lens, case_cpu.scale, block_table=table)
    return out, lse


def errors(got_fp16: torch.Tensor, want: np.ndarray):
    g = got_fp16.numpy().astype(np.float64)
    diff = np.abs(g - want)
    big = np.abs(want) >= REL_FLOOR
    max_abs = float(diff.max()) if diff.size else 0.0
    max_rel = float((diff[big] / np.abs(want[big])).max()) if big.any() else 0.0
    return max_abs, max_rel


def assert_close(got_fp16, want, got_lse=None, want_lse=None, what=""):
    assert torch.isfinite(got_fp16.float()).all(), f"{what}: non-finite output"
    max_abs, max_rel = errors(got_fp16, want)
    assert max_abs <= MAX_ABS, f"{what}: max-abs {max_abs:.3e} > {MAX_ABS}"
    assert max_rel <= MAX_REL, f"{what}: max-rel {max_rel:.3e} > {MAX_REL}"
    if got_lse is not None:
        g = got_lse.numpy().astype(np.float64)
        fin = np.isfinite(want_lse)
        assert np.array_equal(np.isneginf(g), np.isneginf(want_lse)), f"{what}: lse -inf pattern"
        assert np.all(np.abs(g[fin] - want_lse[fin]) <= LSE_ATOL + LSE_RTOL * np.abs(want_lse[fin])), \
            f"{what}: lse off by {np.abs(g[fin] - want_lse[fin]).max():.3e}"
    return max_abs, max_rel
