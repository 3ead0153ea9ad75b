"""Thin ctypes layer over libinstinfer.so: argument marshalling only.

Function names mirror the C ABI (see include/instinfer.h for what each argument means).
Tensors are torch CUDA tensors used as device memory; every step of the path runs in the
library's kernels.  There is no fallback: if the library has not been built, loading fails.
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path
from typing import Optional, Sequence, Union

import torch

# INSTINFER_LIBRARY selects another build of the same library (the bounds-checking one, say).
LIBRARY = Path(os.environ.get("INSTINFER_LIBRARY") or Path(__file__).resolve().parent / "libinstinfer.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA = range(5)
FLAG_SEQ_LEN_RANGE, FLAG_BLOCK_RANGE, FLAG_COPY_TIMEOUT, FLAG_BOUNDS_CHECK = 1, 2, 4, 8
STATIC_WORKSPACE_BYTES = 16 << 20

_lib: Optional[ctypes.CDLL] = None


class InstInferError(RuntimeError):
    def __init__(self, status: int):
        super().__init__(f"instinfer status {status}: {status_string(status)}")
        self.status = status


def load() -> ctypes.CDLL:
    """dlopen the CUDA library; raises if it is missing (build it with paper_2409_04992_b200.build)."""
    global _lib
    if _lib is None:
        if not LIBRARY.exists():
            raise RuntimeError(f"{LIBRARY} is missing: run `python -m paper_2409_04992_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(str(LIBRARY))
        i32, i64, ptr, f32, sz = (ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p,
                                  ctypes.c_float, ctypes.c_size_t)
        lib.instinfer_kv_append.restype = ctypes.c_int
        lib.instinfer_kv_append.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i64,
                                            i32, i32, i32, i32, ptr, ptr]
        lib.instinfer_kv_append_bulk.restype = ctypes.c_int
        lib.instinfer_kv_append_bulk.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i64,
                                                 i32, i32, i32, i32, i32, ptr, ptr]
        lib.instinfer_decode_attention.restype = ctypes.c_int
        lib.instinfer_decode_attention.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i32,
                                                   i32, i32, f32, ptr, sz, ptr, ptr]
        lib.instinfer_decode_attention_paged.restype = ctypes.c_int
        lib.instinfer_decode_attention_paged.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr,
                                                         i32, i32, i32, i32, i32, i64, i32, f32,
                                                         ptr, sz, ptr, ptr]
        lib.instinfer_decode_attention_static.restype = ctypes.c_int
        lib.instinfer_decode_attention_static.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr,
                                                          i32, i32, i32, i32, i32, i32, i64, i32,
                                                          f32, ptr, ptr]
        lib.instinfer_decode_attention_allgather.restype = ctypes.c_int
        lib.instinfer_decode_attention_allgather.argtypes = [ptr, i32, ptr, ptr, ptr, ptr, ptr, ptr,
                                                             i32, i32, i32, i32, i32, i32, i32, i32,
                                                             i64, i32, f32, ptr, sz, ptr, ptr]
        lib.instinfer_allgather_workspace_bytes.restype = sz
        lib.instinfer_allgather_workspace_bytes.argtypes = [i32, i32, i32, i32]
        lib.instinfer_decode_attention_grouped.restype = ctypes.c_int
        lib.instinfer_decode_attention_grouped.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr,
                                                           i32, i32, i32, i32, i32, i32, i32, i32,
                                                           i64, i32, f32, ptr, sz, ptr, ptr]
        lib.instinfer_grouped_workspace_bytes.restype = sz
        lib.instinfer_grouped_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32]
        lib.instinfer_decode_step_host.restype = ctypes.c_int
        lib.instinfer_decode_step_host.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr,
                                                   i32, i32, i64, i32, i32, i32, i32, i32, f32,
                                                   ptr, sz, ptr, ptr]
        lib.instinfer_decode_step_host_overlapped.restype = ctypes.c_int
        lib.instinfer_decode_step_host_overlapped.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr,
                                                              i32, i32, i64, i32, i32, i32, i32, i32, f32,
                                                              ptr, sz, ptr, ptr, ptr, ptr, ptr, ptr]
        lib.instinfer_sparf_append.restype = ctypes.c_int
        lib.instinfer_sparf_append.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i64,
                                               ptr, i32, i32, i64, i32, i32, i32, ptr, ptr]
        lib.instinfer_sparf_append_bulk.restype = ctypes.c_int
        lib.instinfer_sparf_append_bulk.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32,
                                                    i64, ptr, i32, i32, i64, i32, i32, i32, i32, ptr, ptr]
        lib.instinfer_sparf_decode_attention.restype = ctypes.c_int
        lib.instinfer_sparf_decode_attention.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr,
                                                         ptr, ptr, i32, i32, i32, i32, i32, i64,
                                                         ptr, i32, i32, i64,
                                                         i32, i32, i32, i32, f32, ptr, sz, ptr, ptr]
        lib.instinfer_set_sparse_path.restype = ctypes.c_int
        lib.instinfer_set_sparse_path.argtypes = [i32]
        lib.instinfer_set_grouped_path.restype = ctypes.c_int
        lib.instinfer_set_grouped_path.argtypes = [i32]
        lib.instinfer_grouped_path_for.restype = i32
        lib.instinfer_grouped_path_for.argtypes = [i32, i32]
        lib.instinfer_sparf_workspace_bytes.restype = sz
        lib.instinfer_sparf_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
        lib.instinfer_workspace_bytes.restype = sz
        lib.instinfer_workspace_bytes.argtypes = [i32, i32, i32, i32]
        lib.instinfer_plan_chunk_tokens.restype = i32
        lib.instinfer_plan_chunk_tokens.argtypes = [i32, i32, i32]
        lib.instinfer_plan_num_splits.restype = i32
        lib.instinfer_plan_num_splits.argtypes = [i32, i32, i32]
        lib.instinfer_plan_merges_in_cluster.restype = i32
        lib.instinfer_plan_merges_in_cluster.argtypes = [i32, i32, i32]
        lib.instinfer_set_chunk_tokens.restype = ctypes.c_int
        lib.instinfer_set_chunk_tokens.argtypes = [i32]
        lib.instinfer_set_timing_events.restype = ctypes.c_int
        lib.instinfer_set_timing_events.argtypes = [ptr, ptr]
        lib.instinfer_status_string.restype = ctypes.c_char_p
        lib.instinfer_status_string.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream or None


def _check(status: int) -> None:
    if status != OK:
        raise InstInferError(status)


def status_string(status: int) -> str:
    return load().instinfer_status_string(int(status)).decode()


def workspace_bytes(batch: int, heads: int, head_dim: int, max_seq_len: int) -> int:
    return int(load().instinfer_workspace_bytes(batch, heads, head_dim, max_seq_len))


def plan_chunk_tokens(batch: int, heads: int, max_seq_len: int) -> int:
    return int(load().instinfer_plan_chunk_tokens(batch, heads, max_seq_len))


def plan_num_splits(batch: int, heads: int, max_seq_len: int) -> int:
    return int(load().instinfer_plan_num_splits(batch, heads, max_seq_len))


def plan_merges_in_cluster(batch: int, heads: int, max_seq_len: int) -> bool:
    return bool(load().instinfer_plan_merges_in_cluster(batch, heads, max_seq_len))


def set_chunk_tokens(chunk_tokens: int) -> None:
    _check(load().instinfer_set_chunk_tokens(int(chunk_tokens)))


def set_timing_events(before_split: Optional[torch.cuda.Event],
                      after_split: Optional[torch.cuda.Event]) -> None:
    """instinfer_set_timing_events with torch events (already created, i.e. recorded once)."""
    _check(load().instinfer_set_timing_events(
        None if before_split is None else before_split.cuda_event,
        None if after_split is None else after_split.cuda_event))


def kv_append(k_cache: torch.Tensor, v_cache: torch.Tensor, k_new: torch.Tensor,
              v_new: torch.Tensor, seq_lens: torch.Tensor,
              block_table: Optional[torch.Tensor] = None,
              status_flags: Optional[torch.Tensor] = None,
              stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_kv_append.  Caches: [B,H,s_max,D] (block_table None) or pools [P,H,T,D]."""
    batch, heads, head_dim = k_new.shape
    if block_table is None:
        max_blocks, block_tokens, phys, s_max = 0, 0, 0, k_cache.shape[2]
    else:
        max_blocks, block_tokens, phys, s_max = (block_table.shape[1], k_cache.shape[2],
                                                 k_cache.shape[0], 0)
    _check(load().instinfer_kv_append(
        _ptr(k_cache), _ptr(v_cache), _ptr(k_new), _ptr(v_new), _ptr(seq_lens),
        _ptr(block_table), max_blocks, block_tokens, phys, batch, heads, head_dim, s_max,
        _ptr(status_flags), _stream(stream)))


def kv_append_bulk(k_cache: torch.Tensor, v_cache: torch.Tensor, k_new: torch.Tensor,
                   v_new: torch.Tensor, seq_lens: torch.Tensor, new_lens: torch.Tensor,
                   block_table: Optional[torch.Tensor] = None,
                   status_flags: Optional[torch.Tensor] = None,
                   stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_kv_append_bulk: k_new, v_new are [B, max_new, H, D] (token-major)."""
    batch, max_new, heads, head_dim = k_new.shape
    if block_table is None:
        max_blocks, block_tokens, phys, s_max = 0, 0, 0, k_cache.shape[2]
    else:
        max_blocks, block_tokens, phys, s_max = (block_table.shape[1], k_cache.shape[2],
                                                 k_cache.shape[0], 0)
    _check(load().instinfer_kv_append_bulk(
        _ptr(k_cache), _ptr(v_cache), _ptr(k_new), _ptr(v_new), _ptr(seq_lens), _ptr(new_lens),
        _ptr(block_table), max_blocks, block_tokens, phys, batch, max_new, heads, head_dim, s_max,
        _ptr(status_flags), _stream(stream)))


def decode_attention(out: torch.Tensor, lse: Optional[torch.Tensor], q: torch.Tensor,
                     k_cache: torch.Tensor, v_cache: torch.Tensor, seq_lens: torch.Tensor,
                     max_seq_len: int, scale: float, workspace: torch.Tensor,
                     status_flags: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_decode_attention over contiguous caches [B,H,s_max,D]."""
    batch, heads, head_dim = q.shape
    _check(load().instinfer_decode_attention(
        _ptr(out), _ptr(lse), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(seq_lens),
        batch, heads, head_dim, k_cache.shape[2], int(max_seq_len), float(scale),
        _ptr(workspace), workspace.numel() * workspace.element_size(),
        _ptr(status_flags), _stream(stream)))


def decode_attention_paged(out: torch.Tensor, lse: Optional[torch.Tensor], q: torch.Tensor,
                           k_pool: torch.Tensor, v_pool: torch.Tensor,
                           block_table: torch.Tensor, seq_lens: torch.Tensor,
                           max_seq_len: int, scale: float, workspace: torch.Tensor,
                           status_flags: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_decode_attention_paged over pools [P,H,T,D] with block_table [B,M]."""
    batch, heads, head_dim = q.shape
    _check(load().instinfer_decode_attention_paged(
        _ptr(out), _ptr(lse), _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
        _ptr(seq_lens), batch, heads, head_dim, k_pool.shape[2], block_table.shape[1],
        k_pool.shape[0], int(max_seq_len), float(scale), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream(stream)))


def decode_attention_static(out: torch.Tensor, lse: Optional[torch.Tensor], q: torch.Tensor,
                            k_cache: torch.Tensor, v_cache: torch.Tensor,
                            block_table: Optional[torch.Tensor], seq_lens: torch.Tensor,
                            max_seq_len: int, scale: float,
                            status_flags: Optional[torch.Tensor] = None,
                            stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_decode_attention_static: attention in the library's built-in scratch array,
    for callers that cannot provide a workspace (block_table None = contiguous caches)."""
    batch, heads, head_dim = q.shape
    if block_table is None:
        s_max, block_tokens, max_blocks, phys = k_cache.shape[2], 0, 0, 0
    else:
        s_max, block_tokens, max_blocks, phys = (0, k_cache.shape[2], block_table.shape[1],
                                                 k_cache.shape[0])
    _check(load().instinfer_decode_attention_static(
        _ptr(out), _ptr(lse), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
        _ptr(seq_lens), batch, heads, head_dim, s_max, block_tokens, max_blocks, phys,
        int(max_seq_len), float(scale), _ptr(status_flags), _stream(stream)))


def allgather_workspace_bytes(batch: int, heads: int, head_dim: int, max_seq_len: int) -> int:
    return int(load().instinfer_allgather_workspace_bytes(batch, heads, head_dim, max_seq_len))


def decode_attention_allgather(out_all: Sequence[Union[torch.Tensor, int]], lse: Optional[torch.Tensor],
                               q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                               block_table: Optional[torch.Tensor], seq_lens: torch.Tensor,
                               head_offset: int, total_heads: int, max_seq_len: int, scale: float,
                               workspace: torch.Tensor,
                               status_flags: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_decode_attention_allgather: this rank's head shard (q [B, heads, D]), output
    rows stored into every rank's [B, total_heads, D] buffer.  out_all holds one entry per
    rank, a tensor or a raw device address of a peer mapping."""
    batch, heads, head_dim = q.shape
    if block_table is None:
        s_max, block_tokens, max_blocks, phys = k_cache.shape[2], 0, 0, 0
    else:
        s_max, block_tokens, max_blocks, phys = (0, k_cache.shape[2], block_table.shape[1],
                                                 k_cache.shape[0])
    addresses = [t.data_ptr() if isinstance(t, torch.Tensor) else int(t) for t in out_all]
    table = (ctypes.c_void_p * len(addresses))(*addresses)
    _check(load().instinfer_decode_attention_allgather(
        table, len(addresses), _ptr(lse), _ptr(q), _ptr(k_cache), _ptr(v_cache),
        _ptr(block_table), _ptr(seq_lens), batch, heads, int(head_offset), int(total_heads),
        head_dim, s_max, block_tokens, max_blocks, phys, int(max_seq_len), float(scale),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status_flags),
        _stream(stream)))


def grouped_workspace_bytes(batch: int, q_tokens: int, q_heads: int, kv_heads: int, head_dim: int,
                            max_seq_len: int) -> int:
    return int(load().instinfer_grouped_workspace_bytes(batch, q_tokens, q_heads, kv_heads,
                                                        head_dim, max_seq_len))


def decode_attention_grouped(out: torch.Tensor, lse: Optional[torch.Tensor], q: torch.Tensor,
                             k_cache: torch.Tensor, v_cache: torch.Tensor,
                             block_table: Optional[torch.Tensor], seq_lens: torch.Tensor,
                             max_seq_len: int, scale: float, workspace: torch.Tensor,
                             status_flags: Optional[torch.Tensor] = None,
                             stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_decode_attention_grouped: q, out [B, Tq, Hq, D]; caches with Hkv heads
    ([B,Hkv,s_max,D], or pools [P,Hkv,T,D] with block_table)."""
    batch, q_tokens, q_heads, head_dim = q.shape
    kv_heads = k_cache.shape[1]
    if block_table is None:
        s_max, block_tokens, max_blocks, phys = k_cache.shape[2], 0, 0, 0
    else:
        s_max, block_tokens, max_blocks, phys = (0, k_cache.shape[2], block_table.shape[1],
                                                 k_cache.shape[0])
    _check(load().instinfer_decode_attention_grouped(
        _ptr(out), _ptr(lse), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
        _ptr(seq_lens), batch, q_tokens, q_heads, kv_heads, head_dim, s_max, block_tokens,
        max_blocks, phys, int(max_seq_len), float(scale), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream(stream)))


def decode_step_host(out_host: torch.Tensor, qkv_host: torch.Tensor, qkv_dev: torch.Tensor,
                     out_dev: torch.Tensor, lse: Optional[torch.Tensor], k_cache: torch.Tensor,
                     v_cache: torch.Tensor, seq_lens: torch.Tensor,
                     block_table: Optional[torch.Tensor], max_seq_len: int, scale: float,
                     workspace: torch.Tensor, status_flags: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_decode_step_host: qkv_host [3,B,H,D] and out_host [B,H,D] are (pinned) host
    tensors, qkv_dev / out_dev device staging buffers of the same shapes."""
    _, batch, heads, head_dim = qkv_host.shape
    if block_table is None:
        max_blocks, block_tokens, phys, s_max = 0, 0, 0, k_cache.shape[2]
    else:
        max_blocks, block_tokens, phys, s_max = (block_table.shape[1], k_cache.shape[2],
                                                 k_cache.shape[0], 0)
    _check(load().instinfer_decode_step_host(
        _ptr(out_host), _ptr(qkv_host), _ptr(qkv_dev), _ptr(out_dev), _ptr(lse), _ptr(k_cache),
        _ptr(v_cache), _ptr(seq_lens), _ptr(block_table), max_blocks, block_tokens, phys, batch,
        heads, head_dim, s_max, int(max_seq_len), float(scale), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream(stream)))


def decode_step_host_overlapped(out_host: torch.Tensor, qkv_host: torch.Tensor, qkv_dev: torch.Tensor,
                                out_dev: torch.Tensor, lse: Optional[torch.Tensor], k_cache: torch.Tensor,
                                v_cache: torch.Tensor, seq_lens: torch.Tensor,
                                block_table: Optional[torch.Tensor], max_seq_len: int, scale: float,
                                workspace: torch.Tensor, status_flags: Optional[torch.Tensor],
                                compute: torch.cuda.Stream, upload: torch.cuda.Stream,
                                download: torch.cuda.Stream, uploaded: torch.cuda.Event,
                                attended: torch.cuda.Event) -> None:
    """instinfer_decode_step_host_overlapped: as decode_step_host, with the upload on `upload`
    and the download on `download`; `uploaded` and `attended` are events that have been
    recorded at least once (torch creates the CUDA event at its first record)."""
    _, batch, heads, head_dim = qkv_host.shape
    if block_table is None:
        max_blocks, block_tokens, phys, s_max = 0, 0, 0, k_cache.shape[2]
    else:
        max_blocks, block_tokens, phys, s_max = (block_table.shape[1], k_cache.shape[2],
                                                 k_cache.shape[0], 0)
    _check(load().instinfer_decode_step_host_overlapped(
        _ptr(out_host), _ptr(qkv_host), _ptr(qkv_dev), _ptr(out_dev), _ptr(lse), _ptr(k_cache),
        _ptr(v_cache), _ptr(seq_lens), _ptr(block_table), max_blocks, block_tokens, phys, batch,
        heads, head_dim, s_max, int(max_seq_len), float(scale), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status_flags), compute.cuda_stream or None,
        upload.cuda_stream or None, download.cuda_stream or None, uploaded.cuda_event or None,
        attended.cuda_event or None))


def sparf_append(k_pool: torch.Tensor, v_pool: torch.Tensor, kt_pool: torch.Tensor,
                 v_sum: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                 seq_lens: torch.Tensor, block_table: torch.Tensor, kt_block_table: torch.Tensor,
                 status_flags: Optional[torch.Tensor] = None,
                 stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_sparf_append: pools [P,H,T,D], kt_pool [Pk,H,D,Tk] with kt_block_table [B,Mk],
    v_sum fp32 [B,H,D]."""
    batch, heads, head_dim = k_new.shape
    _check(load().instinfer_sparf_append(
        _ptr(k_pool), _ptr(v_pool), _ptr(kt_pool), _ptr(v_sum), _ptr(k_new), _ptr(v_new),
        _ptr(seq_lens), _ptr(block_table), block_table.shape[1], k_pool.shape[2], k_pool.shape[0],
        _ptr(kt_block_table), kt_block_table.shape[1], kt_pool.shape[3], kt_pool.shape[0],
        batch, heads, head_dim, _ptr(status_flags), _stream(stream)))


def sparf_append_bulk(k_pool: torch.Tensor, v_pool: torch.Tensor, kt_pool: torch.Tensor,
                      v_sum: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                      seq_lens: torch.Tensor, new_lens: torch.Tensor, block_table: torch.Tensor,
                      kt_block_table: torch.Tensor, status_flags: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_sparf_append_bulk: k_new, v_new are [B, max_new, H, D] (token-major)."""
    batch, max_new, heads, head_dim = k_new.shape
    _check(load().instinfer_sparf_append_bulk(
        _ptr(k_pool), _ptr(v_pool), _ptr(kt_pool), _ptr(v_sum), _ptr(k_new), _ptr(v_new),
        _ptr(seq_lens), _ptr(new_lens), _ptr(block_table), block_table.shape[1], k_pool.shape[2],
        k_pool.shape[0], _ptr(kt_block_table), kt_block_table.shape[1], kt_pool.shape[3],
        kt_pool.shape[0], batch, max_new, heads, head_dim, _ptr(status_flags), _stream(stream)))


def grouped_path_for(head_dim: int, block_tokens: int) -> int:
    """instinfer_grouped_path_for: 1 warp-level MMAs, 2 tcgen05, 0 unsupported (block_tokens 0: contiguous)."""
    return int(load().instinfer_grouped_path_for(int(head_dim), int(block_tokens)))


def set_grouped_path(path: int) -> None:
    """instinfer_set_grouped_path: 0 automatic, 1 warp-level MMAs, 2 tcgen05 where the shape allows."""
    _check(load().instinfer_set_grouped_path(int(path)))


def set_sparse_path(path: int) -> None:
    """instinfer_set_sparse_path: 0 automatic, 1 chunk-parallel, 2 one block per row."""
    _check(load().instinfer_set_sparse_path(int(path)))


def sparf_workspace_bytes(batch: int, heads: int, head_dim: int, max_seq_len: int, max_k: int) -> int:
    return int(load().instinfer_sparf_workspace_bytes(batch, heads, head_dim, max_seq_len, max_k))


def sparf_decode_attention(out: torch.Tensor, alpha: Optional[torch.Tensor],
                           selected: Optional[torch.Tensor], q: torch.Tensor,
                           k_pool: torch.Tensor, v_pool: torch.Tensor, kt_pool: torch.Tensor,
                           v_sum: torch.Tensor, block_table: torch.Tensor,
                           kt_block_table: torch.Tensor, seq_lens: torch.Tensor,
                           k_tokens: torch.Tensor, max_seq_len: int, max_k: int, r: int,
                           local_window: int, scale: float, workspace: torch.Tensor,
                           status_flags: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> None:
    """instinfer_sparf_decode_attention (Algorithm 1) over paged pools."""
    batch, heads, head_dim = q.shape
    _check(load().instinfer_sparf_decode_attention(
        _ptr(out), _ptr(alpha), _ptr(selected), _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(kt_pool),
        _ptr(v_sum), _ptr(block_table), _ptr(seq_lens), _ptr(k_tokens), batch, heads, head_dim,
        k_pool.shape[2], block_table.shape[1], k_pool.shape[0],
        _ptr(kt_block_table), kt_block_table.shape[1], kt_pool.shape[3], kt_pool.shape[0],
        int(max_seq_len), int(max_k), int(r), int(local_window), float(scale), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream(stream)))


def alloc_workspace(batch: int, heads: int, head_dim: int, max_seq_len: int,
                    device: torch.device | str = "cuda") -> torch.Tensor:
    """A byte tensor of the size the library asks for under the current split plan."""
    need = workspace_bytes(batch, heads, head_dim, max_seq_len)
    if need == 0:
        raise InstInferError(ERR_INVALID_ARG)
    return torch.empty(need, dtype=torch.uint8, device=device)
