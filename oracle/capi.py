"""ctypes front end of the C oracle (test infrastructure; the product never imports this).

Arrays are numpy: fp16 data travels as uint16 bit patterns so nothing is converted on the
way in, results come back as float64.
"""
from __future__ import annotations

import ctypes
from typing import Optional

import numpy as np

from . import build as _build

_lib = None


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(_build.build()))
        i32, i64, ptr = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_num_threads.argtypes = []
        lib.oracle_kv_append.restype = ctypes.c_int
        lib.oracle_kv_append.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i64,
                                         i32, i32, i32, i32]
        lib.oracle_decode_attention.restype = ctypes.c_int
        lib.oracle_decode_attention.argtypes = [ptr, ptr, ptr, i64, ptr, ptr, ptr, ptr, ptr,
                                                i32, i32, i64, i32, i32, i32, i32,
                                                ctypes.c_float]
        lib.oracle_decode_attention_grouped.restype = ctypes.c_int
        lib.oracle_decode_attention_grouped.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32,
                                                        i64, i32, i32, i32, i32, i32, i32,
                                                        ctypes.c_float]
        lib.oracle_kv_append_bulk.restype = ctypes.c_int
        lib.oracle_kv_append_bulk.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i64,
                                              i32, i32, i32, i32, i32]
        lib.oracle_sparf_append.restype = ctypes.c_int
        lib.oracle_sparf_append.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32, i64,
                                            ptr, i32, i32, i64, i32, i32, i32]
        lib.oracle_sparf_append_bulk.restype = ctypes.c_int
        lib.oracle_sparf_append_bulk.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, i32, i32,
                                                 i64, ptr, i32, i32, i64, i32, i32, i32, i32]
        lib.oracle_sparf_attention.restype = ctypes.c_int
        lib.oracle_sparf_attention.argtypes = [ptr, ptr, ptr, i64, ptr, ptr, i64, ptr, ptr, ptr, ptr,
                                               ptr, ptr, ptr, ptr, i32, i32, i64, ptr, i32, i32, i64,
                                               i32, i32, i32, i32, i32, ctypes.c_float]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's (sequence, head) loop runs on."""
    return int(_load().oracle_num_threads())


def _bits(a: np.ndarray, writable: bool = False) -> np.ndarray:
    """View an fp16 / uint16 array as contiguous uint16 bit patterns (no copy if possible)."""
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError(f"expected float16 or uint16 bits, got {a.dtype}")
    if not a.flags.c_contiguous or (writable and not a.flags.writeable):
        raise ValueError("oracle arrays must be C-contiguous (and writable where mutated)")
    return a


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


class OracleError(RuntimeError):
    """Raised with the C oracle's negative return code."""

    def __init__(self, code: int):
        super().__init__({-1: "bad argument", -2: "seq_len out of range",
                          -3: "block id out of range"}.get(code, f"code {code}"))
        self.code = code


def _table(block_table, batch):
    if block_table is None:
        return None, 0
    t = np.ascontiguousarray(block_table, dtype=np.int32)
    if t.ndim != 2 or t.shape[0] != batch:
        raise ValueError("block_table must be [batch, max_blocks_per_seq]")
    return t, t.shape[1]


def kv_append(k_cache: np.ndarray, v_cache: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
              seq_lens: np.ndarray, block_table: Optional[np.ndarray] = None) -> None:
    """In-place append of the new token's k,v at logical position seq_lens[b]-1.

    contiguous: caches are [B,H,s_max,D]; paged: pools are [P,H,T,D] and block_table [B,M].
    """
    kb, vb = _bits(k_cache, True), _bits(v_cache, True)
    kn, vn = _bits(np.ascontiguousarray(k_new)), _bits(np.ascontiguousarray(v_new))
    batch, heads, head_dim = kn.shape
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    if table is None:
        s_max, block_tokens, phys = kb.shape[2], 0, 0
    else:
        s_max, block_tokens, phys = 0, kb.shape[2], kb.shape[0]
    rc = _load().oracle_kv_append(_p(kb), _p(vb), _p(kn), _p(vn), _p(lens), _p(table),
                                  max_blocks, block_tokens, phys, batch, heads, head_dim, s_max)
    if rc:
        raise OracleError(rc)


def kv_append_bulk(k_cache: np.ndarray, v_cache: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                   seq_lens: np.ndarray, new_lens: np.ndarray,
                   block_table: Optional[np.ndarray] = None) -> None:
    """In-place append of new_lens[b] tokens per sequence; k_new, v_new are [B,N,H,D]."""
    kb, vb = _bits(k_cache, True), _bits(v_cache, True)
    kn, vn = _bits(np.ascontiguousarray(k_new)), _bits(np.ascontiguousarray(v_new))
    batch, max_new, heads, head_dim = kn.shape
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    news = np.ascontiguousarray(new_lens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    if table is None:
        s_max, block_tokens, phys = kb.shape[2], 0, 0
    else:
        s_max, block_tokens, phys = 0, kb.shape[2], kb.shape[0]
    rc = _load().oracle_kv_append_bulk(_p(kb), _p(vb), _p(kn), _p(vn), _p(lens), _p(news), _p(table),
                                       max_blocks, block_tokens, phys, batch, max_new, heads,
                                       head_dim, s_max)
    if rc:
        raise OracleError(rc)


def decode_attention(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                     seq_lens: np.ndarray, scale: float,
                     block_table: Optional[np.ndarray] = None, want_weights: bool = False):
    """softmax(scale * q K^T) V per (sequence, head) in fp64.

    Returns (out [B,H,D] float64, lse [B,H] float64, weights [B,H,max(seq_lens)] or None).
    """
    qb = _bits(np.ascontiguousarray(q))
    kb, vb = _bits(k_cache), _bits(v_cache)
    batch, heads, head_dim = qb.shape
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    if table is None:
        s_max, block_tokens, phys = kb.shape[2], 0, 0
    else:
        s_max, block_tokens, phys = 0, kb.shape[2], kb.shape[0]
    out = np.zeros((batch, heads, head_dim), dtype=np.float64)
    lse = np.zeros((batch, heads), dtype=np.float64)
    weights, stride = None, 0
    if want_weights:
        stride = int(lens.max()) if batch else 0
        weights = np.zeros((batch, heads, max(stride, 1)), dtype=np.float64)
        stride = max(stride, 1)
    rc = _load().oracle_decode_attention(_p(out), _p(lse), _p(weights), stride, _p(qb), _p(kb),
                                         _p(vb), _p(lens), _p(table), max_blocks, block_tokens,
                                         phys, batch, heads, head_dim, s_max,
                                         ctypes.c_float(scale))
    if rc:
        raise OracleError(rc)
    return out, lse, weights


def decode_attention_grouped(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                             seq_lens: np.ndarray, scale: float,
                             block_table: Optional[np.ndarray] = None):
    """Grouped-head, multi-token decode attention in fp64: q [B,Tq,Hq,D], caches with Hkv heads
    (Hq a multiple of Hkv); new token t sees positions [0, seq_lens[b] - (Tq-1-t)).

    Returns (out [B,Tq,Hq,D] float64, lse [B,Tq,Hq] float64).
    """
    qb = _bits(np.ascontiguousarray(q))
    kb, vb = _bits(k_cache), _bits(v_cache)
    batch, q_tokens, q_heads, head_dim = qb.shape
    kv_heads = kb.shape[1]
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    if table is None:
        s_max, block_tokens, phys = kb.shape[2], 0, 0
    else:
        s_max, block_tokens, phys = 0, kb.shape[2], kb.shape[0]
    out = np.zeros((batch, q_tokens, q_heads, head_dim), dtype=np.float64)
    lse = np.zeros((batch, q_tokens, q_heads), dtype=np.float64)
    rc = _load().oracle_decode_attention_grouped(_p(out), _p(lse), _p(qb), _p(kb), _p(vb), _p(lens),
                                                 _p(table), max_blocks, block_tokens, phys, batch,
                                                 q_tokens, q_heads, kv_heads, head_dim, s_max,
                                                 ctypes.c_float(scale))
    if rc:
        raise OracleError(rc)
    return out, lse


def sparf_append(k_pool: np.ndarray, v_pool: np.ndarray, kt_pool: np.ndarray, v_sum: np.ndarray,
                 k_new: np.ndarray, v_new: np.ndarray, seq_lens: np.ndarray,
                 block_table: np.ndarray, kt_block_table: Optional[np.ndarray] = None) -> None:
    """In-place append for the SparF state: pools [P,H,T,D], K^T pool [Pk,H,D,Tk] with its own
    table (default: the K/V table, i.e. Tk == T), v_sum f32 [B,H,D]."""
    kb, vb, ktb = _bits(k_pool, True), _bits(v_pool, True), _bits(kt_pool, True)
    kn, vn = _bits(np.ascontiguousarray(k_new)), _bits(np.ascontiguousarray(v_new))
    if v_sum.dtype != np.float32 or not v_sum.flags.c_contiguous:
        raise TypeError("v_sum must be contiguous float32")
    batch, heads, head_dim = kn.shape
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    kt_table, kt_max_blocks = _table(block_table if kt_block_table is None else kt_block_table, batch)
    rc = _load().oracle_sparf_append(_p(kb), _p(vb), _p(ktb), _p(v_sum), _p(kn), _p(vn), _p(lens),
                                     _p(table), max_blocks, kb.shape[2], kb.shape[0],
                                     _p(kt_table), kt_max_blocks, ktb.shape[3], ktb.shape[0],
                                     batch, heads, head_dim)
    if rc:
        raise OracleError(rc)


def sparf_append_bulk(k_pool: np.ndarray, v_pool: np.ndarray, kt_pool: np.ndarray, v_sum: np.ndarray,
                      k_new: np.ndarray, v_new: np.ndarray, seq_lens: np.ndarray, new_lens: np.ndarray,
                      block_table: np.ndarray, kt_block_table: Optional[np.ndarray] = None) -> None:
    """In-place bulk append for the SparF state; k_new, v_new are [B,N,H,D]."""
    kb, vb, ktb = _bits(k_pool, True), _bits(v_pool, True), _bits(kt_pool, True)
    kn, vn = _bits(np.ascontiguousarray(k_new)), _bits(np.ascontiguousarray(v_new))
    if v_sum.dtype != np.float32 or not v_sum.flags.c_contiguous:
        raise TypeError("v_sum must be contiguous float32")
    batch, max_new, heads, head_dim = kn.shape
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    news = np.ascontiguousarray(new_lens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    kt_table, kt_max_blocks = _table(block_table if kt_block_table is None else kt_block_table, batch)
    rc = _load().oracle_sparf_append_bulk(_p(kb), _p(vb), _p(ktb), _p(v_sum), _p(kn), _p(vn), _p(lens),
                                          _p(news), _p(table), max_blocks, kb.shape[2], kb.shape[0],
                                          _p(kt_table), kt_max_blocks, ktb.shape[3], ktb.shape[0],
                                          batch, max_new, heads, head_dim)
    if rc:
        raise OracleError(rc)


def sparf_attention(q: np.ndarray, k_pool: np.ndarray, v_pool: np.ndarray, kt_pool: np.ndarray,
                    v_sum: np.ndarray, seq_lens: np.ndarray, k_tokens: np.ndarray,
                    block_table: np.ndarray, r: int, l: int, scale: float,
                    given: Optional[np.ndarray] = None, want_weights: bool = False,
                    kt_block_table: Optional[np.ndarray] = None):
    """Algorithm 1 per (sequence, head).  Returns (out f64 [B,H,D], alpha f64 [B,H],
    selected int32 [B,H,max k] ascending / -1 padded, approximate weights or None)."""
    qb = _bits(np.ascontiguousarray(q))
    kb, vb, ktb = _bits(k_pool), _bits(v_pool), _bits(kt_pool)
    batch, heads, head_dim = qb.shape
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ks = np.ascontiguousarray(k_tokens, dtype=np.int32)
    table, max_blocks = _table(block_table, batch)
    kt_table, kt_max_blocks = _table(block_table if kt_block_table is None else kt_block_table, batch)
    vs = np.ascontiguousarray(v_sum, dtype=np.float32)
    stride_k = max(int(np.minimum(ks, lens).max()) if batch else 0, 1)
    stride_s = max(int(lens.max()) if batch else 0, 1)
    out = np.zeros((batch, heads, head_dim), dtype=np.float64)
    alpha = np.zeros((batch, heads), dtype=np.float64)
    selected = np.full((batch, heads, stride_k), -1, dtype=np.int32)
    weights = np.zeros((batch, heads, stride_s), dtype=np.float64) if want_weights else None
    giv = None
    if given is not None:
        giv = np.full((batch, heads, stride_k), -1, dtype=np.int32)
        giv[:, :, :min(stride_k, given.shape[2])] = given[:, :, :stride_k]
    rc = _load().oracle_sparf_attention(_p(out), _p(alpha), _p(weights), stride_s, _p(selected),
                                        _p(giv), stride_k, _p(qb), _p(kb), _p(vb), _p(ktb), _p(vs),
                                        _p(lens), _p(ks), _p(table), max_blocks, kb.shape[2],
                                        kb.shape[0], _p(kt_table), kt_max_blocks, ktb.shape[3],
                                        ktb.shape[0], batch, heads, head_dim, int(r), int(l),
                                        ctypes.c_float(scale))
    if rc:
        raise OracleError(rc)
    return out, alpha, selected, weights
