"""Brute-force decode attention in pure Python, for tiny shapes only (test infrastructure).

A second, separately written statement of Sec. II-A's softmax(q K^T / sqrt(d_k)) V for one
query row per head, used to pin the C oracle: Python floats are IEEE binary64, every sum is
`math.fsum` (correctly rounded), fp16 bit patterns are decoded by `struct`.  Nested lists in,
nested lists out; no numpy, no shared code with the C file or with the CUDA library.
"""
from __future__ import annotations

import math
import struct
from typing import List, Optional, Sequence


def half_value(bits: int) -> float:
    """Exact value of an IEEE binary16 bit pattern."""
    return struct.unpack("<e", struct.pack("<H", bits & 0xFFFF))[0]


def _row(cache, b: int, h: int, i: int, table: Optional[Sequence[Sequence[int]]], tokens: int):
    """Row of token i: cache[b][h][i] (contiguous) or pool[table[b][i//T]][h][i%T] (paged)."""
    if table is None:
        return cache[b][h][i]
    return cache[table[b][i // tokens]][h][i % tokens]


def decode_attention(q, k_cache, v_cache, seq_lens: Sequence[int], scale: float,
                     block_table=None, block_tokens: int = 0):
    """q: [B][H][D] fp16 bit patterns; caches likewise.  Returns (out, lse, weights) lists.

    `scale` is first rounded to binary32, as the C ABI carries a float.
    """
    scale = struct.unpack("<f", struct.pack("<f", scale))[0]
    out: List = []
    lse: List = []
    weights: List = []
    for b, length in enumerate(seq_lens):
        out_b, lse_b, w_b = [], [], []
        for h in range(len(q[b])):
            qv = [half_value(x) for x in q[b][h]]
            dim = len(qv)
            if length == 0:
                out_b.append([0.0] * dim)
                lse_b.append(-math.inf)
                w_b.append([])
                continue
            keys = [[half_value(x) for x in _row(k_cache, b, h, i, block_table, block_tokens)]
                    for i in range(length)]
            vals = [[half_value(x) for x in _row(v_cache, b, h, i, block_table, block_tokens)]
                    for i in range(length)]
            logits = [scale * math.fsum(qd * kd for qd, kd in zip(qv, row)) for row in keys]
            top = max(logits)
            expo = [math.exp(s - top) for s in logits]
            z = math.fsum(expo)
            w = [e / z for e in expo]
            out_b.append([math.fsum(w[i] * vals[i][d] for i in range(length))
                          for d in range(dim)])
            lse_b.append(top + math.log(z))
            w_b.append(w)
        out.append(out_b)
        lse.append(lse_b)
        weights.append(w_b)
    return out, lse, weights


def kv_append(k_cache, v_cache, k_new, v_new, seq_lens: Sequence[int],
              block_table=None, block_tokens: int = 0) -> None:
    """In-place list version of the append: position seq_lens[b]-1 receives the new rows."""
    for b, length in enumerate(seq_lens):
        if length == 0:
            continue
        for h in range(len(k_new[b])):
            _row(k_cache, b, h, length - 1, block_table, block_tokens)[:] = list(k_new[b][h])
            _row(v_cache, b, h, length - 1, block_table, block_tokens)[:] = list(v_new[b][h])


def sparf_attention(q, k_rows, v_rows, r: int, k: int, l: int, scale: float):
    """Algorithm 1 (SparF / SparQ arithmetic) for ONE head in pure Python.

    q: [D] fp16 bit patterns; k_rows, v_rows: [S][D] bit patterns (already gathered in token
    order).  vbar is the plain mean of the V rows.  Returns (out [D], alpha, J ascending).
    Ties in both top-k selections go to the lower index.
    """
    scale = struct.unpack("<f", struct.pack("<f", scale))[0]
    qv = [half_value(x) for x in q]
    K = [[half_value(x) for x in row] for row in k_rows]
    V = [[half_value(x) for x in row] for row in v_rows]
    S, D = len(K), len(qv)
    if S == 0:
        return [0.0] * D, 0.0, []
    k = min(k, S)
    l = min(l, k)
    dims = sorted(range(D), key=lambda d: (-abs(qv[d]), d))[:r]
    q_l1 = math.fsum(abs(x) for x in qv)
    ratio = math.fsum(abs(qv[d]) for d in dims) / q_l1 if q_l1 > 0 else 1.0
    approx = [scale / math.sqrt(ratio) * math.fsum(qv[d] * K[i][d] for d in dims) for i in range(S)]
    top = max(approx)
    e = [math.exp(x - top) for x in approx]
    z = math.fsum(e)
    s_hat = [x / z for x in e]
    keyed = [s_hat[i] + (1.0 if i >= S - l else 0.0) for i in range(S)]
    J = sorted(sorted(range(S), key=lambda i: (-keyed[i], i))[:k])
    alpha = math.fsum(s_hat[j] for j in J)
    vbar = [math.fsum(V[i][d] for i in range(S)) / S for d in range(D)]
    if not J:
        return vbar, 0.0, []
    logits = [scale * math.fsum(qv[d] * K[j][d] for d in range(D)) for j in J]
    top = max(logits)
    w = [math.exp(x - top) for x in logits]
    zw = math.fsum(w)
    out = [alpha * math.fsum(w[t] / zw * V[j][d] for t, j in enumerate(J)) + (1.0 - alpha) * vbar[d]
           for d in range(D)]
    return out, alpha, J
