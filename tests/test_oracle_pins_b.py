"""Pins for the CPU oracle, part B: invariants, brute force, a library routine, layouts."""
import math

import numpy as np
import pytest
import torch

from oracle import brute, capi

SCALE = 1.0 / math.sqrt(128.0)


def f16(rng, shape, gain=1.0):
    return (rng.standard_normal(shape) * gain).astype(np.float16)


def grid16(rng, shape, span=8):
    """fp16 multiples of 1/16 in [-span, span): sums and doublings of these stay exact."""
    return (rng.integers(-span * 16, span * 16, size=shape) / 16.0).astype(np.float16)


def paginate(cache, lens, tokens, rng, spare=2):
    """Re-lay a contiguous [B,H,S,D] cache into pools [P,H,T,D] under a random block table."""
    B, H, S, D = cache.shape
    need = [-(-int(n) // tokens) for n in lens]
    P = sum(need) + spare
    perm = rng.permutation(P)
    table = np.full((B, max(max(need), 1)), -1, dtype=np.int32)
    pool = np.full((P, H, tokens, D), np.float16(np.nan), dtype=np.float16)
    at = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[at:at + n]
        at += n
        for j in range(n):
            rows = cache[b, :, j * tokens:(j + 1) * tokens, :]
            pool[table[b, j], :, :rows.shape[1], :] = rows
    return pool, table


def test_logit_shift_leaves_the_output_unchanged():
    rng = np.random.default_rng(11)
    L = 23
    q, k, v = grid16(rng, (1, 2, 128), 2), grid16(rng, (1, 2, L, 128), 4), f16(rng, (1, 2, L, 128))
    c = grid16(rng, (1, 2, 1, 128), 4)
    shifted = (k.astype(np.float32) + c.astype(np.float32)).astype(np.float16)
    assert np.array_equal(shifted.astype(np.float32), k.astype(np.float32) + c.astype(np.float32))
    a, lse_a, _ = capi.decode_attention(q, k, v, np.array([L]), SCALE)
    b, lse_b, _ = capi.decode_attention(q, shifted, v, np.array([L]), SCALE)
    assert np.allclose(a, b, rtol=0, atol=1e-12)
    qc = float(np.float32(SCALE)) * np.einsum("bhd,bhd->bh", q.astype(np.float64),
                                              c[:, :, 0, :].astype(np.float64))
    assert np.allclose(lse_b - lse_a, qc, rtol=0, atol=1e-10)


def test_output_is_linear_in_v():
    rng = np.random.default_rng(12)
    L = 31
    q, k = f16(rng, (1, 3, 128)), f16(rng, (1, 3, L, 128))
    v1, v2 = grid16(rng, (1, 3, L, 128)), grid16(rng, (1, 3, L, 128))
    mix = (2.0 * v1.astype(np.float32) - v2.astype(np.float32)).astype(np.float16)
    lens = np.array([L])
    o1 = capi.decode_attention(q, k, v1, lens, SCALE)[0]
    o2 = capi.decode_attention(q, k, v2, lens, SCALE)[0]
    om = capi.decode_attention(q, k, mix, lens, SCALE)[0]
    assert np.allclose(om, 2.0 * o1 - o2, rtol=0, atol=1e-12)


def test_heads_and_sequences_are_independent():
    rng = np.random.default_rng(13)
    lens = np.array([9, 17])
    q, k, v = f16(rng, (2, 3, 128)), f16(rng, (2, 3, 17, 128)), f16(rng, (2, 3, 17, 128))
    base = capi.decode_attention(q, k, v, lens, SCALE)[0]
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[1, 2], k2[1, 2], v2[1, 2] = 0, 1, -1          # disturb exactly one (b, h)
    other = capi.decode_attention(q2, k2, v2, lens, SCALE)[0]
    keep = np.ones((2, 3), dtype=bool)
    keep[1, 2] = False
    assert np.array_equal(base[keep], other[keep])
    assert not np.array_equal(base[1, 2], other[1, 2])


def test_two_halves_merge_to_the_whole_by_log_sum_exp():
    rng = np.random.default_rng(14)
    L, cut = 45, 14
    q, k, v = f16(rng, (1, 4, 128), 2.0), f16(rng, (1, 4, L, 128), 2.0), f16(rng, (1, 4, L, 128))
    whole, lse, _ = capi.decode_attention(q, k, v, np.array([L]), SCALE)
    o1, l1, _ = capi.decode_attention(q, k[:, :, :cut].copy(), v[:, :, :cut].copy(),
                                      np.array([cut]), SCALE)
    o2, l2, _ = capi.decode_attention(q, k[:, :, cut:].copy(), v[:, :, cut:].copy(),
                                      np.array([L - cut]), SCALE)
    top = np.maximum(l1, l2)
    w1, w2 = np.exp(l1 - top), np.exp(l2 - top)
    merged = (w1[..., None] * o1 + w2[..., None] * o2) / (w1 + w2)[..., None]
    assert np.allclose(merged, whole, rtol=0, atol=1e-13)
    assert np.allclose(top + np.log(w1 + w2), lse, rtol=1e-14)


@pytest.mark.parametrize("tokens", [1, 4, 16])
def test_paged_equals_contiguous_and_ignores_the_block_permutation(tokens):
    rng = np.random.default_rng(15)
    lens = np.array([1, 16, 33, 0, 40])
    q = f16(rng, (5, 2, 128))
    k, v = f16(rng, (5, 2, 40, 128)), f16(rng, (5, 2, 40, 128))
    flat = capi.decode_attention(q, k, v, lens, SCALE)
    state = rng.bit_generator.state
    kp, table = paginate(k, lens, tokens, rng)
    rng.bit_generator.state = state
    vp, table_v = paginate(v, lens, tokens, rng)
    assert np.array_equal(table, table_v)
    paged = capi.decode_attention(q, kp, vp, lens, SCALE, block_table=table)
    assert np.array_equal(flat[0], paged[0]) and np.array_equal(flat[1], paged[1])
    kp2, table2 = paginate(k, lens, tokens, np.random.default_rng(99))
    vp2, _ = paginate(v, lens, tokens, np.random.default_rng(99))
    assert not np.array_equal(table, table2)
    again = capi.decode_attention(q, kp2, vp2, lens, SCALE, block_table=table2)
    assert np.array_equal(paged[0], again[0])


@pytest.mark.parametrize("dim,tokens", [(8, 0), (128, 0), (8, 2), (128, 4)])
def test_brute_force_on_tiny_shapes(dim, tokens):
    rng = np.random.default_rng(16 + dim + tokens)
    lens = np.array([8, 3, 0, 1][: 2 if dim == 128 else 4])
    B, H = len(lens), 2
    q, k, v = f16(rng, (B, H, dim), 2.0), f16(rng, (B, H, 8, dim), 2.0), f16(rng, (B, H, 8, dim))
    table = None
    kk, vv = k, v
    if tokens:
        state = rng.bit_generator.state
        kk, table = paginate(k, lens, tokens, rng)
        rng.bit_generator.state = state
        vv, _ = paginate(v, lens, tokens, rng)
    scale = 1.0 / math.sqrt(dim)
    out, lse, w = capi.decode_attention(q, kk, vv, lens, scale, block_table=table,
                                        want_weights=True)
    bo, bl, bw = brute.decode_attention(
        q.view(np.uint16).tolist(), kk.view(np.uint16).tolist(), vv.view(np.uint16).tolist(),
        lens.tolist(), scale, None if table is None else table.tolist(), tokens)
    assert np.allclose(out, np.array(bo), rtol=0, atol=1e-13)
    for b, L in enumerate(lens):
        for h in range(H):
            if L:
                assert abs(lse[b, h] - bl[b][h]) < 1e-13
                assert np.allclose(w[b, h, :L], bw[b][h], rtol=0, atol=1e-14)
            else:
                assert bl[b][h] == -math.inf and np.isneginf(lse[b, h])


@pytest.mark.parametrize("B,H,lens", [(1, 40, [1024]), (3, 4, [5, 130, 77])])
def test_library_softmax_in_float64_agrees(B, H, lens):
    g = torch.Generator().manual_seed(17)
    S = max(lens)
    q = torch.randn(B, H, 128, generator=g).half()
    k = torch.randn(B, H, S, 128, generator=g).half()
    v = torch.randn(B, H, S, 128, generator=g).half()
    out, lse, _ = capi.decode_attention(q.numpy(), k.numpy(), v.numpy(), np.array(lens), SCALE)
    scale32 = float(np.float32(SCALE))
    for b, L in enumerate(lens):
        logits = torch.einsum("hd,hld->hl", q[b].double(), k[b, :, :L].double()) * scale32
        want = torch.einsum("hl,hld->hd", torch.softmax(logits, dim=-1), v[b, :, :L].double())
        assert np.allclose(out[b], want.numpy(), rtol=0, atol=1e-13)
        assert np.allclose(lse[b], torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-13)
