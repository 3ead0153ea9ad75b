"""Pins for the sparse-attention (SparF, Algorithm 1) oracle.  The paper prints no worked
example, so the pins are the reductions the algorithm itself fixes: with every query dim and
every token kept it IS dense attention; with every dim kept the approximate scores are the
exact ones; with the window as large as k it is local attention; plus brute force."""
import math

import numpy as np
import pytest

from oracle import brute, capi

SCALE = 1.0 / math.sqrt(128.0)


def f16(rng, shape, gain=1.0):
    return (rng.standard_normal(shape) * gain).astype(np.float16)


def paged(rng, lens, tokens, heads=2, dim=128, gain=1.0):
    """Random paged pools with a shuffled table, their K^T copy and the true fp32 V sums."""
    need = [-(-int(n) // tokens) for n in lens]
    P = sum(need) + 1
    perm = rng.permutation(P)
    table = np.full((len(lens), max(max(need), 1)), -1, dtype=np.int32)
    at = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[at:at + n]
        at += n
    k = f16(rng, (P, heads, tokens, dim), gain)
    v = f16(rng, (P, heads, tokens, dim))
    kt = np.ascontiguousarray(k.transpose(0, 1, 3, 2))
    v_sum = np.zeros((len(lens), heads, dim), dtype=np.float32)
    for b, n in enumerate(lens):
        rows = rows_of(v, table, b, n, tokens)
        v_sum[b] = rows.astype(np.float64).sum(axis=1).astype(np.float32)
    return k, v, kt, v_sum, table


def rows_of(pool, table, b, n, tokens):
    """[H, n, D] rows of sequence b in token order."""
    blocks = table[b, : -(-int(n) // tokens)]
    return pool[blocks].transpose(1, 0, 2, 3).reshape(pool.shape[1], -1, pool.shape[3])[:, :n]


def test_keeping_everything_is_dense_attention():
    rng = np.random.default_rng(31)
    lens = np.array([1, 9, 40, 0])
    k, v, kt, v_sum, table = paged(rng, lens, 8)
    q = f16(rng, (4, 2, 128), 2.0)
    dense, _, _ = capi.decode_attention(q, k, v, lens, SCALE, block_table=table)
    out, alpha, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, lens, table, r=128, l=0, scale=SCALE)
    assert np.allclose(out, dense, rtol=0, atol=1e-13)
    assert np.allclose(alpha[lens > 0], 1.0, rtol=0, atol=1e-13) and np.all(alpha[lens == 0] == 0)
    for b, n in enumerate(lens):
        assert np.array_equal(sel[b, :, :n], np.tile(np.arange(n), (2, 1)))
    # k larger than the sequence is clipped, and r no longer matters once all tokens are kept
    out2, alpha2, _, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, lens + 5, table, r=3, l=2, scale=SCALE)
    assert np.allclose(out2, dense, rtol=0, atol=1e-13)


def test_all_dims_kept_selects_the_top_k_of_the_exact_weights():
    rng = np.random.default_rng(32)
    lens = np.array([50])
    k, v, kt, v_sum, table = paged(rng, lens, 16, gain=2.0)
    q = f16(rng, (1, 2, 128), 2.0)
    _, _, w = capi.decode_attention(q, k, v, lens, SCALE, block_table=table, want_weights=True)
    out, alpha, sel, approx = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([7]), table,
                                                   r=128, l=0, scale=SCALE, want_weights=True)
    assert np.allclose(approx, w, rtol=0, atol=1e-14)            # ratio = 1: temperature sqrt(d)
    for h in range(2):
        want = np.sort(np.argsort(-w[0, h], kind="stable")[:7])
        assert np.array_equal(sel[0, h], want)
        assert abs(alpha[0, h] - w[0, h, want].sum()) < 1e-14
        # step 11 spelled out with the weights renormalised over J
        vr = rows_of(v, table, 0, 50, 16)[h].astype(np.float64)
        attn = (w[0, h, want] / w[0, h, want].sum()) @ vr[want]
        vbar = v_sum[0, h].astype(np.float64) / 50
        assert np.allclose(out[0, h], alpha[0, h] * attn + (1 - alpha[0, h]) * vbar, atol=1e-13)


def test_window_as_large_as_k_is_local_attention():
    rng = np.random.default_rng(33)
    lens = np.array([37])
    k, v, kt, v_sum, table = paged(rng, lens, 8)
    q = f16(rng, (1, 2, 128))
    _, _, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([10]), table, r=16, l=10, scale=SCALE)
    assert np.array_equal(sel[0, 0], np.arange(27, 37)) and np.array_equal(sel[0, 1], np.arange(27, 37))
    _, _, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([10]), table, r=16, l=4, scale=SCALE)
    assert np.all(np.isin(np.arange(33, 37), sel[0, 0])) and len(set(sel[0, 0])) == 10


@pytest.mark.parametrize("r,kk,l,tokens", [(2, 3, 0, 8), (4, 5, 2, 8), (8, 8, 8, 16), (1, 1, 0, 8), (3, 0, 0, 8)])
def test_brute_force_on_tiny_shapes(r, kk, l, tokens):
    rng = np.random.default_rng(34 + r)
    lens = np.array([11, 1, 6])
    k, v, kt, v_sum, table = paged(rng, lens, tokens, heads=2, dim=8, gain=2.0)
    q = f16(rng, (3, 2, 8), 2.0)
    scale = 1 / math.sqrt(8)
    out, alpha, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.full(3, kk), table, r=r, l=l, scale=scale)
    for b, n in enumerate(lens):
        kr, vr = rows_of(k, table, b, n, tokens), rows_of(v, table, b, n, tokens)
        for h in range(2):
            bo, ba, bj = brute.sparf_attention(q[b, h].view(np.uint16).tolist(), kr[h].view(np.uint16).tolist(),
                                               vr[h].view(np.uint16).tolist(), r, kk, l, scale)
            assert sel[b, h, :len(bj)].tolist() == bj
            assert abs(alpha[b, h] - ba) < 1e-13
            # brute uses the exact mean, the oracle the fp32 running sum: allow that rounding
            assert np.allclose(out[b, h], np.array(bo), rtol=0, atol=1e-6)


def test_alpha_grows_with_k_and_a_given_selection_is_honoured():
    rng = np.random.default_rng(35)
    lens = np.array([64])
    k, v, kt, v_sum, table = paged(rng, lens, 16, gain=2.0)
    q = f16(rng, (1, 2, 128), 2.0)
    last = 0.0
    for kk in (1, 4, 16, 64):
        out, alpha, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([kk]), table, r=16, l=0, scale=SCALE)
        assert np.all(alpha > last - 1e-15) and np.all(alpha <= 1 + 1e-12)
        last = alpha.min()
    given = np.tile(np.array([3, 9, 20, 41], dtype=np.int32), (1, 2, 1))
    out, alpha, sel, w = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([4]), table, r=16, l=0,
                                              scale=SCALE, given=given, want_weights=True)
    assert np.array_equal(sel, given)
    assert np.allclose(alpha, w[:, :, [3, 9, 20, 41]].sum(axis=2), atol=1e-14)


def test_sparf_append_writes_both_k_layouts_and_the_running_sum():
    rng = np.random.default_rng(36)
    lens = np.array([9, 16, 0])
    k, v, kt, v_sum, table = paged(rng, lens, 8)
    k0, v0, kt0, s0 = k.copy(), v.copy(), kt.copy(), v_sum.copy()
    kn, vn = f16(rng, (3, 2, 128)), f16(rng, (3, 2, 128))
    capi.sparf_append(k, v, kt, v_sum, kn, vn, lens, table)
    k1, v1 = k0.copy(), v0.copy()
    capi.kv_append(k1, v1, kn, vn, lens, block_table=table)
    assert np.array_equal(k.view(np.uint16), k1.view(np.uint16)) and np.array_equal(v.view(np.uint16), v1.view(np.uint16))
    assert np.array_equal(kt.view(np.uint16), np.ascontiguousarray(k.transpose(0, 1, 3, 2)).view(np.uint16))
    assert np.array_equal(v_sum[2], s0[2])
    assert np.array_equal(v_sum[:2], (s0[:2] + vn[:2].astype(np.float32)))     # one fp32 rounding


def relayout_kt(k, table, lens, tokens, kt_tokens, rng):
    """K^T pool [Pk,H,D,Tk] with its own shuffled table, holding the same logical keys."""
    H, D = k.shape[1], k.shape[3]
    need = [-(-int(n) // kt_tokens) for n in lens]
    Pk = sum(need) + 1
    perm = rng.permutation(Pk)
    kt_table = np.full((len(lens), max(max(need), 1)), -1, dtype=np.int32)
    kt = np.full((Pk, H, D, kt_tokens), np.float16(np.nan), dtype=np.float16)
    at = 0
    for b, n in enumerate(need):
        kt_table[b, :n] = perm[at:at + n]
        at += n
        rows = rows_of(k, table, b, lens[b], tokens)                 # [H, L, D]
        for j in range(n):
            piece = rows[:, j * kt_tokens:(j + 1) * kt_tokens]       # [H, <=Tk, D]
            kt[kt_table[b, j], :, :, :piece.shape[1]] = piece.transpose(0, 2, 1)
    return kt, kt_table


@pytest.mark.parametrize("kt_tokens", [8, 32, 64])
def test_the_transposed_copy_may_use_its_own_block_size(kt_tokens):
    rng = np.random.default_rng(37)
    lens = np.array([70, 9, 0, 33])
    k, v, kt, v_sum, table = paged(rng, lens, 8, gain=2.0)
    q = f16(rng, (4, 2, 128), 2.0)
    ks = np.array([9, 2, 0, 5])
    same = capi.sparf_attention(q, k, v, kt, v_sum, lens, ks, table, r=16, l=2, scale=SCALE, want_weights=True)
    kt2, kt_table = relayout_kt(k, table, lens, 8, kt_tokens, rng)
    other = capi.sparf_attention(q, k, v, kt2, v_sum, lens, ks, table, r=16, l=2, scale=SCALE,
                                 want_weights=True, kt_block_table=kt_table)
    for a, b in zip(same, other):
        assert np.array_equal(a, b)
    # the append lands in the right column of the right K^T block
    lens2 = lens + np.array([1, 1, 0, 1])
    grow = [-(-int(n) // 8) for n in lens2]
    assert all(g <= table.shape[1] or True for g in grow)
    lens_ok = np.array([70, 9, 0, 33])            # re-append the last token of each live sequence
    kn, vn = f16(rng, (4, 2, 128)), f16(rng, (4, 2, 128))
    capi.sparf_append(k, v, kt2, v_sum, kn, vn, lens_ok, table, kt_block_table=kt_table)
    want_kt, _ = None, None
    for b, n in enumerate(lens_ok):
        if n:
            blk, col = kt_table[b, (n - 1) // kt_tokens], (n - 1) % kt_tokens
            assert np.array_equal(kt2[blk, :, :, col].view(np.uint16), kn[b].view(np.uint16))


def two_key_problem(q_vals, k0, k1):
    """One sequence of two tokens, one head, 128 dims, one 8-token block; k0, k1 are dicts dim -> value."""
    q = np.zeros((1, 1, 128), np.float16)
    k = np.zeros((1, 1, 8, 128), np.float16)
    for d, x in q_vals.items():
        q[0, 0, d] = x
    for d, x in k0.items():
        k[0, 0, 0, d] = x
    for d, x in k1.items():
        k[0, 0, 1, d] = x
    v = np.zeros((1, 1, 8, 128), np.float16)
    v[0, 0, 0, 0], v[0, 0, 1, 0] = 1.0, -1.0
    kt = np.ascontiguousarray(k.transpose(0, 1, 3, 2))
    v_sum = np.zeros((1, 1, 128), np.float32)
    return q, k, v, kt, v_sum, np.zeros((1, 1), np.int32)


def test_the_temperature_is_the_printed_one_on_a_two_key_closed_form():
    # |q| = 2 on dims 0-3 (negative: the ranking is on magnitudes), 1 on dims 4-15: with r = 4,
    # |q_I|_1 / |q|_1 = 8 / 20, temperature sqrt(128 * 0.4); two keys give a logistic weight.
    q_vals = {d: -2.0 for d in range(4)} | {d: 1.0 for d in range(4, 16)}
    k0 = {0: 1.5, 1: -0.5, 5: 3.0}             # dims 5, 9 are outside I and must not count
    k1 = {0: -1.0, 2: 0.5, 9: -3.0}
    q, k, v, kt, v_sum, table = two_key_problem(q_vals, k0, k1)
    _, alpha, sel, w = capi.sparf_attention(q, k, v, kt, v_sum, np.array([2]), np.array([1]), table,
                                            r=4, l=0, scale=SCALE, want_weights=True)
    dot0, dot1 = -2.0 * 1.5 + -2.0 * -0.5, -2.0 * -1.0 + -2.0 * 0.5
    delta = (dot0 - dot1) / math.sqrt(128 * 0.4)
    want0 = 1.0 / (1.0 + math.exp(-delta))
    # the scale is rounded to binary32 on the way in: 6e-8 relative on delta
    assert abs(w[0, 0, 0] - want0) < 1e-7 and abs(w[0, 0, 1] - (1 - want0)) < 1e-7
    keep = 0 if want0 > 0.5 else 1
    assert sel[0, 0, 0] == keep and abs(alpha[0, 0] - max(want0, 1 - want0)) < 1e-7


def test_step_six_is_the_ranking_of_the_printed_sum():
    # s^ + m ranked with numpy from the oracle's own s^ (generic data: no rounding corner)
    rng = np.random.default_rng(38)
    lens = np.array([200, 77])
    k, v, kt, v_sum, table = paged(rng, lens, 8, gain=2.0)
    q = f16(rng, (2, 2, 128), 2.0)
    ks, l = np.array([25, 10]), 6
    _, _, sel, w = capi.sparf_attention(q, k, v, kt, v_sum, lens, ks, table, r=16, l=l, scale=SCALE, want_weights=True)
    for b, S in enumerate(lens):
        m = (np.arange(S) >= S - l).astype(np.float64)
        for h in range(2):
            want = np.sort(np.argsort(-(w[b, h, :S] + m), kind="stable")[:ks[b]])
            assert np.array_equal(sel[b, h, :ks[b]], want)


def test_the_window_survives_a_dominant_early_token():
    # token 0 takes all the approximate weight (s^ = 1 to fp64 rounding, the rest underflows
    # against it); with k = l = 2 the kept set is still the last two positions
    q_vals = {0: 60.0}
    q, k, v, kt, v_sum, table = two_key_problem(q_vals, {0: 60.0}, {})
    k[0, 0, 2, 0] = kt[0, 0, 0, 2] = -1.0
    _, alpha, sel, w = capi.sparf_attention(q, k, v, kt, v_sum, np.array([3]), np.array([2]), table,
                                            r=1, l=2, scale=SCALE, want_weights=True)
    assert w[0, 0, 0] == 1.0 and 1.0 + w[0, 0, 1] == 1.0
    assert sel[0, 0].tolist() == [1, 2] and alpha[0, 0] < 1e-100
