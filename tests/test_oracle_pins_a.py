"""Pins for the CPU oracle, part A: closed forms and special cases (no GPU).

Each test fixes the oracle against something other than itself: a value the mathematics
gives in closed form, so that a dropped term, a wrong sign, a wrong index or a transposed
operand in the C file fails at least one of them.
"""
import math

import numpy as np
import pytest

from oracle import capi

SCALE = 1.0 / math.sqrt(128.0)


def f16(rng, shape, gain=1.0):
    return (rng.standard_normal(shape) * gain).astype(np.float16)


def test_half_widening_is_exact_for_every_bit_pattern():
    # L = 1 returns the V row itself, so 65536 patterns fit one call: B=1, H=512, D=128.
    bits = np.arange(65536, dtype=np.uint16).reshape(1, 512, 1, 128)
    q = np.zeros((1, 512, 128), dtype=np.float16)
    k = np.zeros((1, 512, 1, 128), dtype=np.float16)
    out, lse, _ = capi.decode_attention(q, k, bits, np.array([1]), SCALE)
    want = bits.view(np.float16).astype(np.float64).reshape(1, 512, 128)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(out), nan)
    assert np.array_equal(out[~nan], want[~nan])
    assert np.all(lse == 0.0)


def test_single_key_returns_its_value_row_and_its_logit():
    rng = np.random.default_rng(1)
    q, k, v = f16(rng, (2, 3, 128)), f16(rng, (2, 3, 1, 128)), f16(rng, (2, 3, 1, 128))
    scale = 0.1                      # not a binary32 value: the oracle must use float(0.1)
    out, lse, w = capi.decode_attention(q, k, v, np.array([1, 1]), scale, want_weights=True)
    assert np.array_equal(out, v[:, :, 0, :].astype(np.float64))
    dots = np.einsum("bhd,bhd->bh", q.astype(np.float64), k[:, :, 0, :].astype(np.float64))
    assert np.allclose(lse, float(np.float32(scale)) * dots, rtol=1e-14, atol=0)
    assert not np.allclose(lse, 0.1 * dots, rtol=1e-10, atol=0)   # double(0.1) is the wrong scale
    assert np.all(w[:, :, 0] == 1.0)


@pytest.mark.parametrize("how", ["identical_keys", "zero_query", "zero_scale"])
def test_uniform_weights_give_the_mean_of_v(how):
    rng = np.random.default_rng(2)
    L = 37
    q, k, v = f16(rng, (1, 2, 128)), f16(rng, (1, 2, L, 128)), f16(rng, (1, 2, L, 128))
    scale = SCALE
    if how == "identical_keys":
        k[:] = k[:, :, :1, :]
    elif how == "zero_query":
        q[:] = 0
    else:
        scale = 0.0
    out, lse, w = capi.decode_attention(q, k, v, np.array([L]), scale, want_weights=True)
    assert np.allclose(out, v.astype(np.float64).mean(axis=2), rtol=0, atol=1e-14)
    assert np.allclose(w, 1.0 / L, rtol=1e-14)
    if how != "identical_keys":
        assert np.allclose(lse, math.log(L), rtol=1e-15)


def test_constant_v_is_returned_whatever_the_keys():
    rng = np.random.default_rng(3)
    L = 50
    q, k = f16(rng, (2, 2, 128), 3.0), f16(rng, (2, 2, L, 128), 3.0)
    v = np.broadcast_to(f16(rng, (2, 2, 1, 128)), (2, 2, L, 128)).copy()
    out, _, _ = capi.decode_attention(q, k, v, np.array([L, L - 7]), SCALE)
    assert np.allclose(out, v[:, :, 0, :].astype(np.float64), rtol=1e-14, atol=0)


def test_weights_are_a_distribution_and_out_is_a_convex_combination():
    rng = np.random.default_rng(4)
    lens = np.array([1, 19, 64])
    q, k, v = f16(rng, (3, 4, 128), 2.0), f16(rng, (3, 4, 64, 128), 2.0), f16(rng, (3, 4, 64, 128))
    out, _, w = capi.decode_attention(q, k, v, lens, SCALE, want_weights=True)
    for b, L in enumerate(lens):
        assert np.all(w[b, :, :L] >= 0)
        assert np.all(w[b, :, L:] == 0)
        assert np.allclose(w[b, :, :L].sum(axis=1), 1.0, rtol=0, atol=1e-12)
        vv = v[b, :, :L, :].astype(np.float64)
        assert np.all(out[b] <= vv.max(axis=1) + 1e-12)
        assert np.all(out[b] >= vv.min(axis=1) - 1e-12)


def test_two_keys_follow_the_logistic_closed_form():
    rng = np.random.default_rng(5)
    q, k, v = f16(rng, (1, 5, 128)), f16(rng, (1, 5, 2, 128)), f16(rng, (1, 5, 2, 128))
    out, lse, _ = capi.decode_attention(q, k, v, np.array([2]), SCALE)
    s = float(np.float32(SCALE)) * np.einsum("hd,hid->hi", q[0].astype(np.float64),
                                             k[0].astype(np.float64))
    w1 = 1.0 / (1.0 + np.exp(s[:, 1] - s[:, 0]))           # sigma(s1 - s2)
    want = w1[:, None] * v[0, :, 0, :].astype(np.float64) + \
        (1.0 - w1)[:, None] * v[0, :, 1, :].astype(np.float64)
    assert np.allclose(out[0], want, rtol=1e-13, atol=1e-15)
    assert np.allclose(lse[0], s[:, 0] + np.log1p(np.exp(s[:, 1] - s[:, 0])), rtol=1e-13)


def test_a_dominant_key_wins():
    rng = np.random.default_rng(6)
    L, star = 33, 20
    q = np.zeros((1, 1, 128), dtype=np.float16)
    q[0, 0, 5] = 16.0
    k = f16(rng, (1, 1, L, 128), 0.25)
    k[0, 0, :, 5] = 0.0
    k[0, 0, star, 5] = 64.0          # logit 16*64/sqrt(128) ~ 90.5 above the rest
    v = f16(rng, (1, 1, L, 128))
    out, _, w = capi.decode_attention(q, k, v, np.array([L]), SCALE, want_weights=True)
    assert abs(w[0, 0, star] - 1.0) < L * math.exp(-50.0)
    assert np.allclose(out[0, 0], v[0, 0, star].astype(np.float64), rtol=0, atol=L * 8 * math.exp(-50.0))


def test_empty_sequence_gives_zero_and_minus_infinity():
    rng = np.random.default_rng(7)
    q, k, v = f16(rng, (2, 2, 128)), f16(rng, (2, 2, 4, 128)), f16(rng, (2, 2, 4, 128))
    out, lse, _ = capi.decode_attention(q, k, v, np.array([0, 3]), SCALE)
    assert np.all(out[0] == 0.0) and np.all(np.isneginf(lse[0]))
    assert np.all(np.isfinite(lse[1]))
