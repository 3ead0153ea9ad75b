"""Pins for the grouped-head / multi-token oracle function.  It is tied to things other than
itself: the already pinned one-query oracle (which it must equal on expanded heads and on
truncated lengths), torch's float64 softmax on the expanded problem, a pure-Python brute
force, and the causal structure."""
import numpy as np
import pytest
import torch

from oracle import brute, capi


def f16(rng, shape):
    return rng.standard_normal(shape).astype(np.float16)


def make(rng, lens, q_tokens, q_heads, kv_heads, tokens=0, dim=128):
    lens = np.asarray(lens)
    B = len(lens)
    if tokens:
        need = [max(1, -(-int(n) // tokens)) for n in lens]
        P = sum(need) + 1
        perm = rng.permutation(P)
        table = np.full((B, max(need)), -1, dtype=np.int32)
        at = 0
        for b, n in enumerate(need):
            table[b, :n] = perm[at:at + n]
            at += n
        k, v = f16(rng, (P, kv_heads, tokens, dim)), f16(rng, (P, kv_heads, tokens, dim))
    else:
        table = None
        k, v = f16(rng, (B, kv_heads, max(int(lens.max()), 1), dim)), f16(rng, (B, kv_heads, max(int(lens.max()), 1), dim))
    q = f16(rng, (B, q_tokens, q_heads, dim))
    return lens, table, q, k, v


def test_one_token_one_group_is_the_plain_oracle_bit_for_bit():
    rng = np.random.default_rng(7)
    lens, table, q, k, v = make(rng, [1, 30, 0, 17], 1, 3, 3, tokens=8)
    out, lse = capi.decode_attention_grouped(q, k, v, lens, 0.1, block_table=table)
    want, want_lse, _ = capi.decode_attention(q[:, 0], k, v, lens, 0.1, block_table=table)
    assert np.array_equal(out[:, 0], want) and np.array_equal(lse[:, 0], want_lse)


@pytest.mark.parametrize("tokens", [0, 8])
@pytest.mark.parametrize("q_tokens,q_heads,kv_heads", [(1, 8, 2), (3, 4, 4), (2, 6, 2), (4, 4, 1)])
def test_equals_plain_oracle_on_expanded_heads_and_truncated_lengths(tokens, q_tokens, q_heads, kv_heads):
    rng = np.random.default_rng(100 * q_tokens + q_heads + tokens)
    lens, table, q, k, v = make(rng, [40, 9, 2, 0, 23], q_tokens, q_heads, kv_heads, tokens)
    out, lse = capi.decode_attention_grouped(q, k, v, lens, 0.09, block_table=table)
    group = q_heads // kv_heads
    k_wide, v_wide = np.repeat(k, group, axis=1), np.repeat(v, group, axis=1)   # head hq <- hq // group
    for t in range(q_tokens):
        visible = np.maximum(lens - (q_tokens - 1 - t), 0)
        want, want_lse, _ = capi.decode_attention(q[:, t], k_wide, v_wide, visible, 0.09, block_table=table)
        assert np.array_equal(out[:, t], want), f"token {t}"
        assert np.array_equal(lse[:, t], want_lse), f"token {t}"


def test_against_torch_float64_softmax():
    rng = np.random.default_rng(11)
    L, Tq, Hq, Hkv, D = 50, 3, 8, 2, 64
    lens, table, q, k, v = make(rng, [L], Tq, Hq, Hkv, dim=D)
    scale = np.float32(1.0 / np.sqrt(D))
    out, lse = capi.decode_attention_grouped(q, k, v, lens, float(scale))
    qt = torch.from_numpy(q.astype(np.float64))[0]                          # [Tq,Hq,D]
    kt = torch.from_numpy(k.astype(np.float64))[0].repeat_interleave(Hq // Hkv, dim=0)   # [Hq,L,D]
    vt = torch.from_numpy(v.astype(np.float64))[0].repeat_interleave(Hq // Hkv, dim=0)
    logits = torch.einsum("thd,hid->thi", qt, kt) * float(scale)
    pos = torch.arange(L)[None, None, :]
    limit = (L - (Tq - 1 - torch.arange(Tq)))[:, None, None]
    logits = logits.masked_fill(pos >= limit, float("-inf"))
    want = torch.einsum("thi,hid->thd", torch.softmax(logits, dim=-1), vt)
    assert np.allclose(out[0], want.numpy(), rtol=1e-12, atol=1e-13)
    assert np.allclose(lse[0], torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-12, atol=1e-12)


def test_against_pure_python_brute_force():
    rng = np.random.default_rng(13)
    Tq, Hq, Hkv, D = 2, 4, 2, 8
    lens, table, q, k, v = make(rng, [5, 1], Tq, Hq, Hkv, tokens=4, dim=D)
    out, lse = capi.decode_attention_grouped(q, k, v, lens, 0.3, block_table=table)
    bits = lambda a: a.view(np.uint16).tolist()
    group = Hq // Hkv
    k_wide, v_wide = bits(np.repeat(k, group, axis=1)), bits(np.repeat(v, group, axis=1))
    for t in range(Tq):
        visible = [max(int(n) - (Tq - 1 - t), 0) for n in lens]
        want, want_lse, _ = brute.decode_attention(bits(np.ascontiguousarray(q[:, t])), k_wide, v_wide,
                                                   visible, 0.3, block_table=table.tolist(), block_tokens=4)
        assert np.allclose(out[:, t], np.array(want), rtol=0, atol=1e-13)
        assert np.allclose(lse[:, t], np.array(want_lse), rtol=1e-13, atol=1e-13)


def test_causal_structure_and_short_sequences():
    rng = np.random.default_rng(17)
    lens, table, q, k, v = make(rng, [20, 2], 3, 2, 1)
    out, lse = capi.decode_attention_grouped(q, k, v, lens, 0.1)
    k2, v2 = k.copy(), v.copy()
    k2[0, :, 19] += np.float16(3.0)                    # the newest token's rows
    v2[0, :, 19] -= np.float16(1.0)
    out2, _ = capi.decode_attention_grouped(q, k2, v2, lens, 0.1)
    assert np.array_equal(out2[0, :2], out[0, :2])     # older new tokens do not see it
    assert not np.array_equal(out2[0, 2], out[0, 2])
    # sequence 1 holds 2 tokens but the step brings 3: the oldest has nothing to attend to,
    # the next sees exactly one row and returns it
    assert np.all(out[1, 0] == 0) and np.all(np.isneginf(lse[1, 0]))
    assert np.array_equal(out[1, 1, 0], v[1, 0, 0].astype(np.float64))


def test_bad_head_counts_are_rejected():
    rng = np.random.default_rng(19)
    lens, table, q, k, v = make(rng, [4], 1, 3, 2)
    with pytest.raises(capi.OracleError) as e:
        capi.decode_attention_grouped(q, k, v, lens, 0.1)
    assert e.value.code == -1
