"""Pins for the bulk (prefill) append of the oracle: it must equal the already pinned
single-token append applied token by token, and touch nothing else."""
import numpy as np
import pytest

from oracle import capi


def f16(rng, shape):
    return rng.standard_normal(shape).astype(np.float16)


def setup(rng, tokens):
    lens = np.array([40, 7, 16, 0, 33])
    news = np.array([40, 3, 16, 0, 1])
    B, H, D, N = len(lens), 2, 128, 40
    if tokens:
        need = [-(-int(n) // tokens) for n in lens]
        P = sum(need) + 2
        perm = rng.permutation(P)
        table = np.full((B, max(need)), -1, dtype=np.int32)
        at = 0
        for b, n in enumerate(need):
            table[b, :n] = perm[at:at + n]
            at += n
        k, v = f16(rng, (P, H, tokens, D)), f16(rng, (P, H, tokens, D))
    else:
        table = None
        k, v = f16(rng, (B, H, 40, D)), f16(rng, (B, H, 40, D))
    return lens, news, table, k, v, f16(rng, (B, N, H, D)), f16(rng, (B, N, H, D))


@pytest.mark.parametrize("tokens", [0, 8, 16])
def test_bulk_append_equals_token_by_token_append(tokens):
    rng = np.random.default_rng(41 + tokens)
    lens, news, table, k, v, kn, vn = setup(rng, tokens)
    k1, v1 = k.copy(), v.copy()
    capi.kv_append_bulk(k, v, kn, vn, lens, news, block_table=table)
    for t in range(int(news.max())):
        active = t < news
        step_lens = np.where(active, lens - news + t + 1, 0)       # length after this token; 0 = skip
        capi.kv_append(k1, v1, kn[:, t], vn[:, t], step_lens, block_table=table)
    assert np.array_equal(k.view(np.uint16), k1.view(np.uint16))
    assert np.array_equal(v.view(np.uint16), v1.view(np.uint16))


def test_bulk_append_rejects_bad_lengths():
    rng = np.random.default_rng(44)
    lens, news, table, k, v, kn, vn = setup(rng, 8)
    for bad in (np.array([41, 3, 16, 0, 1]), np.array([40, 8, 16, 0, 1]), np.array([40, -1, 16, 0, 1])):
        with pytest.raises(capi.OracleError) as e:
            capi.kv_append_bulk(k, v, kn, vn, lens, bad, block_table=table)
        assert e.value.code == -2


def test_sparse_bulk_append_equals_token_by_token_sparse_append():
    rng = np.random.default_rng(45)
    lens, news = np.array([40, 7, 16, 0, 33]), np.array([40, 3, 16, 0, 1])
    B, H, D, N, T, Tk = 5, 2, 128, 40, 8, 32
    need, need_k = [-(-int(n) // T) for n in lens], [-(-int(n) // Tk) for n in lens]
    P, Pk = sum(need) + 1, sum(need_k) + 1
    table = np.full((B, max(need)), -1, dtype=np.int32)
    kt_table = np.full((B, max(need_k)), -1, dtype=np.int32)
    perm, perm_k = rng.permutation(P), rng.permutation(Pk)
    at = at_k = 0
    for b in range(B):
        table[b, :need[b]] = perm[at:at + need[b]]
        kt_table[b, :need_k[b]] = perm_k[at_k:at_k + need_k[b]]
        at, at_k = at + need[b], at_k + need_k[b]
    k, v, kt = f16(rng, (P, H, T, D)), f16(rng, (P, H, T, D)), f16(rng, (Pk, H, D, Tk))
    v_sum = rng.standard_normal((B, H, D)).astype(np.float32)
    kn, vn = f16(rng, (B, N, H, D)), f16(rng, (B, N, H, D))
    k1, v1, kt1, s1 = k.copy(), v.copy(), kt.copy(), v_sum.copy()
    capi.sparf_append_bulk(k, v, kt, v_sum, kn, vn, lens, news, table, kt_block_table=kt_table)
    for t in range(int(news.max())):
        step_lens = np.where(t < news, lens - news + t + 1, 0)
        capi.sparf_append(k1, v1, kt1, s1, kn[:, t], vn[:, t], step_lens, table, kt_block_table=kt_table)
    for a, b_ in ((k, k1), (v, v1), (kt, kt1)):
        assert np.array_equal(a.view(np.uint16), b_.view(np.uint16))
    assert np.array_equal(v_sum.view(np.uint32), s1.view(np.uint32))
