"""Pins for the CPU oracle, part C: the append, error codes, and the paper's sizing figures."""
import math
import os

import numpy as np
import pytest

from oracle import brute, capi
from paper_2409_04992_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "kv_sizing.txt")


def f16(rng, shape):
    return rng.standard_normal(shape).astype(np.float16)


def read_golden():
    table = {}
    with open(GOLDEN) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                key, value = line.split()[:2]
                table[key] = float(value)
    return table


def test_append_contiguous_changes_exactly_the_new_rows():
    rng = np.random.default_rng(21)
    lens = np.array([1, 7, 0, 12])
    k, v = f16(rng, (4, 3, 12, 128)), f16(rng, (4, 3, 12, 128))
    kn, vn = f16(rng, (4, 3, 128)), f16(rng, (4, 3, 128))
    k0, v0 = k.copy(), v.copy()
    capi.kv_append(k, v, kn, vn, lens)
    changed_k = k.view(np.uint16) != k0.view(np.uint16)
    for b, L in enumerate(lens):
        if L == 0:
            assert not changed_k[b].any()
            continue
        assert np.array_equal(k[b, :, L - 1].view(np.uint16), kn[b].view(np.uint16))
        assert np.array_equal(v[b, :, L - 1].view(np.uint16), vn[b].view(np.uint16))
        mask = np.ones(12, dtype=bool)
        mask[L - 1] = False
        assert np.array_equal(k[b][:, mask].view(np.uint16), k0[b][:, mask].view(np.uint16))
        assert np.array_equal(v[b][:, mask].view(np.uint16), v0[b][:, mask].view(np.uint16))


@pytest.mark.parametrize("tokens", [1, 4, 16])
def test_append_paged_matches_the_list_version(tokens):
    rng = np.random.default_rng(22)
    lens = np.array([1, 16, 17, 0, 33])
    need = [-(-int(n) // tokens) for n in lens]
    P = sum(need) + 2
    perm = rng.permutation(P)
    table = np.full((5, max(need)), -1, dtype=np.int32)
    at = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[at:at + n]
        at += n
    k, v = f16(rng, (P, 2, tokens, 128)), f16(rng, (P, 2, tokens, 128))
    kn, vn = f16(rng, (5, 2, 128)), f16(rng, (5, 2, 128))
    kl, vl = k.view(np.uint16).tolist(), v.view(np.uint16).tolist()
    brute.kv_append(kl, vl, kn.view(np.uint16).tolist(), vn.view(np.uint16).tolist(),
                    lens.tolist(), table.tolist(), tokens)
    k0 = k.copy()
    capi.kv_append(k, v, kn, vn, lens, block_table=table)
    assert np.array_equal(k.view(np.uint16), np.array(kl, dtype=np.uint16))
    assert np.array_equal(v.view(np.uint16), np.array(vl, dtype=np.uint16))
    assert (k.view(np.uint16) != k0.view(np.uint16)).sum() <= 4 * 2 * 128
    for b, L in enumerate(lens):
        if L:
            blk, slot = table[b, (L - 1) // tokens], (L - 1) % tokens
            assert np.array_equal(k[blk, :, slot].view(np.uint16), kn[b].view(np.uint16))
            assert np.array_equal(v[blk, :, slot].view(np.uint16), vn[b].view(np.uint16))


def test_new_token_attends_to_itself_after_the_append():
    # A query aligned with its own fresh key, far from all cached keys, must return v_new.
    rng = np.random.default_rng(23)
    L = 9
    k, v = f16(rng, (1, 1, L, 128)) * np.float16(0.1), f16(rng, (1, 1, L, 128))
    kn = np.zeros((1, 1, 128), dtype=np.float16)
    kn[0, 0, 0] = 64.0
    q = np.zeros((1, 1, 128), dtype=np.float16)
    q[0, 0, 0] = 16.0
    vn = f16(rng, (1, 1, 128))
    capi.kv_append(k, v, kn, vn, np.array([L]))
    out, _, w = capi.decode_attention(q, k, v, np.array([L]), 1.0 / math.sqrt(128), want_weights=True)
    assert w[0, 0, L - 1] > 1 - 1e-12
    assert np.allclose(out[0, 0], vn[0, 0].astype(np.float64), atol=1e-10)


def test_errors_are_reported_not_computed():
    rng = np.random.default_rng(24)
    q, k, v = f16(rng, (1, 1, 128)), f16(rng, (3, 1, 4, 128)), f16(rng, (3, 1, 4, 128))
    with pytest.raises(capi.OracleError) as e:
        capi.decode_attention(q, k, v, np.array([5]), 0.1, block_table=np.array([[0, 7]], dtype=np.int32))
    assert e.value.code == -3
    with pytest.raises(capi.OracleError) as e:
        capi.decode_attention(q, k, v, np.array([9]), 0.1, block_table=np.array([[0, 1]], dtype=np.int32))
    assert e.value.code == -2
    with pytest.raises(capi.OracleError) as e:
        capi.kv_append(k, v, q, q, np.array([2]), block_table=np.array([[-1, 1]], dtype=np.int32))
    assert e.value.code == -3
    with pytest.raises(capi.OracleError) as e:
        capi.decode_attention(q, k[:1], v[:1], np.array([5]), 0.1)
    assert e.value.code == -2


def test_sizing_figures_printed_in_the_paper():
    g = read_golden()
    assert workloads.HEAD_DIM_13B * 2 == g["vector_bytes_head128_fp16"]
    assert 4096 // (workloads.HEAD_DIM_13B * 2) == g["tokens_per_4KB_page"]
    assert workloads.HEADS_13B == g["heads_opt13b"]
    assert workloads.kv_bytes_per_token() == 20480
    # 40 layers of 40 x 128: batch 32 at 4K tokens is "approximately 100 GB" ...
    gb = workloads.kv_cache_bytes(32, 4096, 40) / 1e9
    assert abs(gb - g["kv_bs32_ctx4k_13b_approx_GB"]) / g["kv_bs32_ctx4k_13b_approx_GB"] < 0.1
    # ... and batch 128 at 2K tokens is "up to 200 GB".
    gb = workloads.kv_cache_bytes(128, 2048, 40) / 1e9
    assert 0.9 * g["kv_bs128_ctx2k_13b_upto_GB"] < gb <= 1.1 * g["kv_bs128_ctx2k_13b_upto_GB"]


def test_embedding_indexed_layout_and_transfer_figures_printed_in_the_paper():
    import inspect

    import bench
    g = read_golden()
    page = 4096
    # one fp16 embedding per token: a 4 KB page holds 2K tokens; grouping 2-8 embeddings per
    # page leaves 1K-256 tokens per group (the sizes the transposed K copy's blocks may take)
    assert page // 2 == g["tokens_per_4KB_page_one_embedding"]
    assert page // (2 * g["embeddings_per_page_max"]) == g["embedding_group_tokens_min"]
    assert page // (2 * g["embeddings_per_page_min"]) == g["embedding_group_tokens_max"]
    kt_default = inspect.signature(bench.measure_sparse).parameters["kt_block_tokens"].default
    assert g["embedding_group_tokens_min"] <= kt_default <= g["embedding_group_tokens_max"]
    keep_default = inspect.signature(bench.measure_sparse).parameters["keep"].default
    assert keep_default * g["default_compression_ratio_inv"] == 1.0
    # per (sequence, head) and step: the cache holds s rows of K and of V; the decode step moves
    # q, k_new, v_new in and one output row back -- s/2 times less
    row = workloads.HEAD_DIM_13B * 2
    for s_len in (1024, 4096, 131072):
        assert (2 * s_len * row) / (4 * row) == g["transfer_reduction_per_s"] * s_len
    # and the benchmark's end-to-end byte accounting is exactly those four rows per (sequence, head)
    w = workloads.STANDARD[4]
    per_step = w.layers * w.batch * w.heads * row
    assert 3 * per_step == 19660800 and per_step == 6553600
