"""Planted mistakes in the oracle (on the CPU): each mutant of the C source must be caught by
the same kind of pin that guards the real oracle.  This checks that the pins are sharp enough
to notice a dropped term, a wrong sign, a wrong index or a transposed operand."""
import ctypes
import math
import os
import subprocess

import numpy as np
import pytest

from oracle import build as oracle_build, capi

SCALE = 1.0 / math.sqrt(128.0)

MUTANTS = {
    "scale_dropped": ("scores[i] = scale * dot;", "scores[i] = dot;"),
    "no_max_subtraction_sign": ("scores[i] = exp(scores[i] - s_max_val);", "scores[i] = exp(s_max_val - scores[i]);"),
    "v_indexed_by_k_offset_plus_one": ("out_row[d] += p * widen_half(v_cache[off + d]);",
                                       "out_row[d] += p * widen_half(v_cache[off + (d + 1) % D]);"),
    "q_transposed_index": ("dot += widen_half(q_row[d]) * widen_half(k_cache[off + d]);",
                           "dot += widen_half(q_row[D - 1 - d]) * widen_half(k_cache[off + d]);"),
    "normaliser_dropped": ("out_row[d] /= z;", "out_row[d] /= 1.0;"),
    "last_token_skipped": ("for (int32_t i = 0; i < L; ++i) {\n        const int64_t off = row_offset(g, b, h, i);\n        if (off < 0) return -3;",
                           "for (int32_t i = 0; i + 1 < L; ++i) {\n        const int64_t off = row_offset(g, b, h, i);\n        if (off < 0) return -3;"),
    "paged_slot_ignores_head": ("return (((int64_t)phys * H + h) * T + (i % T)) * D;",
                                "return (((int64_t)phys * H) * T + (i % T)) * D;"),
    "append_off_by_one": ("const int64_t dst = row_offset(&g, b, h, L - 1);",
                          "const int64_t dst = row_offset(&g, b, h, L > 1 ? L - 2 : 0);"),
    "subnormal_exponent": ("mag = ldexp((double)frac, -24);", "mag = ldexp((double)frac, -25);"),
    "grouped_head_map_interleaved": ("const int err = attend_one(&g, b, hq / group, visible,",
                                     "const int err = attend_one(&g, b, hq % kv_heads, visible,"),
    "grouped_causal_off_by_one": ("int32_t visible = seq_lens[b] - (q_tokens - 1 - t);",
                                  "int32_t visible = seq_lens[b] - (q_tokens - t);"),
    "grouped_token_order_reversed": ("int32_t visible = seq_lens[b] - (q_tokens - 1 - t);",
                                     "int32_t visible = seq_lens[b] - t;"),
}


# Planted mistakes in the sparse (Algorithm 1) oracle: lists of (old, new) replacements.
SPARF_SOURCE = oracle_build.SOURCES[1]
SPARF_MUTANTS = {
    "window_mask_off_by_one": [("order[i].mask = i >= S - window ? 1 : 0;", "order[i].mask = i > S - window ? 1 : 0;")],
    "temperature_ratio_inverted": [("(double)scale / sqrt(ratio);", "(double)scale * sqrt(ratio);")],
    "alpha_summed_over_all_tokens": [("            if (alpha) alpha[pair] = mass;",
                                      "            mass = 0.0; for (int32_t i = 0; i < S; ++i) mass += a[i];\n"
                                      "            if (alpha) alpha[pair] = mass;")],
    "one_minus_alpha_term_dropped": [("mass * attended + (1.0 - mass) * vbar;", "mass * attended;")],
    "mean_value_divided_by_k": [("(double)v_sum[pair * D + d] / (double)S;",
                                 "(double)v_sum[pair * D + d] / (double)(k > 0 ? k : 1);")],
    "top_r_on_signed_q": [("dims[d].key = fabs(widen(qv[d]));", "dims[d].key = widen(qv[d]);"),
                          ("q_l1 += dims[d].key;", "q_l1 += fabs(dims[d].key);"),
                          ("qi_l1 += dims[t].key;", "qi_l1 += fabs(dims[t].key);")],
    "ties_to_the_higher_position": [("return (a->index > b->index) - (a->index < b->index);",
                                     "return (a->index < b->index) - (a->index > b->index);")],
    "transposed_copy_stored_token_major": [("return (((int64_t)phys * g->heads + h) * g->dim + d) * g->tokens + i % g->tokens;",
                                            "return (((int64_t)phys * g->heads + h) * g->tokens + i % g->tokens) * g->dim + d;")],
    "exact_softmax_not_renormalised_over_J": [("const double attended = k > 0 ? o[d] / zs : 0.0;",
                                               "const double attended = k > 0 ? o[d] : 0.0;")],
    "approximate_scores_unscaled": [("a[i] = approx_scale * dot;", "a[i] = dot;")],
}


def build_mutant(tmp_path, name):
    sources = {src: src.read_text() for src in oracle_build.SOURCES}
    if name in MUTANTS:
        target, edits = oracle_build.SOURCE, [MUTANTS[name]]
    else:
        target, edits = SPARF_SOURCE, SPARF_MUTANTS[name]
    for old, new in edits:
        assert old in sources[target], f"mutation site for {name} not found"
        sources[target] = sources[target].replace(old, new, 1)
    paths = []
    for src, text in sources.items():
        path = tmp_path / f"{name}_{src.name}"
        path.write_text(text)
        paths.append(str(path))
    lib = tmp_path / f"{name}.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", *paths, "-o", str(lib), "-lm"],
                   check=True, capture_output=True)
    return str(lib)


def pins(_unused=None):
    """A compact subset of the pins; returns the names of those that fail."""
    failed = []
    rng = np.random.default_rng(5)

    def f16(shape, gain=1.0):
        return (rng.standard_normal(shape) * gain).astype(np.float16)

    def check(name, ok):
        if not ok:
            failed.append(name)

    # single key: out = V row, lse = scale * q.k
    q, k, v = f16((1, 2, 128)), f16((1, 2, 1, 128)), f16((1, 2, 1, 128))
    out, lse, _ = capi.decode_attention(q, k, v, np.array([1]), SCALE)
    check("single_key", np.array_equal(out, v[:, :, 0].astype(np.float64)) and np.allclose(
        lse, float(np.float32(SCALE)) * np.einsum("bhd,bhd->bh", q.astype(np.float64), k[:, :, 0].astype(np.float64)),
        rtol=1e-13))
    # library softmax in float64 on a ragged case
    lens = np.array([5, 37])
    q, k, v = f16((2, 3, 128), 2.0), f16((2, 3, 37, 128), 2.0), f16((2, 3, 37, 128))
    out, lse, _ = capi.decode_attention(q, k, v, lens, SCALE)
    ok = True
    for b, L in enumerate(lens):
        s = np.einsum("hd,hld->hl", q[b].astype(np.float64), k[b, :, :L].astype(np.float64)) * float(np.float32(SCALE))
        w = np.exp(s - s.max(axis=1, keepdims=True))
        w /= w.sum(axis=1, keepdims=True)
        ok &= np.allclose(out[b], np.einsum("hl,hld->hd", w, v[b, :, :L].astype(np.float64)), atol=1e-12, rtol=0)
    check("library_softmax", ok)
    # paged == contiguous with two heads
    kc, vc = f16((1, 2, 8, 128)), f16((1, 2, 8, 128))
    table = np.array([[1, 0]], dtype=np.int32)
    kp = np.stack([kc[0, :, 4:8], kc[0, :, 0:4]])          # [P=2, H=2, T=4, D]
    vp = np.stack([vc[0, :, 4:8], vc[0, :, 0:4]])
    q = f16((1, 2, 128))
    a = capi.decode_attention(q, kc, vc, np.array([7]), SCALE)[0]
    b_ = capi.decode_attention(q, np.ascontiguousarray(kp), np.ascontiguousarray(vp), np.array([7]), SCALE,
                               block_table=table)[0]
    check("paged_equals_contiguous", np.array_equal(a, b_))
    # append lands in the last slot
    kc2, vc2 = kc.copy(), vc.copy()
    kn, vn = f16((1, 2, 128)), f16((1, 2, 128))
    capi.kv_append(kc2, vc2, kn, vn, np.array([6]))
    check("append_slot", np.array_equal(kc2[0, :, 5].view(np.uint16), kn[0].view(np.uint16)) and
          np.array_equal(kc2[0, :, 4].view(np.uint16), kc[0, :, 4].view(np.uint16)))
    # half widening, subnormals included
    bits = np.arange(65536, dtype=np.uint16).reshape(1, 512, 1, 128)
    out, _, _ = capi.decode_attention(np.zeros((1, 512, 128), np.float16), np.zeros((1, 512, 1, 128), np.float16),
                                      bits, np.array([1]), SCALE)
    want = bits.view(np.float16).astype(np.float64).reshape(1, 512, 128)
    fin = ~np.isnan(want)
    check("half_widening", np.array_equal(out[fin], want[fin]))
    # grouped heads and several new tokens: numpy softmax on the expanded, causally cut problem
    L, Tq, Hq, Hkv = 9, 2, 4, 2
    q, k, v = f16((1, Tq, Hq, 128)), f16((1, Hkv, L, 128)), f16((1, Hkv, L, 128))
    out, _ = capi.decode_attention_grouped(q, k, v, np.array([L]), SCALE)
    ok = True
    for t in range(Tq):
        n = L - (Tq - 1 - t)
        for hq in range(Hq):
            hk = hq // (Hq // Hkv)
            s = k[0, hk, :n].astype(np.float64) @ q[0, t, hq].astype(np.float64) * float(np.float32(SCALE))
            w = np.exp(s - s.max())
            ok &= np.allclose(out[0, t, hq], (w / w.sum()) @ v[0, hk, :n].astype(np.float64), atol=1e-12, rtol=0)
    check("grouped_definition", ok)
    return failed


def sparf_pins():
    """A compact subset of the sparse oracle's pins; returns the names of those that fail."""
    from tests.test_oracle_pins_sparf import paged, rows_of
    from oracle import brute

    failed = []
    rng = np.random.default_rng(11)

    def f16(shape, gain=1.0):
        return (rng.standard_normal(shape) * gain).astype(np.float16)

    def check(name, ok):
        if not ok:
            failed.append(name)

    # every dim and every token kept: dense attention, alpha = 1
    lens = np.array([1, 9, 40])
    k, v, kt, v_sum, table = paged(rng, lens, 8)
    q = f16((3, 2, 128), 2.0)
    dense, _, _ = capi.decode_attention(q, k, v, lens, SCALE, block_table=table)
    out, alpha, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, lens, table, r=128, l=0, scale=SCALE)
    check("dense_reduction", np.allclose(out, dense, rtol=0, atol=1e-13) and np.allclose(alpha, 1.0, atol=1e-13))
    # every dim kept: the approximate weights are the dense weights, J their top-k, step 11 spelled out
    lens = np.array([50])
    k, v, kt, v_sum, table = paged(rng, lens, 16, gain=2.0)
    q = f16((1, 2, 128), 2.0)
    _, _, w = capi.decode_attention(q, k, v, lens, SCALE, block_table=table, want_weights=True)
    out, alpha, sel, approx = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([7]), table,
                                                   r=128, l=0, scale=SCALE, want_weights=True)
    ok = np.allclose(approx, w, rtol=0, atol=1e-14)
    for h in range(2):
        want = np.sort(np.argsort(-w[0, h], kind="stable")[:7])
        ok &= np.array_equal(sel[0, h], want) and abs(alpha[0, h] - w[0, h, want].sum()) < 1e-14
        vr = rows_of(v, table, 0, 50, 16)[h].astype(np.float64)
        attn = (w[0, h, want] / w[0, h, want].sum()) @ vr[want]
        vbar = v_sum[0, h].astype(np.float64) / 50
        ok &= np.allclose(out[0, h], alpha[0, h] * attn + (1 - alpha[0, h]) * vbar, atol=1e-13)
    check("all_dims_kept", bool(ok))
    # window as large as k: local attention
    lens = np.array([37])
    k, v, kt, v_sum, table = paged(rng, lens, 8)
    q = f16((1, 2, 128))
    _, _, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.array([10]), table, r=16, l=10, scale=SCALE)
    check("local_window", np.array_equal(sel[0, 0], np.arange(27, 37)) and np.array_equal(sel[0, 1], np.arange(27, 37)))
    # zero query: every score equal, the cut is by position
    q0 = np.zeros((1, 2, 128), np.float16)
    _, _, sel, _ = capi.sparf_attention(q0, k, v, kt, v_sum, lens, np.array([6]), table, r=16, l=2, scale=SCALE)
    check("ties_by_position", np.array_equal(sel[0, 0], np.array([0, 1, 2, 3, 35, 36])))
    # brute force on tiny shapes
    ok = True
    for r, kk, l in [(2, 3, 0), (4, 5, 2), (3, 6, 1)]:
        lens = np.array([11, 6])
        k, v, kt, v_sum, table = paged(rng, lens, 8, heads=2, dim=8, gain=2.0)
        q = f16((2, 2, 8), 2.0)
        scale = 1 / math.sqrt(8)
        out, alpha, sel, _ = capi.sparf_attention(q, k, v, kt, v_sum, lens, np.full(2, kk), table, r=r, l=l, scale=scale)
        for b, n in enumerate(lens):
            kr, vr = rows_of(k, table, b, n, 8), rows_of(v, table, b, n, 8)
            for h in range(2):
                bo, ba, bj = brute.sparf_attention(q[b, h].view(np.uint16).tolist(), kr[h].view(np.uint16).tolist(),
                                                   vr[h].view(np.uint16).tolist(), r, kk, l, scale)
                ok &= sel[b, h, :len(bj)].tolist() == bj and abs(alpha[b, h] - ba) < 1e-13
                ok &= np.allclose(out[b, h], np.array(bo), rtol=0, atol=1e-6)
    check("brute_force", bool(ok))
    # closed forms and the printed ranking (the pins of the sparse pin file itself)
    from tests import test_oracle_pins_sparf as sparse_pins
    for pin in (sparse_pins.test_the_temperature_is_the_printed_one_on_a_two_key_closed_form,
                sparse_pins.test_step_six_is_the_ranking_of_the_printed_sum,
                sparse_pins.test_the_window_survives_a_dominant_early_token):
        try:
            pin()
        except AssertionError:
            failed.append(pin.__name__)
    # the append keeps the embedding-major copy the transpose of K
    lens = np.array([9, 16])
    k, v, kt, v_sum, table = paged(rng, lens, 8)
    kn, vn = f16((2, 2, 128)), f16((2, 2, 128))
    capi.sparf_append(k, v, kt, v_sum, kn, vn, lens, table)
    check("append_transpose", np.array_equal(kt.view(np.uint16),
                                             np.ascontiguousarray(k.transpose(0, 1, 3, 2)).view(np.uint16)))
    return failed


def test_the_real_oracle_passes_the_compact_pins():
    assert pins(None) == []
    assert sparf_pins() == []


ORACLE_FUNCTIONS = ("oracle_num_threads", "oracle_kv_append", "oracle_decode_attention",
                    "oracle_decode_attention_grouped", "oracle_sparf_append", "oracle_sparf_attention")


def load_mutant(lib_path, monkeypatch):
    real = capi._load()
    mutant = ctypes.CDLL(lib_path)
    for fn in ORACLE_FUNCTIONS:
        getattr(mutant, fn).restype = getattr(real, fn).restype
        getattr(mutant, fn).argtypes = getattr(real, fn).argtypes
    monkeypatch.setattr(capi, "_lib", mutant)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_each_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    load_mutant(build_mutant(tmp_path, name), monkeypatch)
    failed = pins(None)
    assert failed, f"mutant {name} slipped through every pin"


@pytest.mark.parametrize("name", sorted(SPARF_MUTANTS))
def test_each_planted_mistake_in_the_sparse_oracle_is_caught(name, tmp_path, monkeypatch):
    load_mutant(build_mutant(tmp_path, name), monkeypatch)
    failed = sparf_pins()
    assert failed, f"mutant {name} slipped through every pin"
    print(name, "caught by", failed)
