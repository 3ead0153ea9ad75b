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


def build_mutant(tmp_path, name):
    old, new = MUTANTS[name]
    text = oracle_build.SOURCE.read_text()
    assert old in text, f"mutation site for {name} not found"
    src = tmp_path / f"{name}.c"
    src.write_text(text.replace(old, new, 1))
    lib = tmp_path / f"{name}.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", str(src), "-o", str(lib), "-lm"],
                   check=True, capture_output=True)
    return str(lib)


def pins(monkey_lib):
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


def test_the_real_oracle_passes_the_compact_pins():
    assert pins(None) == []


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_each_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    lib_path = build_mutant(tmp_path, name)
    real = capi._load()
    mutant = ctypes.CDLL(lib_path)
    for fn in ("oracle_num_threads", "oracle_kv_append", "oracle_decode_attention",
               "oracle_decode_attention_grouped"):
        getattr(mutant, fn).restype = getattr(real, fn).restype
        getattr(mutant, fn).argtypes = getattr(real, fn).argtypes
    monkeypatch.setattr(capi, "_lib", mutant)
    failed = pins(mutant)
    assert failed, f"mutant {name} slipped through every pin"
