"""The seeded input generator: layout conventions, poison placement, determinism (no GPU)."""
import numpy as np
import pytest
import torch

from oracle import capi
from paper_2409_04992_b200 import workloads as wl


def small(w, **kw):
    return w.replace(**{'heads': 3, **kw})


CASES = [
    small(wl.STANDARD[0], len_lo=70, len_hi=70, s_max=70),
    small(wl.STANDARD[1], batch=4, len_lo=20, len_hi=90, s_max=90),
    small(wl.STANDARD[2], batch=3, len_lo=48, len_hi=48),
    small(wl.STANDARD[3], batch=2, len_lo=130, len_hi=130),
    small(wl.STANDARD[4], batch=4, len_lo=33, len_hi=97, layers=2),
]


def bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def test_standard_list_matches_the_five_configurations():
    names = [(w.batch, w.len_lo, w.len_hi, w.layout, w.block_tokens, w.layers) for w in wl.STANDARD]
    assert names == [(1, 1024, 1024, "contiguous", 0, 1), (16, 2048, 4096, "contiguous", 0, 1),
                     (64, 16384, 16384, "paged", 16, 1), (8, 131072, 131072, "paged", 64, 1),
                     (16, 4096, 8192, "paged", 32, 40)]
    assert all(w.heads == 40 and w.head_dim == 128 for w in wl.STANDARD)
    assert wl.STANDARD[1].s_max == 4096 and wl.STANDARD[3].peaked_fraction == 0.01


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_same_seed_same_bits_and_layers_differ(w):
    a, b = wl.generate(w), wl.generate(w)
    for name in ("q", "k_new", "v_new", "k_cache", "v_cache", "seq_lens"):
        assert torch.equal(getattr(a, name).view(torch.int16) if getattr(a, name).dtype == torch.float16
                           else getattr(a, name),
                           getattr(b, name).view(torch.int16) if getattr(b, name).dtype == torch.float16
                           else getattr(b, name))
    c = wl.generate(w, layer=1)
    assert c.seq_lens_host == a.seq_lens_host
    assert not torch.equal(c.q.view(torch.int16), a.q.view(torch.int16))
    assert all(w.len_lo <= n <= w.len_hi for n in a.seq_lens_host)


@pytest.mark.parametrize("w", [c for c in CASES if c.paged], ids=lambda w: w.name)
def test_block_table_is_one_permutation_with_spares(w):
    c = wl.generate(w)
    T = w.block_tokens
    table = c.block_table.numpy()
    used = []
    for b, n in enumerate(c.seq_lens_host):
        nb = -(-n // T)
        used += table[b, :nb].tolist()
        assert np.all(table[b, nb:] == -1)
    P = c.k_cache.shape[0]
    assert len(set(used)) == len(used) == P - w.spare_blocks
    assert min(used) >= 0 and max(used) < P
    spare = sorted(set(range(P)) - set(used))
    assert all(np.all(bits(c.k_cache[p]) == wl.NAN_BITS) for p in spare)
    assert sorted(used) != used            # physically shuffled


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_poison_sits_exactly_outside_the_attended_range(w):
    c = wl.generate(w)
    q, kn, vn = (t.numpy() for t in (c.q, c.k_new, c.v_new))
    k, v = c.k_cache.numpy().copy(), c.v_cache.numpy().copy()
    table = None if c.block_table is None else c.block_table.numpy()
    lens = np.array(c.seq_lens_host)
    # Before the append the slot of the new token is poisoned: attention sees NaN ...
    out, _, _ = capi.decode_attention(q, k, v, lens, c.scale, block_table=table)
    assert np.isnan(out).all()
    # ... after it, nothing attended is poisoned.
    capi.kv_append(k, v, kn, vn, lens, block_table=table)
    out, lse, _ = capi.decode_attention(q, k, v, lens, c.scale, block_table=table)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    # gather_rows walks the same layout.
    case2 = wl.Case(**{**c.__dict__, "k_cache": torch.from_numpy(k), "v_cache": torch.from_numpy(v)})
    kr, vr = wl.gather_rows(case2, w.batch - 1, 1)
    L = c.seq_lens_host[-1]
    o1, _, _ = capi.decode_attention(q[-1:, 1:2], kr.numpy()[None, None], vr.numpy()[None, None],
                                     np.array([L]), c.scale)
    assert np.array_equal(o1[0, 0], out[-1, 1])


def test_peaked_keys_are_about_one_percent_times_four():
    w = small(wl.STANDARD[3], batch=1, len_lo=64 * 400, len_hi=64 * 400, heads=2)
    c = wl.generate(w, poison=False)
    rms = c.k_cache.float().pow(2).mean(dim=-1).sqrt().flatten()
    share = (rms > 2.5).float().mean().item()
    assert 0.005 < share < 0.015
    assert abs(rms[rms > 2.5].mean().item() - 4.0) < 0.2
    assert abs(c.v_cache.float().std().item() - 1.0) < 0.01


def test_byte_accounting():
    c = wl.generate(CASES[1])
    assert c.kv_tokens == sum(c.seq_lens_host)
    assert c.kv_bytes_read == c.kv_tokens * 3 * 128 * 4
