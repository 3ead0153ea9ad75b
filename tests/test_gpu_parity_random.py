"""GPU parity on randomly drawn configurations (seeded): layouts, block sizes, batch and head
counts, ragged lengths including 0 and 1, forced and automatic split plans, scales and query
gains, for the dense path, the sparse path (both of its forms) and the grouped-head /
multi-token path."""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import binding, workloads as wl
from tests import gpu_util as gu
from tests import test_gpu_grouped as tg
from tests import test_gpu_sparf as sp

pytestmark = pytest.mark.gpu


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    paged = bool(rng.integers(2))
    tokens = int(rng.choice([8, 16, 24, 32, 48, 64, 128])) if paged else 0
    batch, heads = int(rng.integers(1, 7)), int(rng.integers(1, 6))
    top = int(rng.choice([40, 200, 700, 1500]))
    lens = [int(x) for x in rng.integers(0, top + 1, size=batch)]
    if rng.integers(3) == 0:
        lens[int(rng.integers(batch))] = 1
    if max(lens) == 0:
        lens[0] = 5
    chunk = int(rng.choice([0, 0, 64, 128, 256]))
    gain = float(rng.choice([0.5, 1.0, 3.0]))
    scale = float(rng.choice([1 / np.sqrt(128), 0.05, 0.2]))
    return paged, tokens, heads, lens, chunk, gain, scale, int(rng.integers(5))


@pytest.mark.parametrize("seed", range(24))
def test_dense_random_configuration(seed):
    paged, tokens, heads, lens, chunk, gain, scale, index = draw(seed)
    w = wl.Workload("random", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout="paged" if paged else "contiguous", s_max=0 if paged else max(lens) + 2,
                    block_tokens=tokens, heads=heads, peaked_fraction=0.03 if seed % 3 == 0 else 0.0)
    cpu = wl.generate(w, seq_lens=lens)
    cpu.q.mul_(gain)
    cpu.scale = scale
    out, lse, flags = gu.gpu_step(gu.to_device(cpu), chunk_tokens=chunk)
    want, want_lse = gu.oracle_step(cpu)
    assert flags == 0
    gu.assert_close(out, want, lse, want_lse, f"seed {seed}: {w.layout} T={tokens} lens={lens} chunk={chunk}")


@pytest.mark.parametrize("seed", range(12))
def test_sparse_random_configuration(seed):
    _, _, heads, lens, _, gain, scale, index = draw(100 + seed)
    rng = np.random.default_rng(2000 + seed)
    tokens = int(rng.choice([8, 16, 32, 64]))
    r = int(rng.choice([1, 8, 16, 32, 128]))
    window = int(rng.choice([0, 4, 32]))
    keep = float(rng.choice([0.0625, 0.125, 0.5]))
    w = wl.Workload("random_sparse", index, batch=len(lens), len_lo=min(lens), len_hi=max(lens),
                    layout="paged", block_tokens=tokens, heads=heads)
    cpu = wl.generate(w, seq_lens=lens)
    cpu.q.mul_(gain)
    cpu.scale = scale
    state = wl.make_sparf_state(cpu, keep)
    binding.set_sparse_path(1 + seed % 2)            # alternate between the two forms of steps 1-7
    try:
        sp.run_and_check(cpu, state, r, window, f"seed {seed}: T={tokens} r={r} l={window} keep={keep} lens={lens}")
    finally:
        binding.set_sparse_path(0)


@pytest.mark.parametrize("seed", range(24))
def test_grouped_random_configuration(seed):
    rng = np.random.default_rng(3000 + seed)
    paged = bool(rng.integers(2))
    tokens = int(rng.choice([16, 32, 48, 64, 128])) if paged else 0
    dim = int(rng.choice([64, 128, 128, 256]))
    group = int(rng.choice([1, 2, 4, 8, 16]))
    q_tokens = int(rng.integers(1, 16 // group + 1))
    kv_heads = int(rng.integers(1, 4))
    batch = int(rng.integers(1, 6))
    top = int(rng.choice([40, 300, 1200]))
    lens = [int(x) for x in rng.integers(0, top + 1, size=batch)]
    if max(lens) == 0:
        lens[0] = 7
    chunk = int(rng.choice([0, 0, 64, 128, 512]))
    g = tg.make("paged" if paged else "contiguous", tokens, kv_heads, q_tokens, group * kv_heads,
                dim=dim, lens=lens, index=int(rng.integers(5)))
    g.q.mul_(float(rng.choice([0.5, 1.0, 3.0])))
    g.base.scale = float(rng.choice([1 / np.sqrt(dim), 0.05, 0.2]))
    tg.check(g, chunk, f"seed {seed}: {'paged' if paged else 'contiguous'} T={tokens} D={dim} G={group} "
                       f"Tq={q_tokens} Hkv={kv_heads} lens={lens} chunk={chunk}")
