"""Run-to-run determinism on the GPU: the split plan is a function of the shapes only and
every reduction has a fixed order (the selection's atomics only count and collect; ranking
and compaction are order-independent), so two runs on the same bits must agree bit for bit."""
import numpy as np
import pytest
import torch

from paper_2409_04992_b200 import workloads as wl
from tests import gpu_util as gu
from tests import test_gpu_grouped as tg
from tests import test_gpu_sparf as ts

pytestmark = pytest.mark.gpu

LENS = [1, 17, 300, 0, 2049, 5000]


def dense_case(layout, tokens):
    w = wl.Workload("determinism", 6, batch=len(LENS), len_lo=0, len_hi=max(LENS), layout=layout,
                    s_max=max(LENS) if layout == "contiguous" else 0, block_tokens=tokens, heads=5)
    return wl.generate(w, seq_lens=LENS)


@pytest.mark.parametrize("layout,tokens", [("contiguous", 0), ("paged", 16)])
def test_dense_runs_agree_bitwise(layout, tokens):
    runs = [gu.gpu_step(gu.to_device(dense_case(layout, tokens))) for _ in range(3)]
    for out, lse, flags in runs[1:]:
        assert flags == 0
        assert np.array_equal(gu.bits(out), gu.bits(runs[0][0]))
        assert np.array_equal(lse.numpy().view(np.uint32), runs[0][1].numpy().view(np.uint32))


def test_grouped_runs_agree_bitwise():
    runs = [tg.gpu_step(tg.to_device(tg.make("paged", 16, 2, 2, 8, lens=LENS))) for _ in range(3)]
    for out, lse, flags in runs[1:]:
        assert flags == 0
        assert np.array_equal(gu.bits(out), gu.bits(runs[0][0]))
        assert np.array_equal(lse.numpy().view(np.uint32), runs[0][1].numpy().view(np.uint32))


def test_sparse_runs_agree_bitwise():
    runs = []
    for _ in range(3):
        cpu, state = ts.make([1, 17, 300, 0, 2049, 9000], heads=4)
        runs.append(ts.gpu_sparf(gu.to_device(cpu), ts.dev_state(state), r=16, l=16))
    for out, alpha, sel, flags in runs[1:]:
        assert flags == 0
        assert np.array_equal(gu.bits(out), gu.bits(runs[0][0]))
        assert np.array_equal(alpha.view(np.uint32), runs[0][1].view(np.uint32))
        assert np.array_equal(sel, runs[0][2])
