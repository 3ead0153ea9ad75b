"""The benchmark's output contract, on a small workload (one JSON line with the agreed keys)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_prints_one_json_line_with_the_contract_keys():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "1", "--steps", "3", "--warmup", "3",
           "--no-others", "--cpu-seconds", "1"]
    done = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert done.returncode == 0, done.stderr[-2000:]
    lines = [x for x in done.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
                "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 3 and d["value"] > 100
    assert d["config"]["workload"] == "ctx2k-4k_b16_contiguous" and d["vs_baseline"] is None
    assert d["gpu_launches"] == 3 * 3                      # append + split + merge per step
    assert d["e2e"]["h2d_bytes_per_step"] == 3 * 16 * 40 * 128 * 2 and d["e2e"]["value"] > 0
    assert d["roofline"]["bound"] == "hbm" and 0 < d["roofline"]["frac"] < 1.5
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["status_flags"] == 0
