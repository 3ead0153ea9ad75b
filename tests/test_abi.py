"""The C-ABI library: it loads, exports what include/*.h declares, and rejects bad
arguments on the host before anything is enqueued (no GPU needed, no compute calls).

The rejection tests hand the library made-up device addresses.  They are only run in a
process that sees no CUDA device, so that a slip in the order of validation could at worst
end in a launch error, never in a kernel running on a bogus address: on a machine with a GPU
this module re-runs itself in a child process with CUDA_VISIBLE_DEVICES emptied."""
import ctypes
import glob
import os
import re
import subprocess
import sys

import pytest

from paper_2409_04992_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000            # aligned, never dereferenced: every call below fails or no-ops first


def _gpu_visible() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


fake_pointers = pytest.mark.skipif(_gpu_visible(), reason="made-up addresses: run in the GPU-less child instead")


@pytest.mark.skipif(not _gpu_visible(), reason="no GPU here: the tests below run in this process")
def test_rejection_tests_pass_in_a_child_that_sees_no_gpu():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    done = subprocess.run([sys.executable, "-m", "pytest", os.path.abspath(__file__), "-q", "-x",
                           "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True,
                          timeout=600)
    assert done.returncode == 0, done.stdout[-3000:] + done.stderr[-2000:]
    assert " passed" in done.stdout and "skipped" in done.stdout    # only this test is skipped there


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    names = []
    for header in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(header).read(), flags=re.S)
        names += re.findall(r"\b(instinfer_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"instinfer_kv_append", "instinfer_decode_attention",
            "instinfer_decode_attention_paged", "instinfer_workspace_bytes"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    texts = [binding.status_string(s) for s in range(5)]
    assert texts[0] == "ok" and len(set(texts)) == 5
    assert binding.status_string(99) == "unknown status"


def test_plan_and_workspace_are_consistent(lib):
    for batch, heads, L in [(1, 40, 1024), (16, 40, 4096), (64, 40, 16384), (8, 40, 131072), (3, 5, 1)]:
        chunk = binding.plan_chunk_tokens(batch, heads, L)
        assert chunk > 0 and chunk % 64 == 0
        splits = binding.plan_num_splits(batch, heads, L)
        assert splits >= -(-L // chunk)
        need = binding.workspace_bytes(batch, heads, 128, L)
        assert need >= batch * heads * splits * 129 * 4
        assert need % 256 == 0
    assert binding.workspace_bytes(1, 40, 64, 1024) == 0          # unsupported head_dim
    assert binding.workspace_bytes(1, 0, 128, 1024) == 0
    assert binding.workspace_bytes(1, 40, 128, 0) == 0
    binding.set_chunk_tokens(128)
    try:
        assert binding.plan_chunk_tokens(1, 40, 1000) == 128
        assert binding.workspace_bytes(1, 40, 128, 1000) >= 40 * 8 * 129 * 4
    finally:
        binding.set_chunk_tokens(0)
    with pytest.raises(binding.InstInferError):
        binding.set_chunk_tokens(100)


def attn(lib, **kw):
    a = dict(out=FAKE, lse=None, q=FAKE, k=FAKE, v=FAKE, lens=FAKE, batch=2, heads=4, dim=128,
             s_max=256, max_len=256, scale=0.1, ws=FAKE, ws_bytes=1 << 30, flags=None)
    a.update(kw)
    return lib.instinfer_decode_attention(a["out"], a["lse"], a["q"], a["k"], a["v"], a["lens"],
                                          a["batch"], a["heads"], a["dim"], a["s_max"],
                                          a["max_len"], a["scale"], a["ws"], a["ws_bytes"],
                                          a["flags"], None)


def paged(lib, **kw):
    a = dict(out=FAKE, q=FAKE, k=FAKE, v=FAKE, table=FAKE, lens=FAKE, batch=2, heads=4, dim=128,
             T=16, M=16, P=40, max_len=256, scale=0.1, ws=FAKE, ws_bytes=1 << 30)
    a.update(kw)
    return lib.instinfer_decode_attention_paged(a["out"], None, a["q"], a["k"], a["v"], a["table"],
                                                a["lens"], a["batch"], a["heads"], a["dim"], a["T"],
                                                a["M"], a["P"], a["max_len"], a["scale"], a["ws"],
                                                a["ws_bytes"], None, None)


def append(lib, **kw):
    a = dict(kc=FAKE, vc=FAKE, kn=FAKE, vn=FAKE, lens=FAKE, table=None, M=0, T=0, P=0,
             batch=2, heads=4, dim=128, s_max=64)
    a.update(kw)
    return lib.instinfer_kv_append(a["kc"], a["vc"], a["kn"], a["vn"], a["lens"], a["table"], a["M"],
                                   a["T"], a["P"], a["batch"], a["heads"], a["dim"], a["s_max"],
                                   None, None)


@fake_pointers
def test_contiguous_attention_rejects_bad_arguments(lib):
    E = binding
    assert attn(lib, out=None) == E.ERR_INVALID_ARG
    assert attn(lib, q=FAKE + 8) == E.ERR_INVALID_ARG            # misaligned
    assert attn(lib, k=None) == E.ERR_INVALID_ARG
    assert attn(lib, lens=None) == E.ERR_INVALID_ARG
    assert attn(lib, heads=0) == E.ERR_INVALID_ARG
    assert attn(lib, batch=-1) == E.ERR_INVALID_ARG
    assert attn(lib, max_len=0) == E.ERR_INVALID_ARG
    assert attn(lib, max_len=257) == E.ERR_INVALID_ARG           # beyond s_max
    assert attn(lib, scale=float("nan")) == E.ERR_INVALID_ARG
    assert attn(lib, dim=64) == E.ERR_UNSUPPORTED
    assert attn(lib, ws=None) == E.ERR_WORKSPACE
    assert attn(lib, ws_bytes=16) == E.ERR_WORKSPACE
    assert attn(lib, ws=FAKE + 4) == E.ERR_WORKSPACE
    assert attn(lib, batch=0, out=None, q=None) == E.OK          # empty call: nothing enqueued


@fake_pointers
def test_paged_attention_rejects_bad_arguments(lib):
    E = binding
    assert paged(lib, table=None) == E.ERR_INVALID_ARG
    assert paged(lib, T=12) == E.ERR_UNSUPPORTED
    assert paged(lib, T=0) == E.ERR_INVALID_ARG
    assert paged(lib, M=0) == E.ERR_INVALID_ARG
    assert paged(lib, P=0) == E.ERR_INVALID_ARG
    assert paged(lib, max_len=257) == E.ERR_INVALID_ARG          # beyond M*T
    assert paged(lib, dim=256) == E.ERR_UNSUPPORTED
    assert paged(lib, ws_bytes=0) == E.ERR_WORKSPACE
    assert paged(lib, batch=0) == E.OK


@fake_pointers
def test_append_rejects_bad_arguments(lib):
    E = binding
    assert append(lib, kc=None) == E.ERR_INVALID_ARG
    assert append(lib, vn=FAKE + 2) == E.ERR_INVALID_ARG
    assert append(lib, lens=None) == E.ERR_INVALID_ARG
    assert append(lib, s_max=0) == E.ERR_INVALID_ARG
    assert append(lib, dim=96) == E.ERR_UNSUPPORTED
    assert append(lib, table=FAKE, M=4, T=16, P=0) == E.ERR_INVALID_ARG
    assert append(lib, table=FAKE, M=4, T=20, P=9) == E.ERR_UNSUPPORTED
    assert append(lib, batch=0) == E.OK


def grouped(lib, **kw):
    a = dict(out=FAKE, q=FAKE, k=FAKE, v=FAKE, table=None, lens=FAKE, batch=2, tq=1, hq=8, hkv=2,
             dim=128, s_max=256, T=0, M=0, P=0, max_len=256, scale=0.1, ws=FAKE, ws_bytes=1 << 30)
    a.update(kw)
    return lib.instinfer_decode_attention_grouped(a["out"], None, a["q"], a["k"], a["v"], a["table"],
                                                  a["lens"], a["batch"], a["tq"], a["hq"], a["hkv"],
                                                  a["dim"], a["s_max"], a["T"], a["M"], a["P"],
                                                  a["max_len"], a["scale"], a["ws"], a["ws_bytes"],
                                                  None, None)


@fake_pointers
def test_grouped_attention_rejects_bad_arguments(lib):
    E = binding
    assert grouped(lib, out=None) == E.ERR_INVALID_ARG
    assert grouped(lib, hq=7) == E.ERR_INVALID_ARG               # 7 query heads over 2 KV heads
    assert grouped(lib, tq=0) == E.ERR_INVALID_ARG
    assert grouped(lib, max_len=257) == E.ERR_INVALID_ARG        # beyond s_max
    assert grouped(lib, scale=float("inf")) == E.ERR_INVALID_ARG
    assert grouped(lib, hq=34) == E.ERR_UNSUPPORTED              # 17 rows per KV head
    assert grouped(lib, tq=9) == E.ERR_UNSUPPORTED               # 4 x 9 rows
    assert grouped(lib, dim=96) == E.ERR_UNSUPPORTED
    assert grouped(lib, table=FAKE, T=8, M=32, P=9) == E.ERR_UNSUPPORTED      # blocks of 8 tokens
    assert grouped(lib, table=FAKE, T=16, M=4, P=9) == E.ERR_INVALID_ARG      # 256 tokens need 16 blocks
    assert grouped(lib, ws_bytes=64) == E.ERR_WORKSPACE
    assert grouped(lib, batch=0, out=None) == E.OK
    for dim in (64, 128, 256):
        assert binding.grouped_workspace_bytes(2, 2, 8, 2, dim, 4096) > 0
    assert binding.grouped_workspace_bytes(2, 1, 8, 3, 128, 4096) == 0


@fake_pointers
def test_allgather_attention_rejects_bad_arguments(lib):
    import ctypes
    E = binding
    one = (ctypes.c_void_p * 1)(FAKE)

    def call(outs=one, n=1, heads=4, offset=0, total=8, batch=2, ws_bytes=1 << 30, q=FAKE):
        return lib.instinfer_decode_attention_allgather(outs, n, None, q, FAKE, FAKE, None, FAKE, batch,
                                                        heads, offset, total, 128, 256, 0, 0, 0, 256,
                                                        0.1, FAKE, ws_bytes, None, None)

    assert call(outs=None) == E.ERR_INVALID_ARG
    assert call(n=0) == E.ERR_INVALID_ARG
    assert call(n=17) == E.ERR_INVALID_ARG
    assert call(offset=5) == E.ERR_INVALID_ARG                   # heads 5..8 of 8
    assert call(offset=-1) == E.ERR_INVALID_ARG
    assert call(outs=(ctypes.c_void_p * 1)(FAKE + 2)) == E.ERR_INVALID_ARG
    assert call(q=None) == E.ERR_INVALID_ARG
    assert call(ws_bytes=binding.workspace_bytes(2, 4, 128, 256)) == E.ERR_WORKSPACE   # no room for the staged rows
    assert call(batch=0) == E.OK
    assert binding.allgather_workspace_bytes(2, 4, 128, 256) > binding.workspace_bytes(2, 4, 128, 256)


def test_sparse_path_knob(lib):
    for path in (0, 1, 2, 0):
        binding.set_sparse_path(path)
    with pytest.raises(binding.InstInferError):
        binding.set_sparse_path(3)


def test_grouped_path_knob(lib):
    for path in (0, 1, 2, 0):
        binding.set_grouped_path(path)
    with pytest.raises(binding.InstInferError):
        binding.set_grouped_path(3)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIBRARY", tmp_path / "libinstinfer.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load()
