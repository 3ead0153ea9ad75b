"""The public header, used from C: tests/abi_c/abi_check.c is compiled as C99 against
include/instinfer.h alone, linked to the built library and run.  It walks every entry
point's argument-rejection path with the header's prototypes and prints planner / workspace
figures, which must equal what the Python binding's hand-written ctypes signatures return --
a drift between the header and the binding (an int32 and an int64 swapped, an argument
missing) would show here.  The program is run with no CUDA device visible: nothing it calls
may reach the device."""
import os
import subprocess

import pytest

from paper_2409_04992_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def report(tmp_path_factory):
    lib = build.build()
    exe = tmp_path_factory.mktemp("abi_c") / "abi_check"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic",
                    "-I", os.path.join(ROOT, "include"), os.path.join(ROOT, "tests", "abi_c", "abi_check.c"),
                    "-o", str(exe), f"-L{lib.parent}", "-linstinfer", f"-Wl,-rpath,{lib.parent}", "-lm"],
                   check=True, capture_output=True, text=True)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    done = subprocess.run([str(exe)], capture_output=True, text=True, env=env, timeout=120)
    return done


def test_the_c_caller_sees_every_rejection_the_header_promises(report):
    assert report.returncode == 0, report.stdout + report.stderr
    assert "failures 0" in report.stdout and "FAIL" not in report.stdout


def test_the_binding_and_the_c_caller_agree_on_sizes(report):
    figures = dict(line.split() for line in report.stdout.splitlines() if len(line.split()) == 2)
    binding.load()
    assert int(figures["workspace"]) == binding.workspace_bytes(16, 40, 128, 8192) > 0
    assert int(figures["workspace_bad_dim"]) == binding.workspace_bytes(16, 40, 64, 8192) == 0
    assert int(figures["allgather_workspace"]) == binding.allgather_workspace_bytes(16, 5, 128, 8192) > 0
    assert int(figures["grouped_workspace"]) == binding.grouped_workspace_bytes(4, 2, 32, 8, 128, 16384) > 0
    assert int(figures["sparf_workspace"]) == binding.sparf_workspace_bytes(8, 40, 128, 131072, 16384) > 0
    assert int(figures["plan_chunk"]) == binding.plan_chunk_tokens(16, 40, 8192) > 0
    assert int(figures["plan_splits"]) == binding.plan_num_splits(16, 40, 8192) > 0
    assert int(figures["static_bytes"]) == binding.STATIC_WORKSPACE_BYTES
