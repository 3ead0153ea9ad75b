"""Compile the CUDA sources into libinstinfer.so next to this file (sm_100a only)."""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

_HERE = Path(__file__).resolve().parent
CSRC = _HERE / "csrc"
INCLUDE = _HERE.parent / "include"
LIBRARY = _HERE / "libinstinfer.so"
SOURCES = [CSRC / "instinfer_api.cu"]      # it includes the api_*.inl parts
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-Xptxas", "-v"]


def _nvcc() -> str:
    found = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(found):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return found


def _inputs():
    return (list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.inl")) +
            list(INCLUDE.glob("*.h")))


def is_current() -> bool:
    return LIBRARY.exists() and all(LIBRARY.stat().st_mtime >= f.stat().st_mtime for f in _inputs())


def build(force: bool = False, verbose: bool = False) -> Path:
    """nvcc -> libinstinfer.so; skipped when the library is newer than every source."""
    if not force and is_current():
        return LIBRARY
    tmp = LIBRARY.with_suffix(f".{os.getpid()}.tmp.so")
    cmd = [_nvcc(), *NVCC_FLAGS, "-I", str(INCLUDE), *map(str, SOURCES), "-o", str(tmp)]
    done = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or done.returncode:
        print(done.stdout + done.stderr)
    if done.returncode:
        raise RuntimeError("nvcc failed")
    os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force=True, verbose=True))
