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
CHECKED_LIBRARY = _HERE / "libinstinfer_checked.so"     # the bounds-checking build (-DINSTINFER_BOUNDS_CHECK)
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


def is_current(library: Path = LIBRARY) -> bool:
    return library.exists() and all(library.stat().st_mtime >= f.stat().st_mtime for f in _inputs())


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    """nvcc -> libinstinfer.so (or, with checked=True, the bounds-checking build
    libinstinfer_checked.so, in which every data-dependent global offset is tested against the
    extent the call's shapes imply and a violation sets status bit 8 instead of being used);
    skipped when the library is newer than every source."""
    library = CHECKED_LIBRARY if checked else LIBRARY
    if not force and is_current(library):
        return library
    tmp = library.with_suffix(f".{os.getpid()}.tmp.so")
    extra = ["-DINSTINFER_BOUNDS_CHECK"] if checked else []
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-I", str(INCLUDE), *map(str, SOURCES), "-o", str(tmp)]
    done = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or done.returncode:
        print(done.stdout + done.stderr)
    if done.returncode:
        raise RuntimeError("nvcc failed")
    os.replace(tmp, library)
    return library


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, checked=True))
