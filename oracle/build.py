"""Compile the C oracle into a shared object next to its source (test infrastructure).

Building the checker is not using it: only tests, the smoke check and the benchmark's
CPU-baseline leg ever load the result.
"""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

_HERE = Path(__file__).resolve().parent
SOURCE = _HERE / "decode_attention_oracle.c"
SOURCES = [SOURCE, _HERE / "sparf_oracle.c"]
LIBRARY = _HERE / "liboracle.so"


def build(force: bool = False) -> Path:
    """gcc -O2 -fopenmp; rebuilt when the source is newer than the library."""
    if not force and LIBRARY.exists() and all(LIBRARY.stat().st_mtime >= f.stat().st_mtime
                                               for f in SOURCES):
        return LIBRARY
    tmp = LIBRARY.with_suffix(f".{os.getpid()}.tmp.so")
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-fno-fast-math", "-ffp-contract=off", *map(str, SOURCES), "-o", str(tmp), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force=True))
