"""In-tree build of the CUDA library (sm_100a only).

`python -m paper_2109_08751_b200.build` or `build()` compiles csrc/*.cu|cpp into
libsparbit_b200.so next to this file.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libsparbit_b200.so"
SOURCES = [CSRC / "api.cu", CSRC / "multi.cu", CSRC / "schedule.cpp"]
HEADERS = [CSRC / "kernels.cuh", CSRC / "phase_desc.h", CSRC / "schedule.h", CSRC / "plan_access.h",
           HERE.parent / "include" / "sparbit.h"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def _nvcc() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if Path(cand).exists() else "nvcc"


def is_stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(f.stat().st_mtime > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not is_stale():
        return LIB
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = [_nvcc(), *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []),
           *map(str, SOURCES), "-o", str(tmp)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
