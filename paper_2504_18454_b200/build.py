"""Compile the CUDA library in-tree: paper_2504_18454_b200/libpalsgd.so (sm_100a).

nvcc cross-compiles without a GPU.  The runtime is linked statically, so the
library loads (and its pure-host entry points work) on a machine without a
driver; anything that touches the GPU then returns PALSGD_ECUDA.
"""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libpalsgd.so"
SOURCES = [CSRC / "palsgd_api.cu", CSRC / "palsgd_noalloc.cu"]
DEPS = sorted(CSRC.glob("*.cu*")) + [HERE.parent / "include" / "palsgd.h", Path(__file__)]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-fmad=false",                 # belt and braces: the kernels use *_rn intrinsics anyway
    "-Xcompiler", "-fPIC,-O2,-Wall",
    "-cudart", "static",
    "-shared",
]


def nvcc_path() -> str:
    return os.environ.get("NVCC") or shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"


def needs_build() -> bool:
    if not LIB.exists():
        return True
    return LIB.stat().st_mtime < max(p.stat().st_mtime for p in DEPS)


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not needs_build():
        return LIB
    tmp = HERE / f"libpalsgd.{os.getpid()}.tmp.so"
    cmd = [nvcc_path(), *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []),
           *map(str, SOURCES), "-o", str(tmp)]
    env = dict(os.environ)
    env.pop("CC", None); env.pop("CXX", None)
    subprocess.check_call(cmd, env=env)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
