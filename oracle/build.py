"""Compile the C oracle into oracle/libpalsgd_oracle.so (gcc, OpenMP).

Test infrastructure: nothing on the product path imports this package.
`-ffp-contract=off` keeps every binary32 operation a single IEEE operation.
"""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

HERE = Path(__file__).resolve().parent
LIB = HERE / "libpalsgd_oracle.so"
SOURCES = [HERE / "palsgd_oracle_common.c", HERE / "palsgd_oracle_impl.c"]
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
          "-Wall", "-Wextra"]


def needs_build() -> bool:
    if not LIB.exists():
        return True
    newest = max(p.stat().st_mtime for p in SOURCES + [Path(__file__)])
    return LIB.stat().st_mtime < newest


def build(force: bool = False) -> Path:
    if not force and not needs_build():
        return LIB
    # the system gcc (the image's $CC points at a wrapper without libgomp)
    cc = os.environ.get("PALSGD_ORACLE_CC") or shutil.which("gcc", path="/usr/bin:/bin") or "gcc"
    objs = []
    common = HERE / "_oracle_common.o"
    subprocess.check_call([cc, *CFLAGS, "-c", str(SOURCES[0]), "-o", str(common)])
    objs.append(common)
    for real, suffix in (("float", "f32"), ("double", "f64")):
        o = HERE / f"_oracle_impl_{suffix}.o"
        subprocess.check_call([cc, *CFLAGS, f"-DREAL={real}", f"-DSUFFIX={suffix}",
                               "-c", str(SOURCES[1]), "-o", str(o)])
        objs.append(o)
    tmp = HERE / f"libpalsgd_oracle.{os.getpid()}.tmp.so"
    subprocess.check_call([cc, "-shared", "-fopenmp", *map(str, objs), "-lm", "-o", str(tmp)])
    os.replace(tmp, LIB)
    for o in objs:
        o.unlink(missing_ok=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
