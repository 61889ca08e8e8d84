"""Builds ``libjac.so`` (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2210_01238_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libjac.so"
CHECKED_LIB = PKG / "libjac_checked.so"      # the same library with every kernel address checked (tests)
SOURCES = [CSRC / "jac.cu", CSRC / "jac_static.cu"]
HEADERS = [ROOT / "include" / "jac.h", *sorted(CSRC.glob("*.h")), *sorted(CSRC.glob("*.cuh"))]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    "--fmad=false",            # no FMA contraction anywhere (the kernels use _rn intrinsics as well)
    "-shared", "-Xcompiler", "-fPIC",
    "-cudart", "static",
]


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(p.stat().st_mtime > t for p in [*SOURCES, *HEADERS, Path(__file__)])


def build_checked(force: bool = False) -> Path:
    """The checked build (-DJAC_CHECK_BOUNDS): kernels compare every global address with its array."""
    if not force and CHECKED_LIB.exists():
        t = CHECKED_LIB.stat().st_mtime
        if not any(p.stat().st_mtime > t for p in [*SOURCES, *HEADERS, Path(__file__)]):
            return CHECKED_LIB
    return build(out=CHECKED_LIB, defines=["JAC_CHECK_BOUNDS"])


def build(force: bool = False, verbose: bool = False, out: Path | None = None, defines=()) -> Path:
    """Compile the library.  ``out``/``defines`` build a variant (-DNAME=VALUE) somewhere else."""
    LIB = Path(out) if out else globals()["LIB"]
    if not force and not out and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    cmd = [nvcc, *NVCC_FLAGS, f"-I{ROOT / 'include'}", f"-I{CSRC}", *[f"-D{d}" for d in defines]]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", str(tmp), *map(str, SOURCES)]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode:
        raise RuntimeError(f"nvcc failed ({r.returncode}): {' '.join(cmd)}")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    if "--checked" in sys.argv:
        print(build_checked(force="--force" in sys.argv))
