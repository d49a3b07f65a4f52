"""Builds liballocmoe.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2604_08133_b200.build [--force] [--verbose] [--checked]

--checked builds liballocmoe_checked.so instead: the same library with -DALLOCMOE_CHECKED, in which every
device-side index that had to be clamped into range is also reported in the status word.  Load it by setting
ALLOCMOE_LIB to its path.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "liballocmoe.so")
SOURCES = ["api.cu", "gate.cu", "select.cu", "permute.cu", "route.cu", "ffn.cu", "combine.cu", "alloc_l.cpp", "tmap.cpp"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "allocmoe.h")]
    return any(os.path.getmtime(d) > t for d in deps)


LIB_CHECKED = os.path.join(PKG, "liballocmoe_checked.so")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    out = LIB_CHECKED if checked else LIB
    if not force and not needs_build(out):
        return out
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if checked:
        cmd += ["-DALLOCMOE_CHECKED"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", out]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed")
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
