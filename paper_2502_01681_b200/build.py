"""Builds libdg4.so (the CUDA library, sm_100a only) in-tree with nvcc."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB = os.path.join(_HERE, "libdg4.so")
SOURCES = sorted(glob.glob(os.path.join(_HERE, "csrc", "dg4_*.cu")))
HEADERS = (sorted(glob.glob(os.path.join(_HERE, "csrc", "*.h"))) + sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cuh")))
           + [os.path.join(_ROOT, "include", "dg4.h")])


def nvcc_path() -> str:
    p = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(p):
        raise RuntimeError("nvcc not found: libdg4.so cannot be built")
    return p


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-pthread", "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_HERE, "csrc"),
           "-o", LIB] + SOURCES
    # compile-time switches of the kernels (e.g. DG4_BUILD_DEFINES="-DDG4_ATTN_KV_EVICT_LAST=1"), for measured variants
    cmd[1:1] = os.environ.get("DG4_BUILD_DEFINES", "").split()
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
