"""Builds libslidedp.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Usage: python -m paper_2609_34162_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libslidedp.so")
SOURCES = [os.path.join(CSRC, f) for f in ("common.cu", "context.cu", "update.cu", "stream.cu",
                                           "model.cu", "ipc.cu")]
DEPENDS = SOURCES + [os.path.join(CSRC, f) for f in ("kernels.cuh", "cast_kernel.cuh",
                                                     "device_utils.cuh", "types.h", "internal.h")]
DEPENDS.append(os.path.join(ROOT, "include", "slidedp.h"))


def nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def build(force: bool = False, verbose: bool = False) -> str:
    stale = (not os.path.exists(LIB)
             or os.path.getmtime(LIB) < max(os.path.getmtime(p) for p in DEPENDS))
    if force or stale:
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = [nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
               "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
               "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", tmp] + SOURCES
        if verbose:
            cmd.insert(1, "-Xptxas"); cmd.insert(2, "-v")
        subprocess.run(cmd, check=True)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
