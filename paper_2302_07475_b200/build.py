"""Builds libs3gd.so (the C-ABI library) in-tree with nvcc for sm_100a.

Usage: python -m paper_2302_07475_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libs3gd.so")
SOURCES = ["s3gd_api.cu", "s3gd_vote.cu", "s3gd_signplane.cu", "s3gd_filter.cu", "s3gd_select.cu", "s3gd_select_small.cu", "s3gd_noalloc.cu", "s3gd_randk.cu", "s3gd_exchange.cu"]
HEADERS = ["s3gd_common.cuh", "s3gd_tile.cuh", "s3gd_select_emit.inl"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; the CUDA library cannot be built")


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "s3gd.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu file for sm_100a into one shared library; returns its path."""
    if os.environ.get("S3GD_LIBRARY"):          # another build was asked for: leave the in-tree one alone
        return os.environ["S3GD_LIBRARY"]
    if not force and not _stale():
        return LIB
    cmd = [
        _nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-shared",
        "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-DS3GD_NOALLOC_MAX_D=4194304ull",
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libs3gd.so")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
