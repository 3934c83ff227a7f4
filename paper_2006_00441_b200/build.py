"""Builds libdasgd.so in-tree with nvcc for sm_100a.

    python -m paper_2006_00441_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libdasgd.so")
SOURCES = [os.path.join(CSRC, "dasgd_api.cu"), os.path.join(CSRC, "dasgd_noalloc.cu"), os.path.join(CSRC, "dasgd_nccl.cu")]
HEADERS = [os.path.join(CSRC, "dasgd_kernels.cuh"), os.path.join(ROOT, "include", "dasgd.h")]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libdasgd.so cannot be built")
    return exe


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    newest = max(os.path.getmtime(p) for p in SOURCES + HEADERS)
    return os.path.getmtime(LIB) >= newest


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-shared", "-Xcompiler", "-fPIC",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += SOURCES + ["-ldl", "-o", LIB + ".tmp"]
    subprocess.run(cmd, check=True)
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
