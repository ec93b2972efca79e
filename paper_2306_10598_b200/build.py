"""Builds libdropcompute.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
SRC = os.path.join(PKG, "csrc", "dropcompute.cu")
HDRS = (os.path.join(ROOT, "include", "dropcompute.h"), os.path.join(ROOT, "include", "dropcompute_dev.h"))
LIB = os.path.join(PKG, "libdropcompute.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",           # every fp32 operation of the sweep is a single IEEE operation, never contracted
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def _cuda_sources():
    csrc = os.path.dirname(SRC)
    return sorted(os.path.join(csrc, f) for f in os.listdir(csrc) if f.endswith((".cu", ".cuh")))


def source_hash() -> str:
    """Hash of the CUDA sources (names and contents), baked into the library as dc_kernel_version(): a profile
    filed under one hash is never reported for a library built from other kernels."""
    h = hashlib.sha1()
    for path in _cuda_sources():
        h.update(os.path.basename(path).encode())
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in (*_cuda_sources(), *HDRS, os.path.abspath(__file__)))


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, f'-DDC_SOURCE_HASH="{source_hash()}"', "-I", os.path.join(ROOT, "include"),
           "-I", os.path.dirname(SRC), "-o", tmp, SRC]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, LIB)
    if verbose:
        print(res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv))
