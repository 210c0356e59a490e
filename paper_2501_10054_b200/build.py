"""Builds libtardis.so (sm_100a) in-tree with nvcc.  Usage: python -m paper_2501_10054_b200.build"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libtardis.so")
LIB_STAMPS = os.path.join(PKG, "libtardis_stamps.so")
SOURCES = ["api.cu", "fold.cu", "generic.cu", "decode.cu", "fused.cu", "gemm.cu", "batched.cu", "calibrate.cu", "stack.cu", "gptq.cu"]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "tardis.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, stamps: bool = False) -> str:
    """Builds the library.  stamps=True builds libtardis_stamps.so instead: the same sources with
    -DTARDIS_PHASE_STAMPS (the fused decode kernel records its phase boundaries; profiling only)."""
    out = LIB_STAMPS if stamps else LIB
    if not force and not stamps and not needs_build():
        return LIB
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-t", "8", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", out] + (["-DTARDIS_PHASE_STAMPS"] if stamps else []) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
    if verbose:
        print(r.stderr)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, stamps="--stamps" in sys.argv))
