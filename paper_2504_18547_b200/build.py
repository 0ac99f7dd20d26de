"""Builds libvitint.so (sm_100a) in-tree with nvcc.  No GPU is needed to compile."""
from __future__ import annotations

import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libvitint.so"
INCLUDE = PKG.parent / "include"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def sources():
    return sorted(CSRC.glob("*.cu")) + sorted(CSRC.glob("*.cuh")) + [INCLUDE / "vitint.h"]


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(p.stat().st_mtime > t for p in sources())


def build_library(force: bool = False, verbose: bool = False) -> Path:
    if force or needs_build():
        cmd = ["nvcc", *NVCC_FLAGS, f"-I{INCLUDE}", str(CSRC / "vitint_lib.cu"), "-o", str(LIB)]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.run(cmd, check=True)
    return LIB


TRACE_LIB = PKG / "libvitint_trace.so"


def build_trace_library() -> Path:
    """Diagnostic build (-DVITINT_TRACE): the GEMM kernel records a timeline of its warp roles (see trace_gemm.py).
    A separate file; the product library is never built with the flag."""
    cmd = ["nvcc", *NVCC_FLAGS, "-DVITINT_TRACE", f"-I{INCLUDE}", str(CSRC / "vitint_lib.cu"), "-o", str(TRACE_LIB)]
    subprocess.run(cmd, check=True)
    return TRACE_LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
