"""Builds and runs csrc/probe_mma_rate.cu: the rate at which the tensor core retires MMAs of each kind when the
operands are already in shared memory (the ceiling the GEMM's mainloop is measured against).

    python -m paper_2504_18547_b200.probe_mma_rate
"""
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent


def main():
    exe = PKG / "probe_mma_rate.bin"
    src = PKG / "csrc" / "probe_mma_rate.cu"
    subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", f"-I{PKG.parent / 'include'}",
                    f"-I{PKG / 'csrc'}", str(src), "-o", str(exe)], check=True)
    sys.exit(subprocess.call([str(exe)]))


if __name__ == "__main__":
    main()
