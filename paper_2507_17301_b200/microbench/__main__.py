"""Compiles and runs the rate microbenchmark (`rates.cu`) on the current GPU:

    python -m paper_2507_17301_b200.microbench

It measures, in isolation, the costs the convolution kernels are built around: reading a slab row from shared
memory and picking a tile's retained columns in registers, and the issue / execution rate of TF32 tcgen05 MMAs
of several widths from one to four issuing threads.  The library does not use it.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))


def main() -> int:
    exe = os.path.join(HERE, "rates")
    src = os.path.join(HERE, "rates.cu")
    if not os.path.exists(exe) or os.path.getmtime(exe) < os.path.getmtime(src):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-o", exe, src])
    return subprocess.call([exe])


if __name__ == "__main__":
    sys.exit(main())
