"""Build and run the pipe-rate probe behind the issue-bound peak of the search pass:

    python -m paper_2508_21613_b200.pipe_probe [sm_mhz]

Prints, for the fp64 and the int64 recurrence cell, items per clock per SM and scheduler
cycles per warp-item on the GPU it runs on."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_PKG, "csrc", "cm_pipe_probe.cu")
EXE = os.path.join(_PKG, "cm_pipe_probe")


def build() -> str:
    if not os.path.exists(EXE) or os.path.getmtime(EXE) < os.path.getmtime(SRC):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "--fmad=false",
                               "-o", EXE, SRC])
    return EXE


if __name__ == "__main__":
    sys.exit(subprocess.call([build(), *sys.argv[1:]]))
