"""Build and run the copy-engine probes (bench/tma_probe.cu) on the current GPU:

    python -m bench.tma_probe

Prints the issue cost of the asynchronous instructions on one thread, the latency of tiled TMA
loads, and the L2 / HBM -> shared-memory feed rate per SM of a ring of TMA loads.  Every wait in
the probe is a bounded poll."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "tma_probe.cu")
EXE = os.path.join(_HERE, "tma_probe.bin")


def build(force: bool = False) -> str:
    if not force and os.path.exists(EXE) and os.path.getmtime(EXE) >= os.path.getmtime(SRC):
        return EXE
    nvcc = os.environ.get("NVCC") or shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-o", EXE, SRC])
    return EXE


if __name__ == "__main__":
    sys.exit(subprocess.call([build()]))
