"""Build and run the main-loop probe (bench/mainloop_probe.cu) on the current GPU:

    python -m bench.mainloop_probe

A minimal dense INT8 tcgen05 GEMM main loop on the DeiT-B fc2 operands with the parts of its
epilogue switchable (none / tcgen05.ld / + st.shared / + TMA stores / + plain stores / stores into an
L2-resident window) and a loads-only and a stores-only run.  Every wait in the probe is a bounded poll."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
SRC = os.path.join(_HERE, "mainloop_probe.cu")
EXE = os.path.join(_HERE, "mainloop_probe.bin")


def build(force: bool = False) -> str:
    if not force and os.path.exists(EXE) and os.path.getmtime(EXE) >= os.path.getmtime(SRC):
        return EXE
    nvcc = os.environ.get("NVCC") or shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17",
                           "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_ROOT, "paper_2607_12505_b200", "csrc"),
                           "-o", EXE, SRC, "-lcuda"])
    return EXE


if __name__ == "__main__":
    sys.exit(subprocess.call([build()]))
