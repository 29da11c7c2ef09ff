"""Builds libnm_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libnm_b200.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-fvisibility=hidden", "-shared", "-cudart", "static",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(_ROOT, "include", "nm.h")]
    return any(os.path.getmtime(d) > t for d in deps)


TRACE_LIB = os.path.join(_HERE, "libnm_b200_trace.so")
DBG_LIB = os.path.join(_HERE, "libnm_b200_dbg.so")


def build(force: bool = False, verbose: bool = False, trace: bool = False, dbg_modes: bool = False) -> str:
    """trace=True builds a second library with -DNM_TRACE (phase stamps in the tcgen05 kernels, used
    by `python -m bench.trace_phases`); dbg_modes=True a third one with -DNM_DBG_MODES (the NM_DBG timing
    experiments without any stamp code).  The product library contains neither."""
    lib = TRACE_LIB if trace else (DBG_LIB if dbg_modes else LIB)
    if not force and not is_stale(lib):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, "-I", os.path.join(_ROOT, "include"), "-I", CSRC]
    if trace:
        cmd += ["-DNM_TRACE"]
    elif dbg_modes:
        cmd += ["-DNM_DBG_MODES"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", tmp, *sources()]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
