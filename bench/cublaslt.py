"""ctypes wrapper of the cuBLASLt comparator (bench/cublaslt_cmp.cu): a dense library GEMM on the same
buffers, every algorithm the heuristic offers timed, the fastest reported.  Harness only."""
from __future__ import annotations

import ctypes
import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "cublaslt_cmp.cu")
LIB = os.path.join(_HERE, "libcublaslt_cmp.so")
_lib = None


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    nvcc = os.environ.get("NVCC") or shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-std=c++17", "-Xcompiler", "-fPIC,-fvisibility=hidden", "-shared", "-cudart", "shared",
                           "-o", tmp, SRC, "-lcublasLt"])
    os.replace(tmp, LIB)
    return LIB


def lib():
    global _lib
    if _lib is None:
        import torch  # noqa: F401  (loads the CUDA runtime the process shares)
        try:                     # the cuBLASLt that ships with torch, so that both comparators use one library
            import nvidia.cublas
            ctypes.CDLL(os.path.join(os.path.dirname(nvidia.cublas.__file__), "lib", "libcublasLt.so.12"), mode=ctypes.RTLD_GLOBAL)
        except Exception:
            pass
        L = ctypes.CDLL(build())
        L.lt_gemm_sweep.restype = ctypes.c_int
        L.lt_gemm_sweep.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                    ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int)]
        _lib = L
    return _lib


_ws = {}


def sweep(X, W, Y, stream, max_algos: int = 16, reps: int = 10):
    """X [T, K], W [O, K], Y [T, O] torch CUDA tensors (int8 -> int32, or fp16 -> fp16).
    Returns dict(best_us, heuristic_us, algos_timed) or None when cuBLASLt offers nothing."""
    import torch
    T, K = X.shape
    O = W.shape[0]
    dtype = 0 if X.dtype == torch.int8 else 1
    dev = X.device
    if dev not in _ws:
        _ws[dev] = torch.empty(64 << 20, dtype=torch.uint8, device=dev)
    ws = _ws[dev]
    best, first, n = ctypes.c_float(0), ctypes.c_float(0), ctypes.c_int(0)
    rc = lib().lt_gemm_sweep(dtype, T, O, K, X.data_ptr(), W.data_ptr(), Y.data_ptr(), ws.data_ptr(), ws.numel(), max_algos, reps,
                             stream.cuda_stream, ctypes.byref(best), ctypes.byref(first), ctypes.byref(n))
    if rc != 0:
        return None
    return {"best_us": float(best.value), "heuristic_us": float(first.value), "algos_timed": int(n.value)}
