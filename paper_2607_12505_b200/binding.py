"""Thin ctypes binding over libnm_b200.so (the C ABI declared in include/nm.h).

Argument marshalling only: every step of the GEMM runs in the library's CUDA
kernels.  torch is used to own device memory and to supply the current stream.
There is no CPU fallback: if the library cannot be loaded or built, importing
the binding's entry points raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np

from . import build as _build

# ---- enums mirrored from nm.h --------------------------------------------------------
NM_OK, NM_ERR_INVALID_ARG, NM_ERR_SHAPE, NM_ERR_ALIGN, NM_ERR_NOT_NM = 0, 1, 2, 3, 4
NM_ERR_UNSUPPORTED, NM_ERR_WORKSPACE, NM_ERR_ARCH, NM_ERR_CUDA, NM_ERR_TIMEOUT = 5, 6, 7, 8, 9
NM_I8, NM_F16 = 0, 1
NM_OUT_I32, NM_OUT_F32, NM_OUT_F16, NM_OUT_I8 = 0, 1, 2, 3
NM_IMG_CANONICAL, NM_IMG_HW24, NM_IMG_DENSE, NM_IMG_REMAP48, NM_IMG_AUTO = 1, 2, 4, 8, 0x80000000
NM_PATH_SIMT, NM_PATH_UMMA_DENSE, NM_PATH_UMMA_SP24, NM_PATH_UMMA_DECODE, NM_PATH_UMMA_EXPAND, NM_PATH_UMMA_REMAP48 = 0, 1, 2, 3, 4, 5
NM_RES_NONE, NM_RES_X, NM_RES_W = 0, 1, 2
NM_MERGE_WORKSPACE, NM_MERGE_CLUSTER = 0, 1
NM_PLAN_DIAG_STALL = 1

EXPORTS = [
    "nm_packed_size", "nm_compress", "nm_compress_host", "nm_prune_magnitude", "nm_decompress",
    "nm_export_canonical", "nm_plan_create", "nm_plan_shape", "nm_spmm", "nm_latency_table",
    "nm_status_string", "nm_launch_count", "nm_spmm_static_scratch", "nm_spmm_ex",
    "nm_predictor_fit", "nm_predictor_eval", "nm_search", "nm_fitness_separable",
]


class NMWeight(ctypes.Structure):
    _fields_ = [
        ("magic", ctypes.c_uint32), ("version", ctypes.c_uint32),
        ("O", ctypes.c_int32), ("K", ctypes.c_int32), ("n", ctypes.c_int32), ("m", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("images", ctypes.c_uint32),
        ("dev_base", ctypes.c_void_p), ("bytes", ctypes.c_uint64),
        ("off_canonical", ctypes.c_uint64),
        ("off_hw24_values", ctypes.c_uint64), ("off_hw24_meta", ctypes.c_uint64), ("off_dense", ctypes.c_uint64),
        ("hw24_row_bytes", ctypes.c_uint64), ("dense_row_bytes", ctypes.c_uint64),
        ("hw24_meta_kblocks", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("off_remap_values", ctypes.c_uint64), ("off_remap_meta", ctypes.c_uint64), ("remap_row_bytes", ctypes.c_uint64),
        ("remap_meta_kblocks", ctypes.c_int32), ("remap_k", ctypes.c_int32), ("remap_k_main", ctypes.c_int32),
        ("reserved2", ctypes.c_int32),
    ]


class NMPlan(ctypes.Structure):
    _fields_ = [
        ("path", ctypes.c_int32), ("tile_o", ctypes.c_int32), ("tile_t", ctypes.c_int32),
        ("cta_group", ctypes.c_int32), ("split_k", ctypes.c_int32), ("stages", ctypes.c_int32),
        ("image", ctypes.c_uint32), ("resident", ctypes.c_int32),
        ("workspace_bytes", ctypes.c_uint64), ("predicted_us", ctypes.c_float), ("issuers", ctypes.c_int32),
        ("merge", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_ if not k.startswith("reserved")}


class NMEpilogue(ctypes.Structure):
    _fields_ = [("scale_dev", ctypes.c_void_p), ("bias_dev", ctypes.c_void_p), ("relu", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class NMLatencyRow(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in
                ("T", "O", "K", "n", "m", "dtype", "out_dtype", "path", "tile_t", "split_k", "reps", "status")] + \
               [("us_mean", ctypes.c_float), ("us_min", ctypes.c_float)]


class NMSearchConfig(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int32), ("levels", ctypes.c_int32), ("generations", ctypes.c_int32),
                ("offspring", ctypes.c_int32), ("overshoot_k", ctypes.c_int32), ("n_init", ctypes.c_int32),
                ("elitist", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("target_us", ctypes.c_double), ("seed", ctypes.c_uint64)]


class NMSearchResult(ctypes.Structure):
    _fields_ = [("fitness", ctypes.c_double), ("latency_us", ctypes.c_double),
                ("fitness_evals", ctypes.c_uint64), ("latency_evals", ctypes.c_uint64),
                ("feasible", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class NMFitnessSeparableArgs(ctypes.Structure):
    _fields_ = [("gain", ctypes.POINTER(ctypes.c_double)), ("levels", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("noise", ctypes.c_double), ("seed", ctypes.c_uint64)]


FITNESS_FN = ctypes.CFUNCTYPE(ctypes.c_double, ctypes.POINTER(ctypes.c_int32), ctypes.c_int32, ctypes.c_void_p)


class NMError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        name = lib().nm_status_string(status).decode()
        super().__init__(f"{where}: {name}{(' ' + detail) if detail else ''}")


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building if the sources are newer) the CUDA library.  Fails loudly."""
    global _lib
    if _lib is not None:
        return _lib
    if os.environ.get("NM_B200_TRACE") == "1":      # the trace build (phase stamps), for bench.trace_phases only
        path = _build.build(trace=True)
    elif os.environ.get("NM_B200_TRACE") == "2":    # the NM_DBG timing experiments without stamp code (harness only)
        path = _build.build(dbg_modes=True)
    else:
        path = _build.LIB
        if _build.is_stale():
            path = _build.build()
    L = ctypes.CDLL(path)
    vp, i64, i32, u32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_uint32, ctypes.c_size_t
    PW, PP = ctypes.POINTER(NMWeight), ctypes.POINTER(NMPlan)
    L.nm_packed_size.restype = sz
    L.nm_packed_size.argtypes = [i32, i32, i32, i32, i32, u32]
    L.nm_compress.argtypes = [vp, i64, i32, i32, i32, i32, i32, u32, vp, sz, vp, PW,
                              ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.nm_compress_host.argtypes = [vp, i64, i32, i32, i32, i32, i32, u32, vp, sz, PW,
                                   ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.nm_prune_magnitude.argtypes = [vp, i64, i32, i32, i32, i32, i32]
    L.nm_decompress.argtypes = [PW, vp, i64, vp]
    L.nm_export_canonical.argtypes = [PW, vp, ctypes.POINTER(sz), vp]
    L.nm_plan_create.argtypes = [i32, PW, i32, i32, PP]
    L.nm_plan_shape.argtypes = [i32, i32, i32, i32, i32, i32, i32, u32, i32, PP]
    L.nm_spmm.argtypes = [vp, i64, i32, PW, PP, vp, i64, i32, vp, sz, vp, vp]
    L.nm_spmm_ex.argtypes = [vp, i64, i32, PW, PP, vp, i64, i32, ctypes.POINTER(NMEpilogue), vp, sz, vp, vp]
    L.nm_spmm_static_scratch.argtypes = [vp, i64, i32, PW, PP, vp, i64, i32, vp, vp]
    L.nm_latency_table.argtypes = [vp, i32, vp, i32, i32, i32, i32, vp, vp, sz, vp, vp, sz,
                                   ctypes.POINTER(NMLatencyRow), vp]
    L.nm_status_string.restype = ctypes.c_char_p
    L.nm_status_string.argtypes = [i32]
    L.nm_launch_count.restype = ctypes.c_uint64
    L.nm_launch_count.argtypes = []
    dp = ctypes.POINTER(ctypes.c_double)
    L.nm_predictor_fit.argtypes = [dp, dp, i32, i32, dp, dp, dp]
    L.nm_predictor_eval.argtypes = [dp, ctypes.c_double, dp, i32, i32, dp]
    L.nm_search.argtypes = [ctypes.POINTER(NMSearchConfig), dp, dp, ctypes.c_double, ctypes.c_void_p, vp,
                            ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(NMSearchResult)]
    L.nm_fitness_separable.restype = ctypes.c_double
    L.nm_fitness_separable.argtypes = [ctypes.POINTER(ctypes.c_int32), i32, vp]
    _lib = L
    return L


def _np_dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.int8:
        return NM_I8
    if a.dtype == np.float16:
        return NM_F16
    raise TypeError(f"weights/activations must be int8 or float16, got {a.dtype}")


def _check(status: int, where: str, detail: str = ""):
    if status != NM_OK:
        raise NMError(status, where, detail)


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


# ---- packing ----------------------------------------------------------------------------
def nm_packed_size(O: int, K: int, n: int, m: int, dtype: int, images: int = NM_IMG_AUTO) -> int:
    return int(lib().nm_packed_size(O, K, n, m, dtype, images))


@dataclass
class PackedWeight:
    """A packed weight: the nm_weight descriptor plus the buffer that backs it."""
    desc: NMWeight
    buf: object            # torch.uint8 device tensor, or numpy uint8 array for host blobs

    @property
    def shape(self):
        return (self.desc.O, self.desc.K)


def nm_compress_host(W: np.ndarray, n: int, m: int, images: int = NM_IMG_AUTO) -> PackedWeight:
    """Pack on the host only (no GPU needed); returns the blob as a numpy array."""
    W = np.ascontiguousarray(W)
    O, K = W.shape
    dt = _np_dtype_code(W)
    cap = nm_packed_size(O, K, n, m, dt, images)
    if cap == 0:
        _check(lib().nm_plan_shape(1, O, K, n, m, dt, NM_OUT_I32 if dt == NM_I8 else NM_OUT_F32, 1, 0,
                                   ctypes.byref(NMPlan())), "nm_compress_host")
    buf = np.zeros(cap, dtype=np.uint8)
    desc = NMWeight()
    br, bg = ctypes.c_int64(-1), ctypes.c_int64(-1)
    st = lib().nm_compress_host(W.ctypes.data, K, O, K, n, m, dt, images, buf.ctypes.data, cap,
                                ctypes.byref(desc), ctypes.byref(br), ctypes.byref(bg))
    _check(st, "nm_compress_host", f"(row {br.value}, group {bg.value})" if st == NM_ERR_NOT_NM else "")
    return PackedWeight(desc, buf[:desc.bytes])


def nm_compress(W: np.ndarray, n: int, m: int, images: int = NM_IMG_AUTO, device="cuda", stream=None) -> PackedWeight:
    """Pack a dense pruned weight (numpy int8 / float16 [O, K]) into device memory."""
    import torch
    W = np.ascontiguousarray(W)
    O, K = W.shape
    dt = _np_dtype_code(W)
    cap = nm_packed_size(O, K, n, m, dt, images)
    if cap == 0:
        raise NMError(NM_ERR_SHAPE, "nm_packed_size", f"O={O} K={K} n={n} m={m}")
    buf = torch.empty(cap + 256, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 256
    desc = NMWeight()
    br, bg = ctypes.c_int64(-1), ctypes.c_int64(-1)
    st = lib().nm_compress(W.ctypes.data, K, O, K, n, m, dt, images, buf.data_ptr() + off, cap,
                           _stream_ptr(stream), ctypes.byref(desc), ctypes.byref(br), ctypes.byref(bg))
    _check(st, "nm_compress", f"(row {br.value}, group {bg.value})" if st == NM_ERR_NOT_NM else "")
    return PackedWeight(desc, buf)


def nm_prune_magnitude(W: np.ndarray, n: int, m: int) -> np.ndarray:
    W = np.array(W, copy=True, order="C")
    O, K = W.shape
    _check(lib().nm_prune_magnitude(W.ctypes.data, K, O, K, n, m, _np_dtype_code(W)), "nm_prune_magnitude")
    return W


def nm_decompress(w: PackedWeight, stream=None) -> np.ndarray:
    d = w.desc
    W = np.zeros((d.O, d.K), dtype=np.int8 if d.dtype == NM_I8 else np.float16)
    _check(lib().nm_decompress(ctypes.byref(d), W.ctypes.data, d.K, _stream_ptr(stream)), "nm_decompress")
    return W


def nm_export_canonical(w: PackedWeight, stream=None) -> np.ndarray:
    nbytes = ctypes.c_size_t(0)
    _check(lib().nm_export_canonical(ctypes.byref(w.desc), None, ctypes.byref(nbytes), _stream_ptr(stream)),
           "nm_export_canonical")
    out = np.zeros(nbytes.value, dtype=np.uint8)
    _check(lib().nm_export_canonical(ctypes.byref(w.desc), out.ctypes.data, ctypes.byref(nbytes), _stream_ptr(stream)),
           "nm_export_canonical")
    return out


# ---- planning ---------------------------------------------------------------------------
def nm_plan_create(T: int, w: PackedWeight, out_dtype: int, device: int = -1) -> NMPlan:
    p = NMPlan()
    _check(lib().nm_plan_create(T, ctypes.byref(w.desc), out_dtype, device, ctypes.byref(p)), "nm_plan_create")
    return p


def nm_plan_shape(T, O, K, n, m, dtype, out_dtype, images, n_sms: int = 0) -> NMPlan:
    p = NMPlan()
    _check(lib().nm_plan_shape(T, O, K, n, m, dtype, out_dtype, images, n_sms, ctypes.byref(p)), "nm_plan_shape")
    return p


# ---- the GEMM ---------------------------------------------------------------------------
def _out_torch_dtype(od: int):
    import torch
    return {NM_OUT_I32: torch.int32, NM_OUT_F32: torch.float32, NM_OUT_F16: torch.float16, NM_OUT_I8: torch.int8}[od]


def nm_spmm(X, w: PackedWeight, plan: NMPlan | None = None, out=None, out_dtype: int | None = None,
            workspace=None, status=None, stream=None, scale=None, bias=None, relu: bool = False):
    """Y = X W~^T.  X: torch int8/float16 [T, K] on the GPU (row stride = pitch).

    Returns Y (allocated here with torch when ``out`` is None).  ``workspace`` is a
    torch uint8 tensor of at least plan.workspace_bytes; it is allocated here when the
    plan needs one and none is passed.  Only enqueues work on the stream.
    """
    import torch
    d = w.desc
    assert X.is_cuda and X.dim() == 2 and X.stride(1) == 1, "X must be a row-major CUDA matrix"
    T, K = X.shape
    if K != d.K:
        raise NMError(NM_ERR_SHAPE, "nm_spmm", f"X has K={K}, weight has K={d.K}")
    if out_dtype is None:
        out_dtype = (NM_OUT_I8 if scale is not None else NM_OUT_I32) if d.dtype == NM_I8 else NM_OUT_F16
    if out is None:
        out = torch.empty((T, d.O), dtype=_out_torch_dtype(out_dtype), device=X.device)
    assert out.is_cuda and out.stride(1) == 1 and out.shape == (T, d.O)
    if plan is None:
        plan = nm_plan_create(T, w, out_dtype, X.device.index if X.device.index is not None else 0)
    ws_ptr, ws_bytes = None, 0
    if plan.workspace_bytes:
        if workspace is None:
            workspace = torch.empty(int(plan.workspace_bytes), dtype=torch.uint8, device=X.device)
        ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    epi = None
    if scale is not None:          # requantising epilogue: int8 out = sat(rint((acc + bias) * scale))
        assert scale.is_cuda and scale.dtype == torch.float32 and scale.numel() == d.O
        assert bias is None or (bias.is_cuda and bias.dtype == torch.int32 and bias.numel() == d.O)
        epi = ctypes.byref(NMEpilogue(scale.data_ptr(), bias.data_ptr() if bias is not None else None, 1 if relu else 0, 0))
    st = lib().nm_spmm_ex(X.data_ptr(), X.stride(0), T, ctypes.byref(d), ctypes.byref(plan),
                          out.data_ptr(), out.stride(0), out_dtype, epi, ws_ptr, ws_bytes,
                          status.data_ptr() if status is not None else None, _stream_ptr(stream))
    _check(st, "nm_spmm")
    return out


def nm_spmm_raw(x_ptr: int, ldx: int, T: int, w: PackedWeight, plan, y_ptr: int, ldy: int, out_dtype: int,
                ws_ptr: int = 0, ws_bytes: int = 0, status_ptr: int = 0, stream_ptr: int = 0) -> int:
    """Direct call with raw device addresses; returns the nm_status (no exception)."""
    return lib().nm_spmm(x_ptr, ldx, T, ctypes.byref(w.desc), ctypes.byref(plan) if plan is not None else None,
                         y_ptr, ldy, out_dtype, ws_ptr or None, ws_bytes, status_ptr or None, stream_ptr or None)


NM_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def nm_spmm_static_scratch_raw(x_ptr: int, ldx: int, T: int, w: PackedWeight, plan, y_ptr: int, ldy: int,
                               out_dtype: int, status_ptr: int = 0, stream_ptr: int = 0) -> int:
    """nm_spmm for callers that cannot allocate: split-K partial sums go to the library's
    built-in 16 MiB scratch array instead of a caller workspace.  Returns the nm_status."""
    return lib().nm_spmm_static_scratch(x_ptr, ldx, T, ctypes.byref(w.desc),
                                        ctypes.byref(plan) if plan is not None else None,
                                        y_ptr, ldy, out_dtype, status_ptr or None, stream_ptr or None)


def nm_latency_table(shapes, nm_pairs, dtype: int, out_dtype: int, reps: int = 20, device="cuda"):
    """Per-operator latency LUT rows for the layer-wise sparsity search (list of dicts)."""
    import torch
    shapes = np.ascontiguousarray(shapes, dtype=np.int32).reshape(-1, 3)
    pairs = np.ascontiguousarray(nm_pairs, dtype=np.int32).reshape(-1, 2)
    eb = 1 if dtype == NM_I8 else 2
    ob = 2 if out_dtype == NM_OUT_F16 else 4
    max_x = int(max(int(T) * int(K) for T, O, K in shapes)) * eb
    max_y = int(max(int(T) * int(O) for T, O, K in shapes)) * ob
    max_w = max(nm_packed_size(int(O), int(K), int(n), int(m), dtype) for T, O, K in shapes for n, m in pairs) + 256
    max_ws = 0
    for T, O, K in shapes:
        for n, m in pairs:
            # the plan depends on which images nm_compress will build; take the largest scratch.
            # Shapes the library rejects simply report their status in their row.
            for imgs in (NM_IMG_CANONICAL | NM_IMG_HW24, NM_IMG_CANONICAL | NM_IMG_DENSE):
                p = NMPlan()
                if lib().nm_plan_shape(int(T), int(O), int(K), int(n), int(m), dtype, out_dtype, imgs, 0,
                                       ctypes.byref(p)) == NM_OK:
                    max_ws = max(max_ws, int(p.workspace_bytes))
    X = torch.zeros(max_x, dtype=torch.uint8, device=device)
    Y = torch.empty(max_y, dtype=torch.uint8, device=device)
    Wp = torch.empty(max_w, dtype=torch.uint8, device=device)
    ws = torch.empty(max(max_ws, 256), dtype=torch.uint8, device=device)
    woff = (-Wp.data_ptr()) % 256
    rows = (NMLatencyRow * (len(shapes) * len(pairs)))()
    _check(lib().nm_latency_table(shapes.ctypes.data, len(shapes), pairs.ctypes.data, len(pairs), dtype, out_dtype,
                                  reps, X.data_ptr(), Wp.data_ptr() + woff, max_w - woff, Y.data_ptr(),
                                  ws.data_ptr(), ws.numel(), rows, _stream_ptr()), "nm_latency_table")
    return [{k: getattr(r, k) for k, _ in NMLatencyRow._fields_} for r in rows]


def _dptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def nm_predictor_fit(lut_us, measured_us):
    """Calibrate Eq. (1) by non-negative least squares: returns (gamma[L], b, residual norm)."""
    A = np.ascontiguousarray(lut_us, dtype=np.float64)
    y = np.ascontiguousarray(measured_us, dtype=np.float64)
    if A.ndim != 2 or y.shape != (A.shape[0],):
        raise ValueError("lut_us must be [S, L] and measured_us [S]")
    S, L = A.shape
    gamma = np.zeros(L, dtype=np.float64)
    b, rn = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().nm_predictor_fit(_dptr(A), _dptr(y), S, L, _dptr(gamma), ctypes.byref(b), ctypes.byref(rn)), "nm_predictor_fit")
    return gamma, float(b.value), float(rn.value)


def nm_predictor_eval(gamma, b, t_us):
    """Eq. (1) for a batch of configurations: t_us [n_cfg, L] -> predicted latencies [n_cfg]."""
    g = np.ascontiguousarray(gamma, dtype=np.float64)
    t = np.ascontiguousarray(t_us, dtype=np.float64)
    if t.ndim == 1:
        t = t[None, :]
    if t.shape[1] != g.shape[0]:
        raise ValueError("t_us must be [n_cfg, L]")
    out = np.zeros(t.shape[0], dtype=np.float64)
    _check(lib().nm_predictor_eval(_dptr(g), float(b), _dptr(t), t.shape[0], t.shape[1], _dptr(out)), "nm_predictor_eval")
    return out


def nm_search(table_us, gamma, b, target_us, generations, offspring, overshoot_k=2, n_init=4, seed=0,
              fitness=None, separable_gain=None, noise=0.0, fitness_seed=0, elitist=False):
    """Algorithm 1.  `table_us` is [L, levels].  The fitness is either a Python callable taking a
    list of levels (1-based) or, with `separable_gain` [L, levels], the library's synthetic
    separable-plus-noise fitness.  Returns (y, result dict, status): status is NM_OK or
    NM_ERR_UNSUPPORTED (no uniform configuration fits the budget)."""
    tab = np.ascontiguousarray(table_us, dtype=np.float64)
    Lyr, levels = tab.shape
    g = np.ascontiguousarray(gamma, dtype=np.float64)
    if g.shape != (Lyr,):
        raise ValueError("gamma must be [L]")
    cfg = NMSearchConfig(Lyr, levels, generations, offspring, overshoot_k, n_init, 1 if elitist else 0, 0, float(target_us), seed)
    y = np.zeros(Lyr, dtype=np.int32)
    res = NMSearchResult()
    keep = []
    if separable_gain is not None:
        gain = np.ascontiguousarray(separable_gain, dtype=np.float64)
        if gain.shape != (Lyr, levels):
            raise ValueError("separable_gain must be [L, levels]")
        args = NMFitnessSeparableArgs(_dptr(gain), levels, 0, float(noise), fitness_seed)
        keep += [gain, args]
        fn_ptr = ctypes.cast(lib().nm_fitness_separable, ctypes.c_void_p)
        user = ctypes.cast(ctypes.pointer(args), ctypes.c_void_p)
    elif fitness is not None:
        cb = FITNESS_FN(lambda yp, n, _u: float(fitness([int(yp[i]) for i in range(n)])))
        keep.append(cb)
        fn_ptr = ctypes.cast(cb, ctypes.c_void_p)
        user = ctypes.c_void_p(0)
    else:
        raise ValueError("give a fitness callable or separable_gain")
    st = lib().nm_search(ctypes.byref(cfg), _dptr(tab), _dptr(g), float(b), fn_ptr, user,
                         y.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), ctypes.byref(res))
    if st not in (NM_OK, NM_ERR_UNSUPPORTED):
        _check(st, "nm_search")
    out = {k: getattr(res, k) for k, _ in NMSearchResult._fields_ if k != "reserved"}
    return y.tolist(), out, st


def launch_count() -> int:
    return int(lib().nm_launch_count())
