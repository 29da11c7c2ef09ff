"""Shared helpers of the GPU parity tests: run nm_spmm through the C ABI and compare with
the CPU oracle element by element (all rows, or a deterministic row sample at sizes the
oracle cannot finish in seconds)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import nm_oracle as orc
from paper_2607_12505_b200 import binding as nm
from paper_2607_12505_b200 import inputs

FP16_REL_TOL = 1e-3       # |Y - Yref| <= 1e-3 * sum_k |x||w| per output element


def sample_rows(T: int, tile: int = 128, frac: float = 0.02, seed: int = 7, cap: int = 2048) -> np.ndarray:
    """First two and last two token tiles (incl. the ragged one) plus seeded-random rows."""
    if T <= 4 * tile + 64:
        return np.arange(T, dtype=np.int64)
    head = np.arange(0, 2 * tile)
    tail = np.arange(max(0, (T - 1) // tile * tile - tile), T)
    rng = np.random.default_rng(seed)
    extra = rng.choice(T, size=min(cap, max(16, int(T * frac))), replace=False)
    return np.unique(np.concatenate([head, tail, extra])).astype(np.int64)


def make_plan(T, w, od, **over):
    plan = nm.nm_plan_create(T, w, od, 0)
    for k, v in over.items():
        setattr(plan, k, v)
    if "merge" not in over and any(k in over for k in ("tile_t", "split_k", "cta_group", "path", "resident")):
        plan.merge = nm.NM_MERGE_WORKSPACE                   # the planner's on-chip merge is tied to its own tile and split
    # the scratch requirement depends on tile, split and merge
    t_pad = -(-T // plan.tile_t) * plan.tile_t               # slices hold whole token tiles
    on_chip = plan.merge == nm.NM_MERGE_CLUSTER
    plan.workspace_bytes = 0 if (plan.split_k <= 1 or on_chip or plan.path == nm.NM_PATH_SIMT) else plan.split_k * t_pad * w.desc.O * 4
    if plan.path == nm.NM_PATH_UMMA_REMAP48:                 # the gathered third-chunk activations sit at the head
        eb = 1 if w.desc.dtype == nm.NM_I8 else 2
        plan.workspace_bytes = -(-(T * (-(-(w.desc.K // 2 * eb) // 16) * 16)) // 256) * 256
        plan.split_k, plan.cta_group, plan.resident = 1, 1, nm.NM_RES_NONE
    if plan.path == nm.NM_PATH_UMMA_EXPAND:                  # the dense copy sits at the head of the workspace
        eb = 1 if w.desc.dtype == nm.NM_I8 else 2
        plan.workspace_bytes += -(-(w.desc.O * (-(-(w.desc.K * eb) // 16) * 16)) // 256) * 256
    return plan


def gpu_spmm(X: np.ndarray, W: np.ndarray, n: int, m: int, od: int | None = None, images=nm.NM_IMG_AUTO, **plan_over):
    """Returns (Y numpy, plan dict, packed weight).  Raises on a device-side timeout."""
    if plan_over.get("path") == nm.NM_PATH_UMMA_REMAP48 and images == nm.NM_IMG_AUTO:
        images = nm.NM_IMG_AUTO | nm.NM_IMG_REMAP48         # only built on request
    if plan_over.get("path") == nm.NM_PATH_UMMA_SP24 and images == nm.NM_IMG_AUTO:
        images = nm.NM_IMG_AUTO | nm.NM_IMG_HW24            # short rows get only the dense image by default
    w = nm.nm_compress(W, n, m, images=images)
    Xd = torch.from_numpy(X).cuda()
    if od is None:
        od = nm.NM_OUT_I32 if X.dtype == np.int8 else nm.NM_OUT_F32
    plan = make_plan(X.shape[0], w, od, **plan_over)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    if plan_over:
        Y = nm.nm_spmm(Xd, w, plan=plan, out_dtype=od, status=status)
    else:
        # no override: let the library plan by itself (it degrades to the CUDA-core path
        # when X cannot be read by TMA) and hand it scratch for whatever it picks
        Y = torch.empty((X.shape[0], w.desc.O), dtype=nm._out_torch_dtype(od), device="cuda")
        ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
        st = nm.nm_spmm_raw(Xd.data_ptr(), Xd.stride(0), X.shape[0], w, None, Y.data_ptr(), Y.stride(0), od,
                            ws.data_ptr(), ws.numel(), status.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert st == nm.NM_OK, nm.lib().nm_status_string(st)
    torch.cuda.synchronize()
    st = int(status[0].item())
    assert st == 0, f"device status word {st:#x} (plan {plan.as_dict()})"
    return Y.cpu().numpy(), plan.as_dict(), w


def check_against_oracle(X, W, n, m, Y, rows=None, out_f16=False):
    """Element-by-element comparison on `rows` (None = all)."""
    packed = orc.compress(W, n, m)
    Ysub = Y if rows is None else Y[rows]
    if X.dtype == np.int8:
        ref = orc.spmm_packed(X, packed, rows=rows)
        bad = np.argwhere(ref != Ysub)
        assert bad.size == 0, f"{len(bad)} int32 mismatches, first at {bad[0].tolist()}: got {Ysub[tuple(bad[0])]} want {ref[tuple(bad[0])]}"
        return
    ref, S = orc.spmm_packed(X, packed, rows=rows)
    err = np.abs(Ysub.astype(np.float64) - ref)
    bound = FP16_REL_TOL * S
    if Ysub.dtype == np.float16:
        # a binary16 OUTPUT cannot resolve better than half its subnormal spacing (2^-24): results
        # below the normal range (|y| < 6.1e-5, only reachable with very short K) carry that much
        bound = bound + 2.0 ** -25
    bad = np.argwhere(err > bound)
    assert bad.size == 0, f"{len(bad)} fp16 outputs beyond 1e-3*sum|x||w|, first {bad[0].tolist()}: err {err[tuple(bad[0])]} bound {bound[tuple(bad[0])]}"
    assert (Ysub[S == 0] == 0).all()


def run_case(T, O, K, n, m, dtype="i8", od=None, at_most=False, key="case", rows="auto", images=nm.NM_IMG_AUTO, **plan_over):
    spec = dict(T=T, O=O, K=K, n=n, m=m, dtype=dtype, name=key)
    X, W = inputs.make_layer(spec, at_most=at_most)
    Y, plan, _ = gpu_spmm(X, W, n, m, od=od, images=images, **plan_over)
    r = sample_rows(T) if rows == "auto" else rows
    if r is not None and len(r) == T:
        r = None
    check_against_oracle(X, W, n, m, Y, rows=r)
    return Y, plan
