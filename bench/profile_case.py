"""Run one GEMM shape through nm_spmm repeatedly (for timing sweeps and ncu captures).

    python -m bench.profile_case --T 12608 --O 1152 --K 384 --nm 2:4 \
        [--dtype i8|f16] [--out i32|f32|f16] [--reps 20] [--rotate 4] [--tile-t 128] \
        [--stages 2] [--split-k 1] [--path simt|dense|sp24]

Prints one JSON line: microseconds per call (CUDA events on the launching stream, buffers
rotated over `--rotate` sets so that consecutive calls do not hit L2), achieved GB/s on the
algorithmic bytes (X once, Y once, packed W once) and dense-equivalent T(FL)OPS.

With NM_B200_TRACE=2 in the environment the binding loads the timing build of the library
(-DNM_DBG_MODES), in which NM_DBG switches parts of the tcgen05 kernels off at run time (bit 1: no
MMAs, 2: no stores, 4: the ring is loaded once; results are then wrong by construction).
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--T", type=int, required=True)
    ap.add_argument("--O", type=int, required=True)
    ap.add_argument("--K", type=int, required=True)
    ap.add_argument("--nm", default="2:4")
    ap.add_argument("--dtype", default="i8", choices=["i8", "f16"])
    ap.add_argument("--out", default=None, choices=[None, "i32", "f32", "f16", "i8"])
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--rotate", type=int, default=0, help="buffer sets (0 = enough to exceed 256 MB)")
    ap.add_argument("--tile-t", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--split-k", type=int, default=0)
    ap.add_argument("--resident", type=int, default=-1)
    ap.add_argument("--cta-group", type=int, default=0)
    ap.add_argument("--issuers", type=int, default=0)
    ap.add_argument("--merge", default=None, choices=[None, "workspace", "cluster"], help="split-K merge (default: the planner's, or workspace under overrides)")
    ap.add_argument("--path", default=None, choices=[None, "simt", "dense", "sp24", "decode", "expand", "remap"])
    ap.add_argument("--eager", action="store_true", help="time eager launches instead of one CUDA graph")
    ap.add_argument("--cublas", action="store_true", help="also time dense cuBLAS (torch._int_mm / torch.matmul) on the same buffers")
    ap.add_argument("--images", default="auto", choices=["auto", "all", "canonical"])
    args = ap.parse_args()

    import torch
    from paper_2607_12505_b200 import binding as nm
    from paper_2607_12505_b200 import inputs

    n, m = (int(v) for v in args.nm.split(":"))
    spec = dict(T=args.T, O=args.O, K=args.K, n=n, m=m, dtype=args.dtype, name="profile")
    X, W = inputs.make_layer(spec)
    od = {"i32": nm.NM_OUT_I32, "f32": nm.NM_OUT_F32, "f16": nm.NM_OUT_F16, "i8": nm.NM_OUT_I8, None: None}[args.out]
    if od is None:
        od = nm.NM_OUT_I32 if args.dtype == "i8" else nm.NM_OUT_F16
    images = {"auto": nm.NM_IMG_AUTO, "all": nm.NM_IMG_AUTO | nm.NM_IMG_DENSE | nm.NM_IMG_HW24, "canonical": nm.NM_IMG_CANONICAL}[args.images]
    if args.path == "remap":
        images |= nm.NM_IMG_REMAP48
    w = nm.nm_compress(W, n, m, images=images)
    plan = nm.nm_plan_create(args.T, w, od, 0)
    if args.path:
        plan.path = {"simt": nm.NM_PATH_SIMT, "dense": nm.NM_PATH_UMMA_DENSE, "sp24": nm.NM_PATH_UMMA_SP24, "decode": nm.NM_PATH_UMMA_DECODE, "expand": nm.NM_PATH_UMMA_EXPAND, "remap": nm.NM_PATH_UMMA_REMAP48}[args.path]
        if args.path == "remap":
            plan.split_k, plan.cta_group, plan.resident = 1, 1, nm.NM_RES_NONE
        if args.path == "decode":
            plan.resident = nm.NM_RES_W
    if args.tile_t:
        plan.tile_t = args.tile_t
    if args.stages:
        plan.stages = args.stages
    if args.split_k:
        plan.split_k = args.split_k
    if args.resident >= 0:
        plan.resident = args.resident
    if args.cta_group:
        plan.cta_group = args.cta_group
    if args.issuers:
        plan.issuers = args.issuers
    if args.merge:
        plan.merge = nm.NM_MERGE_CLUSTER if args.merge == "cluster" else nm.NM_MERGE_WORKSPACE
    elif args.tile_t or args.split_k or args.cta_group or args.path or args.resident >= 0:
        plan.merge = nm.NM_MERGE_WORKSPACE
    t_pad = -(-args.T // plan.tile_t) * plan.tile_t
    plan.workspace_bytes = 0 if (plan.split_k <= 1 or plan.merge == nm.NM_MERGE_CLUSTER) else plan.split_k * t_pad * args.O * 4
    if plan.path == nm.NM_PATH_UMMA_REMAP48:         # the gathered third-chunk activations sit at the head of the workspace
        plan.workspace_bytes = -(-(args.T * (-(-(args.K // 2 * (1 if args.dtype == "i8" else 2)) // 16) * 16)) // 256) * 256
    if plan.path == nm.NM_PATH_UMMA_EXPAND:          # the dense copy sits at the head of the workspace
        plan.workspace_bytes += -(-(args.O * (-(-(args.K * (1 if args.dtype == "i8" else 2)) // 16) * 16)) // 256) * 256

    eb = 1 if args.dtype == "i8" else 2
    ob = 2 if od == nm.NM_OUT_F16 else (1 if od == nm.NM_OUT_I8 else 4)
    scale = torch.full((args.O,), 1e-4, dtype=torch.float32, device="cuda") if od == nm.NM_OUT_I8 else None
    b = 0 if n == m else int(np.ceil(np.log2(m)))
    kept = args.O * args.K * n / m
    alg_bytes = args.T * args.K * eb + args.T * args.O * ob + kept * eb + kept * b / 8
    per_set = args.T * args.K * eb + args.T * args.O * ob
    R = args.rotate or max(1, int(np.ceil(256e6 / per_set)))
    Xs = [torch.from_numpy(X).cuda() for _ in range(R)]
    Ys = [torch.empty((args.T, args.O), dtype=nm._out_torch_dtype(od), device="cuda") for _ in range(R)]
    ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")

    def call(i):
        nm.nm_spmm(Xs[i % R], w, plan=plan, out=Ys[i % R], out_dtype=od, workspace=ws, status=status, scale=scale)

    for i in range(args.warmup):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.Stream()
    graph = None
    with torch.cuda.stream(stream):
        if not args.eager:
            # one graph holding `reps` back-to-back calls: host launch cost stays out of the timing
            call(0)
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(args.reps):
                    call(i)
            graph.replay()
            stream.synchronize()
        e0.record(stream)
        if graph is not None:
            graph.replay()
        else:
            for i in range(args.reps):
                call(i)
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.reps
    cublas_us = None
    if args.cublas:
        # comparator only (never on the product path): dense library GEMM on the masked dense W
        Wd = torch.from_numpy(W).cuda()
        outs = [None] * R

        def dense(i):
            if args.dtype == "i8":
                outs[i % R] = torch._int_mm(Xs[i % R], Wd.t())
            else:
                outs[i % R] = torch.matmul(Xs[i % R], Wd.t()) if ob == 2 else torch.matmul(Xs[i % R], Wd.t()).float()
        with torch.cuda.stream(stream):
            for i in range(3):
                dense(i)
            stream.synchronize()
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2, stream=stream):
                for i in range(args.reps):
                    dense(i)
            g2.replay()
            stream.synchronize()
            e0.record(stream)
            g2.replay()
            e1.record(stream)
            stream.synchronize()
        cublas_us = e0.elapsed_time(e1) * 1e3 / args.reps
    print(json.dumps({
        "T": args.T, "O": args.O, "K": args.K, "nm": args.nm, "dtype": args.dtype, "out": ob, "us": round(us, 2),
        "gbs": round(alg_bytes / us / 1e3, 1), "dense_tops": round(2.0 * args.T * args.O * args.K / us / 1e6, 1),
        "cublas_dense_us": None if cublas_us is None else round(cublas_us, 2),
        "speedup_vs_cublas": None if cublas_us is None else round(cublas_us / us, 3),
        "plan": plan.as_dict(), "rotate": R, "status": int(status[0].item()),
    }))


if __name__ == "__main__":
    main()
