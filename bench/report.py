"""Per-shape performance report over the benchmark configurations (one B200).

    python -m bench.report [--configs cfg1,cfg2,cfg4] [--reps 20] [--out report.json]

For every distinct (layer shape, n:m, dtype) of the selected configurations it times nm_spmm
under the library's own plan and dense cuBLAS (torch._int_mm / torch.matmul) on the same
buffers -- each as one CUDA graph of `reps` back-to-back calls over rotating buffer sets
larger than L2 -- and prints microseconds, useful and dense-equivalent T(FL)OPS, GB/s on the
algorithmic bytes, and the fraction of the HBM and tensor rooflines.  The tensor peaks are
measured in the same run (dense library GEMM 8192^3; the sparse peak is taken as twice that).
It also times the small-batch weight-streaming case as a stack: the 72 distinct linear layers
of ViT-L at batch 1 in one graph, bytes over time.  The SM clock and the throttle reasons seen
while each configuration was timed are printed and stored with its rows (a group taken under a
thermal or hardware slowdown is to be re-run).
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np


def _graph_time(torch, fn, reps, stream):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for i in range(2):
            fn(i)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(reps):
                fn(i)
        g.replay()
        stream.synchronize()
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps


def image_read_bytes(nm, w, plan):
    """Bytes of the packed weight one call of `plan` actually reads (the image its path uses)."""
    d = w.desc
    if plan.path == nm.NM_PATH_UMMA_SP24:
        return d.O * d.hw24_row_bytes + -(-d.O // 128) * d.hw24_meta_kblocks * 2048
    if plan.path == nm.NM_PATH_UMMA_DENSE and d.n != d.m:
        return d.O * d.dense_row_bytes
    eb = 1 if d.dtype == nm.NM_I8 else 2
    return nm.nm_packed_size(d.O, d.K, d.n, d.m, d.dtype, nm.NM_IMG_CANONICAL)


def measure_peaks(torch, stream):
    """Dense library GEMM peaks (8192^3, best of 5 graph replays of 5 calls)."""
    n = 8192
    a8 = torch.randint(-128, 127, (n, n), dtype=torch.int8, device="cuda")
    b8 = torch.randint(-128, 127, (n, n), dtype=torch.int8, device="cuda")
    a16 = torch.randn(n, n, dtype=torch.float16, device="cuda")
    b16 = torch.randn(n, n, dtype=torch.float16, device="cuda")
    out = {}
    for name, fn in (("int8_dense_tops", lambda i: torch._int_mm(a8, b8.t())), ("fp16_dense_tflops", lambda i: torch.matmul(a16, b16.t()))):
        best = min(_graph_time(torch, fn, 5, stream) for _ in range(5))
        out[name] = 2.0 * n ** 3 / best / 1e6
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="cfg0,cfg1,cfg2,cfg3,cfg4")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--out", default=None)
    ap.add_argument("--stack-only", action="store_true", help="only the small-batch ViT-L layer stack")
    ap.add_argument("--max-shapes", type=int, default=0, help="cap per config (0 = all distinct shapes)")
    args = ap.parse_args()

    import torch
    from paper_2607_12505_b200 import binding as nm
    from paper_2607_12505_b200 import inputs

    from bench.clocks import ClockSampler
    stream = torch.cuda.Stream()
    sampler = ClockSampler(torch.cuda.current_device()).start()
    clock_groups = {}
    hbm = 6450.9
    peaks_file = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(peaks_file):
        hbm = float(json.load(open(peaks_file))["hbm_gbs"])
    peaks = measure_peaks(torch, stream)
    print(json.dumps({"hbm_gbs_measured_copy": hbm, **{k: round(v, 1) for k, v in peaks.items()}}))

    cfgs = {
        "cfg0": [dict(inputs.cfg0(), name="cfg0")],
        "cfg1": inputs.cfg1_layers(),
        "cfg2": inputs.cfg2_layers("i8") + inputs.cfg2_layers("f16"),
        "cfg3": inputs.cfg3_layers(),
        "cfg4": inputs.cfg4_layers(),
    }
    rows = []
    for cname in ([] if args.stack_only else args.configs.split(",")):
        seen = set()
        count = 0
        mark = sampler.mark()
        for s in cfgs[cname]:
            key = (s["T"], s["K"], s["O"], s["n"], s["m"], s["dtype"])
            if key in seen:
                continue
            seen.add(key)
            if args.max_shapes and count >= args.max_shapes:
                break
            count += 1
            T, K, O, n, m, dt = key
            eb = 1 if dt == "i8" else 2
            od = nm.NM_OUT_I32 if dt == "i8" else nm.NM_OUT_F16
            ob = 4 if dt == "i8" else 2
            X, W = inputs.make_layer(s, "report")
            w = nm.nm_compress(W, n, m)
            plan = nm.nm_plan_create(T, w, od, 0)
            per_set = T * K * eb + T * O * ob
            R = max(1, min(8, int(np.ceil(256e6 / per_set))))
            Xs = [torch.from_numpy(X).cuda() for _ in range(R)]
            Ys = [torch.empty((T, O), dtype=nm._out_torch_dtype(od), device="cuda") for _ in range(R)]
            ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
            us = _graph_time(torch, lambda i: nm.nm_spmm(Xs[i % R], w, plan=plan, out=Ys[i % R], out_dtype=od, workspace=ws), args.reps, stream)
            Wd = torch.from_numpy(W).cuda()
            cb = None
            if T > 16:
                if dt == "i8":
                    cb = _graph_time(torch, lambda i: torch._int_mm(Xs[i % R], Wd.t()), args.reps, stream)
                else:
                    cb = _graph_time(torch, lambda i: torch.matmul(Xs[i % R], Wd.t()), args.reps, stream)
            b = 0 if n == m else int(np.ceil(np.log2(m)))
            kept = O * K * n / m
            alg = T * K * eb + T * O * ob + kept * eb + kept * b / 8
            dense_ops = 2.0 * T * O * K
            sparse_hw = plan.path == nm.NM_PATH_UMMA_SP24
            tensor_peak = (peaks["int8_dense_tops"] if dt == "i8" else peaks["fp16_dense_tflops"]) * (2.0 if sparse_hw else 1.0)
            t_hbm, t_mma = alg / hbm / 1e3, dense_ops / tensor_peak / 1e6
            row = dict(config=cname, name=s.get("name", ""), T=T, K=K, O=O, nm=f"{n}:{m}", dtype=dt, us=round(us, 2),
                       cublas_dense_us=None if cb is None else round(cb, 2), speedup=None if cb is None else round(cb / us, 3),
                       dense_tops=round(dense_ops / us / 1e6, 1), useful_tops=round(dense_ops * n / m / us / 1e6, 1),
                       gbs=round(alg / us / 1e3, 1), frac_hbm=round(alg / us / 1e3 / hbm, 3),
                       frac_tensor=round(dense_ops / us / 1e6 / tensor_peak, 3), bound="hbm" if t_hbm >= t_mma else "tensor",
                       frac_roofline=round(max(t_hbm, t_mma) / us, 3),
                       plan={k: v for k, v in plan.as_dict().items() if k in ("path", "tile_t", "stages", "split_k", "cta_group", "issuers", "resident")})
            rows.append(row)
            print(json.dumps(row))
            del Xs, Ys, Wd, w
        # clocks and throttle reasons seen while this configuration's rows were timed (read-only query)
        clock_groups[cname] = sampler.summary(since=mark)
        print(json.dumps({"clocks": cname, **clock_groups[cname]}))

    # ---- the fused requantising epilogue (INT8 in, INT8 out) on the INT8 2:4 layers of cfg1 / cfg2:
    # one byte per output instead of four moves these GEMMs from the HBM towards the tensor roofline
    if not args.stack_only and not args.max_shapes:
        seen = set()
        mark = sampler.mark()
        for cname in [c for c in args.configs.split(",") if c in ("cfg1", "cfg2")]:
            for s in cfgs[cname]:
                key = (s["T"], s["K"], s["O"])
                if s["dtype"] != "i8" or (s["n"], s["m"]) != (2, 4) or key in seen:
                    continue
                seen.add(key)
                T, K, O = key
                X, W = inputs.make_layer(s, "report")
                w = nm.nm_compress(W, 2, 4)
                plan = nm.nm_plan_create(T, w, nm.NM_OUT_I8, 0)
                R = max(1, min(8, int(np.ceil(256e6 / (T * K + T * O)))))
                Xs = [torch.from_numpy(X).cuda() for _ in range(R)]
                Ys = [torch.empty((T, O), dtype=torch.int8, device="cuda") for _ in range(R)]
                scale = torch.full((O,), 1e-4, dtype=torch.float32, device="cuda")
                ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
                us = _graph_time(torch, lambda i: nm.nm_spmm(Xs[i % R], w, plan=plan, out=Ys[i % R], out_dtype=nm.NM_OUT_I8,
                                                             workspace=ws, scale=scale), args.reps, stream)
                i32 = [r for r in rows if (r["T"], r["K"], r["O"], r["nm"], r["dtype"]) == (T, K, O, "2:4", "i8")]
                kept = O * K / 2
                alg = T * K + T * O + kept + kept * 2 / 8
                dense_ops = 2.0 * T * O * K
                t_hbm, t_mma = alg / hbm / 1e3, dense_ops / (2.0 * peaks["int8_dense_tops"]) / 1e6
                row = dict(config=cname + ".int8_out", name=s.get("name", ""), T=T, K=K, O=O, nm="2:4", dtype="i8->i8", us=round(us, 2),
                           us_int32_out=i32[0]["us"] if i32 else None, dense_tops=round(dense_ops / us / 1e6, 1),
                           gbs=round(alg / us / 1e3, 1), bound="hbm" if t_hbm >= t_mma else "tensor",
                           frac_roofline=round(max(t_hbm, t_mma) / us, 3),
                           plan={k: v for k, v in plan.as_dict().items() if k in ("path", "tile_t", "split_k", "cta_group", "issuers")})
                rows.append(row)
                print(json.dumps(row))
                del Xs, Ys, w
        clock_groups["int8_out"] = sampler.summary(since=mark)
        print(json.dumps({"clocks": "int8_out", **clock_groups["int8_out"]}))

    # ---- small-batch weight streaming measured over a stack of distinct layers (ViT-L, batch 1)
    stack = None
    if "cfg4" in args.configs or args.stack_only:
        T = 197
        mark = sampler.mark()
        for (n, m) in [(2, 4), (1, 8)]:
            layers = []
            for blk in range(24):
                for (name, K, O) in [("qkv", 1024, 3072), ("fc1", 1024, 4096), ("fc2", 4096, 1024)]:
                    Wn = inputs.w_i8(O, K, n, m, "stack", blk, name)
                    w = nm.nm_compress(Wn, n, m)
                    plan = nm.nm_plan_create(T, w, nm.NM_OUT_I32, 0)
                    Xd = torch.from_numpy(inputs.x_i8(T, K, "stack", name)).cuda()
                    Yd = torch.empty((T, O), dtype=torch.int32, device="cuda")
                    ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
                    layers.append((Xd, w, plan, Yd, ws, K, O))

            def run_stack(i):
                for (Xd, w, plan, Yd, ws, K, O) in layers:
                    nm.nm_spmm(Xd, w, plan=plan, out=Yd, workspace=ws)
            us = _graph_time(torch, run_stack, 5, stream)
            b = int(np.ceil(np.log2(m)))
            native = sum(T * K + T * O * 4 + O * K * n / m * (1 + b / 8) for (*_, K, O) in layers)
            image = sum(T * K + T * O * 4 + image_read_bytes(nm, w, plan) for (_x, w, plan, _y, _ws, K, O) in layers)
            stack = dict(workload="vit_l_batch1_72_layers", nm=f"{n}:{m}", us=round(us, 1), us_per_layer=round(us / len(layers), 2),
                         gbs_native_bytes=round(native / us / 1e3, 1), gbs_image_bytes=round(image / us / 1e3, 1),
                         frac_hbm_native=round(native / us / 1e3 / hbm, 3), frac_hbm_image=round(image / us / 1e3 / hbm, 3),
                         weights_read_mb=round(sum(image_read_bytes(nm, w, plan) for (_x, w, plan, *_r) in layers) / 1e6, 1))
            print(json.dumps(stack))
            rows.append(stack)
            del layers
        clock_groups["vit_l_b1_stack"] = sampler.summary(since=mark)
        print(json.dumps({"clocks": "vit_l_b1_stack", **clock_groups["vit_l_b1_stack"]}))
    sampler.stop()
    if args.out:
        json.dump(dict(hbm_gbs=hbm, peaks=peaks, clocks=clock_groups, rows=rows), open(args.out, "w"))


if __name__ == "__main__":
    main()
