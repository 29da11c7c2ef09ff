"""Planner quality on the paper's kernel-evaluation grid (Section 6.1, Table 1).

For every shape of the grid T in {64,128,256,512}, O, K in {128,256,512,1024} and every
sparsity level (50 %, 75 %, 87.5 %) this times nm_spmm under each admissible split-K value
and compares the planner's choice with the sweep's optimum, reporting the three Table-1
statistics -- top-1 hit rate, average and worst normalised performance (t_best / t_planner)
-- plus the speed-up over dense cuBLAS (torch._int_mm) on the same shapes.

    python -m bench.planner_quality [--reps 20] [--out table.json] [--quick]

Timing: CUDA events around one CUDA graph holding `reps` back-to-back calls; the SM clock and the
throttle reasons seen while each sparsity level was measured are stored with its statistics.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np

SPARSITY = {"50%": (2, 4), "75%": (2, 8), "87.5%": (1, 8)}
SPLITS = (1, 2, 4, 8, 16)


def _time_graph(torch, fn, reps, stream):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        fn()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                fn()
        g.replay()
        stream.synchronize()
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps


def evaluate(Ts=(64, 128, 256, 512), OKs=(128, 256, 512, 1024), reps=20, sparsity=None):
    """Times the grid; returns dict(grid, clocks, summary, rows)."""
    import torch
    from paper_2607_12505_b200 import binding as nm
    from paper_2607_12505_b200 import inputs
    from bench.clocks import ClockSampler

    sparsity = sparsity or SPARSITY
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(torch.cuda.current_device()).start()
    clocks = {}
    for label, (n, m) in sparsity.items():
        mark = sampler.mark()
        for T in Ts:
            for O in OKs:
                for K in OKs:
                    X = torch.from_numpy(inputs.x_i8(T, K, "pq")).cuda()
                    Wn = inputs.w_i8(O, K, n, m, "pq")
                    w = nm.nm_compress(Wn, n, m)
                    Wd = torch.from_numpy(Wn).cuda()
                    Y = torch.empty((T, O), dtype=torch.int32, device="cuda")
                    chosen = nm.nm_plan_create(T, w, nm.NM_OUT_I32, 0)
                    ksteps = -(-(K // 2) // 128)
                    times = {}
                    for s in SPLITS:
                        if s > 1 and s > ksteps:
                            continue
                        # both ways of merging the slices: through the workspace, and on chip where the
                        # kernel supports it (narrow tiles, up to 8 slices)
                        for merge in (nm.NM_MERGE_WORKSPACE, nm.NM_MERGE_CLUSTER):
                            if merge == nm.NM_MERGE_CLUSTER and (s == 1 or s > 8 or chosen.tile_t > 64 or chosen.cta_group != 1):
                                continue
                            plan = nm.nm_plan_create(T, w, nm.NM_OUT_I32, 0)
                            plan.split_k = s
                            plan.merge = merge
                            t_pad = -(-T // plan.tile_t) * plan.tile_t
                            plan.workspace_bytes = 0 if (s == 1 or merge == nm.NM_MERGE_CLUSTER) else s * t_pad * O * 4
                            ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
                            key = f"{s}" if merge == nm.NM_MERGE_WORKSPACE else f"{s}c"
                            times[key] = _time_graph(torch, lambda: nm.nm_spmm(X, w, plan=plan, out=Y, workspace=ws), reps, stream)
                    t_cublas = _time_graph(torch, lambda: torch._int_mm(X, Wd.t()), reps, stream) if T > 16 else None
                    best = min(times, key=times.get)
                    mine = f"{int(chosen.split_k)}" + ("c" if chosen.split_k > 1 and chosen.merge == nm.NM_MERGE_CLUSTER else "")
                    rows.append(dict(sparsity=label, T=T, O=O, K=K, planner_split=mine, best_split=best,
                                     t_planner_us=round(times[mine], 3), t_best_us=round(times[best], 3),
                                     cublas_dense_us=None if t_cublas is None else round(t_cublas, 3),
                                     times_us={k: round(v, 3) for k, v in times.items()}))
        clocks[label] = sampler.summary(since=mark)
    sampler.stop()
    summary = {}
    for label in sparsity:
        sub = [r for r in rows if r["sparsity"] == label]
        norm = [r["t_best_us"] / r["t_planner_us"] for r in sub]
        # a choice within 2 % of the optimum counts as a hit (timer noise on ~5 us kernels)
        hits = [1.0 if (r["planner_split"] == r["best_split"] or r["t_best_us"] / r["t_planner_us"] > 0.98) else 0.0 for r in sub]
        sp = [r["cublas_dense_us"] / r["t_planner_us"] for r in sub if r["cublas_dense_us"]]
        summary[label] = dict(shapes=len(sub), top1_hit_rate=round(float(np.mean(hits)), 3),
                              avg_norm_perf=round(float(np.mean(norm)), 3), worst_norm_perf=round(float(np.min(norm)), 3),
                              geomean_speedup_vs_cublas_dense=round(float(np.exp(np.mean(np.log(sp)))), 3) if sp else None,
                              min_speedup=round(min(sp), 3) if sp else None, max_speedup=round(max(sp), 3) if sp else None,
                              clocks=clocks[label])
    return dict(grid=dict(T=list(Ts), O=list(OKs), K=list(OKs)), summary=summary, rows=rows)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--out", default=None)
    ap.add_argument("--quick", action="store_true", help="a 2x2x2 corner of the grid")
    args = ap.parse_args()
    Ts = (64, 512) if args.quick else (64, 128, 256, 512)
    OKs = (128, 1024) if args.quick else (128, 256, 512, 1024)
    out = evaluate(Ts, OKs, args.reps)
    print(json.dumps(out["summary"], indent=1))
    if args.out:
        json.dump(out, open(args.out, "w"))


if __name__ == "__main__":
    main()
