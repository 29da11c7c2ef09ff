"""The planner's choice against an exhaustive sweep over (CTA group, token tile, issuing warps).

    python -m bench.plan_sweep [--out sweep.json] [--reps 20]

For 40 shapes drawn from the benchmark configurations (DeiT-S / DeiT-B / Swin-T / ViT-L layers, INT8 and
FP16, ratios on the sparse and on the dense tensor-core path, 1576 to 200704 tokens) every combination
of CTA group in {1, 2}, token tile in {64, 96, ..., 256} and 1 or 2 issuing warps that the kernels accept
is timed as one CUDA graph of `reps` calls over rotating buffers (> 256 MB), next to the plan
nm_plan_create picks.  Prints one line per shape and the totals; clocks are sampled while it runs.
"""
from __future__ import annotations

import argparse
import itertools
import json

import numpy as np

SHAPES = [  # (T, O, K, n, m, dtype)
    (12608, 1152, 384, 2, 4, "i8"), (12608, 384, 384, 2, 4, "i8"), (12608, 1536, 384, 2, 4, "i8"), (12608, 384, 1536, 2, 4, "i8"),
    (25216, 2304, 768, 2, 4, "i8"), (25216, 768, 768, 2, 4, "i8"), (25216, 3072, 768, 2, 4, "i8"), (25216, 768, 3072, 2, 4, "i8"),
    (25216, 768, 3072, 4, 4, "i8"), (25216, 3072, 768, 4, 4, "i8"), (25216, 768, 768, 4, 4, "i8"),
    (25216, 2304, 768, 2, 4, "f16"), (25216, 768, 3072, 2, 4, "f16"), (25216, 768, 3072, 4, 4, "f16"),
    (1576, 3072, 1024, 2, 4, "i8"), (1576, 4096, 1024, 2, 4, "i8"), (1576, 1024, 4096, 2, 4, "i8"), (1576, 3072, 1024, 4, 8, "i8"),
    (1576, 3072, 1024, 2, 4, "f16"), (1576, 4096, 1024, 2, 4, "f16"), (1576, 1024, 4096, 2, 4, "f16"),
    (1576, 3072, 1024, 4, 8, "f16"), (1576, 4096, 1024, 4, 8, "f16"),
    (3136, 2304, 768, 2, 4, "i8"), (3136, 768, 3072, 2, 4, "i8"), (3136, 768, 768, 2, 4, "i8"), (3136, 3072, 768, 4, 8, "i8"),
    (50176, 768, 192, 2, 4, "i8"), (50176, 576, 192, 2, 4, "i8"), (50176, 192, 768, 2, 4, "i8"),
    (12544, 1536, 384, 2, 4, "i8"), (12544, 1152, 384, 4, 8, "i8"), (200704, 288, 96, 2, 4, "i8"), (200704, 96, 384, 2, 4, "i8"),
    (50432, 1024, 4096, 2, 4, "i8"), (50432, 4096, 1024, 2, 4, "i8"), (12608, 3072, 1024, 2, 4, "i8"),
    (12608, 4096, 1024, 2, 4, "f16"), (12608, 1024, 4096, 4, 8, "f16"), (12608, 3072, 1024, 4, 8, "i8"),
]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--reps", type=int, default=20)
    args = ap.parse_args()

    import torch
    from paper_2607_12505_b200 import binding as nm
    from paper_2607_12505_b200 import inputs
    from bench.clocks import ClockSampler

    stream = torch.cuda.Stream()
    sampler = ClockSampler(torch.cuda.current_device()).start()

    def timeit(fn):
        with torch.cuda.stream(stream):
            fn(0)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(args.reps):
                    fn(i)
            g.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) * 1e3 / args.reps

    rows = []
    for (T, O, K, n, m, dt) in SHAPES:
        i8 = dt == "i8"
        od = nm.NM_OUT_I32 if i8 else nm.NM_OUT_F16
        W = (inputs.w_i8 if i8 else inputs.w_f16)(O, K, n, m, "plan_sweep")
        w = nm.nm_compress(W, n, m)
        per_set = T * K * (1 if i8 else 2) + T * O * (4 if i8 else 2)
        R = max(1, min(8, int(np.ceil(256e6 / per_set))))
        Xs = [(torch.randint(-128, 128, (T, K), dtype=torch.int8, device="cuda") if i8 else
               (torch.randn((T, K), device="cuda") * 0.02).half()) for _ in range(R)]
        Ys = [torch.empty((T, O), dtype=nm._out_torch_dtype(od), device="cuda") for _ in range(R)]
        base = nm.nm_plan_create(T, w, od, 0)

        def run(plan):
            ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
            return timeit(lambda i: nm.nm_spmm(Xs[i % R], w, plan=plan, out=Ys[i % R], out_dtype=od, workspace=ws, stream=stream))
        t_plan = run(base)
        res = {}
        for cg, tt, iss in itertools.product((1, 2), (64, 96, 128, 160, 192, 224, 256), (1, 2)):
            if tt > ((T + 31) // 32) * 32 or (cg == 2 and O <= 128):
                continue
            if iss == 2 and (cg == 2 or 2 * tt + (64 if base.path == nm.NM_PATH_UMMA_SP24 else 0) > 512):
                continue
            p = nm.nm_plan_create(T, w, od, 0)
            p.cta_group, p.tile_t, p.issuers, p.split_k, p.workspace_bytes = cg, tt, iss, 1, 0
            try:
                res[f"g{cg}t{tt}i{iss}"] = round(run(p), 2)
            except nm.NMError:
                continue
        best = min(res, key=res.get)
        t_best = min(res[best], t_plan)
        rows.append(dict(T=T, O=O, K=K, nm=f"{n}:{m}", dtype=dt, planner=f"g{base.cta_group}t{base.tile_t}i{base.issuers}s{base.split_k}",
                         t_planner_us=round(t_plan, 2), best=best, t_best_us=t_best, times_us=res))
        print(f"{T}x{K}->{O} {n}:{m} {dt}: planner {rows[-1]['planner']} {t_plan:.2f} us | best of sweep {best} {res[best]:.2f} us | "
              f"planner / best {t_plan / t_best:.3f}", flush=True)
    ratios = [r["t_planner_us"] / r["t_best_us"] for r in rows]
    summary = dict(shapes=len(rows), geomean_planner_over_best=round(float(np.exp(np.mean(np.log(ratios)))), 4),
                   worst=round(max(ratios), 3), total_planner_us=round(sum(r["t_planner_us"] for r in rows), 1),
                   total_best_us=round(sum(r["t_best_us"] for r in rows), 1), clocks=sampler.stop())
    print(json.dumps(summary))
    if args.out:
        json.dump(dict(summary=summary, rows=rows), open(args.out, "w"))


if __name__ == "__main__":
    main()
