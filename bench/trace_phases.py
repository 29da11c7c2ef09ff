"""Where the time of a launch goes: wall-clock stamps of the pipeline phases of every CTA.

    python -m bench.trace_phases --stack vit_l_b1 [--nm 2:4] [--dtype i8]
    python -m bench.trace_phases --T 1576 --O 3072 --K 1024 --nm 4:8 --dtype f16 [--reps 6]

Uses the trace build of the library (compiled with -DNM_TRACE; the product library has no stamps):
each CTA of the tcgen05 kernels writes %globaltimer at kernel entry, end of prologue, release of
the grid-dependency wait, first ring stage full, last commit of its first and of its last tile,
first accumulator ready, last store of its first and of its last tile, staging patch free, and
just before tensor memory is freed.  The launches are replayed as one CUDA graph (dependent
launches, as in a model); the table gives, per layer of the last replay, the earliest / median /
latest CTA for every phase relative to the release of the grid-dependency wait, and the gap
between the end of one layer and the release of the next one's wait.

Timing experiments of the trace build (environment variable NM_DBG, read at launch): 1 = the issuing
warp issues no MMAs (stages are recycled at once), 2 = the epilogue stores nothing, 3 = both, i.e. only
the operand loads run; 4 (CTA-pair kernel only) = the ring is loaded once and the K loops run over it
without further loads, so 6 = the MMAs alone.  Results are wrong by construction; only the times mean
something.  For timing these modes use `NM_B200_TRACE=2 python -m bench.profile_case ...`: that library
has the switches without the stamp code, which slows the inner loops by itself.
"""
from __future__ import annotations

import argparse
import json
import os

os.environ["NM_B200_TRACE"] = "1"

import numpy as np  # noqa: E402

SLOTS = ["entry", "prologue_done", "wait_released", "first_stage_full", "first_tile_committed", "last_tile_committed",
         "first_acc_ready", "first_tile_stored", "last_tile_stored", "patch_free", "before_dealloc"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--stack", default=None, choices=[None, "vit_l_b1", "vit_l_b8"])
    ap.add_argument("--T", type=int, default=1576)
    ap.add_argument("--O", type=int, default=3072)
    ap.add_argument("--K", type=int, default=1024)
    ap.add_argument("--nm", default="2:4")
    ap.add_argument("--dtype", default="i8", choices=["i8", "f16"])
    ap.add_argument("--reps", type=int, default=6, help="single shape: back-to-back calls on rotating buffers in the graph")
    ap.add_argument("--stages", type=int, default=0, help="override the ring depth of every plan (0: the planner's)")
    ap.add_argument("--tile-t", type=int, default=0, help="override the token tile of every plan (0: the planner's)")
    ap.add_argument("--split-k", type=int, default=0, help="override split-K of every plan that splits (0: the planner's)")
    ap.add_argument("--issuers", type=int, default=0)
    ap.add_argument("--cta-group", type=int, default=0)
    ap.add_argument("--out", default=None)
    args = ap.parse_args()

    import ctypes
    import torch
    from paper_2607_12505_b200 import binding as nm
    from paper_2607_12505_b200 import inputs

    n, m = (int(v) for v in args.nm.split(":"))
    i8 = args.dtype == "i8"
    od = nm.NM_OUT_I32 if i8 else nm.NM_OUT_F16
    if args.stack:
        T = 197 * (1 if args.stack == "vit_l_b1" else 8)
        specs = [dict(name=f"{blk}.{nme}", T=T, K=K, O=O) for blk in range(24)
                 for (nme, K, O) in [("qkv", 1024, 3072), ("fc1", 1024, 4096), ("fc2", 4096, 1024)]]
    else:
        specs = [dict(name=f"call{i}", T=args.T, K=args.K, O=args.O) for i in range(args.reps)]
    L = nm.lib()
    L.nm_trace_set_buffer.argtypes = [ctypes.c_void_p]
    L.nm_trace_set_buffer.restype = None
    layers = []
    for s in specs:
        W = (inputs.w_i8 if i8 else inputs.w_f16)(s["O"], s["K"], n, m, "trace", s["name"])
        X = (inputs.x_i8 if i8 else inputs.x_f16)(s["T"], s["K"], "trace", s["name"])
        w = nm.nm_compress(W, n, m)
        plan = nm.nm_plan_create(s["T"], w, od, 0)
        if args.stages:
            plan.stages = args.stages
        if args.issuers:
            plan.issuers = args.issuers
        if args.cta_group:
            plan.cta_group = args.cta_group
        if args.tile_t or args.split_k:
            plan.tile_t = args.tile_t or plan.tile_t
            if args.split_k:
                plan.split_k = args.split_k
            t_pad = -(-s["T"] // plan.tile_t) * plan.tile_t
            plan.workspace_bytes = plan.split_k * t_pad * s["O"] * 4 if plan.split_k > 1 else 0
        Xd = torch.from_numpy(X).cuda()
        Yd = torch.empty((s["T"], s["O"]), dtype=nm._out_torch_dtype(od), device="cuda")
        ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
        tr = torch.zeros((2 * 148 + 8, 16), dtype=torch.int64, device="cuda")
        layers.append(dict(spec=s, w=w, plan=plan, Xd=Xd, Yd=Yd, ws=ws, tr=tr))
    stream = torch.cuda.Stream()

    def run():
        for Lr in layers:
            L.nm_trace_set_buffer(Lr["tr"].data_ptr())
            nm.nm_spmm(Lr["Xd"], Lr["w"], plan=Lr["plan"], out=Lr["Yd"], out_dtype=od, workspace=Lr["ws"], stream=stream)
        L.nm_trace_set_buffer(None)

    with torch.cuda.stream(stream):
        run()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            run()
        for _ in range(3):
            g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    total_us = e0.elapsed_time(e1) * 1e3
    rows = []
    prev_end = None
    for Lr in layers:
        t = Lr["tr"].cpu().numpy().astype(np.int64)
        t = t[t[:, 0] > 0]                       # CTAs that ran
        rel = t[:, 2].min()                      # first CTA past the grid-dependency wait
        row = dict(name=Lr["spec"]["name"], ctas=int(t.shape[0]), tiles_per_cta_max=int(t[:, 12].max()),
                   plan={k: v for k, v in Lr["plan"].as_dict().items() if k in ("path", "tile_t", "cta_group", "split_k", "issuers")})
        for i, name in enumerate(SLOTS):
            col = t[:, i][t[:, i] > 0]
            if col.size:
                row[name] = [round(float(v - rel) / 1e3, 2) for v in (col.min(), np.median(col), col.max())]
        # cycles inside waits (per CTA; median over CTAs), shown as microseconds at 1.9 GHz
        for slot, name in ((13, "issuer_waits_stage_us"), (14, "issuer_waits_drain_us"), (15, "producer_waits_free_stage_us"), (11, "epilogue_waits_acc_us")):
            col = t[:, slot][t[:, slot] > 0]             # CTAs that have the role (the peer of a CTA pair issues nothing)
            row[name] = round(float(np.median(col)) / 1900.0, 2) if col.size else 0.0
        end = t[:, 10].max()
        row["launch_span_us"] = round(float(end - rel) / 1e3, 2)
        row["gap_prev_end_to_release_us"] = None if prev_end is None else round(float(rel - prev_end) / 1e3, 2)
        prev_end = end
        rows.append(row)
    out = dict(total_us=round(total_us, 2), us_per_launch=round(total_us / len(layers), 2), layers=rows)
    cols = ["entry", "wait_released", "first_stage_full", "first_tile_committed", "last_tile_committed", "first_acc_ready",
            "last_tile_stored", "before_dealloc"]
    print(f"graph replay: {total_us:.1f} us, {total_us / len(layers):.2f} us per launch (stamps cost a little)")
    print("us relative to the first CTA's release from the grid-dependency wait; earliest/median/latest CTA")
    print("| layer | CTAs | " + " | ".join(cols) + " | span | gap before |")
    print("|---|---|" + "---|" * (len(cols) + 2))
    for r in rows[:12] + rows[-3:] if len(rows) > 15 else rows:
        print(f"| {r['name']} | {r['ctas']} | " + " | ".join("/".join(f"{v:.2f}" for v in r.get(c, [0, 0, 0])) for c in cols) +
              f" | {r['launch_span_us']} | {r['gap_prev_end_to_release_us']} |")
    print("time inside waits, median CTA (us at 1.9 GHz): issuing warp for a loaded stage / for a drained accumulator; producer for a free stage; epilogue warp for an accumulator")
    for r in (rows[:6] if len(rows) > 6 else rows):
        print(f"  {r['name']}: {r['issuer_waits_stage_us']} / {r['issuer_waits_drain_us']} ; {r['producer_waits_free_stage_us']} ; {r['epilogue_waits_acc_us']}  (span {r['launch_span_us']})")
    if len(rows) > 3:
        body = rows[2:]
        print("mean over layers (from the third on): span %.2f us, gap %.2f us" % (
            np.mean([r["launch_span_us"] for r in body]), np.mean([r["gap_prev_end_to_release_us"] for r in body])))
        for c in cols:
            print(f"  {c}: median-CTA mean {np.mean([r[c][1] for r in body if c in r]):.2f} us")
    if args.out:
        json.dump(out, open(args.out, "w"))


if __name__ == "__main__":
    main()
