"""Sustained throughput of tensor-bound GEMMs under the board power limit, with the clocks seen.

    python -m bench.sustained [--seconds 4] [--out sustained.json]

A graph of 20 back-to-back calls lasts a few milliseconds: short enough for the GPU to run it at
its maximum clock.  A kernel that keeps the tensor cores busy for seconds is throttled to the
board power limit instead (`sw_power_cap`), and what it then delivers depends on the energy it
spends per multiply-accumulate -- including the energy of toggling real data, which an all-zero
operand does not spend.  For each shape this replays a graph of 50 calls for `--seconds` while a
thread samples `nvidia-smi` (SM clock, power, throttle reasons; read-only queries), for nm_spmm
under its own plan, for nm_spmm on an all-zero X, and for dense cuBLAS on the same operands.
"""
from __future__ import annotations

import argparse
import json
import subprocess
import threading
import time

import numpy as np

SHAPES = [  # (label, T, K, O, n, m, dtype, out)
    ("vit_l.b256.fc2 f16 2:4", 50432, 4096, 1024, 2, 4, "f16", "f16"),
    ("deit_b.qkv f16 2:4", 25216, 768, 2304, 2, 4, "f16", "f16"),
    ("deit_b.fc1 f16 2:4", 25216, 768, 3072, 2, 4, "f16", "f16"),
    ("vit_l.b256.fc2 i8 2:4", 50432, 4096, 1024, 2, 4, "i8", "i32"),
    ("deit_b.fc2 i8 2:4", 25216, 3072, 768, 2, 4, "i8", "i32"),
]
QUERY = "clocks.sm,power.draw,clocks_event_reasons.sw_power_cap,clocks_event_reasons.hw_slowdown,clocks_event_reasons.sw_thermal_slowdown"


def _sampler(stop, rows, index):
    while not stop.is_set():
        r = subprocess.run(["nvidia-smi", f"--query-gpu={QUERY}", "--format=csv,noheader,nounits", "-i", str(index)],
                           capture_output=True, text=True)
        if r.returncode == 0 and r.stdout.strip():
            rows.append([c.strip() for c in r.stdout.strip().split(",")])
        time.sleep(0.1)


def _sustain(torch, fn, seconds, stream, index):
    with torch.cuda.stream(stream):
        fn()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(50):
                fn()
        g.replay()
        stream.synchronize()
        stop, rows = threading.Event(), []
        th = threading.Thread(target=_sampler, args=(stop, rows, index))
        th.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0, reps = time.time(), 0
        e0.record(stream)
        while time.time() - t0 < seconds:
            g.replay()
            reps += 1
            if reps % 20 == 0:
                stream.synchronize()
        e1.record(stream)
        stream.synchronize()
        stop.set()
        th.join()
    rows = rows[3:] if len(rows) > 6 else rows          # the first samples see the ramp
    clk = [float(r[0]) for r in rows]
    pw = [float(r[1]) for r in rows]
    return dict(us=e0.elapsed_time(e1) * 1e3 / (reps * 50), sm_mhz=float(np.median(clk)) if clk else None,
                watts=float(np.median(pw)) if pw else None,
                power_cap=float(np.mean([r[2] == "Active" for r in rows])) if rows else None,
                slowdown=any(r[3] == "Active" or r[4] == "Active" for r in rows))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seconds", type=float, default=4.0)
    ap.add_argument("--out", default=None)
    args = ap.parse_args()

    import torch
    from paper_2607_12505_b200 import binding as nm
    from paper_2607_12505_b200 import inputs

    stream = torch.cuda.Stream()
    index = torch.cuda.current_device()
    out = []
    for (label, T, K, O, n, m, dt, o) in SHAPES:
        od = {"i32": nm.NM_OUT_I32, "f16": nm.NM_OUT_F16, "f32": nm.NM_OUT_F32}[o]
        X, W = inputs.make_layer(dict(T=T, O=O, K=K, n=n, m=m, dtype=dt, name="sustained"))
        w = nm.nm_compress(W, n, m)
        plan = nm.nm_plan_create(T, w, od, 0)
        Xd, Xz = torch.from_numpy(X).cuda(), torch.zeros((T, K), dtype=torch.int8 if dt == "i8" else torch.float16, device="cuda")
        Wd = torch.from_numpy(W).cuda()
        Y = torch.empty((T, O), dtype=nm._out_torch_dtype(od), device="cuda")
        ops = 2.0 * T * K * O
        row = dict(shape=label, T=T, K=K, O=O, nm=f"{n}:{m}", dtype=dt, plan={k: v for k, v in plan.as_dict().items() if k in ("path", "tile_t", "cta_group", "split_k", "issuers")})
        for key, fn in (("nm_spmm", lambda: nm.nm_spmm(Xd, w, plan=plan, out=Y, out_dtype=od)),
                        ("nm_spmm_zero_x", lambda: nm.nm_spmm(Xz, w, plan=plan, out=Y, out_dtype=od)),
                        ("cublas_dense", (lambda: torch._int_mm(Xd, Wd.t())) if dt == "i8" else (lambda: torch.matmul(Xd, Wd.t())))):
            r = _sustain(torch, fn, args.seconds, stream, index)
            r["dense_equiv_tops"] = round(ops / r["us"] / 1e6, 1)
            r["us"] = round(r["us"], 2)
            row[key] = r
        print(json.dumps(row), flush=True)
        out.append(row)
    if args.out:
        json.dump(out, open(args.out, "w"))


if __name__ == "__main__":
    main()
