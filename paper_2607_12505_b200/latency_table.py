"""Export the per-operator sparsity-latency lookup table (Section 5.1) to a file.

    python -m paper_2607_12505_b200.latency_table --model deit_b --batch 64 --out lut.csv [--dtype i8|f16] [--json]

One row per (operator shape, N:8 ratio): T, K, O, n, m, path, tile_t, split_k, mean and minimum
microseconds, measured by nm_latency_table (graph-replayed back-to-back calls).  The table is what
nm_predictor_fit / nm_search consume as t_l(s_l).
"""
from __future__ import annotations

import argparse
import csv
import json

from .inputs import MODELS, layer_shapes

FIELDS = ["T", "K", "O", "n", "m", "dtype", "out_dtype", "path", "tile_t", "split_k", "reps", "status", "us_mean", "us_min"]


def export(model: str, batch: int, dtype: str = "i8", reps: int = 20, ratios=None):
    from . import binding as nm
    T = batch * MODELS[model][2]
    shapes = sorted({(K, O) for (_, K, O) in layer_shapes(model)})
    ratios = ratios or [(n, 8) for n in range(1, 9)]
    dt, od = (nm.NM_I8, nm.NM_OUT_I32) if dtype == "i8" else (nm.NM_F16, nm.NM_OUT_F16)
    return nm.nm_latency_table([(T, O, K) for (K, O) in shapes], ratios, dtype=dt, out_dtype=od, reps=reps)


def write(rows, path: str, as_json: bool = False):
    if as_json:
        with open(path, "w") as f:
            json.dump([{k: r[k] for k in FIELDS} for r in rows], f, indent=1)
        return
    with open(path, "w", newline="") as f:
        w = csv.DictWriter(f, fieldnames=FIELDS)
        w.writeheader()
        for r in rows:
            w.writerow({k: (round(r[k], 3) if isinstance(r[k], float) else r[k]) for k in FIELDS})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="deit_b", choices=sorted(MODELS))
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--dtype", default="i8", choices=["i8", "f16"])
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--out", required=True)
    ap.add_argument("--json", action="store_true")
    args = ap.parse_args()
    rows = export(args.model, args.batch, args.dtype, args.reps)
    write(rows, args.out, args.json)
    print(f"{len(rows)} rows -> {args.out}")


if __name__ == "__main__":
    main()
