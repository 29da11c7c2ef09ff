"""Calibrate and validate the latency predictor of Section 5.1 on one B200.

    python -m bench.predictor_eval [--model deit_b] [--batch 64] [--fit 40] [--test 24]

1. Table: nm_latency_table over the model's operator shapes x the ratios N:8, N = 1..8
   (INT8 -> INT32), i.e. the (shape, sparsity) lookup table.
2. Measurements: random layer-wise configurations y[l] in 1..8; for each, the model's whole stack
   of linear layers (every layer with its own packed weight and activation buffers) is captured
   in one CUDA graph and timed by replay -- the stand-in for a "full-model measurement".
3. nm_predictor_fit (non-negative least squares, Eq. (1)) on the first --fit configurations;
   relative error of nm_predictor_eval on the remaining --test configurations, next to the plain
   sum of table latencies (gamma = 1, b = 0).
Prints one JSON object.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from paper_2607_12505_b200.inputs import MODELS, layer_shapes  # noqa: E402,F401


class Stack:
    """The linear layers of a ViT-family model on the GPU: the (shape, ratio) latency table and a
    way to measure a whole layer-wise configuration as one replayed CUDA graph."""

    def __init__(self, model="deit_b", batch=64, reps=20, blocks=None):
        import torch
        from paper_2607_12505_b200 import binding as nm
        from paper_2607_12505_b200 import inputs
        self.torch, self.nm, self.inputs = torch, nm, inputs
        self.reps = reps
        self.T = batch * MODELS[model][2]
        self.layers = layer_shapes(model)
        if blocks is not None:
            self.layers = self.layers[:4 * blocks]
        self.L = len(self.layers)
        self.shapes = sorted({(K, O) for (_, K, O) in self.layers})
        ratios = [(n, 8) for n in range(1, 9)]
        rows = nm.nm_latency_table([(self.T, O, K) for (K, O) in self.shapes], ratios, dtype=nm.NM_I8,
                                   out_dtype=nm.NM_OUT_I32, reps=reps)
        self.lut = {}
        for r in rows:
            if r["status"] != 0:
                raise RuntimeError(f"latency table row failed: {r}")
            self.lut[(r["K"], r["O"], r["n"])] = float(r["us_mean"])
        self.stream = torch.cuda.Stream()
        self.packed = {}
        self.Xs = {K: torch.from_numpy(inputs.x_i8(self.T, K, "predictor", K)).cuda() for K in {K for (_, K, _) in self.layers}}
        self.Ys = [torch.empty((self.T, O), dtype=torch.int32, device="cuda") for (_, _, O) in self.layers]

    def table(self):
        """[L, 8]: table latency of every layer at every level N = 1..8."""
        return np.array([[self.lut[(K, O, n)] for n in range(1, 9)] for (_, K, O) in self.layers])

    def table_row(self, cfg):
        return np.array([self.lut[(self.layers[li][1], self.layers[li][2], int(n))] for li, n in enumerate(cfg)])

    def _weight(self, li, n):
        key = (li, n)
        if key not in self.packed:
            nm, torch = self.nm, self.torch
            _, K, O = self.layers[li]
            W = self.inputs.w_i8(O, K, n, 8, "predictor", li, n)
            w = nm.nm_compress(W, n, 8)
            plan = nm.nm_plan_create(self.T, w, nm.NM_OUT_I32, 0)
            ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device="cuda")
            self.packed[key] = (w, plan, ws)
        return self.packed[key]

    def measure(self, cfg):
        """Microseconds of one pass over all layers under configuration cfg (levels 1..8)."""
        nm, torch, stream = self.nm, self.torch, self.stream
        entries = [self._weight(li, int(n)) for li, n in enumerate(cfg)]

        def run():
            for li, (w, plan, ws) in enumerate(entries):
                nm.nm_spmm(self.Xs[self.layers[li][1]], w, plan=plan, out=self.Ys[li], workspace=ws)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            run()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run()
            for _ in range(3):
                g.replay()
            stream.synchronize()
            e0.record(stream)
            for _ in range(self.reps):
                g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) * 1e3 / self.reps

    def operator_columns(self, table_rows):
        """Sum the per-layer table latencies of each operator type: [S, L] -> [S, 4]."""
        kinds = sorted({name.split(".")[1] for (name, _, _) in self.layers})
        idx = [[i for i, (name, _, _) in enumerate(self.layers) if name.split(".")[1] == k] for k in kinds]
        return np.stack([table_rows[:, ix].sum(axis=1) for ix in idx], axis=1), kinds, idx


def evaluate(model="deit_b", batch=64, fit=40, test=24, group="layer", reps=20, seed=0, blocks=None):
    """Runs the three steps; returns (summary dict, design matrix [S, n_coef], measured [S])."""
    import argparse as _ap
    args = _ap.Namespace(model=model, batch=batch, fit=fit, test=test, group=group, reps=reps, seed=seed)
    from paper_2607_12505_b200 import binding as nm
    stack = Stack(model, batch, reps, blocks)
    T, L, layers, lut, shapes, measure = stack.T, stack.L, stack.layers, stack.lut, stack.shapes, stack.measure

    rng = np.random.default_rng(args.seed)
    n_cfg = args.fit + args.test
    cfgs = rng.integers(1, 9, size=(n_cfg, L))
    # a few structured configurations among the calibration set: uniform levels
    for i, n in enumerate(range(1, 9)):
        if i < args.fit:
            cfgs[i, :] = n
    measured = np.array([measure(c) for c in cfgs])
    table = np.array([[lut[(layers[li][1], layers[li][2], int(n))] for li, n in enumerate(c)] for c in cfgs])

    # ---- 3. calibrate and validate
    if args.group == "operator":
        cols, _, _ = stack.operator_columns(table)
    else:
        cols = table
    A_fit, y_fit, A_te, y_te = cols[:args.fit], measured[:args.fit], cols[args.fit:], measured[args.fit:]
    gamma, b, rnorm = nm.nm_predictor_fit(A_fit, y_fit)
    pred_te = nm.nm_predictor_eval(gamma, b, A_te)
    pred_fit = nm.nm_predictor_eval(gamma, b, A_fit)
    err_te = np.abs(pred_te - y_te) / y_te
    err_fit = np.abs(pred_fit - y_fit) / y_fit
    naive_te = np.abs(table[args.fit:].sum(axis=1) - y_te) / y_te
    out = {
        "model": args.model, "batch": args.batch, "tokens": T, "layers": L, "group": args.group,
        "coefficients": int(cols.shape[1]) + 1, "fit_configs": args.fit, "test_configs": args.test,
        "table_us": {f"{K}x{O}": [round(lut[(K, O, n)], 2) for n in range(1, 9)] for (K, O) in shapes},
        "measured_us_range": [round(float(measured.min()), 1), round(float(measured.max()), 1)],
        "gamma_nonzero": int(np.count_nonzero(gamma)), "gamma_range": [round(float(gamma.min()), 3), round(float(gamma.max()), 3)],
        "b_us": round(b, 2), "fit_rnorm": round(rnorm, 3),
        "fit_err_mean": round(float(err_fit.mean()), 4), "fit_err_max": round(float(err_fit.max()), 4),
        "test_err_mean": round(float(err_te.mean()), 4), "test_err_max": round(float(err_te.max()), 4),
        "naive_sum_test_err_mean": round(float(naive_te.mean()), 4), "naive_sum_test_err_max": round(float(naive_te.max()), 4),
    }
    return out, cols, measured


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="deit_b", choices=sorted(MODELS))
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--fit", type=int, default=40)
    ap.add_argument("--test", type=int, default=24)
    ap.add_argument("--group", default="layer", choices=["layer", "operator"],
                    help="one coefficient per layer (Eq. (1)) or one per operator type")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--out", default=None)
    args = ap.parse_args()
    out, _, _ = evaluate(args.model, args.batch, args.fit, args.test, args.group, args.reps, args.seed)
    print(json.dumps(out))
    if args.out:
        json.dump(out, open(args.out, "w"))


if __name__ == "__main__":
    main()
