"""Close the loop of Section 5 on one B200: table -> calibrated predictor -> Algorithm 1 ->
measure what the search chose.

    python -m bench.search_eval [--model deit_b] [--batch 64] [--budgets 0.8,0.85,0.9,0.95]

The fitness is synthetic (the paper's is the accuracy inherited from a trained supernet, which
needs ImageNet and trained weights): separable, increasing and concave in the level of each
layer with a random per-layer sensitivity, plus a small configuration-dependent perturbation.
For each budget (a fraction of the measured all-dense stack latency) it reports the chosen
configuration, its predicted and measured latency, and its fitness next to two baselines under
the same budget: the densest uniform configuration, and the best of as many random feasible
configurations as the search evaluated.
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="deit_b")
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--budgets", default="0.8,0.85,0.9,0.95")
    ap.add_argument("--generations", type=int, default=30)
    ap.add_argument("--offspring", type=int, default=8)
    ap.add_argument("--overshoot-k", type=int, default=3)
    ap.add_argument("--fit", type=int, default=32)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--out", default=None)
    args = ap.parse_args()

    from paper_2607_12505_b200 import binding as nm
    from bench.predictor_eval import Stack

    stack = Stack(args.model, args.batch, args.reps)
    L = stack.L
    rng = np.random.default_rng(args.seed)

    # ---- calibrate Eq. (1), one coefficient per operator type, on random + uniform configurations
    cfgs = rng.integers(1, 9, size=(args.fit, L))
    for i, n in enumerate(range(1, 9)):
        cfgs[i, :] = n
    measured = np.array([stack.measure(c) for c in cfgs])
    rows = np.array([stack.table_row(c) for c in cfgs])
    cols, kinds, idx = stack.operator_columns(rows)
    g_op, b, _ = nm.nm_predictor_fit(cols, measured)
    gamma = np.zeros(L)
    for k, ix in enumerate(idx):
        gamma[ix] = g_op[k]
    table = stack.table()
    dense_us = float(measured[7])                       # the uniform 8:8 configuration

    # ---- synthetic fitness: sum_l s_l * log2(1 + level) (+ perturbation)
    sens = rng.uniform(0.2, 1.0, size=L)
    gain = sens[:, None] * np.log2(1.0 + np.arange(1, 9))[None, :]
    noise = 0.02

    def fitness_of(y):
        args_f = nm.NMFitnessSeparableArgs(gain.ctypes.data_as(nm.ctypes.POINTER(nm.ctypes.c_double)), 8, 0, noise, 11)
        ya = np.asarray(y, dtype=np.int32)
        return float(nm.lib().nm_fitness_separable(ya.ctypes.data_as(nm.ctypes.POINTER(nm.ctypes.c_int32)), L,
                                                   nm.ctypes.cast(nm.ctypes.pointer(args_f), nm.ctypes.c_void_p)))

    results = []
    for frac in [float(v) for v in args.budgets.split(",")]:
        target = frac * dense_us
        y, res, st = nm.nm_search(table, gamma, b, target, args.generations, args.offspring, overshoot_k=args.overshoot_k,
                                  n_init=4, seed=args.seed, separable_gain=gain, noise=noise, fitness_seed=11)
        row = {"budget_frac": frac, "target_us": round(target, 1), "status": st}
        if st == nm.NM_OK:
            meas = stack.measure(y)
            pred = float(nm.nm_predictor_eval(gamma, b, table[np.arange(L), np.array(y) - 1])[0])
            # baselines under the same predicted budget
            uni = None
            for n in range(8, 0, -1):
                if float(nm.nm_predictor_eval(gamma, b, table[:, n - 1])[0]) <= target:
                    uni = [n] * L
                    break
            best_rand, tried = -np.inf, 0
            while tried < int(res["fitness_evals"]):
                c = rng.integers(1, 9, size=L)
                tried += 1
                if float(nm.nm_predictor_eval(gamma, b, table[np.arange(L), c - 1])[0]) <= target:
                    best_rand = max(best_rand, fitness_of(c))
            row.update({"config": y, "levels_hist": np.bincount(y, minlength=9)[1:].tolist(),
                        "predicted_us": round(pred, 1), "measured_us": round(meas, 1),
                        "measured_over_target": round(meas / target, 4), "pred_err": round(abs(pred - meas) / meas, 4),
                        "fitness": round(res["fitness"], 4), "fitness_uniform": None if uni is None else round(fitness_of(uni), 4),
                        "fitness_best_random_feasible": None if best_rand == -np.inf else round(best_rand, 4),
                        "fitness_evals": int(res["fitness_evals"]), "latency_evals": int(res["latency_evals"])})
        results.append(row)
        print(json.dumps(row))
    out = {"model": args.model, "batch": args.batch, "layers": L, "dense_us": round(dense_us, 1),
           "gamma_per_operator": dict(zip(kinds, [round(float(v), 3) for v in g_op])), "b_us": round(b, 2), "results": results}
    if args.out:
        json.dump(out, open(args.out, "w"))


if __name__ == "__main__":
    main()
