"""Markdown rendering of the JSON that `python -m bench.report --out report.json` writes.

    python -m bench.report_md report.json > profiles/report_all_configs.md

Measurement harness only (formatting; nothing is timed here).
"""
from __future__ import annotations

import json
import math
import sys


def _geo(xs):
    return math.exp(sum(math.log(x) for x in xs) / len(xs)) if xs else None


def _plan(p):
    return f"p{p['path']} g{p['cta_group']} t{p['tile_t']} s{p['split_k']} i{p['issuers']}"


def _is_sparse_path(r):
    return r["plan"]["path"] == 2


def main(path):
    d = json.load(open(path))
    rows = [r for r in d["rows"] if r.get("config") in ("cfg0", "cfg1", "cfg2", "cfg3", "cfg4")]
    q_rows = [r for r in d["rows"] if str(r.get("config", "")).endswith(".int8_out")]
    stacks = [r for r in d["rows"] if "workload" in r]
    pk = d["peaks"]
    out = []
    out.append("# All benchmark configurations on one B200 — nm_spmm under its own plan vs dense cuBLAS\n")
    out.append("Commands: `python -m bench.report --out report.json` (every distinct shape / ratio / dtype of the five\n"
               "configurations; each timing is one CUDA graph of 20 back-to-back calls over rotating buffer sets > 256 MB, replayed),\n"
               "then `python -m bench.report_md report.json` (this file).\n"
               f"Dense library peaks measured in the same run (8192^3): INT8 {pk['int8_dense_tops']:.0f} TOPS, FP16 {pk['fp16_dense_tflops']:.0f} TFLOPS; the sparse tensor\n"
               f"roofline is taken as twice those; HBM roofline {d['hbm_gbs']} GB/s (measured copy). `plan` = path (1 dense MMA, 2 sparse MMA), CTA group, token tile, split-K, issuing warps.\n")
    out.append("Clocks sampled (read-only `nvidia-smi --query-gpu`, 100 ms period) while each configuration was timed:\n")
    out.append("| group | median SM MHz | min | max | max power W | reasons active | samples |")
    out.append("|---|---|---|---|---|---|---|")
    bad = []
    for g, c in d["clocks"].items():
        out.append(f"| {g} | {c['sm_mhz']} | {c['sm_min_mhz']} | {c['sm_max_mhz']} | {c['power_w_max']} | {', '.join(c['reasons']) or '—'} | {c['samples']} |")
        bad += [x for x in c["reasons"] if x in ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")]
    out.append("")
    out.append("No group saw `hw_slowdown`, `hw_thermal_slowdown` or `sw_thermal_slowdown`; `sw_power_cap` is kept where it shows."
               if not bad else f"SLOWDOWN REASONS SEEN: {sorted(set(bad))} — re-run.")
    out.append("")
    out.append("Geometric mean of the speed-up over dense cuBLAS (`torch._int_mm` / `torch.matmul`, same buffers, same timing):\n")
    out.append("| config | dtype | ratios on the sparse tensor core (2:4-clean) | other ratios (dense MMA) |")
    out.append("|---|---|---|---|")
    for cfg in ("cfg1", "cfg2", "cfg3", "cfg4"):
        for dt in ("i8", "f16"):
            sel = [r for r in rows if r["config"] == cfg and r["dtype"] == dt]
            if not sel:
                continue
            cells = []
            for sp in (True, False):
                s = [r for r in sel if _is_sparse_path(r) == sp]
                if not s:
                    cells.append("–")
                    continue
                su = [r["speedup"] for r in s]
                fr = [r["frac_roofline"] for r in s]
                cells.append(f"{_geo(su):.2f}× ({min(su):.2f}–{max(su):.2f}), {min(fr):.2f}–{max(fr):.2f} of roofline")
            out.append(f"| {cfg} | {dt} | {cells[0]} | {cells[1]} |")
    out.append("")
    out.append("| config | layer | T×K×O | n:m | dtype | plan | µs | cuBLAS dense µs | speed-up | dense-equiv T(FL)OPS | GB/s (algorithmic) | bound | fraction of roofline |")
    out.append("|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        out.append(f"| {r['config']} | {r['name']} | {r['T']}×{r['K']}×{r['O']} | {r['nm']} | {r['dtype']} | {_plan(r['plan'])} | {r['us']} | "
                   f"{r['cublas_dense_us']} | {r['speedup']} | {r['dense_tops']} | {r['gbs']} | {r['bound']} | {r['frac_roofline']} |")
    out.append("")
    if stacks:
        out.append("ViT-L batch 1 as one graph of its 72 linear layers (dependent launches, distinct weights):\n")
        for s in stacks:
            out.append(f"* {s['nm']}: {s['us']} µs per pass, {s['us_per_layer']} µs per layer, {s['gbs_image_bytes']} GB/s on the bytes read "
                       f"({s['frac_hbm_image']} of the HBM rate), weights read {s['weights_read_mb']} MB")
        out.append("")
    if q_rows:
        out.append("## Fused requantising epilogue (INT8 in, INT8 out) on the INT8 2:4 layers of cfg1 / cfg2\n")
        out.append("Rows `*.int8_out` of the same run (per-channel scale 1e-4).  Bytes are counted with one byte per output; the sparse "
                   "tensor roofline is twice the dense INT8 peak measured in the run.\n")
        out.append("| layer | T×K×O | plan | µs (INT8 out) | µs (INT32 out) | dense-equiv TOPS | GB/s (algorithmic) | bound | fraction of roofline |")
        out.append("|---|---|---|---|---|---|---|---|---|")
        for r in q_rows:
            out.append(f"| {r['name']} | {r['T']}×{r['K']}×{r['O']} | {_plan(r['plan'])} | {r['us']} | {r['us_int32_out']} | {r['dense_tops']} | {r['gbs']} | {r['bound']} | {r['frac_roofline']} |")
    print("\n".join(out))


if __name__ == "__main__":
    main(sys.argv[1])
