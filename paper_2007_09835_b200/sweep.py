"""Sparsity / group-size sweep on a synthesized layer (Section 3 of the paper: the group size is
"determined offline with actual ... testings using synthesized CNN layers").

    python -m paper_2007_09835_b200.sweep [--json out.json] [--iters 30]

Layer: C_in = C_out = 256, T = 8, H = W = 14, 3x3x3, batch 32, bf16 (config 4 of the baseline).
For every group size g_m x g_n and FLOPs pruning rate it times rt3d_conv3d_sparse with a KGS
mask (exact number of kept (group, location) pairs) and with a vanilla mask (whole groups), and
reports time, speedup over rt3d_conv3d_dense on the same shape, and speedup / pruning rate
(the paper's 3.43x at 3.6x is 0.95 on a phone).  Group sizes beyond the paper's 4..8 show
where that ratio holds on B200: when a kernel group is as wide as a tensor-core bundle and as
deep as a 64-channel K chunk, a pruned location is a K step that is never issued.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

import rt3d_synth as synth
from paper_2007_09835_b200 import binding as B, nets

PAPER_GROUPS = [(4, 4), (8, 4), (8, 8)]
WIDE_GROUPS = [(16, 16), (32, 16), (64, 64), (128, 64), (256, 64)]
RATES = [1, 2, 3, 4, 6, 8]


def time_layer(layer, x, y, iters, algo=B.ALGO_AUTO):
    for _ in range(5):
        layer(x, y, algo=algo)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        layer(x, y, algo=algo)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3        # microseconds


def run(iters=30, groups=None, rates=None, algo=B.ALGO_AUTO, schemes=("kgs", "vanilla")):
    spec = synth.ConvSpec("sweep", 256, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    x = nets.to_device(synth.make_input(4, (32, 8, 14, 14, 256)))
    base = synth.make_layer(spec, 4, 0, 4, 4, "none", None)
    dense = nets.ConvLayer(spec, base["w"], base["bias"], None, dtype=torch.bfloat16, dense=True)
    y = dense.alloc_out(x)
    dense_us = time_layer(dense, x, y, iters)
    _, dense_macs, _ = dense.cost(x)
    rows = [{"scheme": "dense", "g_m": 0, "g_n": 0, "rate": 1.0, "us": dense_us, "speedup": 1.0, "ratio": 1.0,
             "tflops_actual": 2 * dense_macs / dense_us / 1e6, "kernel": B.rt3d_last_plan()["kernel"]}]
    for g_m, g_n in (groups or PAPER_GROUPS + WIDE_GROUPS):
        P, Q = synth.n_groups(256, 256, g_m, g_n)
        for rate in (rates or RATES):
            for scheme in schemes:
                if scheme == "vanilla" and (rate == 1 or round(P * Q / rate) < 1):
                    continue
                if scheme == "kgs":
                    L = synth.make_layer(spec, 4, g_m * 1000 + g_n * 10 + rate, g_m, g_n, "exact_total",
                                         round(P * Q * 27 / rate))
                else:
                    L = synth.make_layer(spec, 4, g_m * 1000 + g_n * 10 + rate, g_m, g_n, "vanilla_total",
                                         round(P * Q / rate))
                lay = nets.ConvLayer(spec, base["w"], base["bias"], L["mask"], g_m, g_n, torch.bfloat16)
                us = time_layer(lay, x, y, iters, algo)
                plan = B.rt3d_last_plan()
                kept, _, _ = lay.cost(x)
                real_rate = dense_macs / kept
                rows.append({"scheme": scheme, "g_m": g_m, "g_n": g_n, "rate": real_rate, "us": us,
                             "speedup": dense_us / us, "ratio": dense_us / us / real_rate,
                             "tflops_actual": 2 * kept / us / 1e6, "kernel": plan["kernel"]})
                lay.packed.free()
    if B.rt3d_last_device_status() != B.OK:
        raise RuntimeError("device reported a bounded-wait timeout")
    return rows


def as_markdown(rows) -> str:
    names = {0: "CUDA cores", 1: "single CTA", 2: "CTA pair", 3: "small C_in", 4: "halo", 6: "sub-tile"}
    out = ["| scheme | group | FLOPs pruning rate | time (us) | speedup vs dense | speedup / rate | actual TFLOP/s | kernel |",
           "|---|---|---|---|---|---|---|---|"]
    for r in rows:
        g = "-" if r["scheme"] == "dense" else f'{r["g_m"]}x{r["g_n"]}'
        out.append(f'| {r["scheme"]} | {g} | {r["rate"]:.2f} | {r["us"]:.1f} | {r["speedup"]:.2f} | {r["ratio"]:.2f} | '
                   f'{r["tflops_actual"]:.0f} | {names.get(r.get("kernel"), r.get("kernel"))} |')
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--json", default=None)
    ap.add_argument("--groups", default=None, help="comma-separated g_m x g_n list, e.g. 8x8,16x16 (default: all)")
    ap.add_argument("--rates", default=None, help="comma-separated FLOPs pruning rates (default: 1,2,3,4,6,8)")
    ap.add_argument("--algo", default="auto", choices=["auto", "pair", "sub"], help="kernel family for the pruned rows")
    args = ap.parse_args()
    groups = [tuple(int(v) for v in g.split("x")) for g in args.groups.split(",")] if args.groups else None
    rates = [int(v) for v in args.rates.split(",")] if args.rates else None
    algo = {"auto": B.ALGO_AUTO, "pair": B.ALGO_UMMA_PAIR, "sub": B.ALGO_UMMA_SUB}[args.algo]
    rows = run(args.iters, groups, rates, algo)
    print(as_markdown(rows))
    if args.json:
        with open(args.json, "w") as f:
            json.dump(rows, f, indent=1)


if __name__ == "__main__":
    main()
