"""Runs the forward pass of one of the network-shaped workloads through the C ABI and prints one JSON line.

    python -m paper_2007_09835_b200.net_bench --net r2plus1d --batch 8

--net c3d | c3d_fc (with the fully connected tail) | r2plus1d | s3d; synthetic clips and KGS-pruned layers from the seeded generators of rt3d_synth
(4x4 groups; keep probability 1/3.6, 0.4 and 1/2.1 as in the paper's Table 2 rates).  By default the pass is
captured in a CUDA graph and replayed `--iters` times between CUDA events; `--eager` launches the kernels one
by one instead (what a profiler should see: `--eager --iters 1 --warmup 2` gives one forward pass to capture).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import rt3d_synth as synth  # noqa: E402
from paper_2007_09835_b200 import binding as B  # noqa: E402
from paper_2007_09835_b200 import nets  # noqa: E402


def build(net: str, dense: bool = False, pair_fusion: bool = True):
    """Returns (network object, clip shape (t, h, w, c))."""
    def layer(sp, cfg, i, density):
        L = synth.make_layer(sp, cfg, i, 4, 4, "none" if dense else "bernoulli", None if dense else density)
        return nets.ConvLayer(sp, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16, dense=dense)

    if net in ("c3d", "c3d_fc"):
        plan = synth.c3d_plan()
        layers = {op.name: layer(op, 2, i, 1 / 3.6) for i, op in enumerate(plan) if isinstance(op, synth.ConvSpec)}
        fc = None
        if net == "c3d_fc":                     # with the three (unpruned) fully connected layers after pool5
            fc = []
            for i, sp in enumerate(synth.c3d_fc_tail()):
                L = synth.make_layer(sp, 2, 100 + i, 4, 4, "none", None)
                fc.append(nets.ConvLayer(sp, L["w"], L["bias"], None, 4, 4, torch.bfloat16, dense=True))
        return nets.C3DNet(plan, layers, fuse_pool=True, fc_layers=fc), (16, 112, 112, 3)
    if net == "r2plus1d":
        stem, blocks = synth.r2plus1d18_plan()
        specs = list(stem)
        for blk in blocks:
            specs += list(blk.convs) + ([blk.shortcut] if blk.shortcut is not None else [])
        layers = {sp.name: layer(sp, 3, i, 0.4) for i, sp in enumerate(specs)}
        return nets.R2Plus1DNet(stem, blocks, layers, fuse_residual=True, fuse_pairs=pair_fusion), (16, 112, 112, 3)
    if net == "s3d":
        plan = synth.s3d_plan()
        layers = {sp.name: layer(sp, 5, i, 1 / 2.1) for i, sp in enumerate(synth.s3d_convs(plan))}
        return nets.S3DNet(plan, layers), (16, 224, 224, 3)
    raise ValueError(net)


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--net", choices=["c3d", "c3d_fc", "r2plus1d", "s3d"], required=True)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--dense", action="store_true", help="unpruned weights through the dense path")
    ap.add_argument("--eager", action="store_true", help="no CUDA graph")
    ap.add_argument("--no-pair-fusion", action="store_true",
                    help="r2plus1d: run every factorised pair as two launches (default: one launch where the library fuses it)")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args(argv)

    net, clip = build(a.net, a.dense, not a.no_pair_fusion)
    x = nets.to_device(synth.make_input(7, (a.batch,) + clip))
    fwd = (lambda: net.forward(x)) if a.eager else nets.GraphedForward(net, x)
    for _ in range(a.warmup):
        fwd()
    torch.cuda.synchronize()
    launches0 = B.rt3d_launch_count()
    if a.eager:
        net.forward(x)
        launches = B.rt3d_launch_count() - launches0
    else:
        launches = None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        fwd()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    print(json.dumps({"net": a.net, "batch": a.batch, "dense": a.dense, "graph": not a.eager, "ms_per_forward": ms,
                      "clips_per_s": a.batch / ms * 1e3, "conv_launches_per_forward": launches,
                      "status": B.rt3d_last_device_status()}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
