"""Times one synthetic convolution layer through the C ABI (CUDA events) and prints one JSON line.

    python -m paper_2007_09835_b200.layer_bench --cin 64 --cout 144 --k 1 3 3 --x 8 16 56 56

The layer is drawn by the seeded generators of rt3d_synth (KGS mask with independent keep probability
`--density` per (group, location), 4x4 groups by default, or `--dense`); input values are uniform in
(-1, 1).  Useful for profiling a single kernel: `--iters 3 --warmup 3` keeps an ncu capture short.
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


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--cin", type=int, required=True)
    ap.add_argument("--cout", type=int, required=True)
    ap.add_argument("--k", type=int, nargs=3, default=(3, 3, 3), metavar=("KT", "KH", "KW"))
    ap.add_argument("--stride", type=int, nargs=3, default=(1, 1, 1))
    ap.add_argument("--pad", type=int, nargs=3, default=None, help="default: k // 2 per axis")
    ap.add_argument("--x", type=int, nargs=4, required=True, metavar=("N", "T", "H", "W"))
    ap.add_argument("--group", type=int, nargs=2, default=(4, 4), metavar=("G_M", "G_N"))
    ap.add_argument("--density", type=float, default=0.4)
    ap.add_argument("--dense", action="store_true")
    ap.add_argument("--algo", type=int, default=B.ALGO_AUTO)
    ap.add_argument("--pool", type=int, nargs=3, default=(1, 1, 1), help="fused max-pool window")
    ap.add_argument("--temporal-cout", type=int, default=0,
                    help="follow the (1 x Kh x Kw) layer by a 3x1x1 conv to this many channels, fused into ONE launch "
                         "(rt3d_conv2plus1d_fused); --separate runs the same pair as two launches")
    ap.add_argument("--separate", action="store_true")
    ap.add_argument("--residual", action="store_true", help="with --temporal-cout: add a residual tensor before the final ReLU")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args(argv)

    pad = tuple(k // 2 for k in a.k) if a.pad is None else tuple(a.pad)
    spec = synth.ConvSpec("layer", a.cin, a.cout, tuple(a.k), tuple(a.stride), pad, True)
    L = synth.make_layer(spec, 3, 1, a.group[0], a.group[1], "none" if a.dense else "bernoulli", None if a.dense else a.density)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], a.group[0], a.group[1], torch.bfloat16, dense=a.dense)
    n, t, h, w = a.x
    x = (torch.rand((n, t, h, w, nets.pitch_for(a.cin, torch.bfloat16)), device="cuda") - 0.5).to(torch.bfloat16)
    x[..., a.cin:] = 0
    pooled = tuple(a.pool) != (1, 1, 1)
    lay_t = None
    if a.temporal_cout:
        spec_t = synth.ConvSpec("temporal", a.cout, a.temporal_cout, (3, 1, 1), (1, 1, 1), (1, 0, 0), True)
        Lt = synth.make_layer(spec_t, 3, 2, a.group[0], a.group[1], "none" if a.dense else "bernoulli", None if a.dense else a.density)
        lay_t = nets.ConvLayer(spec_t, Lt["w"], Lt["bias"], Lt["mask"], a.group[0], a.group[1], torch.bfloat16, dense=a.dense)
        y = torch.zeros((n, t, h, w, nets.pitch_for(a.temporal_cout, torch.bfloat16)), dtype=torch.bfloat16, device="cuda")
        res = (torch.rand_like(y, dtype=torch.float32) - 0.5).to(torch.bfloat16) if a.residual else None
        if a.separate:
            mid = lay.alloc_out(x)

            def run():
                lay(x, mid, x_pad_zero=True)
                lay_t.fused(mid, y, residual=res)
        else:
            xd, yd = B.tensor_desc(x, a.cin), B.tensor_desc(y, a.temporal_cout)
            rd = None if res is None else B.tensor_desc(res, a.temporal_cout)

            def run():
                B.rt3d_conv2plus1d_fused(xd, lay.packed, lay.bias, pad, True, lay_t.packed, lay_t.bias, (1, 0, 0), True, yd,
                                         residual=rd)
    elif pooled:
        to, ho, wo = spec.out_extent(t, h, w)
        y = torch.zeros((n, to // a.pool[0], ho // a.pool[1], wo // a.pool[2], nets.pitch_for(a.cout, torch.bfloat16)),
                        dtype=torch.bfloat16, device="cuda")
        run = lambda: lay.fused(x, y, pool=tuple(a.pool), algo=a.algo, x_pad_zero=True)  # noqa: E731
    else:
        y = lay.alloc_out(x)
        run = lambda: lay(x, y, algo=a.algo, x_pad_zero=True)  # noqa: E731
    for _ in range(a.warmup):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / a.iters * 1e3
    kept, dense_macs, alg_bytes = lay.cost(x)
    if lay_t is not None:                # the pair: MACs of both layers; bytes = input + output (+ residual) + both weight sets
        k2, d2, b2 = lay_t.cost(lay.alloc_out(x))
        mid_bytes = n * t * h * w * a.cout * 2
        kept, dense_macs = kept + k2, dense_macs + d2
        alg_bytes = alg_bytes + b2 - 2 * mid_bytes + (n * t * h * w * a.temporal_cout * 2 if a.residual else 0)
    print(json.dumps({"us_per_call": us, "plan": B.rt3d_last_plan(), "kept_gmac": kept / 1e9, "dense_gmac": dense_macs / 1e9,
                      "executed_tflops": 2 * dense_macs / us / 1e6, "algorithmic_tflops": 2 * kept / us / 1e6,
                      "algorithmic_gbs": alg_bytes / us / 1e3, "status": B.rt3d_last_device_status()}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
