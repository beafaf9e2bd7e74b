#!/usr/bin/env python
"""Benchmark of the RT3D conv3d hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]
    python bench.py layer --cin 64 --cout 144 --k 1 3 3 --x 8 16 56 56      (one layer or fused pair, see layer_main)
    python bench.py net --net r2plus1d --batch 8                             (one network forward pass, see net_main)
    python bench.py ncu-traffic --csv RAW.csv --kernel REGEX --out profiles/X.json   (DRAM bytes per launch from an ncu export)

Workload (config 1 of the baseline): one C3D-conv3a-shaped layer, batch 8, C_in=128,
C_out=256, T=8, H=W=28, 3x3x3, stride 1, pad 1, bf16 in / fp32 accumulate / bf16 out,
KGS-pruned with 4x4 kernel groups at about 2.5x FLOPs pruning, fused bias + ReLU.
A step is one rt3d_conv3d_sparse call on one batch.  Inputs are seeded synthetic tensors
(no dataset).  Each step uses the next of several input/output buffer sets whose total size
exceeds twice the L2 capacity, so no step finds its operands in L2 from the previous one.

The JSON line reports actual TFLOP/s (2 x kept multiply-accumulates / time); the same run
also times the library's dense path on the same shape (speedup vs dense, to be compared with
the FLOPs pruning rate as the paper does), an end-to-end variant through the host-buffer entry
point, the CPU oracle on the machine's host cores, and the roofline fraction of the kernel.
With torchrun and N > 1 every rank runs the same per-GPU workload on its own batch (weak
scaling, no collective on the data path); times are the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np

import rt3d_synth as synth

CFG = dict(n=8, t=8, h=28, w=28, cin=128, cout=256, k=(3, 3, 3), stride=(1, 1, 1), pad=(1, 1, 1),
           g_m=4, g_n=4, density=0.4)
L2_BYTES = 126 * 1024 * 1024
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "conv3d_umma_pair_cfg1.json")   # written by `bench.py ncu-traffic`
WORKLOAD = "cfg1: C3D conv3a-shaped layer, batch 8, 128->256, 8x28x28, 3x3x3 s1 p1, KGS 4x4 ~2.5x, bf16"


def make_workload():
    spec = synth.ConvSpec("conv3a", CFG["cin"], CFG["cout"], CFG["k"], CFG["stride"], CFG["pad"], True)
    L = synth.make_layer(spec, 1, 0, CFG["g_m"], CFG["g_n"], "bernoulli", CFG["density"])
    x = synth.make_input(1, (CFG["n"], CFG["t"], CFG["h"], CFG["w"], CFG["cin"]))
    return spec, L, x


def dram_traffic_per_launch():
    """DRAM bytes (read + write) of one launch of the timed kernel on this workload: the mean over the launches of
    one ncu capture, stored beside its summary under profiles/ by `bench.py ncu-traffic`.  None if absent."""
    try:
        rec = json.load(open(TRAFFIC_JSON))
        return float(rec["dram_bytes_read_per_launch"]) + float(rec["dram_bytes_write_per_launch"])
    except (OSError, KeyError, ValueError):
        return None


def ncu_traffic_main(argv=None) -> int:
    """`python bench.py ncu-traffic --csv RAW.csv --kernel REGEX --out profiles/X.json --command "..."`: reads the raw
    page of an ncu report exported as CSV (`ncu -i report.ncu-rep --page raw --csv > RAW.csv`) and stores the mean
    dram__bytes_read.sum / dram__bytes_write.sum per launch of the kernels matching REGEX."""
    import csv
    import re
    ap = argparse.ArgumentParser(prog="bench.py ncu-traffic")
    ap.add_argument("--csv", required=True)
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--out", required=True)
    ap.add_argument("--workload", default=WORKLOAD)
    ap.add_argument("--command", default="", help="the command that produced the report (kept for the record)")
    a = ap.parse_args(argv)
    rows = list(csv.reader(open(a.csv)))
    hdr, units = rows[0], rows[1]
    ik, ir, iw = hdr.index("Kernel Name"), hdr.index("dram__bytes_read.sum"), hdr.index("dram__bytes_write.sum")
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    sel = [r for r in rows[2:] if re.search(a.kernel, r[ik])]
    if not sel:
        raise SystemExit("no launch matches the kernel pattern")
    rd = sum(float(r[ir]) for r in sel) / len(sel) * scale[units[ir]]
    wr = sum(float(r[iw]) for r in sel) / len(sel) * scale[units[iw]]
    rec = {"kernel": sel[0][ik], "workload": a.workload, "launches": len(sel), "dram_bytes_read_per_launch": rd,
           "dram_bytes_write_per_launch": wr, "command": a.command}
    with open(a.out, "w") as f:
        json.dump(rec, f, indent=1)
        f.write("\n")
    print(json.dumps(rec))
    return 0


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.active = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            if self.active.is_set():
                try:
                    self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                    try:
                        r = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                    except Exception:
                        r = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                    for bit, name in self.REASONS.items():
                        if r & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
            time.sleep(0.0005)

    def stop(self):
        self._stop_evt.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_timed(spec, L, x, clips: int):
    """Times the CPU oracle, as it stands, on the first `clips` clips of the batch."""
    import oracle
    xs = np.ascontiguousarray(x[:clips])
    t0 = time.perf_counter()
    oracle.conv3d(xs, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    return time.perf_counter() - t0


def time_networks(torch, rt3d, nets, dev, iters=20):
    """Forward passes of the C3D-shaped (cfg2: batch 1 and 16, KGS ~3.6x and dense) and R(2+1)D-18-shaped
    (cfg3: batch 8, KGS ~2.5x) networks, each captured in a CUDA graph; clips per second."""
    out = {}

    def timed(fwd):
        for _ in range(3):
            fwd()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fwd()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    plan = synth.c3d_plan()
    specs = [(i, op) for i, op in enumerate(plan) if isinstance(op, synth.ConvSpec)]
    raw = {op.name: synth.make_layer(op, 2, i, 4, 4, "bernoulli", 1 / 3.6) for i, op in specs}
    for mode in ("kgs", "dense"):
        layers = {op.name: nets.ConvLayer(op, raw[op.name]["w"], raw[op.name]["bias"],
                                          None if mode == "dense" else raw[op.name]["mask"], 4, 4, torch.bfloat16,
                                          dense=(mode == "dense"), device=dev) for _, op in specs}
        net = nets.C3DNet(plan, layers, fuse_pool=True)
        for batch in (1, 16):
            x = nets.to_device(synth.make_input(2, (batch, 16, 112, 112, 3)), torch.bfloat16, device=dev)
            ms = timed(nets.GraphedForward(net, x))
            out[f"c3d_{mode}_b{batch}_clips_per_s"] = batch / ms * 1e3
            out[f"c3d_{mode}_b{batch}_ms"] = ms
        if mode == "kgs":
            kept = dense = 0
            t, h, w = 16, 112, 112
            for op in plan:
                if isinstance(op, synth.ConvSpec):
                    k, d, _ = layers[op.name].cost(torch.empty((1, t, h, w, nets.pitch_for(op.cin, torch.bfloat16)),
                                                               dtype=torch.bfloat16, device=dev))
                    kept += k; dense += d
                    t, h, w = op.out_extent(t, h, w)
                else:
                    t, h, w = [(dd + 2 * p - kk) // s + 1 for dd, p, kk, s in zip((t, h, w), op.pad, op.k, op.stride)]
            out["c3d_flops_pruning_rate"] = dense / kept
            out["c3d_dense_gmac_per_clip"] = dense / 1e9
        del net, layers
    out["c3d_b16_speedup_vs_dense"] = out["c3d_dense_b16_ms"] / out["c3d_kgs_b16_ms"]
    del raw

    stem, blocks = synth.r2plus1d18_plan()
    rspecs = list(stem)
    for blk in blocks:
        rspecs += list(blk.convs) + ([blk.shortcut] if blk.shortcut is not None else [])
    rlayers = {}
    for i, sp in enumerate(rspecs):
        L = synth.make_layer(sp, 3, i, 4, 4, "bernoulli", 0.4)
        rlayers[sp.name] = nets.ConvLayer(sp, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16, device=dev)
    rnet = nets.R2Plus1DNet(stem, blocks, rlayers, fuse_residual=True, fuse_pairs=True)
    x = nets.to_device(synth.make_input(3, (8, 16, 112, 112, 3)), torch.bfloat16, device=dev)
    ms = timed(nets.GraphedForward(rnet, x))
    out["r2plus1d_kgs_b8_clips_per_s"] = 8 / ms * 1e3
    out["r2plus1d_kgs_b8_ms"] = ms
    out["r2plus1d_launches"] = rnet.n_launches()
    del rnet, rlayers

    # S3D-shaped network (separable 3-D Inception, 16 x 224 x 224 clips, KGS about 2.1x), batch 8
    splan = synth.s3d_plan()
    slayers = {}
    for i, sp in enumerate(synth.s3d_convs(splan)):
        L = synth.make_layer(sp, 5, i, 4, 4, "bernoulli", 1 / 2.1)
        slayers[sp.name] = nets.ConvLayer(sp, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16, device=dev)
    snet = nets.S3DNet(splan, slayers)
    x = nets.to_device(synth.make_input(5, (8, 16, 224, 224, 3)), torch.bfloat16, device=dev)
    ms = timed(nets.GraphedForward(snet, x))
    out["s3d_kgs_b8_clips_per_s"] = 8 / ms * 1e3
    out["s3d_kgs_b8_ms"] = ms
    return out


def network_cost(torch, nets, convs_in_order, dev):
    """Sums rt3d_conv3d_cost over (layer, input extents) pairs: kept MACs, dense MACs, algorithmic bytes per clip."""
    kept = dense = nbytes = 0
    for layer, (t, h, w) in convs_in_order:
        k, d, b = layer.cost(torch.empty((1, t, h, w, nets.pitch_for(layer.spec.cin, torch.bfloat16)), dtype=torch.bfloat16, device=dev))
        kept += k; dense += d; nbytes += b
    return kept, dense, nbytes


def roofline_of(ms, batch, kept, dense, nbytes, pk):
    """Achieved-vs-bound figures of one forward pass: the bound is the slower of the kept FLOPs at the measured sustained
    bf16 rate and the algorithmic bytes (activations once per layer, weights once per pass) at the measured HBM rate."""
    t = ms * 1e-3
    sustained = pk["bf16_tflops_sustained"] or pk["bf16_tflops"]
    tensor_ms = 2.0 * kept * batch / (sustained * 1e12) * 1e3
    hbm_ms = nbytes * batch / (pk["hbm_gbs"] * 1e9) * 1e3
    bound_ms = max(tensor_ms, hbm_ms)
    return {"ms": ms, "kept_tflops": 2.0 * kept * batch / t / 1e12, "executed_tflops": 2.0 * dense * batch / t / 1e12,
            "kept_frac_of_sustained": 2.0 * kept * batch / t / 1e12 / sustained,
            "executed_frac_of_sustained": 2.0 * dense * batch / t / 1e12 / sustained,
            "alg_gbs": nbytes * batch / t / 1e9, "tensor_bound_ms": tensor_ms, "hbm_bound_ms": hbm_ms,
            "bound": "tensor" if tensor_ms >= hbm_ms else "hbm", "achieved": bound_ms / ms, "peak": 1.0, "frac": bound_ms / ms,
            "unit": "bound time / measured time", "peak_source": pk["source"] + " (sustained bf16, HBM copy)"}


def time_configs(torch, rt3d, nets, dev, pk, net_times):
    """Per-config figures beside the cfg1 headline: cfg0 (fp32 layer, launch-bound), cfg2 / cfg3 rooflines from the timed
    forward passes, and a subset of the cfg4 sweep with speedup over the dense path against the pruning rate."""
    out = {}

    def timed(fn, iters=50, warm=5):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3          # microseconds

    # cfg0: 16 -> 32 channels, 8x28x28, 3x3x3, fp32, 14 of 27 locations kept per 4x4 group: 0.09 GFLOP, launch-bound
    spec0 = synth.ConvSpec("cfg0", 16, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L0 = synth.make_layer(spec0, 0, 0, 4, 4, "exact_per_group", 14)
    lay0 = nets.ConvLayer(spec0, L0["w"], L0["bias"], L0["mask"], 4, 4, torch.float32, device=dev)
    x0 = nets.to_device(synth.make_input(0, (1, 8, 28, 28, 16)), torch.float32, device=dev)
    y0 = lay0.alloc_out(x0)
    def graphed_us(fn, calls=20):
        """Mean time of one call when `calls` of them are captured into one CUDA graph: the device-side launch
        interval, without the host-side cost of the binding."""
        fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(calls):
                fn()
        return timed(g.replay, iters=20, warm=3) / calls

    us0 = graphed_us(lambda: lay0(x0, y0))
    tiny = torch.zeros((1, 1, 1, 1, 4), dtype=torch.float32, device=dev)
    floor = graphed_us(lambda: nets.add_relu(tiny, tiny, 4, True, tiny))     # launch interval of a trivial kernel
    k0, d0, b0 = lay0.cost(x0)
    alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12                           # fp32 FFMA peak of the device, TFLOP/s
    out["cfg0"] = {"workload": "cfg0: 16->32, 8x28x28, 3x3x3, fp32, KGS 4x4 14/27 (20 calls per CUDA graph)", "us_per_call": us0,
                   "launch_floor_us": floor, "bound": "launch", "achieved": floor / us0, "peak": 1.0, "frac": floor / us0,
                   "unit": "launch interval of a trivial kernel / measured", "kept_gflops": 2.0 * k0 / us0 / 1e3,
                   "alu_frac": 2.0 * k0 / us0 / 1e6 / alu_peak, "alg_gbs": b0 / us0 / 1e3}
    del lay0

    # cfg2 / cfg3: cost of the networks per clip, with the forward times measured by time_networks
    plan = synth.c3d_plan()
    convs, (t, h, w) = [], (16, 112, 112)
    raw = {}
    for i, op in enumerate(plan):
        if isinstance(op, synth.ConvSpec):
            L = synth.make_layer(op, 2, i, 4, 4, "bernoulli", 1 / 3.6)
            convs.append((nets.ConvLayer(op, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16, device=dev), (t, h, w)))
            t, h, w = op.out_extent(t, h, w)
        else:
            t, h, w = [(dd + 2 * p - kk) // s + 1 for dd, p, kk, s in zip((t, h, w), op.pad, op.k, op.stride)]
    kept, dense, nbytes = network_cost(torch, nets, convs, dev)
    w_bytes = sum(int(l.packed.view()["nnz"]) * 16 * 2 for l, _ in convs)        # packed weights are read once per pass, not per clip
    for b in (1, 16):
        per_clip = nbytes - w_bytes + w_bytes / b
        out[f"cfg2_c3d_b{b}"] = roofline_of(net_times[f"c3d_kgs_b{b}_ms"], b, kept, dense, per_clip, pk)
        out[f"cfg2_c3d_b{b}"]["workload"] = f"cfg2: C3D-shaped forward, batch {b}, KGS 4x4 ~3.6x"
    del convs
    stem, blocks = synth.r2plus1d18_plan()
    seq, (t, h, w) = [], (16, 112, 112)
    idx = 0

    def add(sp, ext):
        nonlocal idx
        L = synth.make_layer(sp, 3, idx, 4, 4, "bernoulli", 0.4)
        idx += 1
        seq.append((nets.ConvLayer(sp, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16, device=dev), ext))
        return sp.out_extent(*ext)
    ext = (t, h, w)
    for sp in stem:
        ext = add(sp, ext)
    for blk in blocks:
        inp = ext
        for sp in blk.convs:
            ext = add(sp, ext)
        if blk.shortcut is not None:
            add(blk.shortcut, inp)
    kept, dense, nbytes = network_cost(torch, nets, seq, dev)
    w_bytes = sum(int(l.packed.view()["nnz"]) * 16 * 2 for l, _ in seq)
    out["cfg3_r2plus1d_b8"] = roofline_of(net_times["r2plus1d_kgs_b8_ms"], 8, kept, dense, nbytes - w_bytes + w_bytes / 8, pk)
    out["cfg3_r2plus1d_b8"]["workload"] = "cfg3: R(2+1)D-18-shaped forward, batch 8, KGS 4x4 ~2.5x (bytes: every layer's input and output once)"
    del seq

    # cfg4 subset: speedup over the dense path against the FLOPs pruning rate
    from paper_2007_09835_b200 import sweep
    rows = sweep.run(iters=20, groups=[(4, 4), (8, 8), (128, 64), (256, 64)], rates=[2, 4, 8], schemes=("kgs",))
    sustained = pk["bf16_tflops_sustained"] or pk["bf16_tflops"]
    out["cfg4"] = [{"scheme": r["scheme"], "group": f'{r["g_m"]}x{r["g_n"]}' if r["g_m"] else "-", "rate": r["rate"], "us": r["us"],
                    "speedup_vs_dense": r["speedup"], "speedup_over_rate": r["ratio"], "kept_tflops": r["tflops_actual"],
                    "frac": r["tflops_actual"] / sustained, "bound": "tensor", "peak": sustained, "achieved": r["tflops_actual"]}
                   for r in rows]
    return out


def time_pruning_step(torch, rt3d, dev, hbm_gbs, iters=20):
    """Device-side pruning step (group norms -> penalties + keep mask) on a weight tensor larger than L2:
    2048 x 1024 x 3x3x3 fp32 = 226 MB, 4x4 groups.  Bound: HBM (the weights are read once)."""
    M, N, k = 2048, 1024, (3, 3, 3)
    w = torch.randn((M, N) + k, device=dev, dtype=torch.float32) * 0.05
    P, Q, Ks = M // 4, N // 4, 27
    norms = torch.empty((P, Q, Ks), device=dev, dtype=torch.float32)
    pen = torch.empty_like(norms)
    keep = torch.empty((P, Q, Ks), device=dev, dtype=torch.uint8)

    def step():
        rt3d.rt3d_kgs_group_norms(w, 4, 4, 2, norms)
        rt3d.rt3d_kgs_reweight(norms, 1e-3, 0.2, pen, keep)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    nbytes = w.numel() * 4 + norms.numel() * (4 + 4 + 4 + 1)
    gbs = nbytes / ms / 1e6
    return {"ms": ms, "alg_bytes": nbytes, "achieved_gbs": gbs, "hbm_peak_gbs": hbm_gbs, "frac": gbs / hbm_gbs,
            "workload": "group norms + reweight, 2048x1024x3x3x3 fp32, 4x4 groups"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    spec, L, x = make_workload()
    clips = 1
    kept_macs = spec.dense_macs(clips, CFG["t"], CFG["h"], CFG["w"]) * float(L["mask"].mean())
    for _ in range(args.warmup):
        oracle_timed(spec, L, x, clips)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_timed(spec, L, x, clips)
    dt = time.perf_counter() - t0
    value = 2.0 * kept_macs * args.steps / dt / 1e12
    sample = f"{clips} of {CFG['n']} clips of the batch per step (masked dense weights, fp64 accumulation)"
    print(json.dumps({
        "impl": "reference", "metric": "sparse_conv3d_actual_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def layer_main(argv=None) -> int:
    """`python bench.py layer ...`: times one synthetic convolution layer (or a fused spatial->temporal pair) through the
    C ABI with CUDA events and prints one JSON line.  The layer is drawn by the seeded generators (KGS mask with
    independent keep probability --density per (group, location), 4x4 groups by default, or --dense); input values are
    uniform in (-1, 1).  `--iters 3 --warmup 3` keeps a profiler capture short."""
    import torch
    from paper_2007_09835_b200 import binding as B, nets
    ap = argparse.ArgumentParser(prog="bench.py layer")
    ap.add_argument("--cin", type=int, required=True)
    ap.add_argument("--cout", type=int, required=True)
    ap.add_argument("--k", type=int, nargs=3, default=(3, 3, 3), metavar=("KT", "KH", "KW"))
    ap.add_argument("--stride", type=int, nargs=3, default=(1, 1, 1))
    ap.add_argument("--pad", type=int, nargs=3, default=None, help="default: k // 2 per axis")
    ap.add_argument("--x", type=int, nargs=4, required=True, metavar=("N", "T", "H", "W"))
    ap.add_argument("--group", type=int, nargs=2, default=(4, 4), metavar=("G_M", "G_N"))
    ap.add_argument("--density", type=float, default=0.4)
    ap.add_argument("--dense", action="store_true")
    ap.add_argument("--algo", type=int, default=0, help="rt3d_algo value (0 = automatic)")
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



def build_network(net: str, dense: bool = False, pair_fusion: bool = True):
    """Returns (network object, clip shape (t, h, w, c)) of a network-shaped workload: synthetic KGS-pruned layers from the
    seeded generators (4x4 groups; keep probability 1/3.6, 0.4 and 1/2.1 as in the paper's Table 2 rates)."""
    import torch
    from paper_2007_09835_b200 import nets
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



def net_main(argv=None) -> int:
    """`python bench.py net --net c3d|c3d_fc|r2plus1d|s3d --batch B`: one forward pass of a network-shaped workload through
    the C ABI, one JSON line.  By default the pass is captured in a CUDA graph and replayed --iters times between CUDA
    events; --eager launches the kernels one by one (`--eager --iters 1 --warmup 2` gives a profiler one pass)."""
    import torch
    from paper_2007_09835_b200 import binding as B, nets
    ap = argparse.ArgumentParser(prog="bench.py net")
    ap.add_argument("--net", choices=["c3d", "c3d_fc", "r2plus1d", "s3d"], required=True)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--dense", action="store_true", help="unpruned weights through the dense path")
    ap.add_argument("--eager", action="store_true", help="no CUDA graph")
    ap.add_argument("--no-pair-fusion", action="store_true",
                    help="r2plus1d: run every factorised pair as two launches (default: one launch where the library fuses it)")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args(argv)

    net, clip = build_network(a.net, a.dense, not a.no_pair_fusion)
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




def main():
    if len(sys.argv) > 1 and sys.argv[1] == "layer":
        return layer_main(sys.argv[2:])
    if len(sys.argv) > 1 and sys.argv[1] == "net":
        return net_main(sys.argv[2:])
    if len(sys.argv) > 1 and sys.argv[1] == "ncu-traffic":
        return ncu_traffic_main(sys.argv[2:])
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--l2-warm", action="store_true", help="reuse one buffer set (operands stay in L2); default rotates sets")
    ap.add_argument("--no-networks", action="store_true", help="skip the C3D / R(2+1)D-shaped forward passes")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2007_09835_b200 as rt3d
    from paper_2007_09835_b200 import nets, dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    group = dist.init(world, rank, "nccl") if world > 1 else None
    dev = torch.device("cuda", local)

    spec, L, x = make_workload()
    sparse = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], CFG["g_m"], CFG["g_n"], torch.bfloat16, device=dev)
    dense = nets.ConvLayer(spec, L["w"], L["bias"], None, dtype=torch.bfloat16, dense=True, device=dev)
    x0 = nets.to_device(x, torch.bfloat16, device=dev)
    y0 = sparse.alloc_out(x0)
    set_bytes = x0.numel() * 2 + y0.numel() * 2
    n_sets = 1 if args.l2_warm else max(2, -(-int(2.5 * L2_BYTES) // set_bytes))
    xs = [x0] + [x0.clone() for _ in range(n_sets - 1)]
    ys = [y0] + [torch.zeros_like(y0) for _ in range(n_sets - 1)]
    kept_macs, dense_macs, alg_bytes = sparse.cost(x0)
    algo = rt3d.rt3d_conv3d_query_algo(rt3d.tensor_desc(x0, spec.cin), sparse.packed, rt3d.tensor_desc(y0, spec.cout),
                                       spec.stride, spec.pad)

    def timed(layer, steps, warmup, sampler=None):
        for i in range(warmup):
            layer(xs[i % n_sets], ys[i % n_sets])
        torch.cuda.synchronize()
        dist.barrier(group)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = rt3d.rt3d_launch_count()
        if sampler:
            sampler.active.set()
        e0.record()
        for i in range(steps):
            layer(xs[i % n_sets], ys[i % n_sets])
        e1.record()
        torch.cuda.synchronize()
        if sampler:
            sampler.active.clear()
        dist.barrier(group)
        ms = dist.max_over_ranks(e0.elapsed_time(e1), group, dev)
        return ms, rt3d.rt3d_launch_count() - l0

    sampler = ClockSampler(local)
    sampler.start()
    sparse_ms, launches = timed(sparse, args.steps, args.warmup, sampler)
    dense_ms, _ = timed(dense, args.steps, args.warmup, sampler)
    if rt3d.rt3d_last_device_status() != rt3d.OK:
        raise SystemExit("device reported a bounded-wait timeout")

    # end to end through the host-buffer entry point: pinned host input -> device -> conv -> pinned host output
    xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    yh = torch.zeros((CFG["n"], CFG["t"], CFG["h"], CFG["w"], CFG["cout"]), dtype=torch.bfloat16).pin_memory()
    bh = torch.from_numpy(L["bias"]).pin_memory()
    xhd, yhd = rt3d.tensor_desc(xh), rt3d.tensor_desc(yh)
    e2e_steps = max(3, min(args.steps, 50))
    for _ in range(3):
        rt3d.rt3d_conv3d_host(xhd, sparse.packed, bh, yhd, spec.stride, spec.pad, True)
    torch.cuda.synchronize()
    dist.barrier(group)
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        rt3d.rt3d_conv3d_host(xhd, sparse.packed, bh, yhd, spec.stride, spec.pad, True)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = dist.max_over_ranks(e0.elapsed_time(e1), group, dev) / e2e_steps
    sampler.stop()

    networks = configs = None
    if not args.no_networks:
        networks = time_networks(torch, rt3d, nets, dev)
        networks["pruning_step"] = time_pruning_step(torch, rt3d, dev, peaks()["hbm_gbs"])
        configs = time_configs(torch, rt3d, nets, dev, peaks(), networks) if world == 1 else None

    flops_kept = 2.0 * kept_macs
    per_step_ms = sparse_ms / args.steps
    value = world * flops_kept / (per_step_ms * 1e-3) / 1e12
    pk = peaks()
    ach = flops_kept / (per_step_ms * 1e-3) / 1e12
    out = {
        "metric": "sparse_conv3d_actual_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "global_batch": CFG["n"] * world, "parallelism": f"batch replicas x{world}",
                   "l2": ("warm: one buffer set reused every step" if args.l2_warm else
                          f"rotating {n_sets} input/output buffer sets ({n_sets * set_bytes / 2**20:.0f} MiB > 2x L2)"),
                   "kernel": "tcgen05" if algo == rt3d.ALGO_UMMA else "cuda-core"},
        "dense_equiv_tflops": world * 2.0 * dense_macs / (per_step_ms * 1e-3) / 1e12,
        "dense_path_tflops": world * 2.0 * dense_macs / (dense_ms / args.steps * 1e-3) / 1e12,
        "speedup_vs_dense": dense_ms / sparse_ms,
        "flops_pruning_rate": dense_macs / kept_macs,
        "dense_ms_per_step": dense_ms / args.steps,
        "clocks": sampler.summary(),
        "e2e": {"value": world * flops_kept / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                "ms_per_step": e2e_ms, "h2d_bytes_per_step": xh.numel() * 2 + bh.numel() * 4,
                "d2h_bytes_per_step": yh.numel() * 2},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": ach / pk["bf16_tflops"], "traffic": dram_traffic_per_launch() if algo == rt3d.ALGO_UMMA else None, "peak_source": pk["source"] + " (burst)",
                     "executed_tflops": 2.0 * dense_macs / (per_step_ms * 1e-3) / 1e12,
                     "alg_bytes_per_launch": alg_bytes},
    }
    if networks is not None:
        out["networks"] = networks
    if configs is not None:
        out["configs"] = configs
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        clips = CFG["n"]
        oracle_timed(spec, L, x, 1)                       # first call: builds / loads the oracle, warms the caches
        passes, total = 0, 0.0
        while total < 10.0 and passes < 32:               # about 10-15 s of CPU work
            total += oracle_timed(spec, L, x, clips)
            passes += 1
        dt = total / passes
        out["cpu_baseline"] = {"value": flops_kept / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(),
                               "kind": "oracle", "seconds": total,
                               "sample": f"all {clips} clips of one batch, mean of {passes} passes "
                                         f"(masked dense weights, fp64 accumulation)"}
    if rank == 0:
        print(json.dumps(out))
    dist.shutdown(group)


if __name__ == "__main__":
    raise SystemExit(main() or 0)
