#!/usr/bin/env python
"""Benchmark of the RT3D conv3d hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

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
# DRAM bytes (read + write) of one launch of the timed kernel on this workload, from the ncu capture
# summarised in profiles/conv3d_umma_pair_cfg1.md (14.68 MB read + 0.01 MB written; the output stays in L2).
DRAM_TRAFFIC_PER_LAUNCH = 14.69e6
WORKLOAD = "cfg1: C3D conv3a-shaped layer, batch 8, 128->256, 8x28x28, 3x3x3 s1 p1, KGS 4x4 ~2.5x, bf16"


def make_workload():
    spec = synth.ConvSpec("conv3a", CFG["cin"], CFG["cout"], CFG["k"], CFG["stride"], CFG["pad"], True)
    L = synth.make_layer(spec, 1, 0, CFG["g_m"], CFG["g_n"], "bernoulli", CFG["density"])
    x = synth.make_input(1, (CFG["n"], CFG["t"], CFG["h"], CFG["w"], CFG["cin"]))
    return spec, L, x


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


def main():
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

    networks = None
    if not args.no_networks:
        networks = time_networks(torch, rt3d, nets, dev)
        networks["pruning_step"] = time_pruning_step(torch, rt3d, dev, peaks()["hbm_gbs"])

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
                     "frac": ach / pk["bf16_tflops"], "traffic": DRAM_TRAFFIC_PER_LAUNCH if algo == rt3d.ALGO_UMMA else None, "peak_source": pk["source"] + " (burst)",
                     "executed_tflops": 2.0 * dense_macs / (per_step_ms * 1e-3) / 1e12,
                     "alg_bytes_per_launch": alg_bytes},
    }
    if networks is not None:
        out["networks"] = networks
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
    main()
