"""Planning mode (rt3d_plan_begin / rt3d_plan_end) and the bounded-wait error path.

Planning: one pass over a network's calls in planning mode must leave nothing to allocate or upload for the real
passes that follow: the library's allocation counter stands still across C3D-shaped forward passes at batch 1 and
batch 16 (kernel choice, K splits, tail split and fused pools included), and the results are those of an unplanned
run.

Bounded waits: every wait inside the kernels gives up after a limit, records an error word and lets the kernel
finish.  The test shortens the limit of the single-CTA kernel to about a millisecond and makes its producer skip
the loads of the last pipeline stage (a load that never comes: nothing faults, nothing spins for ever); the kernel
must return by itself, rt3d_last_device_status must report the timeout once, and the next ordinary call must be
correct again.
"""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

import netref

pytestmark = pytest.mark.gpu


def test_no_allocation_after_planning():
    plan, layers = netref.make_c3d_layers(2, 1 / 3.6)
    specs = [op for op in plan if isinstance(op, synth.ConvSpec)]
    dl = {sp.name: nets.ConvLayer(sp, layers[sp.name]["w"], layers[sp.name]["bias"], layers[sp.name]["mask"], 4, 4,
                                  torch.bfloat16) for sp in specs}
    net = nets.C3DNet(plan, dl, fuse_pool=True)
    x16 = nets.to_device(oracle.bf16_round(synth.make_input(2, (16, 16, 112, 112, 3))))
    x1 = x16[:1].contiguous()
    launches = rt3d.rt3d_launch_count()
    with rt3d.planning():                       # the larger batch first: workspaces only ever grow
        net.forward(x16)
        net.forward(x1)
    assert rt3d.rt3d_launch_count() == launches          # planning launches nothing
    torch.cuda.synchronize()
    allocs = rt3d.rt3d_alloc_count()
    plans16, plans1 = {}, {}
    y16 = net.forward(x16, plan_log=plans16).clone()
    y1 = net.forward(x1, plan_log=plans1).clone()
    torch.cuda.synchronize()
    assert rt3d.rt3d_alloc_count() == allocs, "a compute call allocated after planning"
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert any(p["n_splits"] > 1 for p in plans1.values())            # batch 1 splits K (needs scratch)
    assert any(p["tail_workers"] > 0 for p in plans16.values())       # batch 16 uses the tail split (needs scratch)
    # same bits as an unplanned network built from the same weights
    dl2 = {sp.name: nets.ConvLayer(sp, layers[sp.name]["w"], layers[sp.name]["bias"], layers[sp.name]["mask"], 4, 4,
                                   torch.bfloat16) for sp in specs}
    net2 = nets.C3DNet(plan, dl2, fuse_pool=True)
    assert torch.equal(net2.forward(x16), y16)
    assert torch.equal(net2.forward(x1), y1)


def test_no_allocation_after_planning_other_networks():
    """The same for the R(2+1)D-shaped network with its fused pairs and side-stream projections, and for the
    S3D-shaped network with its parallel branches writing into channel slices."""
    def dev(layers, specs):
        return {sp.name: nets.ConvLayer(sp, layers[sp.name]["w"], layers[sp.name]["bias"], layers[sp.name]["mask"], 4, 4,
                                        torch.bfloat16) for sp in specs}
    stem, blocks, layers = netref.make_r2plus1d_layers(3, 0.4)
    specs = list(stem)
    for blk in blocks:
        specs += list(blk.convs) + ([blk.shortcut] if blk.shortcut is not None else [])
    plan_s, layers_s = netref.make_s3d_layers(5, 1 / 2.1)
    specs_s = synth.s3d_convs(plan_s)
    cases = [
        (lambda: nets.R2Plus1DNet(stem, blocks, dev(layers, specs), fuse_residual=True, fuse_pairs=True),
         oracle.bf16_round(synth.make_input(3, (4, 16, 112, 112, 3)))),
        (lambda: nets.S3DNet(plan_s, dev(layers_s, specs_s)), oracle.bf16_round(synth.make_input(5, (2, 16, 224, 224, 3)))),
    ]
    for make, x in cases:
        net = make()
        xd = nets.to_device(x)
        with rt3d.planning():
            net.forward(xd)
        torch.cuda.synchronize()
        allocs = rt3d.rt3d_alloc_count()
        y = net.forward(xd).clone()
        torch.cuda.synchronize()
        assert rt3d.rt3d_alloc_count() == allocs, "a compute call allocated after planning"
        assert rt3d.rt3d_last_device_status() == rt3d.OK
        assert torch.equal(make().forward(xd), y)                 # same bits as an unplanned network


def test_bounded_wait_times_out_and_the_library_recovers():
    spec = synth.ConvSpec("to", 64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 9, 4, 4, 4, "bernoulli", 0.5)
    x = synth.make_input(31, (1, 2, 8, 8, 64))                          # 128 voxels: one tile, one CTA
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(x)
    y = nets.to_numpy(lay(xd, algo=rt3d.ALGO_UMMA), 64)
    assert rt3d.rt3d_last_plan()["kernel"] == 1 and rt3d.rt3d_last_device_status() == rt3d.OK
    assert float(np.abs(y - ref).max() / np.abs(ref).max()) <= 2e-2
    try:
        rt3d.rt3d_debug_set(rt3d.DEBUG_WAIT_CYCLES, 2_000_000)           # about one millisecond of SM clocks
        rt3d.rt3d_debug_set(rt3d.DEBUG_DROP_LAST_LOAD, 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lay(xd, algo=rt3d.ALGO_UMMA)
        e1.record()
        torch.cuda.synchronize()                                         # the kernel returns by itself
        assert e0.elapsed_time(e1) < 500.0                               # milliseconds: well under the default limit
        assert rt3d.rt3d_last_device_status() == rt3d.ERR_TIMEOUT
        assert rt3d.rt3d_last_device_status() == rt3d.OK                 # reported once, then cleared
    finally:
        rt3d.rt3d_debug_set(rt3d.DEBUG_DROP_LAST_LOAD, 0)
        rt3d.rt3d_debug_set(rt3d.DEBUG_WAIT_CYCLES, 0)
    y = nets.to_numpy(lay(xd, algo=rt3d.ALGO_UMMA), 64)                  # the context and the handle are fine
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert float(np.abs(y - ref).max() / np.abs(ref).max()) <= 2e-2
    # a K-split call after the timeout: its arrival counters were cleared with the error word
    spec5 = synth.ConvSpec("to5", 512, 512, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L5 = synth.make_layer(spec5, 9, 5, 4, 4, "bernoulli", 0.3)
    x5 = synth.make_input(32, (1, 2, 7, 7, 512))
    lay5 = nets.ConvLayer(spec5, L5["w"], L5["bias"], L5["mask"], 4, 4, torch.bfloat16)
    y5 = nets.to_numpy(lay5(nets.to_device(x5)), 512)
    assert rt3d.rt3d_last_plan()["n_splits"] > 1
    ref5 = oracle.conv3d(x5, L5["w"], L5["mask"], L5["bias"], spec5.stride, spec5.pad, True, round_bf16=True)
    assert float(np.abs(y5 - ref5).max() / np.abs(ref5).max()) <= 2e-2
