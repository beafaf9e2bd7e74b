"""GPU parity on the network-shaped workloads (C3D-shaped, R(2+1)D-18-shaped) and the sparsity sweep.

Per layer the CUDA library receives exactly the input the oracle consumed (teacher forcing),
so every conv output is held to max|err| <= 2e-2 * max|ref| and every pool / add output must be
bit-identical.  The free-running forward pass (the library feeding itself) is compared at the
network output with the same norm and the same 2e-2: the two data flows round each layer's output to
bf16 independently, so a one-ulp rounding difference (2^-8 relative) of an activation perturbs the
next layer's input, but the measured errors (4e-3 to 1e-2, recorded by record_error) stay well inside.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

import netref

pytestmark = pytest.mark.gpu
TOL = 2e-2
TOL_FREE = 2e-2


def rel_err(y, ref):
    assert np.isfinite(y).all()
    return float(np.abs(y - ref).max() / np.abs(ref).max())


def record_error(name, err, tol):
    """Keeps the measured error of a free-running forward pass on record (one line per case appended to
    parity_errors.txt in the folder RT3D_PARITY_LOG_DIR names, if it is set and exists): the distance from the
    2e-2 single-layer tolerance is otherwise invisible behind a passing assertion."""
    folder = os.environ.get("RT3D_PARITY_LOG_DIR", "")
    if folder and os.path.isdir(folder):
        with open(os.path.join(folder, "parity_errors.txt"), "a") as f:
            f.write(f"{name}: max|err|/max|ref| = {err:.4e} (asserted <= {tol:g})\n")


def device_layers(layers, specs, dense=False):
    return {sp.name: nets.ConvLayer(sp, layers[sp.name]["w"], layers[sp.name]["bias"], layers[sp.name]["mask"],
                                    4, 4, torch.bfloat16, dense=dense) for sp in specs}


# ------------------------------------------------------------------------------- C3D-shaped
@pytest.fixture(scope="module")
def c3d():
    plan, layers = netref.make_c3d_layers(2, 1 / 3.6)
    specs = [op for op in plan if isinstance(op, synth.ConvSpec)]
    x2 = oracle.bf16_round(synth.make_input(2, (2, 16, 112, 112, 3)))     # stands for clips 0 and 15 of a batch
    rec, final = netref.c3d_reference(plan, layers, x2)
    return plan, layers, specs, x2, rec, final


def test_c3d_layers_teacher_forced(c3d):
    plan, layers, specs, x2, rec, final = c3d
    dl = device_layers(layers, specs)
    dense_macs = kept_macs = 0
    for op in plan:
        inp, ref = rec[op.name]
        c_in = inp.shape[-1]
        xd = nets.to_device(inp[:1])
        if isinstance(op, synth.ConvSpec):
            y = nets.to_numpy(dl[op.name](xd), op.cout)
            assert (ref[:1] != 0).mean() > 0.10, op.name
            e = rel_err(y, ref[:1])
            assert e <= TOL, (op.name, e)
            k, d, _ = dl[op.name].cost(xd)
            kept_macs += k; dense_macs += d
        else:
            y = nets.to_numpy(nets.maxpool(xd, c_in, op), c_in)
            np.testing.assert_array_equal(y, ref[:1])
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert abs(dense_macs / 1e9 - 38.497) < 0.01                 # dense conv work of the C3D-shaped stack per clip
    assert 3.2 < dense_macs / kept_macs < 4.0                    # about 3.6x FLOPs pruning overall


@pytest.mark.parametrize("batch,fuse", [(1, False), (16, False), (1, True), (16, True), (5, True)])
def test_c3d_free_running_forward(c3d, batch, fuse):
    plan, layers, specs, x2, rec, final = c3d
    dl = device_layers(layers, specs)
    net = nets.C3DNet(plan, dl, fuse_pool=fuse)
    if batch == 1:
        x = x2[:1]
        pick = [0]
    else:                                                        # the first and the last clip are the oracle's two
        filler = oracle.bf16_round(synth.make_input(22, (batch - 2, 16, 112, 112, 3)))
        x = np.concatenate([x2[:1], filler, x2[1:]], axis=0)
        pick = [0, batch - 1]
    y = nets.to_numpy(net.forward(nets.to_device(x)), 512)
    assert y.shape == (batch, 1, 4, 4, 512)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    ref = final[: len(pick)]
    assert (ref != 0).mean() > 0.10
    e = rel_err(y[pick], ref)
    record_error(f"C3D-shaped free-running forward, batch {batch}, fused pools {fuse}", e, TOL_FREE)
    assert e <= TOL_FREE, e
    if fuse:
        assert any(net.fused_ok.values())                        # at least conv1/conv2 really ran fused


def test_c3d_layers_teacher_forced_at_the_batch16_plan(c3d):
    """The eight conv layers once more, each called exactly as the batch-16 forward pass calls it (same shapes, fused
    pools where that forward fuses them), so that the kernel plans a large batch selects (CTA-pair kernel, tail
    split, pooling epilogue) are checked per layer against the oracle and not only at the network output.  The
    batch is made of the oracle's two clips in an irregular order: clips are independent, so EVERY clip of the
    batch has a full reference (a superset of sampling outputs on the clips between the first and the last)."""
    plan, layers, specs, x2, rec, final = c3d
    dl = device_layers(layers, specs)
    net = nets.C3DNet(plan, dl, fuse_pool=True)
    order = [0, 1, 1, 0, 1, 0, 0, 1, 0, 0, 1, 1, 1, 0, 0, 1]
    x16 = x2[order]
    plans_fwd = {}
    net.forward(nets.to_device(x16), plan_log=plans_fwd)          # what the real forward pass runs per layer
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert plans_fwd["conv3a"]["kernel"] in (2, 7) and plans_fwd["conv1"]["kernel"] == 3
    assert plans_fwd["conv1"]["fused_pool"] == 1 and plans_fwd["conv2"]["fused_pool"] == 1
    assert any(p["tail_workers"] > 0 for p in plans_fwd.values())  # the batch-16 pass does use the tail split
    for i, op in enumerate(plan):
        if not isinstance(op, synth.ConvSpec):
            continue
        inp, ref = rec[op.name]
        xd = nets.to_device(inp[order])
        nxt = plan[i + 1] if i + 1 < len(plan) else None
        fused = plans_fwd[op.name]["fused_pool"] == 1
        if fused:
            y = net._try_fused(op, nxt, xd, rt3d.ALGO_AUTO, None, i == 0)
            assert y is not None
            expect = rec[nxt.name][1]                             # the oracle's pooled tensor
        else:
            y = dl[op.name](xd, x_pad_zero=(i == 0))
            expect = ref
        assert rt3d.rt3d_last_plan() == plans_fwd[op.name], (op.name, rt3d.rt3d_last_plan(), plans_fwd[op.name])
        got = nets.to_numpy(y, op.cout)
        e = rel_err(got, expect[order])
        assert e <= TOL, (op.name, e)
    assert rt3d.rt3d_last_device_status() == rt3d.OK


def test_c3d_fc_tail(c3d):
    """fc6-fc8 as dense 1x1x1 convolutions over the flattened pool5 block: teacher-forced per layer, then the
    whole stack (convs + pools + FC) free-running against the oracle's logits."""
    plan, layers, specs, x2, rec, final = c3d
    fc = netref.make_c3d_fc_layers(2)
    fc_rec, logits = netref.c3d_fc_reference(fc, final)
    fc_specs = synth.c3d_fc_tail()
    fc_dl = [nets.ConvLayer(sp, fc[sp.name]["w"], fc[sp.name]["bias"], None, 4, 4, torch.bfloat16, dense=True) for sp in fc_specs]
    for sp, lay in zip(fc_specs, fc_dl):
        inp, ref = fc_rec[sp.name]
        y = nets.to_numpy(lay(nets.to_device(inp)), sp.cout)
        assert rel_err(y, ref) <= TOL, sp.name
    net = nets.C3DNet(plan, device_layers(layers, specs), fuse_pool=True, fc_layers=fc_dl)
    y = nets.to_numpy(net.forward(nets.to_device(x2)), 101)
    assert y.shape == (2, 1, 1, 1, 101)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    e = rel_err(y, logits)
    record_error("C3D-shaped + FC tail, free-running, 2 clips", e, TOL_FREE)
    assert e <= TOL_FREE


def test_c3d_dense_path_forward():
    plan, layers = netref.make_c3d_layers(2, 1.0, dense=True)
    specs = [op for op in plan if isinstance(op, synth.ConvSpec)]
    x = oracle.bf16_round(synth.make_input(2, (1, 16, 112, 112, 3)))
    rec, final = netref.c3d_reference(plan, layers, x)
    net = nets.C3DNet(plan, device_layers(layers, specs, dense=True))
    keep = {}
    y = nets.to_numpy(net.forward(nets.to_device(x), keep=keep), 512)
    e1 = rel_err(nets.to_numpy(keep["conv1"], 64), rec["conv1"][1])
    assert e1 <= TOL, e1
    assert rel_err(y, final) <= TOL_FREE


# -------------------------------------------------------------------------- R(2+1)D-shaped
@pytest.fixture(scope="module")
def r21d():
    stem, blocks, layers = netref.make_r2plus1d_layers(3, 0.4)
    x2 = oracle.bf16_round(synth.make_input(3, (2, 16, 112, 112, 3)))     # stands for clips 0 and 7 of a batch of 8
    rec, final = netref.r2plus1d_reference(stem, blocks, layers, x2)
    specs = list(stem)
    for blk in blocks:
        specs += list(blk.convs) + ([blk.shortcut] if blk.shortcut is not None else [])
    return stem, blocks, layers, specs, x2, rec, final


def test_r2plus1d_layers_teacher_forced(r21d):
    stem, blocks, layers, specs, x2, rec, final = r21d
    dl = device_layers(layers, specs)
    dense_macs = kept_macs = 0
    for sp in specs:
        inp, ref = rec[sp.name]
        xd = nets.to_device(inp)
        y = nets.to_numpy(dl[sp.name](xd), sp.cout)
        e = rel_err(y, ref)
        assert e <= TOL, (sp.name, e)
        k, d, _ = dl[sp.name].cost(xd)
        kept_macs += k; dense_macs += d
    for blk in blocks:
        (a, b), ref = rec[blk.name + ".out"]
        c = a.shape[-1]
        y = nets.to_numpy(nets.add_relu(nets.to_device(a), nets.to_device(b), c, True), c)
        np.testing.assert_array_equal(y, oracle.bf16_round(ref))
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert abs(dense_macs / 2 / 1e9 - 40.519) < 0.01             # dense conv work per clip
    assert 2.2 < dense_macs / kept_macs < 2.8                    # about 2.5x


@pytest.mark.parametrize("batch,fuse", [(8, False), (8, True), (8, "pairs"), (3, "pairs")])
def test_r2plus1d_free_running(r21d, batch, fuse):
    stem, blocks, layers, specs, x2, rec, final = r21d
    net = nets.R2Plus1DNet(stem, blocks, device_layers(layers, specs), fuse_residual=bool(fuse), fuse_pairs=fuse == "pairs")
    filler = oracle.bf16_round(synth.make_input(33, (batch - 2, 16, 112, 112, 3)))
    x = np.concatenate([x2[:1], filler, x2[1:]], axis=0)
    y = nets.to_numpy(net.forward(nets.to_device(x)), 512)
    assert y.shape == (batch, 2, 7, 7, 512)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert (final != 0).mean() > 0.10
    e = rel_err(y[[0, batch - 1]], final)
    record_error(f"R(2+1)D-shaped free-running forward, batch {batch}, fusion {fuse}", e, TOL_FREE)
    assert e <= TOL_FREE, e
    if fuse == "pairs":       # the two stage-2 blocks run their four factorised pairs as one launch each
        assert net.pairs_fused == {"s2b1.c1.s", "s2b1.c2.s", "s2b2.c1.s", "s2b2.c2.s"}, (net.pairs_fused, net.pairs_declined)
        launches = rt3d.rt3d_launch_count()
        net.forward(nets.to_device(x))
        assert rt3d.rt3d_launch_count() - launches == net.n_launches()


# ------------------------------------------------------------------------------ S3D-shaped
@pytest.fixture(scope="module")
def s3d():
    plan, layers = netref.make_s3d_layers(5, 1 / 2.1)
    x = oracle.bf16_round(synth.make_input(5, (1, 16, 224, 224, 3)))
    rec, final = netref.s3d_reference(plan, layers, x)
    return plan, layers, x, rec, final


def test_s3d_layers_teacher_forced(s3d):
    plan, layers, x, rec, final = s3d
    specs = synth.s3d_convs(plan)
    dl = device_layers(layers, specs)
    dense_macs = kept_macs = 0
    for sp in specs:
        inp, ref = rec[sp.name]
        xd = nets.to_device(inp)
        y = nets.to_numpy(dl[sp.name](xd), sp.cout)
        assert (ref != 0).mean() > 0.10, sp.name
        e = rel_err(y, ref)
        assert e <= TOL, (sp.name, e)
        k, d, _ = dl[sp.name].cost(xd)
        kept_macs += k; dense_macs += d
    for op in plan:
        pools = [op] if isinstance(op, synth.PoolSpec) else ([op.pool] if isinstance(op, synth.InceptionSpec) else [])
        for ps in pools:
            inp, ref = rec[ps.name]
            c = inp.shape[-1]
            y = nets.to_numpy(nets.maxpool(nets.to_device(inp), c, ps), c)
            np.testing.assert_array_equal(y, ref)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert abs(dense_macs / 1e9 - 17.978) < 0.01                 # dense conv work of the S3D-shaped stack per clip
    assert 1.9 < dense_macs / kept_macs < 2.3                    # about 2.1x FLOPs pruning (Table 2)


def test_s3d_free_running_forward(s3d):
    plan, layers, x, rec, final = s3d
    net = nets.S3DNet(plan, device_layers(layers, synth.s3d_convs(plan)))
    keep = {}
    y = nets.to_numpy(net.forward(nets.to_device(x), keep=keep), 1024)
    assert y.shape == (1, 2, 7, 7, 1024)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    # the first Inception block: every branch landed in its channel slice
    blk = nets.to_numpy(keep["mixed3b"], 256)
    assert rel_err(blk, rec["mixed3b"][1]) <= TOL_FREE
    assert (final != 0).mean() > 0.10
    e = rel_err(y, final)
    record_error("S3D-shaped free-running forward, batch 1", e, TOL_FREE)
    assert e <= TOL_FREE


# --------------------------------------------------------------------------- sparsity sweep
SWEEP_SPEC = synth.ConvSpec("sweep", 256, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)


def sweep_variants():
    out = [("dense", 4, 4, 1)]
    for g_m, g_n in ((4, 4), (8, 4), (8, 8)):
        for rate in (1, 2, 3, 4, 6, 8):
            out.append(("kgs", g_m, g_n, rate))
            if rate > 1:
                out.append(("vanilla", g_m, g_n, rate))
    return out


@pytest.fixture(scope="module")
def sweep_input():
    x = oracle.bf16_round(synth.make_input(4, (32, 8, 14, 14, 256)))
    return x, nets.to_device(x)


@pytest.mark.parametrize("scheme,g_m,g_n,rate", sweep_variants())
def test_sparsity_sweep_clips_0_and_31(sweep_input, scheme, g_m, g_n, rate):
    x, xd = sweep_input
    sp = SWEEP_SPEC
    P, Q = synth.n_groups(256, 256, g_m, g_n)
    layer_id = g_m * 100 + g_n * 10 + rate
    if scheme == "dense":
        L = synth.make_layer(sp, 4, layer_id, g_m, g_n, "none", None)
    elif scheme == "kgs":
        L = synth.make_layer(sp, 4, layer_id, g_m, g_n, "exact_total", round(P * Q * 27 / rate))
    else:
        L = synth.make_layer(sp, 4, layer_id, g_m, g_n, "vanilla_total", round(P * Q / rate))
    lay = nets.ConvLayer(sp, L["w"], L["bias"], L["mask"], g_m, g_n, torch.bfloat16, dense=(scheme == "dense"))
    y = nets.to_numpy(lay(xd), 256)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    ref = oracle.conv3d(x[[0, 31]], L["w"], L["mask"], L["bias"], sp.stride, sp.pad, True, round_bf16=True)
    assert (ref != 0).mean() > 0.10
    e = rel_err(y[[0, 31]], ref)
    assert e <= TOL, e
    kept, dense_macs, _ = lay.cost(xd)
    assert abs(dense_macs / kept - rate) < 0.01 * rate


@pytest.mark.parametrize("g_m,g_n", [(4, 4), (8, 4), (8, 8)])
def test_sparsity_sweep_full_batch_one_variant_per_group_size(sweep_input, g_m, g_n):
    x, xd = sweep_input
    sp = SWEEP_SPEC
    P, Q = synth.n_groups(256, 256, g_m, g_n)
    L = synth.make_layer(sp, 4, 900 + g_m + g_n, g_m, g_n, "exact_total", round(P * Q * 27 / 4))
    lay = nets.ConvLayer(sp, L["w"], L["bias"], L["mask"], g_m, g_n, torch.bfloat16)
    y = nets.to_numpy(lay(xd), 256)
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], sp.stride, sp.pad, True, round_bf16=True)
    assert rel_err(y, ref) <= TOL


# ------------------------------------------------------------------------------ CUDA-graph replay
@pytest.mark.parametrize("which", ["c3d", "r2plus1d", "s3d"])
def test_graph_replay_matches_eager(which, request):
    """The forward passes are timed as captured CUDA graphs (dependent launches, side streams as parallel branches):
    a replay must give the bits of the eager pass, also after new clips were copied into the captured input buffer."""
    if which == "c3d":
        plan, layers, specs, x2, rec, final = request.getfixturevalue("c3d")
        make = lambda: nets.C3DNet(plan, device_layers(layers, specs), fuse_pool=True)
    elif which == "r2plus1d":
        stem, blocks, layers, specs, x2, rec, final = request.getfixturevalue("r21d")
        make = lambda: nets.R2Plus1DNet(stem, blocks, device_layers(layers, specs), fuse_residual=True, fuse_pairs=True)
    else:
        plan, layers, x2, rec, final = request.getfixturevalue("s3d")
        make = lambda: nets.S3DNet(plan, device_layers(layers, synth.s3d_convs(plan)))
    xa = nets.to_device(x2)
    xb = nets.to_device(oracle.bf16_round(synth.make_input(77, x2.shape)))
    eager = make()
    ya, yb = eager.forward(xa).clone(), eager.forward(xb).clone()
    g = nets.GraphedForward(make(), xa.clone())
    assert torch.equal(g().clone(), ya)
    g.x.copy_(xb)
    assert torch.equal(g().clone(), yb)
    g.x.copy_(xa)
    assert torch.equal(g().clone(), ya)
    assert rt3d.rt3d_last_device_status() == rt3d.OK


def test_c3d_batch1_graph_replays_give_the_same_bits(c3d):
    """1500 replays of the batch-1 forward, each compared with the first.  Before the small-C_in kernel's unused K half
    was given an in-image window, about 2 % of such replays differed in one pooled voxel of pool1: for the tile's last
    voxel that half read 16 bytes past the staged image, shared memory that no load writes; whatever an earlier
    kernel had left there, if a NaN or an infinity, became NaN x 0 in that voxel's accumulators and the max-pool
    dropped it without a trace.  (Other shapes and batch sizes never showed it in thousands of replays.)"""
    plan, layers, specs, x2, rec, final = c3d
    net = nets.C3DNet(plan, device_layers(layers, specs), fuse_pool=True)
    g = nets.GraphedForward(net, nets.to_device(x2[:1]))
    y0 = g().clone()
    torch.cuda.synchronize()
    bad = 0
    for _ in range(1500):
        y = g()
        torch.cuda.synchronize()
        bad += 0 if torch.equal(y, y0) else 1
    assert bad == 0, f"{bad} of 1500 replays differ from the first"
    assert rt3d.rt3d_last_device_status() == rt3d.OK
