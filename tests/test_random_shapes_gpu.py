"""GPU parity on seeded RANDOM layer shapes: what the hand-picked cases of the other files may have missed.

Each case draws channels, kernel, strides, padding, extents, kernel-group size, density, activation, an optional
residual and an optional fused pool from a fixed seed, runs the library (AUTO or a forced kernel family) and
compares the whole output with the CPU oracle at the bf16 tolerance, max|err| <= 2e-2 * max|ref|; a second run must
give the same bits.  Where the library declines a convolution call (RT3D_ERR_UNSUPPORTED: a fusion or a forced kernel
family that does not apply to the drawn shape) the case runs the convolution through AUTO and the pool as a launch of
its own, as a caller would; a factorised pair that the one-launch kernel does not take is skipped.  (A draw of this
kind found the pooled small-C_in call whose trailing half piece was stored unpooled.)
"""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu

TOL = 2e-2
GROUPS = [(4, 4), (8, 4), (8, 8), (16, 16), (64, 64), (128, 64)]


def draw_conv_case(rng):
    cin = int(rng.choice([8, 16, 24, 45, 64, 96, 128, 144, 192, 230, 256, 320]))
    cout = int(rng.choice([16, 32, 48, 64, 80, 112, 128, 144, 160, 192, 256, 288, 384, 512]))
    k = tuple(int(rng.choice([1, 2, 3, 3, 3, 5])) for _ in range(3))
    if k[0] * k[1] * k[2] * cin > 40000:
        k = (k[0], 1, 1)
    stride = tuple(int(rng.choice([1, 1, 1, 2])) for _ in range(3))
    pad = tuple(int(rng.integers(0, q // 2 + 1)) for q in k)
    n = int(rng.integers(1, 9))
    t = int(rng.integers(max(1, k[0] - 2 * pad[0]), 17))
    h = int(rng.integers(max(4, k[1]), 60))
    w = int(rng.integers(max(4, k[2]), 60))
    if n * t * h * w * cin * cout * k[0] * k[1] * k[2] > 1.5e11:      # keep the oracle within about a second
        n, t = min(n, 2), min(t, 6)
    g_m, g_n = GROUPS[int(rng.integers(0, len(GROUPS)))]
    dens = float(rng.choice([0.15, 0.4, 0.7]))
    kind = "bernoulli" if rng.random() < 0.85 else "none"
    dense = kind == "none" and rng.random() < 0.5
    relu = bool(rng.random() < 0.7)
    algo = [rt3d.ALGO_AUTO, rt3d.ALGO_AUTO, rt3d.ALGO_UMMA, rt3d.ALGO_UMMA_PAIR, rt3d.ALGO_UMMA_HALO][int(rng.integers(0, 5))]
    use_res = bool(rng.random() < 0.5)
    pool = [(1, 1, 1), (1, 1, 1), (1, 2, 2), (2, 2, 2)][int(rng.integers(0, 4))]
    return cin, cout, k, stride, pad, (n, t, h, w), (g_m, g_n), kind, dens, dense, relu, algo, use_res, pool


@pytest.mark.parametrize("case", range(48))
def test_random_conv_layers_against_oracle(case):
    rng = np.random.default_rng(77000 + case)
    cin, cout, k, stride, pad, (n, t, h, w), (g_m, g_n), kind, dens, dense, relu, algo, use_res, pool = draw_conv_case(rng)
    spec = synth.ConvSpec("r", cin, cout, k, stride, pad, relu)
    L = synth.make_layer(spec, 31, case, g_m, g_n, kind, None if kind == "none" else dens)
    x = synth.make_input(3100 + case, (n, t, h, w, cin))
    mask = None if dense else L["mask"]
    lin = oracle.conv3d(x, L["w"], mask, L["bias"], stride, pad, False, round_bf16=False).astype(np.float64)
    res = synth.make_input(5100 + case, lin.shape) if use_res else None
    if use_res:
        lin = lin + oracle.bf16_round(res)
    act = oracle.bf16_round((np.maximum(lin, 0) if relu else lin).astype(np.float32))
    pool = tuple(p if d >= p else 1 for p, d in zip(pool, act.shape[1:4]))
    ref = oracle.maxpool3d(act, pool, pool) if pool != (1, 1, 1) else act
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], g_m, g_n, torch.bfloat16, dense=dense)
    xd = nets.to_device(x)
    rd = nets.to_device(res) if use_res else None
    ys = []
    for _ in range(2):
        y = torch.full(ref.shape[:4] + (nets.pitch_for(cout, torch.bfloat16),), 7.0, dtype=torch.bfloat16, device="cuda")
        try:
            lay.fused(xd, y, residual=rd, pool=pool, algo=algo)
        except rt3d.Rt3dError as e:
            # declined (a fusion or a forced kernel family that does not apply to this shape): what a caller does
            # then, the convolution through AUTO and the pool as a launch of its own
            assert e.status == rt3d.ERR_UNSUPPORTED, e
            full = torch.full(act.shape[:4] + (nets.pitch_for(cout, torch.bfloat16),), 7.0, dtype=torch.bfloat16, device="cuda")
            lay.fused(xd, full, residual=rd)
            y = full if pool == (1, 1, 1) else nets.maxpool(full, cout, synth.PoolSpec("p", pool, pool, (0, 0, 0)), y)
        ys.append(y)
    torch.cuda.synchronize()
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    got = nets.to_numpy(ys[0], cout)
    assert np.isfinite(got).all()
    scale = np.abs(ref).max()
    assert scale > 0
    assert np.abs(got - ref).max() <= TOL * scale, (rt3d.rt3d_last_plan(), np.abs(got - ref).max() / scale)
    assert torch.equal(ys[0], ys[1])                               # fixed summation order: repeatable bits


@pytest.mark.parametrize("case", range(16))
def test_random_factorised_pairs_against_oracle(case):
    rng = np.random.default_rng(78000 + case)
    cin = int(rng.choice([3, 8, 16, 32, 45, 64]))
    cmid = int(rng.choice([16, 48, 64, 80, 96, 112, 144, 160, 200]))
    cout = int(rng.choice([16, 32, 48, 64, 80, 96, 128]))
    kh, kw = int(rng.choice([1, 3, 3, 5])), int(rng.choice([1, 3, 3, 5]))
    n, t = int(rng.integers(1, 5)), int(rng.integers(1, 20))
    h, w = int(rng.integers(kh, 50)), int(rng.integers(kw, 50))
    dens = None if rng.random() < 0.15 else float(rng.choice([0.2, 0.5, 0.8]))
    with_res, relu_s, relu_t = bool(rng.random() < 0.5), bool(rng.random() < 0.7), bool(rng.random() < 0.7)
    pad_s = (0, kh // 2, kw // 2)
    sp_s = synth.ConvSpec("s", cin, cmid, (1, kh, kw), (1, 1, 1), pad_s, relu_s)
    sp_t = synth.ConvSpec("t", cmid, cout, (3, 1, 1), (1, 1, 1), (1, 0, 0), relu_t)
    kind = "none" if dens is None else "bernoulli"
    Ls = synth.make_layer(sp_s, 41, case, 4, 4, kind, dens)
    Lt = synth.make_layer(sp_t, 42, case, 4, 4, kind, dens)
    x = synth.make_input(4100 + case, (n, t, h, w, cin))
    res = synth.make_input(4101 + case, (n, t, h, w, cout)) if with_res else None
    mid = oracle.bf16_round(oracle.conv3d(x, Ls["w"], Ls["mask"], Ls["bias"], (1, 1, 1), pad_s, relu_s, round_bf16=True))
    out = oracle.conv3d(mid, Lt["w"], Lt["mask"], Lt["bias"], (1, 1, 1), (1, 0, 0), False, round_bf16=True).astype(np.float64)
    if res is not None:
        out = out + oracle.bf16_round(res)
    ref = (np.maximum(out, 0) if relu_t else out).astype(np.float32)
    ls = nets.ConvLayer(sp_s, Ls["w"], Ls["bias"], Ls["mask"], 4, 4, torch.bfloat16, dense=dens is None)
    lt = nets.ConvLayer(sp_t, Lt["w"], Lt["bias"], Lt["mask"], 4, 4, torch.bfloat16, dense=dens is None)
    xd = nets.to_device(x)
    rd = nets.to_device(res) if with_res else None
    ys = []
    try:
        for _ in range(2):
            y = torch.full((n, t, h, w, nets.pitch_for(cout, torch.bfloat16)), 55.0, dtype=torch.bfloat16, device="cuda")
            rt3d.rt3d_conv2plus1d_fused(rt3d.tensor_desc(xd, cin), ls.packed, ls.bias, pad_s, relu_s, lt.packed, lt.bias,
                                        (1, 0, 0), relu_t, rt3d.tensor_desc(y, cout),
                                        residual=None if rd is None else rt3d.tensor_desc(rd, cout))
            ys.append(y)
    except rt3d.Rt3dError as e:
        assert e.status == rt3d.ERR_UNSUPPORTED, e
        pytest.skip(f"declined: {e}")
    torch.cuda.synchronize()
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    got = nets.to_numpy(ys[0], cout)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL * np.abs(ref).max()
    assert torch.equal(ys[0], ys[1])


@pytest.mark.parametrize("case", range(24))
def test_random_max_pools_bit_exact(case):
    rng = np.random.default_rng(79000 + case)
    c = int(rng.choice([3, 8, 16, 45, 64, 100, 128, 192, 256, 480]))
    k = tuple(int(rng.choice([1, 2, 3])) for _ in range(3))
    s = tuple(int(rng.choice([1, 2])) for _ in range(3))
    p = tuple(int(rng.integers(0, kk // 2 + 1)) for kk in k)
    n, t = int(rng.integers(1, 4)), int(rng.integers(k[0], 12))
    h, w = int(rng.integers(k[1], 40)), int(rng.integers(k[2], 40))
    x = oracle.bf16_round(synth.make_input(4300 + case, (n, t, h, w, c)))
    ref = oracle.maxpool3d(x, k, s, p)
    y = nets.maxpool(nets.to_device(x), c, synth.PoolSpec("p", k, s, p))
    torch.cuda.synchronize()
    got = nets.to_numpy(y, c)
    assert got.shape == ref.shape and np.array_equal(got, ref)


@pytest.mark.parametrize("case", range(24))
def test_random_channel_slices_against_oracle(case):
    """Input and output as channel slices of wider tensors (the way an Inception block's branches read a shared input
    and write into their part of the concatenation): the result matches the oracle and the neighbouring channels of
    the output tensor keep their contents."""
    from paper_2007_09835_b200 import binding as B
    rng = np.random.default_rng(80000 + case)
    cin = int(rng.choice([8, 16, 24, 64, 96, 128, 192, 256]))
    cout = int(rng.choice([16, 32, 48, 64, 96, 128, 160, 192, 256, 384]))
    k = tuple(int(rng.choice([1, 1, 3, 3])) for _ in range(3))
    stride = tuple(int(rng.choice([1, 1, 2])) for _ in range(3))
    pad = tuple(q // 2 for q in k)
    n, t = int(rng.integers(1, 5)), int(rng.integers(1, 9))
    h, w = int(rng.integers(4, 40)), int(rng.integers(4, 40))
    xl, xr = 8 * int(rng.integers(0, 4)), 8 * int(rng.integers(0, 4))
    yl, yr = 8 * int(rng.integers(0, 5)), 8 * int(rng.integers(0, 5))
    relu = bool(rng.random() < 0.7)
    algo = [rt3d.ALGO_AUTO, rt3d.ALGO_AUTO, rt3d.ALGO_UMMA, rt3d.ALGO_UMMA_PAIR, rt3d.ALGO_SIMT][int(rng.integers(0, 5))]
    spec = synth.ConvSpec("s", cin, cout, k, stride, pad, relu)
    L = synth.make_layer(spec, 95, case, 4, 4, "bernoulli", float(rng.choice([0.2, 0.5])))
    x = synth.make_input(9500 + case, (n, t, h, w, cin))
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], stride, pad, relu, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xw = torch.full((n, t, h, w, xl + cin + xr), 77.0, dtype=torch.bfloat16, device="cuda")    # junk beside the input slice
    xw[..., xl:xl + cin] = torch.from_numpy(x).to(torch.bfloat16).cuda()
    yw = torch.full(tuple(ref.shape[:4]) + (yl + cout + yr,), 9.0, dtype=torch.bfloat16, device="cuda")
    try:
        lay.run_desc(B.channel_slice_desc(xw, xl, cin), B.channel_slice_desc(yw, yl, cout), algo=algo)
    except rt3d.Rt3dError as e:
        assert e.status == rt3d.ERR_UNSUPPORTED, e
        lay.run_desc(B.channel_slice_desc(xw, xl, cin), B.channel_slice_desc(yw, yl, cout))
    torch.cuda.synchronize()
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    got = yw[..., yl:yl + cout].float().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL * np.abs(ref).max(), rt3d.rt3d_last_plan()
    assert (yw[..., :yl] == 9.0).all() and (yw[..., yl + cout:] == 9.0).all()
