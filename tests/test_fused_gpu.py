"""GPU parity of the fused layer boundaries (residual add before the ReLU, max-pool after it) against
the oracle's composition of the separate steps.  Same norm and tolerance as the plain convolution:
max|err| <= 2e-2 * max|ref| (bf16), 1e-3 (fp32)."""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu

RES_CASES = [
    # cin, cout, k, stride, pad, (n,t,h,w), algo, dtype
    (64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (4, 8, 16, 16), rt3d.ALGO_AUTO, torch.bfloat16),      # pair kernel, TMA stores
    (144, 64, (3, 1, 1), (1, 1, 1), (1, 0, 0), (2, 8, 28, 28), rt3d.ALGO_AUTO, torch.bfloat16),     # R(2+1)D block end
    (230, 128, (3, 1, 1), (1, 1, 1), (1, 0, 0), (1, 4, 14, 14), rt3d.ALGO_UMMA, torch.bfloat16),    # few tiles: K split
    (64, 45, (1, 3, 3), (1, 1, 1), (0, 1, 1), (1, 3, 9, 11), rt3d.ALGO_UMMA, torch.bfloat16),       # ragged channels, direct stores
    (64, 230, (1, 3, 3), (1, 2, 2), (0, 1, 1), (2, 4, 28, 28), rt3d.ALGO_AUTO, torch.bfloat16),     # strided, 16-column tail
    (3, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 32, 24), rt3d.ALGO_AUTO, torch.bfloat16),       # small-C_in kernel
    (24, 40, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 7, 9), rt3d.ALGO_SIMT, torch.bfloat16),
    (16, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 8, 8), rt3d.ALGO_SIMT, torch.float32),
]


@pytest.mark.parametrize("case", RES_CASES)
@pytest.mark.parametrize("relu", [True, False])
def test_residual_add_fused_into_the_epilogue(case, relu):
    cin, cout, k, stride, pad, (n, t, h, w), algo, dtype = case
    spec = synth.ConvSpec("f", cin, cout, k, stride, pad, relu)
    L = synth.make_layer(spec, 11, cin + cout, 4, 4, "bernoulli", 0.4)
    x = synth.make_input(1100, (n, t, h, w, cin))
    bf = dtype == torch.bfloat16
    conv = oracle.conv3d(x, L["w"], L["mask"], L["bias"], stride, pad, False, round_bf16=bf)
    res = synth.make_input(1101, conv.shape)
    res_r = oracle.bf16_round(res) if bf else res
    ref = conv.astype(np.float64) + res_r
    if relu:
        ref = np.maximum(ref, 0)
    ref = ref.astype(np.float32)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, dtype)
    xd, rd = nets.to_device(x, dtype), nets.to_device(res, dtype)
    y = torch.full(lay.out_shape(xd), 55.0, dtype=dtype, device="cuda")
    rt3d.rt3d_conv3d_sparse_fused(rt3d.tensor_desc(xd, cin), lay.packed, lay.bias, rt3d.tensor_desc(y, cout), stride, pad,
                                  relu, residual=rt3d.tensor_desc(rd, cout), algo=algo)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    got = nets.to_numpy(y, cout)
    assert np.isfinite(got).all()
    tol = 2e-2 if bf else 1e-3
    assert np.abs(got - ref).max() <= tol * np.abs(ref).max()
    assert (y[..., cout:] == 55.0).all()
    # and it equals the two-step path within one bf16 rounding of the intermediate
    y2 = nets.add_relu(lay(xd, relu=False, algo=algo), rd, cout, relu)
    assert np.abs(nets.to_numpy(y2, cout) - got).max() <= tol * np.abs(ref).max()


POOL_CASES = [
    # cin, cout, k, (n,t,h,w), pool
    (3, 64, (3, 3, 3), (2, 4, 48, 40), (1, 2, 2)),        # C3D conv1 + pool1 (small-C_in kernel)
    (64, 128, (3, 3, 3), (2, 8, 24, 24), (2, 2, 2)),      # conv2 + pool2 (pair kernel, two K steps per stage)
    (128, 256, (3, 3, 3), (4, 4, 12, 12), (2, 2, 2)),     # conv3b + pool3 shape class
    (64, 64, (3, 3, 3), (3, 5, 13, 9), (2, 2, 2)),        # odd extents: last windows are dropped
    (64, 256, (1, 3, 3), (2, 3, 16, 16), (1, 2, 2)),
    (64, 64, (3, 3, 3), (2, 6, 10, 12), (2, 1, 2)),
    (8, 96, (3, 3, 3), (1, 5, 23, 21), (1, 2, 2)),        # small-C_in kernel, odd extents, three whole pieces
]


@pytest.mark.parametrize("algo", ["umma", "pair"])
@pytest.mark.parametrize("case", POOL_CASES)
def test_max_pool_fused_into_the_epilogue(case, algo):
    cin, cout, k, (n, t, h, w), pool = case
    if algo == "pair" and cin < 16:
        pytest.skip("the small-C_in kernel has no CTA-pair form")
    algo = rt3d.ALGO_UMMA if algo == "umma" else rt3d.ALGO_UMMA_PAIR
    pad = tuple(kk // 2 for kk in k)
    spec = synth.ConvSpec("p", cin, cout, k, (1, 1, 1), pad, True)
    L = synth.make_layer(spec, 12, cin + cout, 4, 4, "bernoulli", 0.4)
    x = synth.make_input(1200, (n, t, h, w, cin))
    conv = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, pad, True, round_bf16=True)
    ref = oracle.maxpool3d(oracle.bf16_round(conv), pool, pool)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(x)
    y = torch.full(ref.shape[:4] + (nets.pitch_for(cout, torch.bfloat16) + 8,), 33.0, dtype=torch.bfloat16, device="cuda")
    lay.fused(xd, y, pool=pool, algo=algo)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    got = nets.to_numpy(y, cout)
    assert (ref != 0).mean() > 0.1
    assert np.abs(got - ref).max() <= 2e-2 * np.abs(ref).max()
    assert (y[..., cout:] == 33.0).all()
    # pooling commutes with the activation and the bf16 rounding: same as conv followed by the pool kernel
    # (bit for bit when both runs use the same K split; the unfused run may split K on small shapes)
    y2 = nets.maxpool(lay(xd), cout, synth.PoolSpec("p", pool, pool, (0, 0, 0)))
    assert np.abs(nets.to_numpy(y2, cout) - got).max() <= 1e-2 * np.abs(ref).max()
    if n * t * h * w >= 148 * 128:
        assert torch.equal(y2[..., :cout], y[..., :cout])


def test_auto_declines_pooling_where_it_would_split_k():
    spec = synth.ConvSpec("p", 256, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 12, 9, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(synth.make_input(5, (1, 2, 14, 14, 256)))                     # 392 voxels: 4 output tiles
    y = torch.zeros((1, 1, 7, 7, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rt3d.Rt3dError) as e:
        lay.fused(xd, y, pool=(2, 2, 2))
    assert e.value.status == rt3d.ERR_UNSUPPORTED
    lay.fused(xd, y, pool=(2, 2, 2), algo=rt3d.ALGO_UMMA)                             # explicit choice: fuses
    ref = nets.maxpool(lay(xd), 256, synth.PoolSpec("p", (2, 2, 2), (2, 2, 2), (0, 0, 0)))
    err = (y.float() - ref.float()).abs().max().item()
    assert err <= 1e-2 * ref.float().abs().max().item()


def test_fused_pool_refusals():
    spec = synth.ConvSpec("p", 64, 48, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)        # bundle width 48: not whole pieces
    L = synth.make_layer(spec, 12, 3, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(synth.make_input(3, (1, 4, 8, 8, 64)))
    y = torch.zeros((1, 2, 4, 4, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rt3d.Rt3dError) as e:
        lay.fused(xd, y, pool=(2, 2, 2), algo=rt3d.ALGO_UMMA)
    assert e.value.status == rt3d.ERR_UNSUPPORTED
    # the same on the small-C_in kernel: 112 channels = three pieces and a half (the call used to write the half
    # piece unpooled, at the unpooled voxel's offset: beyond the pooled tensor)
    spec1 = synth.ConvSpec("p", 8, 112, (3, 3, 5), (1, 2, 1), (0, 1, 0), True)
    L1 = synth.make_layer(spec1, 12, 5, 4, 4, "bernoulli", 0.3)
    lay1 = nets.ConvLayer(spec1, L1["w"], L1["bias"], L1["mask"], 4, 4, torch.bfloat16)
    xd1 = nets.to_device(synth.make_input(4, (1, 15, 22, 56, 8)))
    with pytest.raises(rt3d.Rt3dError) as e:
        lay1.fused(xd1, torch.zeros((1, 13, 5, 26, 112), dtype=torch.bfloat16, device="cuda"), pool=(1, 2, 2))
    assert e.value.status == rt3d.ERR_UNSUPPORTED
    spec2 = synth.ConvSpec("p", 64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L2 = synth.make_layer(spec2, 12, 4, 4, 4, "bernoulli", 0.4)
    lay2 = nets.ConvLayer(spec2, L2["w"], L2["bias"], L2["mask"], 4, 4, torch.bfloat16)
    with pytest.raises(rt3d.Rt3dError) as e:                                           # wrong pooled extents
        lay2.fused(xd, torch.zeros((1, 4, 4, 4, 64), dtype=torch.bfloat16, device="cuda"), pool=(2, 2, 2))
    assert e.value.status == rt3d.ERR_SHAPE
    with pytest.raises(rt3d.Rt3dError) as e:                                           # CUDA-core kernel has no pooled epilogue
        lay2.fused(xd, torch.zeros((1, 2, 4, 4, 64), dtype=torch.bfloat16, device="cuda"), pool=(2, 2, 2), algo=rt3d.ALGO_SIMT)
    assert e.value.status == rt3d.ERR_UNSUPPORTED


def test_fused_argument_errors():
    spec = synth.ConvSpec("f", 64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 11, 1, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(synth.make_input(1, (1, 2, 8, 8, 64)))
    y = lay.alloc_out(xd)
    bad = torch.zeros((1, 2, 8, 7, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rt3d.Rt3dError) as e:
        rt3d.rt3d_conv3d_sparse_fused(rt3d.tensor_desc(xd), lay.packed, lay.bias, rt3d.tensor_desc(y), spec.stride, spec.pad,
                                      True, residual=rt3d.tensor_desc(bad))
    assert e.value.status == rt3d.ERR_SHAPE
    with pytest.raises(rt3d.Rt3dError) as e:                       # residual must not alias the output
        rt3d.rt3d_conv3d_sparse_fused(rt3d.tensor_desc(xd), lay.packed, lay.bias, rt3d.tensor_desc(y), spec.stride, spec.pad,
                                      True, residual=rt3d.tensor_desc(y))
    assert e.value.status == rt3d.ERR_INVALID_ARG
    with pytest.raises(rt3d.Rt3dError) as e:
        rt3d.rt3d_conv3d_sparse_fused(rt3d.tensor_desc(xd), lay.packed, lay.bias, rt3d.tensor_desc(y), spec.stride, spec.pad,
                                      True, pool=(3, 1, 1))
    assert e.value.status == rt3d.ERR_INVALID_ARG
