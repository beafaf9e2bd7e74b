"""GPU parity of the one-launch factorised (2+1)D convolution (spatial 1xKhxKw conv, ReLU, bf16 rounding,
temporal 3x1x1 conv, residual, ReLU) against the oracle's composition of the two convolutions with the
intermediate tensor rounded to bf16, exactly as the two separate launches store it.  Same norm and tolerance
as the plain convolution: max|err| <= 2e-2 * max|ref|."""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu

ST_CASES = [
    # cin, mid, cout, (kh, kw), (n, t, h, w), density, residual, relu_s, relu_t
    (64, 144, 64, (3, 3), (2, 16, 56, 56), 0.4, True, True, True),      # R(2+1)D stage-2 block end: cut mid-clip across pairs
    (64, 144, 64, (3, 3), (1, 5, 20, 13), 0.4, False, True, True),      # ragged patches, dummy second patch
    (64, 144, 64, (3, 3), (3, 1, 16, 8), 0.5, True, True, False),       # a single frame: only the centre tap contributes
    (45, 64, 64, (3, 3), (2, 2, 17, 9), 0.6, False, False, True),       # ragged input channels, two frames
    (32, 80, 48, (1, 1), (1, 9, 16, 24), 0.7, True, True, True),        # pointwise spatial conv, 16-column tails
    (64, 96, 96, (3, 1), (2, 7, 33, 10), 0.5, False, True, False),
    (16, 160, 64, (3, 3), (1, 4, 12, 12), None, True, True, True),      # dense weights
    (64, 144, 64, (3, 3), (1, 40, 16, 8), 0.4, True, True, True),       # one patch, 40 frames: every CTA pair gets one frame of a cut clip
    (48, 112, 64, (3, 3), (2, 37, 24, 16), 0.5, False, True, True),     # long clips cut at odd places
]


def _reference(x, Ls, Lt, pad_s, relu_s, relu_t, res):
    mid = oracle.conv3d(x, Ls["w"], Ls["mask"], Ls["bias"], (1, 1, 1), pad_s, relu_s, round_bf16=True)
    mid = oracle.bf16_round(mid)                 # the intermediate tensor is a bf16 tensor
    out = oracle.conv3d(mid, Lt["w"], Lt["mask"], Lt["bias"], (1, 1, 1), (1, 0, 0), False, round_bf16=True)
    out = out.astype(np.float64)
    if res is not None:
        out = out + oracle.bf16_round(res)
    if relu_t:
        out = np.maximum(out, 0)
    return out.astype(np.float32)


@pytest.mark.parametrize("case", ST_CASES)
def test_spatial_then_temporal_in_one_launch(case):
    cin, cmid, cout, (kh, kw), (n, t, h, w), density, with_res, relu_s, relu_t = case
    pad_s = (0, kh // 2, kw // 2)
    sp_s = synth.ConvSpec("s", cin, cmid, (1, kh, kw), (1, 1, 1), pad_s, relu_s)
    sp_t = synth.ConvSpec("t", cmid, cout, (3, 1, 1), (1, 1, 1), (1, 0, 0), relu_t)
    kind = "none" if density is None else "bernoulli"
    Ls = synth.make_layer(sp_s, 21, cin + cmid, 4, 4, kind, density)
    Lt = synth.make_layer(sp_t, 22, cmid + cout, 4, 4, kind, density)
    x = synth.make_input(2100 + cin, (n, t, h, w, cin))
    res = synth.make_input(2101, (n, t, h, w, cout)) if with_res else None
    ref = _reference(x, Ls, Lt, pad_s, relu_s, relu_t, res)
    assert (ref != 0).mean() > 0.1

    ls = nets.ConvLayer(sp_s, Ls["w"], Ls["bias"], Ls["mask"], 4, 4, torch.bfloat16, dense=density is None)
    lt = nets.ConvLayer(sp_t, Lt["w"], Lt["bias"], Lt["mask"], 4, 4, torch.bfloat16, dense=density is None)
    xd = nets.to_device(x)
    rd = nets.to_device(res) if with_res else None
    y = torch.full((n, t, h, w, nets.pitch_for(cout, torch.bfloat16)), 55.0, dtype=torch.bfloat16, device="cuda")
    launches = rt3d.rt3d_launch_count()
    rt3d.rt3d_conv2plus1d_fused(rt3d.tensor_desc(xd, cin), ls.packed, ls.bias, pad_s, relu_s, lt.packed, lt.bias, (1, 0, 0),
                                relu_t, rt3d.tensor_desc(y, cout),
                                residual=None if rd is None else rt3d.tensor_desc(rd, cout))
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert rt3d.rt3d_launch_count() - launches == 1
    assert rt3d.rt3d_last_plan()["kernel"] == 5
    got = nets.to_numpy(y, cout)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 2e-2 * np.abs(ref).max()
    assert (y[..., cout:] == 55.0).all()
    # against the two separate launches: same intermediate rounding, so only summation order differs
    mid = ls(xd)
    y2 = torch.zeros_like(y)
    lt.fused(mid, y2, residual=rd, relu=relu_t)
    assert np.abs(nets.to_numpy(y2, cout) - got).max() <= 1e-2 * np.abs(ref).max()
    # repeatable bit for bit
    y3 = torch.zeros_like(y)
    rt3d.rt3d_conv2plus1d_fused(rt3d.tensor_desc(xd, cin), ls.packed, ls.bias, pad_s, relu_s, lt.packed, lt.bias, (1, 0, 0),
                                relu_t, rt3d.tensor_desc(y3, cout),
                                residual=None if rd is None else rt3d.tensor_desc(rd, cout))
    torch.cuda.synchronize()
    assert torch.equal(y3[..., :cout], y[..., :cout])


def test_pairs_the_fused_kernel_does_not_take_are_declined():
    def layers(cin, cmid, cout, ks, kt):
        sp_s = synth.ConvSpec("s", cin, cmid, ks, (1, 1, 1), (0, ks[1] // 2, ks[2] // 2), True)
        sp_t = synth.ConvSpec("t", cmid, cout, kt, (1, 1, 1), (kt[0] // 2, 0, 0), True)
        Ls = synth.make_layer(sp_s, 23, 1, 4, 4, "bernoulli", 0.5)
        Lt = synth.make_layer(sp_t, 24, 2, 4, 4, "bernoulli", 0.5)
        return (nets.ConvLayer(sp_s, Ls["w"], Ls["bias"], Ls["mask"]), nets.ConvLayer(sp_t, Lt["w"], Lt["bias"], Lt["mask"]))

    def call(ls, lt, cin, cout, shape, pad_t=(1, 0, 0)):
        x = torch.zeros(shape + (nets.pitch_for(cin, torch.bfloat16),), dtype=torch.bfloat16, device="cuda")
        y = torch.zeros(shape + (nets.pitch_for(cout, torch.bfloat16),), dtype=torch.bfloat16, device="cuda")
        rt3d.rt3d_conv2plus1d_fused(rt3d.tensor_desc(x, cin), ls.packed, ls.bias, ls.spec.pad, True, lt.packed, lt.bias, pad_t,
                                    True, rt3d.tensor_desc(y, cout))

    before = rt3d.rt3d_launch_count()
    for cin, cmid, cout, ks, kt in [(128, 144, 64, (1, 3, 3), (3, 1, 1)),      # more than 64 input channels
                                    (64, 230, 128, (1, 3, 3), (3, 1, 1)),      # 2*240 + 3*128 TMEM columns
                                    (64, 144, 64, (1, 3, 3), (1, 1, 1))]:      # temporal kernel is not 3
        ls, lt = layers(cin, cmid, cout, ks, kt)
        with pytest.raises(rt3d.Rt3dError) as e:
            call(ls, lt, cin, cout, (1, 4, 16, 16), (kt[0] // 2, 0, 0))
        assert e.value.status == rt3d.ERR_UNSUPPORTED
    ls, lt = layers(64, 144, 64, (1, 3, 3), (3, 1, 1))
    with pytest.raises(rt3d.Rt3dError) as e:                                   # wrong output extent: a shape error
        call(ls, lt, 64, 64, (1, 4, 16, 16), (0, 0, 0))
    assert e.value.status == rt3d.ERR_SHAPE
    assert rt3d.rt3d_launch_count() == before
