"""GPU parity of the CTA-pair kernel's t-grouped variant (plan kernel 7) against the CPU oracle.

In that variant the steps that differ only in kt share ONE staged input tile that is Kt - 1 frames deeper, each
step reading it through a descriptor that starts kt frames in (with a temporal stride of 2: one deeper tile per
phase of the stride, tap kt reading tile kt % 2 from frame kt / 2 on); the step order, the unit of the tail split and the
two issuing threads' halves all change with it, so it gets its own cases: 2- and 3-deep kernels, dense and sparse
lists, lists with pruned steps (groups of one or two steps), ragged boxes and channels, spatial strides, the tail
split in both forms, fused pooling and residual.  Tolerance as everywhere: max|err| <= 2e-2 * max|ref| (bf16).
"""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu

CASES = [
    # cin, cout, k, stride, (n,t,h,w), (g_m, g_n), mask kind, dense, wants a tail split
    (64, 128, (3, 3, 3), (1, 1, 1), (2, 8, 24, 24), (4, 4), "bernoulli", False, False),
    (64, 128, (3, 3, 3), (1, 1, 1), (2, 8, 24, 24), (4, 4), "none", True, False),          # computed steps
    (96, 80, (2, 3, 3), (1, 1, 1), (4, 9, 30, 30), (4, 4), "bernoulli", False, False),      # two-deep kernel, 2 chunks
    (144, 64, (3, 1, 1), (1, 1, 1), (2, 8, 28, 28), (4, 4), "bernoulli", False, False),     # temporal factor, 3 chunks
    (128, 128, (3, 3, 3), (1, 1, 1), (3, 7, 27, 29), (4, 4), "bernoulli", False, False),    # ragged boxes
    (160, 112, (3, 3, 3), (1, 1, 1), (2, 6, 20, 20), (8, 4), "bernoulli", False, False),    # ragged chunk and bundle
    (128, 128, (3, 3, 3), (1, 1, 1), (2, 8, 24, 24), (128, 64), "bernoulli", False, False), # pruned steps: short groups
    (64, 128, (3, 3, 3), (1, 1, 1), (4, 8, 28, 28), (4, 4), "bernoulli", False, True),      # 98 items on 74 pairs
    (128, 128, (3, 3, 3), (1, 1, 1), (1, 8, 28, 28), (4, 4), "bernoulli", False, True),     # 25 items: all of them split
    (64, 128, (3, 3, 3), (1, 2, 2), (2, 8, 32, 32), (4, 4), "bernoulli", False, False),     # spatial stride
    (64, 64, (7, 1, 1), (2, 1, 1), (2, 16, 40, 40), (4, 4), "bernoulli", False, False),     # temporal stride 2: two phase tiles
    (64, 96, (5, 3, 3), (2, 1, 1), (2, 16, 20, 20), (4, 4), "bernoulli", False, True),      # the same, five taps, every tile split
]


def run(case, pair_only=True):
    cin, cout, k, stride, (n, t, h, w), (g_m, g_n), kind, dense, _ = case
    pad = tuple(q // 2 for q in k)
    spec = synth.ConvSpec("tg", cin, cout, k, stride, pad, True)
    L = synth.make_layer(spec, 14, cin + cout, g_m, g_n, kind, None if kind == "none" else 0.4)
    x = synth.make_input(1400 + cin, (n, t, h, w, cin))
    ref = oracle.conv3d(x, L["w"], None if dense else L["mask"], L["bias"], stride, pad, True, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], g_m, g_n, torch.bfloat16, dense=dense)
    xd = nets.to_device(x)
    return spec, lay, xd, ref


@pytest.mark.parametrize("case", CASES)
def test_t_grouped_pair_kernel_against_oracle(case):
    spec, lay, xd, ref = run(case)
    y = torch.full(lay.out_shape(xd)[:4] + (nets.pitch_for(spec.cout, torch.bfloat16) + 8,), 21.0, dtype=torch.bfloat16,
                   device="cuda")
    lay(xd, y, algo=rt3d.ALGO_UMMA_PAIR)
    plan = rt3d.rt3d_last_plan()
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert plan["kernel"] == 7, plan
    if case[-1]:
        assert plan["tail_workers"] > 0, plan
    got = nets.to_numpy(y, spec.cout)
    assert np.isfinite(got).all() and (ref != 0).mean() > 0.1
    assert np.abs(got - ref).max() <= 2e-2 * np.abs(ref).max()
    assert (y[..., spec.cout:] == 21.0).all()                      # nothing written beyond the real channels
    # a second run gives the same bits (fixed summation order of the two issuing threads' halves and of the shares)
    y2 = torch.full_like(y, 21.0)
    lay(xd, y2, algo=rt3d.ALGO_UMMA_PAIR)
    assert torch.equal(y, y2)
    # and the step-per-location form of the same kernel agrees to one bf16 rounding
    rt3d.rt3d_debug_set(rt3d.DEBUG_T_GROUPS, 0)
    try:
        y3 = lay(xd, algo=rt3d.ALGO_UMMA_PAIR)
        assert rt3d.rt3d_last_plan()["kernel"] == 2
    finally:
        rt3d.rt3d_debug_set(rt3d.DEBUG_T_GROUPS, 1)
    assert np.abs(nets.to_numpy(y3, spec.cout) - got).max() <= 1e-2 * np.abs(ref).max()


def test_t_grouped_with_fused_pool_and_residual():
    # conv2 + pool2 of the C3D-shaped network, and a residual add before the ReLU
    spec = synth.ConvSpec("tgp", 64, 128, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 14, 7, 4, 4, "bernoulli", 0.4)
    x = synth.make_input(1407, (2, 8, 24, 24, 64))
    conv = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(x)
    pool = (2, 2, 2)
    ref = oracle.maxpool3d(oracle.bf16_round(conv), pool, pool)
    y = torch.zeros(ref.shape[:4] + (128,), dtype=torch.bfloat16, device="cuda")
    lay.fused(xd, y, pool=pool, algo=rt3d.ALGO_UMMA_PAIR)
    plan = rt3d.rt3d_last_plan()
    assert plan["kernel"] == 7 and plan["fused_pool"] == 1, plan
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert np.abs(nets.to_numpy(y, 128) - ref).max() <= 2e-2 * np.abs(ref).max()

    lin = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, False, round_bf16=True)
    res = synth.make_input(1408, lin.shape)
    ref2 = np.maximum(lin.astype(np.float64) + oracle.bf16_round(res), 0).astype(np.float32)
    rd = nets.to_device(res)
    y2 = torch.zeros(lay.out_shape(xd), dtype=torch.bfloat16, device="cuda")
    rt3d.rt3d_conv3d_sparse_fused(rt3d.tensor_desc(xd, 64), lay.packed, lay.bias, rt3d.tensor_desc(y2, 128), spec.stride,
                                  spec.pad, True, residual=rt3d.tensor_desc(rd, 128), algo=rt3d.ALGO_UMMA_PAIR)
    assert rt3d.rt3d_last_plan()["kernel"] == 7
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert np.abs(nets.to_numpy(y2, 128) - ref2).max() <= 2e-2 * np.abs(ref2).max()
