"""Sub-tile kernel (RT3D_ALGO_UMMA_SUB): the tensor-core path that skips pruned kernel locations per block of
16 output x 16 input channels, against the CPU oracle at the bf16 tolerance.  The cases span several tiles
with a ragged tail, ragged channel counts on both sides, strides, every group size of the paper plus wider
ones, a bundle split (M > 256), all-pruned bundles and residual fusion; rt3d_last_plan proves the kernel ran."""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _run(shape, cin, cout, k, g_m, g_n, density, stride=(1, 1, 1), relu=True, seed=5, mask_edit=None):
    spec = synth.ConvSpec("sub", cin, cout, k, stride, tuple(kk // 2 for kk in k), relu)
    L = synth.make_layer(spec, 9, seed, g_m, g_n, "bernoulli", density)
    mask = L["mask"] if mask_edit is None else mask_edit(L["mask"].copy())
    x = synth.make_input(700 + seed, shape + (cin,))
    ref = oracle.conv3d(x, L["w"], mask, L["bias"], spec.stride, spec.pad, relu, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], mask, g_m, g_n, torch.bfloat16)
    y = lay(nets.to_device(x), algo=rt3d.ALGO_UMMA_SUB)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert rt3d.rt3d_last_plan()["kernel"] == 6
    got = nets.to_numpy(y, cout)
    err = float(np.abs(got - ref).max() / np.abs(ref).max())
    assert (ref != 0).mean() > 0.1
    assert err <= TOL, err
    return lay, y


@pytest.mark.parametrize("shape,cin,cout,k,g_m,g_n,density,stride", [
    ((1, 2, 8, 8), 64, 64, (1, 1, 1), 8, 8, 0.5, (1, 1, 1)),
    ((2, 4, 9, 7), 128, 256, (3, 3, 3), 8, 8, 0.125, (1, 1, 1)),       # 504 voxels: 4 tiles, ragged tail
    ((2, 4, 9, 7), 72, 230, (1, 3, 3), 8, 4, 0.3, (1, 1, 1)),          # ragged channels on both sides
    ((1, 4, 14, 14), 256, 300, (3, 3, 3), 16, 16, 0.25, (1, 1, 1)),    # two bundles of 160
    ((2, 5, 13, 11), 64, 96, (3, 3, 3), 4, 4, 0.4, (1, 2, 2)),         # the paper's 4 x 4 groups, strided
    ((1, 3, 12, 12), 192, 128, (3, 1, 1), 64, 64, 0.5, (1, 1, 1)),
    ((4, 8, 14, 14), 256, 256, (3, 3, 3), 8, 8, 0.125, (1, 1, 1)),     # 49 tiles on the persistent grid
])
def test_sub_kernel_against_oracle(shape, cin, cout, k, g_m, g_n, density, stride):
    _run(shape, cin, cout, k, g_m, g_n, density, stride)


def test_sub_kernel_pruned_ranges_and_bundles():
    # output channels 16..47 keep nothing (their ranges get zero blocks), and the whole second bundle of 256 is
    # pruned (no steps at all): both must come out as act(bias)
    def edit(mask):
        mask[16:48] = 0
        mask[256:] = 0
        return mask
    _run((2, 2, 8, 8), 64, 300, (3, 3, 3), 8, 8, 0.3, mask_edit=edit, relu=False)


def test_sub_kernel_repeatable_and_residual():
    lay, y1 = _run((2, 4, 9, 7), 128, 256, (3, 3, 3), 8, 8, 0.2, seed=7)
    x = nets.to_device(synth.make_input(707, (2, 4, 9, 7, 128)))
    y2 = lay(x, algo=rt3d.ALGO_UMMA_SUB)
    assert torch.equal(y1, y2)                                         # fixed accumulation order per output
    res = nets.to_device(synth.make_input(99, (2, 4, 9, 7, 256)))
    y3 = lay.fused(x, lay.alloc_out(x), residual=res, algo=rt3d.ALGO_UMMA_SUB)
    assert rt3d.rt3d_last_plan()["kernel"] == 6
    y4 = lay.fused(x, lay.alloc_out(x), residual=res, algo=rt3d.ALGO_UMMA_PAIR)
    scale = float(y4.float().abs().max())
    assert float((y3.float() - y4.float()).abs().max()) <= 1e-2 * scale


def test_sub_kernel_refusals():
    spec = synth.ConvSpec("sub", 64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 9, 1, 4, 4, "none", None)
    dense = nets.ConvLayer(spec, L["w"], L["bias"], None, dtype=torch.bfloat16, dense=True)
    x = nets.to_device(synth.make_input(3, (1, 2, 8, 8, 64)))
    with pytest.raises(rt3d.Rt3dError) as e:
        dense(x, algo=rt3d.ALGO_UMMA_SUB)
    assert e.value.status == rt3d.ERR_UNSUPPORTED
