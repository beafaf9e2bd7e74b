"""Tensors beyond 2^31 elements (outputs of 4.9 GB): index arithmetic, tensor-map extents and work-item counts at
sizes the oracle cannot follow.  The batch is two seeded clips repeated, so every clip has a reference: the same
layer run on the two clips alone (itself covered by the oracle tests); the first, middle and last clips of the
large run must match it (to 1e-2 of the largest value for the convolutions, whose grid may cut K differently at the
larger size; bit for bit for pools and adds).  Needs about 10 GB."""
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu

CASES = [
    # name, cin, cout, kernel, pad, clip extents, batch, fused pool
    ("first layer, small-C_in kernel", 3, 64, (3, 3, 3), (1, 1, 1), (16, 112, 112), 192, (1, 1, 1)),
    ("3x3x3 on the CTA-pair kernel", 64, 128, (3, 3, 3), (1, 1, 1), (16, 56, 56), 384, (1, 1, 1)),
    ("the same with the pool fused", 64, 128, (3, 3, 3), (1, 1, 1), (16, 56, 56), 384, (2, 2, 2)),
    ("pointwise 480 -> 192", 480, 192, (1, 1, 1), (0, 0, 0), (16, 28, 28), 1024, (1, 1, 1)),
]


def picks(batch):
    return (0, 1, batch // 2, batch // 2 + 1, batch - 2, batch - 1)


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_conv_outputs_beyond_2_31_elements(case):
    if torch.cuda.mem_get_info()[0] < 16 * 2**30:
        pytest.skip("needs 16 GB of free device memory")
    _, cin, cout, k, pad, clip, batch, pool = case
    spec = synth.ConvSpec("big", cin, cout, k, (1, 1, 1), pad, True)
    L = synth.make_layer(spec, 71, 1, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    two = nets.to_device(oracle.bf16_round(synth.make_input(7100, (2,) + clip + (cin,))))
    x = two.repeat((batch // 2, 1, 1, 1, 1)).contiguous()
    o = lay.out_shape(two)
    shape2 = (2, o[1] // pool[0], o[2] // pool[1], o[3] // pool[2], o[4])
    y2 = torch.zeros(shape2, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((batch,) + shape2[1:], dtype=torch.bfloat16, device="cuda")
    lay.fused(two, y2, pool=pool)
    lay.fused(x, y, pool=pool)
    torch.cuda.synchronize()
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    if pool == (1, 1, 1):
        assert y.numel() > 2**31
    assert float(y2.float().abs().max()) > 0
    scale = float(y2.float().abs().max())
    for i in picks(batch):          # equal up to the summation order of a K split the larger grid may choose
        assert float((y[i].float() - y2[i % 2].float()).abs().max()) <= 1e-2 * scale, i
    del x, y
    torch.cuda.empty_cache()


def test_pools_and_add_beyond_2_31_elements():
    if torch.cuda.mem_get_info()[0] < 16 * 2**30:
        pytest.skip("needs 16 GB of free device memory")
    two = nets.to_device(oracle.bf16_round(synth.make_input(7200, (2, 16, 112, 112, 64))))
    x = two.repeat((96, 1, 1, 1, 1)).contiguous()
    assert x.numel() > 2**31
    for ps in (synth.PoolSpec("p", (1, 2, 2), (1, 2, 2), (0, 0, 0)), synth.PoolSpec("p", (3, 3, 3), (1, 1, 1), (1, 1, 1))):
        y2, y = nets.maxpool(two, 64, ps), nets.maxpool(x, 64, ps)
        torch.cuda.synchronize()
        for i in picks(192):
            assert torch.equal(y[i], y2[i % 2]), (ps.k, i)
        del y
    a2, a = nets.add_relu(two, two, 64), nets.add_relu(x, x, 64)
    torch.cuda.synchronize()
    for i in picks(192):
        assert torch.equal(a[i], a2[i % 2]), i
    del a, x
    torch.cuda.empty_cache()
