"""rt3d_conv3d_sparse_noalloc: the convolution entry point for callers that cannot allocate.

Who needs it: code that runs a layer from inside a real-time / latency-critical loop, or from a
thread that must never block on the CUDA allocator (cudaMalloc synchronises the whole device), or
in a process whose device memory is budgeted by another component.  Such a caller prepares the
weights once up front and afterwards uses this entry point, whose K-split scratch is a fixed array
inside the library.  The test calls it through the C ABI twice in a row and compares with the
regular entry point; it also checks the two refusals (workspace too small, handle not prepared).
This file sorts last on purpose, so a run that stops at the first failure has already run
every other test; it does not depend on any of them.
"""
import numpy as np
import pytest
import torch

import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu


def _layer(cin, cout, k, seed):
    spec = synth.ConvSpec("na", cin, cout, k, (1, 1, 1), tuple(kk // 2 for kk in k), True)
    L = synth.make_layer(spec, 8, seed, 4, 4, "bernoulli", 0.4)
    return spec, nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)


def _call_noalloc(lay, spec, x, y):
    rt3d.rt3d_conv3d_sparse_noalloc(rt3d.tensor_desc(x, spec.cin), lay.packed, lay.bias, rt3d.tensor_desc(y, spec.cout),
                                    spec.stride, spec.pad, spec.relu)


@pytest.mark.parametrize("shape,cin,cout", [((2, 2, 7, 7), 512, 512),      # 4 output tiles, 216 K steps: split 8 ways
                                            ((1, 4, 14, 14), 256, 230),    # 7 tiles, ragged channels
                                            ((8, 8, 28, 28), 128, 256)])   # 392 tiles: no split, no scratch
def test_noalloc_matches_regular_entry_point_twice(shape, cin, cout):
    spec, lay = _layer(cin, cout, (3, 3, 3), cin + cout)
    x = nets.to_device(synth.make_input(801, shape + (cin,)))
    y_ref = lay(x)                                      # regular entry point (allocates on first use)
    lay.packed.prepare()                                # everything that needs an allocation happens here
    torch.cuda.synchronize()
    scale = float(y_ref.float().abs().max())
    assert scale > 0
    outs = []
    for _ in range(2):                                  # two calls in a row share the library's workspace
        y = torch.full_like(y_ref, 123.0)
        _call_noalloc(lay, spec, x, y)
        torch.cuda.synchronize()
        assert rt3d.rt3d_last_device_status() == rt3d.OK
        err = float((y[..., :cout].float() - y_ref[..., :cout].float()).abs().max())
        assert err <= 2e-2 * scale, err
        assert (y[..., cout:] == 123.0).all()           # channel-pitch padding stays untouched
        outs.append(y)
    assert torch.equal(outs[0], outs[1])


def test_noalloc_refuses_what_it_cannot_do():
    # 26 output tiles x 5 splits x 128 KiB partial tiles = 16.25 MiB: more than the 16 MiB workspace
    spec, lay = _layer(1152, 512, (3, 3, 3), 7)
    x = nets.to_device(synth.make_input(802, (4, 2, 14, 14, 1152)))
    y = lay.alloc_out(x)
    with pytest.raises(rt3d.Rt3dError) as e:            # handle not prepared on this device yet
        _call_noalloc(lay, spec, x, y)
    assert e.value.status == rt3d.ERR_NOT_PREPARED
    lay.packed.prepare()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    tiles, steps = 13 * 2, 27 * 18
    splits = max(1, min(8, sms // tiles, steps // 8))
    if tiles * splits * 128 * 256 * 4 > 16 * 2 ** 20:
        with pytest.raises(rt3d.Rt3dError) as e:
            _call_noalloc(lay, spec, x, y)
        assert e.value.status == rt3d.ERR_WORKSPACE
    y_ok = lay(x)                                       # the allocating entry point has no such limit
    assert torch.isfinite(y_ok.float()).all()
    spec32, _ = _layer(16, 32, (3, 3, 3), 9)            # fp32 handles are outside this entry point
    L = synth.make_layer(spec32, 8, 9, 4, 4, "bernoulli", 0.5)
    lay32 = nets.ConvLayer(spec32, L["w"], L["bias"], L["mask"], 4, 4, torch.float32)
    x32 = nets.to_device(synth.make_input(803, (1, 2, 8, 8, 16)), torch.float32)
    lay32(x32)
    with pytest.raises(rt3d.Rt3dError) as e:
        _call_noalloc(lay32, spec32, x32, lay32.alloc_out(x32))
    assert e.value.status == rt3d.ERR_UNSUPPORTED
