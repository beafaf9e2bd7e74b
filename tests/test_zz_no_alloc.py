"""rt3d_conv3d_sparse_noalloc: the convolution entry point for callers that cannot allocate.

Who needs it: code that runs a layer from inside a real-time / latency-critical loop, or from a
thread that must never block on the CUDA allocator (cudaMalloc synchronises the whole device), or
in a process whose device memory is budgeted by another component.  Such a caller prepares the
weights once up front and afterwards uses this entry point, whose K-split scratch is a fixed array
inside the library.  The test calls it through the C ABI twice in a row and compares with the
regular entry point and, for one case, with the CPU oracle; it checks that device memory does not move
across the first call, that the K-split path through the fixed workspace really ran, and the two refusals
(workspace too small, handle not prepared).
This file sorts last on purpose, so a run that stops at the first failure has already run
every other test; it does not depend on any of them.
"""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu


def _layer(cin, cout, k, seed, raw=False):
    spec = synth.ConvSpec("na", cin, cout, k, (1, 1, 1), tuple(kk // 2 for kk in k), True)
    L = synth.make_layer(spec, 8, seed, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    return (spec, lay, L) if raw else (spec, lay)


def _call_noalloc(lay, spec, x, y):
    rt3d.rt3d_conv3d_sparse_noalloc(rt3d.tensor_desc(x, spec.cin), lay.packed, lay.bias, rt3d.tensor_desc(y, spec.cout),
                                    spec.stride, spec.pad, spec.relu)


@pytest.mark.parametrize("shape,cin,cout,split", [((2, 2, 7, 7), 512, 512, True),      # 4 output tiles, 216 K steps: split 8 ways
                                                  ((1, 4, 14, 14), 256, 230, True),    # 7 tiles, ragged channels
                                                  ((8, 8, 28, 28), 128, 256, False)])  # 392 tiles: no split, no scratch
def test_noalloc_matches_regular_entry_point_twice(shape, cin, cout, split):
    spec, lay, L = _layer(cin, cout, (3, 3, 3), cin + cout, raw=True)
    x_host = synth.make_input(801, shape + (cin,))
    x = nets.to_device(x_host)
    y_ref = lay(x)                                      # regular entry point (allocates on first use)
    lay(x, algo=rt3d.ALGO_UMMA)                         # the single-CTA kernel's code is on the device (the runtime loads a kernel at its first launch)
    lay.packed.prepare()                                # everything that needs an allocation or a set-up happens here
    torch.cuda.synchronize()
    scale = float(y_ref.float().abs().max())
    assert scale > 0
    outs = []
    for rep in range(2):                                # two calls in a row share the library's workspace
        y = torch.full_like(y_ref, 123.0)
        torch.cuda.synchronize()
        free_before, allocs_before = torch.cuda.mem_get_info()[0], rt3d.rt3d_alloc_count()
        _call_noalloc(lay, spec, x, y)
        torch.cuda.synchronize()
        # neither the library nor the CUDA runtime on its behalf took device memory during the call
        assert torch.cuda.mem_get_info()[0] == free_before and rt3d.rt3d_alloc_count() == allocs_before
        assert rt3d.rt3d_last_device_status() == rt3d.OK
        plan = rt3d.rt3d_last_plan()
        assert plan["kernel"] == 1 and (plan["n_splits"] > 1) == split, plan
        err = float((y[..., :cout].float() - y_ref[..., :cout].float()).abs().max())
        assert err <= 2e-2 * scale, err
        assert (y[..., cout:] == 123.0).all()           # channel-pitch padding stays untouched
        outs.append(y)
    assert torch.equal(outs[0], outs[1])
    if cin == 256:                                      # and against the definition: the CPU oracle, bf16 tolerance
        ref = oracle.conv3d(x_host, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
        got = nets.to_numpy(outs[0], cout)
        assert float(np.abs(got - ref).max() / np.abs(ref).max()) <= 2e-2


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
    if tiles * splits * 128 * 256 * 4 <= 16 * 2 ** 20:
        pytest.skip(f"with {sms} SMs this shape splits {splits} ways and fits the fixed workspace: refusal not reachable")
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
