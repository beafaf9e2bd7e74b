"""Host-side argument validation of the compute entry points (no GPU, nothing is launched):
every shape / dtype / alignment error is reported before any CUDA call is made."""
import ctypes

import numpy as np
import pytest

import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import binding as B

FAKE = 0x10000     # a 16-byte aligned, never dereferenced address


def tensor(n, t, h, w, c, cs=None, dtype=B.RT3D_BF16, data=FAKE):
    return B.Tensor(data, n, t, h, w, c, c if cs is None else cs, dtype)


@pytest.fixture(scope="module")
def packed():
    spec = synth.ConvSpec("v", 16, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1))
    L = synth.make_layer(spec, 5, 0, 4, 4, "bernoulli", 0.5)
    return B.rt3d_pack_kgs(L["w"], L["mask"], 4, 4, B.RT3D_BF16)


def call(packed, x, y, stride=(1, 1, 1), pad=(1, 1, 1), algo=0, fn="rt3d_conv3d_sparse"):
    p = B.ConvParams(*stride, *pad, 1, algo)
    return getattr(B.lib(), fn)(ctypes.byref(x), packed.handle, None, ctypes.byref(p), ctypes.byref(y), None)


def test_conv_argument_errors(packed):
    good_x, good_y = tensor(1, 4, 8, 8, 16), tensor(1, 4, 8, 8, 32)
    assert call(packed, tensor(1, 4, 8, 8, 24), good_y) == B.ERR_SHAPE                 # channels != N
    assert call(packed, good_x, tensor(1, 4, 8, 8, 16)) == B.ERR_SHAPE                 # channels != M
    assert call(packed, good_x, tensor(1, 4, 8, 7, 32)) == B.ERR_SHAPE                 # wrong output extent
    assert call(packed, tensor(1, 4, 8, 8, 16, dtype=B.RT3D_F32), good_y) == B.ERR_SHAPE   # dtype != handle's
    assert call(packed, good_x, good_y, stride=(0, 1, 1)) == B.ERR_INVALID_ARG
    assert call(packed, good_x, good_y, pad=(-1, 1, 1)) == B.ERR_INVALID_ARG
    assert call(packed, good_x, good_y, algo=9) == B.ERR_INVALID_ARG
    assert call(packed, tensor(1, 4, 8, 8, 16, data=0), good_y) == B.ERR_INVALID_ARG   # NULL data
    assert call(packed, tensor(1, 4, 8, 8, 16, cs=12), good_y) == B.ERR_INVALID_ARG    # pitch < channels
    assert call(packed, tensor(1, 4, 8, 8, 16, cs=20), good_y) == B.ERR_INVALID_ARG    # pitch not a multiple of 8
    assert call(packed, tensor(1, 4, 8, 8, 16, data=FAKE + 2), good_y) == B.ERR_INVALID_ARG   # misaligned
    assert call(packed, good_x, good_y) == B.ERR_INVALID_ARG                           # x and y overlap
    assert call(packed, tensor(1, 1, 1, 1, 16), tensor(1, 1, 1, 1, 32), pad=(0, 0, 0)) == B.ERR_SHAPE   # smaller than kernel
    far_y = tensor(1, 4, 8, 8, 32, data=FAKE + (1 << 24))
    assert call(packed, good_x, far_y, fn="rt3d_conv3d_dense") == B.ERR_INVALID_ARG    # dense entry needs a dense handle


def test_cost_needs_no_device(packed):
    k, d, b = B.rt3d_conv3d_cost(tensor(2, 4, 8, 8, 16), packed, (1, 1, 1), (1, 1, 1))
    assert d == 2 * 4 * 8 * 8 * 32 * 16 * 27 and 0 < k < d and b > 0


def test_pool_and_add_argument_errors():
    x = tensor(1, 4, 8, 8, 16)
    y = tensor(1, 2, 4, 4, 16, data=FAKE + (1 << 24))
    lib = B.lib()
    bad = tensor(1, 2, 4, 5, 16, data=FAKE + (1 << 24))
    assert lib.rt3d_maxpool3d(ctypes.byref(x), 2, 2, 2, 2, 2, 2, 0, 0, 0, ctypes.byref(bad), None) == B.ERR_SHAPE
    assert lib.rt3d_maxpool3d(ctypes.byref(x), 2, 2, 2, 2, 2, 2, 2, 0, 0, ctypes.byref(y), None) == B.ERR_INVALID_ARG
    assert lib.rt3d_maxpool3d(ctypes.byref(x), 0, 2, 2, 2, 2, 2, 0, 0, 0, ctypes.byref(y), None) == B.ERR_INVALID_ARG
    a, b = tensor(1, 2, 4, 4, 16), tensor(1, 2, 4, 4, 24)
    assert lib.rt3d_add_relu(ctypes.byref(a), ctypes.byref(b), 1, ctypes.byref(a), None) == B.ERR_SHAPE


def test_fused_call_argument_errors_need_no_device(packed):
    lib = B.lib()
    x, y = tensor(1, 4, 8, 8, 16), tensor(1, 4, 8, 8, 32, data=FAKE + (1 << 24))
    p = B.ConvParams(1, 1, 1, 1, 1, 1, 1, 0)

    def fused(fz, yy=y):
        return lib.rt3d_conv3d_sparse_fused(ctypes.byref(x), packed.handle, None, ctypes.byref(p), ctypes.byref(fz),
                                            ctypes.byref(yy), None)

    assert fused(B.Fusion(None, 3, 1, 1)) == B.ERR_INVALID_ARG                         # window must be 1 or 2
    assert fused(B.Fusion(None, 1, 0, 1)) == B.ERR_INVALID_ARG
    assert fused(B.Fusion(None, 2, 2, 2)) == B.ERR_SHAPE                               # y is not the pooled extent
    pooled = tensor(1, 2, 4, 4, 32, data=FAKE + (1 << 24))
    res = tensor(1, 4, 8, 8, 32, data=FAKE + (1 << 25))
    assert fused(B.Fusion(ctypes.pointer(res), 2, 2, 2), pooled) == B.ERR_UNSUPPORTED  # residual and pooling together
    bad_res = tensor(1, 4, 8, 7, 32, data=FAKE + (1 << 25))
    assert fused(B.Fusion(ctypes.pointer(bad_res), 1, 1, 1)) == B.ERR_SHAPE


def test_fused_pair_argument_errors_need_no_device():
    """rt3d_conv2plus1d_fused: argument and shape errors as the two separate calls would give them, and the
    refusals that depend on the layers alone, all before any CUDA call."""
    def pack(cin, cout, k, dtype=B.RT3D_BF16):
        spec = synth.ConvSpec("p", cin, cout, k, (1, 1, 1), tuple(kk // 2 for kk in k))
        L = synth.make_layer(spec, 6, cin + cout, 4, 4, "bernoulli", 0.5)
        return B.rt3d_pack_kgs(L["w"], L["mask"], 4, 4, dtype)

    ws, wt = pack(16, 48, (1, 3, 3)), pack(48, 32, (3, 1, 1))
    lib = B.lib()
    x, y = tensor(1, 4, 8, 8, 16), tensor(1, 4, 8, 8, 32, data=FAKE + (1 << 24))
    ps, pt = B.ConvParams(1, 1, 1, 0, 1, 1, 1, 0), B.ConvParams(1, 1, 1, 1, 0, 0, 1, 0)

    def pair(xx=x, yy=y, w1=ws, w2=wt, p1=ps, p2=pt, res=None):
        return lib.rt3d_conv2plus1d_fused(ctypes.byref(xx), w1.handle, None, ctypes.byref(p1), w2.handle, None,
                                          ctypes.byref(p2), None if res is None else ctypes.byref(res), ctypes.byref(yy), None)

    assert pair(xx=tensor(1, 4, 8, 8, 24)) == B.ERR_SHAPE                              # x channels != w_s->N
    assert pair(yy=tensor(1, 4, 8, 8, 48, data=FAKE + (1 << 24))) == B.ERR_SHAPE       # y channels != w_t->M
    assert pair(yy=tensor(1, 2, 8, 8, 32, data=FAKE + (1 << 24))) == B.ERR_SHAPE       # wrong output extent
    assert pair(w2=pack(40, 32, (3, 1, 1))) == B.ERR_SHAPE                             # w_t->N != w_s->M
    assert pair(p2=B.ConvParams(0, 1, 1, 1, 0, 0, 1, 0)) == B.ERR_INVALID_ARG          # stride 0
    assert pair(yy=tensor(1, 4, 8, 8, 32)) == B.ERR_INVALID_ARG                        # y overlaps x
    assert pair(res=tensor(1, 4, 8, 7, 32, data=FAKE + (1 << 25))) == B.ERR_SHAPE      # residual extent
    assert pair(res=y) == B.ERR_INVALID_ARG                                            # residual overlaps y
    # layer pairs the one-kernel path does not take: refused on the host, nothing launched
    assert pair(w1=pack(16, 48, (3, 3, 3)), p1=B.ConvParams(1, 1, 1, 1, 1, 1, 1, 0)) == B.ERR_UNSUPPORTED    # not 1xKhxKw
    assert pair(yy=tensor(1, 4, 4, 4, 32, data=FAKE + (1 << 24)), p1=B.ConvParams(1, 2, 2, 0, 1, 1, 1, 0)) == B.ERR_UNSUPPORTED   # strided
    f32s, f32t = pack(16, 48, (1, 3, 3), B.RT3D_F32), pack(48, 32, (3, 1, 1), B.RT3D_F32)
    xf = tensor(1, 4, 8, 8, 16, dtype=B.RT3D_F32)
    yf = tensor(1, 4, 8, 8, 32, dtype=B.RT3D_F32, data=FAKE + (1 << 24))
    assert pair(xx=xf, yy=yf, w1=f32s, w2=f32t) == B.ERR_UNSUPPORTED                   # fp32


def test_last_plan_before_any_convolution():
    import threading
    out = {}

    def worker():                                   # the record is per thread: a fresh thread has none
        out["null"] = B.lib().rt3d_last_plan(None)
        out["fresh"] = B.lib().rt3d_last_plan(ctypes.byref(B.PlanInfo()))

    th = threading.Thread(target=worker)
    th.start(); th.join()
    assert out == {"null": B.ERR_INVALID_ARG, "fresh": B.ERR_INVALID_ARG}


def test_channel_slice_descriptor():
    import torch
    t = torch.zeros((1, 2, 3, 4, 64), dtype=torch.bfloat16)
    d = B.channel_slice_desc(t, 16, 24)
    assert (d.c, d.c_stride, d.n, d.t, d.h, d.w) == (24, 64, 1, 2, 3, 4)
    assert d.data == t.data_ptr() + 32
    with pytest.raises(ValueError):
        B.channel_slice_desc(t, 48, 24)             # runs past the pitch
    with pytest.raises(ValueError):
        B.channel_slice_desc(t[..., :32], 0, 8)     # not a dense tensor
