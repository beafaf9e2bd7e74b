"""Thin ctypes binding of librt3d.so: argument marshalling only.

Function names mirror the C ABI in include/rt3d.h.  Tensors are torch tensors used purely
as device (or pinned host) memory: NDHWC, contiguous in the last dimension, optionally with
a channel pitch wider than the channel count.  Every numerical step runs inside the CUDA
library; there is no fallback: if librt3d.so is missing the import of this module fails.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("RT3D_LIB") or os.path.join(_HERE, "librt3d.so")   # RT3D_LIB: alternative build of the same library

RT3D_F32, RT3D_BF16 = 0, 1
ALGO_AUTO, ALGO_SIMT, ALGO_UMMA, ALGO_UMMA_PAIR, ALGO_UMMA_HALO, ALGO_UMMA_SUB = 0, 1, 2, 3, 4, 5
OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_MASK_NOT_GROUP_UNIFORM, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT = range(8)
ERR_WORKSPACE, ERR_NOT_PREPARED = 8, 9


class Rt3dError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        msg = _lib.rt3d_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{where}: {msg} (status {int(status)})")


class Tensor(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("n", ctypes.c_int32), ("t", ctypes.c_int32), ("h", ctypes.c_int32),
                ("w", ctypes.c_int32), ("c", ctypes.c_int32), ("c_stride", ctypes.c_int32), ("dtype", ctypes.c_int32)]


class ConvParams(ctypes.Structure):
    _fields_ = [("st", ctypes.c_int32), ("sh", ctypes.c_int32), ("sw", ctypes.c_int32),
                ("pt", ctypes.c_int32), ("ph", ctypes.c_int32), ("pw", ctypes.c_int32),
                ("relu", ctypes.c_int32), ("algo", ctypes.c_int32), ("x_pad_zero", ctypes.c_int32),
                ("concurrent", ctypes.c_int32)]


class Fusion(ctypes.Structure):
    _fields_ = [("residual", ctypes.POINTER(Tensor)), ("pool_t", ctypes.c_int32), ("pool_h", ctypes.c_int32),
                ("pool_w", ctypes.c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in ("kernel", "n_tile", "n_splits", "tail_workers", "fused_pool")]


class PackedView(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in ("M", "N", "Kt", "Kh", "Kw", "g_m", "g_n", "P", "Q", "Ks",
                                              "dtype", "is_vanilla", "is_dense")] + \
               [("nnz", ctypes.c_int64), ("group_ptr", ctypes.POINTER(ctypes.c_int32)),
                ("pos_idx", ctypes.POINTER(ctypes.c_uint16)), ("tiles", ctypes.c_void_p)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2007_09835_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, f32p, u8p = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_uint8)
    TP, CP = ctypes.POINTER(Tensor), ctypes.POINTER(ConvParams)
    lib.rt3d_pack_kgs.argtypes = [f32p, u8p, i, i, i, i, i, i, i, i, ctypes.POINTER(vp)]
    lib.rt3d_pack_dense.argtypes = [f32p, i, i, i, i, i, i, ctypes.POINTER(vp)]
    lib.rt3d_packed_view_get.argtypes = [vp, ctypes.POINTER(PackedView)]
    lib.rt3d_unpack_to_dense.argtypes = [vp, f32p]
    lib.rt3d_unpack_device_layout.argtypes = [vp, i, f32p]
    lib.rt3d_unpack_device_layout_tgroups.argtypes = [vp, i, f32p]
    lib.rt3d_unpack_sub_layout.argtypes = [vp, i, f32p]
    lib.rt3d_packed_prepare.argtypes = [vp]
    lib.rt3d_packed_free.argtypes = [vp]
    lib.rt3d_packed_free.restype = None
    for name in ("rt3d_conv3d_sparse", "rt3d_conv3d_dense", "rt3d_conv3d_host", "rt3d_conv3d_sparse_noalloc"):
        getattr(lib, name).argtypes = [TP, vp, vp, CP, TP, vp]
    lib.rt3d_conv3d_sparse_fused.argtypes = [TP, vp, vp, CP, ctypes.POINTER(Fusion), TP, vp]
    lib.rt3d_conv2plus1d_fused.argtypes = [TP, vp, vp, CP, vp, vp, CP, TP, TP, vp]
    lib.rt3d_kgs_group_norms.argtypes = [vp, i, i, i, i, i, i, i, i, vp, vp]
    lib.rt3d_kgs_reweight.argtypes = [vp, ctypes.c_int64, ctypes.c_float, ctypes.c_float, vp, vp, vp]
    lib.rt3d_kgs_expand_mask.argtypes = [vp, i, i, i, i, i, i, i, vp, vp]
    lib.rt3d_maxpool3d.argtypes = [TP] + [i] * 9 + [TP, vp]
    lib.rt3d_add_relu.argtypes = [TP, TP, i, TP, vp]
    i64p = ctypes.POINTER(ctypes.c_int64)
    lib.rt3d_conv3d_cost.argtypes = [TP, vp, CP, i64p, i64p, i64p]
    lib.rt3d_conv3d_query_algo.argtypes = [TP, vp, CP, TP, ctypes.POINTER(ctypes.c_int)]
    lib.rt3d_last_plan.argtypes = [ctypes.POINTER(PlanInfo)]
    lib.rt3d_last_device_status.argtypes = [vp]
    lib.rt3d_launch_count.restype = ctypes.c_int64
    lib.rt3d_alloc_count.restype = ctypes.c_int64
    lib.rt3d_plan_begin.restype = None
    lib.rt3d_plan_end.restype = None
    lib.rt3d_debug_set.argtypes = [i, ctypes.c_longlong]
    lib.rt3d_status_string.restype = ctypes.c_char_p
    lib.rt3d_status_string.argtypes = [i]
    lib.rt3d_version.restype = ctypes.c_char_p
    return lib


_lib = None
_lib = _load()


def lib():
    """The loaded ctypes library (for callers that want the raw C ABI)."""
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise Rt3dError(status, where)


class Packed:
    """Owner of an rt3d_packed handle."""

    def __init__(self, handle: int):
        self.handle = ctypes.c_void_p(handle)

    def view(self) -> dict:
        v = PackedView()
        _check(_lib.rt3d_packed_view_get(self.handle, ctypes.byref(v)), "rt3d_packed_view_get")
        PQ = v.P * v.Q
        out = {k: getattr(v, k) for k in ("M", "N", "Kt", "Kh", "Kw", "g_m", "g_n", "P", "Q", "Ks", "dtype",
                                          "is_vanilla", "is_dense", "nnz")}
        out["group_ptr"] = np.ctypeslib.as_array(v.group_ptr, shape=(PQ + 1,)).copy()
        if v.nnz:
            out["pos_idx"] = np.ctypeslib.as_array(v.pos_idx, shape=(v.nnz,)).copy()
            ty = ctypes.c_uint16 if v.dtype == RT3D_BF16 else ctypes.c_float
            arr = ctypes.cast(v.tiles, ctypes.POINTER(ty))
            out["tiles"] = np.ctypeslib.as_array(arr, shape=(v.nnz, v.g_m, v.g_n)).copy()
        else:
            out["pos_idx"] = np.zeros(0, np.uint16)
            out["tiles"] = np.zeros((0, v.g_m, v.g_n), np.uint16 if v.dtype == RT3D_BF16 else np.float32)
        return out

    def unpack_to_dense(self) -> np.ndarray:
        v = self.view()
        out = np.empty((v["M"], v["N"], v["Kt"], v["Kh"], v["Kw"]), np.float32)
        _check(_lib.rt3d_unpack_to_dense(self.handle, out.ctypes.data_as(ctypes.POINTER(ctypes.c_float))),
               "rt3d_unpack_to_dense")
        return out

    def unpack_device_layout(self, n_tile: int = 0, t_groups: bool = False) -> np.ndarray:
        v = self.view()
        out = np.empty((v["M"], v["N"], v["Kt"], v["Kh"], v["Kw"]), np.float32)
        fn = _lib.rt3d_unpack_device_layout_tgroups if t_groups else _lib.rt3d_unpack_device_layout
        _check(fn(self.handle, int(n_tile), out.ctypes.data_as(ctypes.POINTER(ctypes.c_float))),
               "rt3d_unpack_device_layout")
        return out

    def unpack_sub_layout(self, n_tile: int = 0) -> np.ndarray:
        v = self.view()
        out = np.empty((v["M"], v["N"], v["Kt"], v["Kh"], v["Kw"]), np.float32)
        _check(_lib.rt3d_unpack_sub_layout(self.handle, int(n_tile), out.ctypes.data_as(ctypes.POINTER(ctypes.c_float))),
               "rt3d_unpack_sub_layout")
        return out

    def prepare(self):
        _check(_lib.rt3d_packed_prepare(self.handle), "rt3d_packed_prepare")

    def free(self):
        if self.handle:
            _lib.rt3d_packed_free(self.handle)
            self.handle = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def _np_f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def rt3d_pack_kgs(w, mask, g_m: int, g_n: int, compute_dtype: int) -> Packed:
    """w: numpy [M,N,Kt,Kh,Kw] float32 (host); mask: numpy uint8 of the same shape or None."""
    w = _np_f32(w)
    M, N, Kt, Kh, Kw = w.shape
    mp = None
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        if mask.shape != w.shape:
            raise ValueError("mask shape must equal weight shape")
        mp = mask.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8))
    h = ctypes.c_void_p()
    _check(_lib.rt3d_pack_kgs(w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), mp, M, N, Kt, Kh, Kw,
                              int(g_m), int(g_n), int(compute_dtype), ctypes.byref(h)), "rt3d_pack_kgs")
    return Packed(h.value)


def rt3d_pack_dense(w, compute_dtype: int) -> Packed:
    w = _np_f32(w)
    M, N, Kt, Kh, Kw = w.shape
    h = ctypes.c_void_p()
    _check(_lib.rt3d_pack_dense(w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), M, N, Kt, Kh, Kw,
                                int(compute_dtype), ctypes.byref(h)), "rt3d_pack_dense")
    return Packed(h.value)


def tensor_desc(t, c: int | None = None) -> Tensor:
    """Describe a torch tensor [n,t,h,w,c_stride] (last dim contiguous) as an rt3d_tensor with
    `c` logical channels (default: all of the last dimension)."""
    import torch
    if t.dim() != 5 or t.stride(4) != 1:
        raise ValueError("expected a 5-D NDHWC tensor with unit channel stride")
    n, tt, h, w, cs = t.shape
    if t.stride() != (tt * h * w * cs, h * w * cs, w * cs, cs, 1):
        raise ValueError("tensor must be dense in (n,t,h,w) with pitch = size of last dimension")
    dt = {torch.float32: RT3D_F32, torch.bfloat16: RT3D_BF16}[t.dtype]
    return Tensor(t.data_ptr(), n, tt, h, w, cs if c is None else int(c), cs, dt)


def channel_slice_desc(t, offset: int, c: int) -> Tensor:
    """Channels [offset, offset + c) of a dense NDHWC torch tensor as an rt3d_tensor (same voxel pitch): lets a
    layer write its output straight into its place of a channel concatenation.  offset must keep the data
    pointer 16-byte aligned (a multiple of 8 bf16 / 4 fp32 channels)."""
    d = tensor_desc(t)
    if offset < 0 or c < 1 or offset + c > d.c_stride:
        raise ValueError("channel slice out of range")
    es = 2 if d.dtype == RT3D_BF16 else 4
    return Tensor(t.data_ptr() + offset * es, d.n, d.t, d.h, d.w, int(c), d.c_stride, d.dtype)


_concurrent = threading.local()


@contextlib.contextmanager
def concurrent_kernels():
    """Convolution calls made by this thread inside the block tell the library that other kernels may run on the
    device at the same time (parallel streams): it then avoids plans whose CTAs wait for one another."""
    prev = getattr(_concurrent, "on", False)
    _concurrent.on = True
    try:
        yield
    finally:
        _concurrent.on = prev


@contextlib.contextmanager
def planning():
    """Planning mode (rt3d_plan_begin / rt3d_plan_end): compute calls inside the block choose their kernels, upload
    their weight layouts and size their workspaces but launch nothing."""
    _lib.rt3d_plan_begin()
    try:
        yield
    finally:
        _lib.rt3d_plan_end()


def _params(stride, pad, relu, algo, x_pad_zero=False) -> ConvParams:
    return ConvParams(int(stride[0]), int(stride[1]), int(stride[2]), int(pad[0]), int(pad[1]), int(pad[2]),
                      int(bool(relu)), int(algo), int(bool(x_pad_zero)), int(getattr(_concurrent, "on", False)))


def _stream_ptr(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return ctypes.c_void_p(int(stream))


def _bias_ptr(bias):
    return None if bias is None else ctypes.c_void_p(bias.data_ptr())


def rt3d_conv3d_sparse(x: Tensor, w: Packed, bias, y: Tensor, stride=(1, 1, 1), pad=(0, 0, 0), relu=False,
                       algo=ALGO_AUTO, stream=None, x_pad_zero=False):
    """x, y: Tensor descriptors (device); bias: torch float32 device tensor [M] or None."""
    _check(_lib.rt3d_conv3d_sparse(ctypes.byref(x), w.handle, _bias_ptr(bias),
                                   ctypes.byref(_params(stride, pad, relu, algo, x_pad_zero)), ctypes.byref(y),
                                   _stream_ptr(stream)), "rt3d_conv3d_sparse")


def rt3d_conv3d_sparse_noalloc(x: Tensor, w: Packed, bias, y: Tensor, stride=(1, 1, 1), pad=(0, 0, 0), relu=False,
                               algo=ALGO_AUTO, stream=None):
    """rt3d_conv3d_sparse for callers that must not allocate device memory at call time (a real-time
    loop, a thread that may not block on the allocator): the handle must have been prepared on this
    device (`w.prepare()`), the K-split scratch is a fixed 16 MiB array inside the library, and a call
    that would need more raises Rt3dError with status ERR_WORKSPACE."""
    _check(_lib.rt3d_conv3d_sparse_noalloc(ctypes.byref(x), w.handle, _bias_ptr(bias),
                                           ctypes.byref(_params(stride, pad, relu, algo)), ctypes.byref(y),
                                           _stream_ptr(stream)), "rt3d_conv3d_sparse_noalloc")


def rt3d_conv3d_sparse_fused(x: Tensor, w: Packed, bias, y: Tensor, stride=(1, 1, 1), pad=(0, 0, 0), relu=False,
                             residual: Tensor | None = None, pool=(1, 1, 1), algo=ALGO_AUTO, stream=None,
                             x_pad_zero=False):
    """y = pool(act(bias + conv(x) + residual)); residual: descriptor of a device tensor with the un-pooled
    output's extents or None; pool: (1|2, 1|2, 1|2) max-pool window = stride applied after the activation."""
    fz = Fusion(ctypes.pointer(residual) if residual is not None else None, int(pool[0]), int(pool[1]), int(pool[2]))
    _check(_lib.rt3d_conv3d_sparse_fused(ctypes.byref(x), w.handle, _bias_ptr(bias),
                                         ctypes.byref(_params(stride, pad, relu, algo, x_pad_zero)), ctypes.byref(fz),
                                         ctypes.byref(y), _stream_ptr(stream)), "rt3d_conv3d_sparse_fused")


def rt3d_conv2plus1d_fused(x: Tensor, w_s: Packed, bias_s, pad_s, relu_s, w_t: Packed, bias_t, pad_t, relu_t,
                           y: Tensor, residual: Tensor | None = None, stream=None):
    """Spatial 1xKhxKw conv then temporal 3x1x1 conv in one launch (all strides 1); Rt3dError with status
    ERR_UNSUPPORTED when the pair does not fit the fused kernel (run the two layers separately then)."""
    res = ctypes.pointer(residual) if residual is not None else None
    _check(_lib.rt3d_conv2plus1d_fused(ctypes.byref(x), w_s.handle, _bias_ptr(bias_s),
                                       ctypes.byref(_params((1, 1, 1), pad_s, relu_s, ALGO_AUTO)), w_t.handle,
                                       _bias_ptr(bias_t), ctypes.byref(_params((1, 1, 1), pad_t, relu_t, ALGO_AUTO)),
                                       res, ctypes.byref(y), _stream_ptr(stream)), "rt3d_conv2plus1d_fused")


def rt3d_conv3d_dense(x: Tensor, w: Packed, bias, y: Tensor, stride=(1, 1, 1), pad=(0, 0, 0), relu=False,
                       algo=ALGO_AUTO, stream=None, x_pad_zero=False):
    _check(_lib.rt3d_conv3d_dense(ctypes.byref(x), w.handle, _bias_ptr(bias),
                                  ctypes.byref(_params(stride, pad, relu, algo, x_pad_zero)), ctypes.byref(y),
                                  _stream_ptr(stream)), "rt3d_conv3d_dense")


def rt3d_conv3d_host(x: Tensor, w: Packed, bias, y: Tensor, stride=(1, 1, 1), pad=(0, 0, 0), relu=False,
                     algo=ALGO_AUTO, stream=None):
    """x, y describe HOST buffers (pinned recommended); bias is a host float32 tensor or None."""
    _check(_lib.rt3d_conv3d_host(ctypes.byref(x), w.handle, _bias_ptr(bias),
                                 ctypes.byref(_params(stride, pad, relu, algo)), ctypes.byref(y),
                                 _stream_ptr(stream)), "rt3d_conv3d_host")


def rt3d_maxpool3d(x: Tensor, k, stride, pad, y: Tensor, stream=None):
    _check(_lib.rt3d_maxpool3d(ctypes.byref(x), *map(int, k), *map(int, stride), *map(int, pad), ctypes.byref(y),
                               _stream_ptr(stream)), "rt3d_maxpool3d")


def rt3d_add_relu(a: Tensor, b: Tensor, relu: bool, y: Tensor, stream=None):
    _check(_lib.rt3d_add_relu(ctypes.byref(a), ctypes.byref(b), int(bool(relu)), ctypes.byref(y),
                              _stream_ptr(stream)), "rt3d_add_relu")


def rt3d_kgs_group_norms(w, g_m: int, g_n: int, norm: int, norms, stream=None):
    """w: torch float32 device tensor [M,N,Kt,Kh,Kw]; norms: torch float32 device tensor [P,Q,Kt*Kh*Kw] (output)."""
    M, N, Kt, Kh, Kw = w.shape
    _check(_lib.rt3d_kgs_group_norms(ctypes.c_void_p(w.data_ptr()), M, N, Kt, Kh, Kw, int(g_m), int(g_n), int(norm),
                                     ctypes.c_void_p(norms.data_ptr()), _stream_ptr(stream)), "rt3d_kgs_group_norms")


def rt3d_kgs_reweight(norms, eps: float, threshold: float, penalty=None, keep=None, stream=None):
    """norms: float32 device tensor; penalty (float32) / keep (uint8): device tensors of the same size or None."""
    _check(_lib.rt3d_kgs_reweight(ctypes.c_void_p(norms.data_ptr()), norms.numel(), float(eps), float(threshold),
                                  None if penalty is None else ctypes.c_void_p(penalty.data_ptr()),
                                  None if keep is None else ctypes.c_void_p(keep.data_ptr()), _stream_ptr(stream)),
           "rt3d_kgs_reweight")


def rt3d_kgs_expand_mask(group_mask, M, N, Kt, Kh, Kw, g_m, g_n, mask, stream=None):
    """group_mask: uint8 device [P,Q,Ks]; mask: uint8 device [M,N,Kt,Kh,Kw] (output)."""
    _check(_lib.rt3d_kgs_expand_mask(ctypes.c_void_p(group_mask.data_ptr()), M, N, Kt, Kh, Kw, int(g_m), int(g_n),
                                     ctypes.c_void_p(mask.data_ptr()), _stream_ptr(stream)), "rt3d_kgs_expand_mask")


def rt3d_conv3d_cost(x: Tensor, w: Packed, stride=(1, 1, 1), pad=(0, 0, 0)):
    """(kept MACs, dense MACs, algorithmic bytes) of one call."""
    k, d, b = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.rt3d_conv3d_cost(ctypes.byref(x), w.handle, ctypes.byref(_params(stride, pad, False, 0)),
                                 ctypes.byref(k), ctypes.byref(d), ctypes.byref(b)), "rt3d_conv3d_cost")
    return k.value, d.value, b.value


def rt3d_conv3d_query_algo(x: Tensor, w: Packed, y: Tensor, stride=(1, 1, 1), pad=(0, 0, 0), algo=ALGO_AUTO) -> int:
    a = ctypes.c_int()
    _check(_lib.rt3d_conv3d_query_algo(ctypes.byref(x), w.handle, ctypes.byref(_params(stride, pad, False, algo)),
                                       ctypes.byref(y), ctypes.byref(a)), "rt3d_conv3d_query_algo")
    return a.value


def rt3d_last_plan() -> dict:
    """How this thread's most recent convolution call was run (kernel, n_tile, n_splits, tail_workers, fused_pool)."""
    info = PlanInfo()
    _check(_lib.rt3d_last_plan(ctypes.byref(info)), "rt3d_last_plan")
    return {name: int(getattr(info, name)) for name, _ in PlanInfo._fields_}


def rt3d_last_device_status(stream=None) -> int:
    return int(_lib.rt3d_last_device_status(_stream_ptr(stream)))


def rt3d_launch_count() -> int:
    return int(_lib.rt3d_launch_count())


def rt3d_alloc_count() -> int:
    return int(_lib.rt3d_alloc_count())


DEBUG_WAIT_CYCLES, DEBUG_DROP_LAST_LOAD, DEBUG_T_GROUPS, DEBUG_POISON = 1, 2, 3, 4


def rt3d_debug_get(what: int) -> int:
    _lib.rt3d_debug_get.restype = ctypes.c_longlong
    _lib.rt3d_debug_get.argtypes = [ctypes.c_int]
    return int(_lib.rt3d_debug_get(int(what)))


DEBUG_WAIT_SITE = 1


def rt3d_debug_set(what: int, value: int):
    _check(_lib.rt3d_debug_set(int(what), int(value)), "rt3d_debug_set")


def rt3d_version() -> str:
    return _lib.rt3d_version().decode()
