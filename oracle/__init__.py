"""Python face of the CPU oracle (oracle/rt3d_oracle.c).

TEST INFRASTRUCTURE ONLY.  Importers allowed: tests/, __graft_entry__.smoke() and the
cpu_baseline / reference legs of bench.py.  The CUDA library and its binding never import
this package, and this package imports nothing from them.

The C file is compiled on first use with gcc (-O2, OpenMP) into
oracle/librt3d_oracle.so; `build()` forces a rebuild check.  All functions take and return
numpy arrays; activations are NDHWC float32, weights [M][N][Kt][Kh][Kw] float32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rt3d_oracle.c")
_SO = os.path.join(_HERE, "librt3d_oracle.so")
_lib = None

_f32p = ctypes.POINTER(ctypes.c_float)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_u16p = ctypes.POINTER(ctypes.c_uint16)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than the source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_bf16_bits.restype = ctypes.c_uint16
        _lib.oracle_bf16_bits.argtypes = [ctypes.c_float]
        _lib.oracle_bf16_widen.restype = ctypes.c_float
        _lib.oracle_bf16_widen.argtypes = [ctypes.c_uint16]
    return _lib


def threads() -> int:
    """Number of threads the OpenMP loops of the oracle will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a, typ):
    return None if a is None else a.ctypes.data_as(typ)


def out_shape(x_shape, M, k, stride, pad):
    n, t, h, w, _ = x_shape
    ext = [(d + 2 * p - kk) // s + 1 for d, p, kk, s in zip((t, h, w), pad, k, stride)]
    return (n, ext[0], ext[1], ext[2], M)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 array to bfloat16 bit patterns (uint16), ties to even."""
    lib = _load()
    a = _f32(a)
    out = np.empty(a.shape, dtype=np.uint16)
    lib.oracle_bf16_round_array(_ptr(a, _f32p), _ptr(out, _u16p), ctypes.c_int64(a.size))
    return out


def bf16_widen(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_round(a: np.ndarray) -> np.ndarray:
    return bf16_widen(bf16_bits(a))


def conv3d(x, w, mask=None, bias=None, stride=(1, 1, 1), pad=(0, 0, 0), relu=False,
           round_bf16=False) -> np.ndarray:
    """Direct 3-D convolution with masked dense weights (gather form, double accumulation)."""
    lib = _load()
    x, w = _f32(x), _f32(w)
    n, t, h, ww, c = x.shape
    M, N, Kt, Kh, Kw = w.shape
    assert N == c, "weight input channels must equal activation channels"
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        assert mask.shape == w.shape
    if bias is not None:
        bias = _f32(bias)
    y = np.empty(out_shape(x.shape, M, (Kt, Kh, Kw), stride, pad), dtype=np.float32)
    rc = lib.oracle_conv3d(_ptr(x, _f32p), n, t, h, ww, c, _ptr(w, _f32p), _ptr(mask, _u8p),
                           _ptr(bias, _f32p), M, Kt, Kh, Kw, *map(int, stride), *map(int, pad),
                           int(relu), int(round_bf16), _ptr(y, _f32p))
    if rc != 0:
        raise ValueError("oracle_conv3d: bad arguments")
    return y


def conv3d_scatter(x, w, mask=None, bias=None, stride=(1, 1, 1), pad=(0, 0, 0), relu=False) -> np.ndarray:
    """Brute-force scatter-form convolution (tiny shapes only)."""
    lib = _load()
    x, w = _f32(x), _f32(w)
    n, t, h, ww, c = x.shape
    M, N, Kt, Kh, Kw = w.shape
    assert N == c
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
    if bias is not None:
        bias = _f32(bias)
    y = np.empty(out_shape(x.shape, M, (Kt, Kh, Kw), stride, pad), dtype=np.float32)
    rc = lib.oracle_conv3d_scatter(_ptr(x, _f32p), n, t, h, ww, c, _ptr(w, _f32p), _ptr(mask, _u8p),
                                   _ptr(bias, _f32p), M, Kt, Kh, Kw, *map(int, stride), *map(int, pad),
                                   int(relu), _ptr(y, _f32p))
    if rc != 0:
        raise ValueError("oracle_conv3d_scatter: bad arguments")
    return y


def conv2d(x, w, bias=None, stride=(1, 1), pad=(0, 0), relu=False) -> np.ndarray:
    """Independent 2-D convolution: x [n,h,w,c], w [M,N,Kh,Kw]."""
    lib = _load()
    x, w = _f32(x), _f32(w)
    n, h, ww, c = x.shape
    M, N, Kh, Kw = w.shape
    assert N == c
    if bias is not None:
        bias = _f32(bias)
    Ho = (h + 2 * pad[0] - Kh) // stride[0] + 1
    Wo = (ww + 2 * pad[1] - Kw) // stride[1] + 1
    y = np.empty((n, Ho, Wo, M), dtype=np.float32)
    rc = lib.oracle_conv2d(_ptr(x, _f32p), n, h, ww, c, _ptr(w, _f32p), _ptr(bias, _f32p), M, Kh, Kw,
                           int(stride[0]), int(stride[1]), int(pad[0]), int(pad[1]), int(relu), _ptr(y, _f32p))
    if rc != 0:
        raise ValueError("oracle_conv2d: bad arguments")
    return y


class MaskNotGroupUniform(ValueError):
    """The mask differs inside one (kernel group, kernel location): not a KGS mask."""


def pack_kgs(w, mask, g_m: int, g_n: int, to_bf16: bool = False) -> dict:
    """Canonical packed form: dict(group_ptr int32[P*Q+1], pos_idx uint16[nnz],
    tiles [nnz,g_m,g_n] float32 or uint16 (bf16 bits), nnz, is_vanilla, P, Q, Ks)."""
    lib = _load()
    w = _f32(w)
    M, N, Kt, Kh, Kw = w.shape
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        assert mask.shape == w.shape
    P, Q = -(-M // g_m), -(-N // g_n)
    nnz = ctypes.c_int64(0)
    van = ctypes.c_int(0)
    rc = lib.oracle_pack_kgs(_ptr(w, _f32p), _ptr(mask, _u8p), M, N, Kt, Kh, Kw, g_m, g_n, int(to_bf16),
                             None, None, None, ctypes.byref(nnz), ctypes.byref(van))
    if rc == 1:
        raise MaskNotGroupUniform("mask is not uniform inside a kernel group")
    if rc != 0:
        raise ValueError("oracle_pack_kgs: bad arguments")
    group_ptr = np.zeros(P * Q + 1, dtype=np.int32)
    pos_idx = np.zeros(nnz.value, dtype=np.uint16)
    tiles = np.zeros((nnz.value, g_m, g_n), dtype=np.uint16 if to_bf16 else np.float32)
    rc = lib.oracle_pack_kgs(_ptr(w, _f32p), _ptr(mask, _u8p), M, N, Kt, Kh, Kw, g_m, g_n, int(to_bf16),
                             _ptr(group_ptr, _i32p), _ptr(pos_idx, _u16p),
                             ctypes.c_void_p(tiles.ctypes.data), ctypes.byref(nnz), ctypes.byref(van))
    assert rc == 0
    return {"group_ptr": group_ptr, "pos_idx": pos_idx, "tiles": tiles, "nnz": int(nnz.value),
            "is_vanilla": bool(van.value), "P": P, "Q": Q, "Ks": Kt * Kh * Kw}


def unpack_kgs(packed: dict, M, N, Kt, Kh, Kw, g_m, g_n) -> np.ndarray:
    lib = _load()
    out = np.empty((M, N, Kt, Kh, Kw), dtype=np.float32)
    tiles = packed["tiles"]
    lib.oracle_unpack_kgs(_ptr(packed["group_ptr"], _i32p), _ptr(packed["pos_idx"], _u16p),
                          ctypes.c_void_p(tiles.ctypes.data), M, N, Kt, Kh, Kw, g_m, g_n,
                          int(tiles.dtype == np.uint16), _ptr(out, _f32p))
    return out


def maxpool3d(x, k, stride, pad=(0, 0, 0)) -> np.ndarray:
    lib = _load()
    x = _f32(x)
    n, t, h, ww, c = x.shape
    ext = [(d + 2 * p - kk) // s + 1 for d, p, kk, s in zip((t, h, ww), pad, k, stride)]
    y = np.empty((n, ext[0], ext[1], ext[2], c), dtype=np.float32)
    rc = lib.oracle_maxpool3d(_ptr(x, _f32p), n, t, h, ww, c, *map(int, k), *map(int, stride),
                              *map(int, pad), _ptr(y, _f32p))
    if rc != 0:
        raise ValueError("oracle_maxpool3d: bad arguments")
    return y


def add_relu(a, b, relu=True) -> np.ndarray:
    lib = _load()
    a, b = _f32(a), _f32(b)
    assert a.shape == b.shape
    y = np.empty_like(a)
    lib.oracle_add_relu(_ptr(a, _f32p), _ptr(b, _f32p), ctypes.c_int64(a.size), int(relu), _ptr(y, _f32p))
    return y


def group_norms(w, g_m: int, g_n: int, g: int = 2) -> np.ndarray:
    """Group-lasso norm per (kernel group, kernel location): float32 [P, Q, Ks]; g = 1 or 2."""
    lib = _load()
    w = _f32(w)
    M, N = w.shape[:2]
    Ks = int(np.prod(w.shape[2:]))
    P, Q = -(-M // g_m), -(-N // g_n)
    out = np.empty((P, Q, Ks), dtype=np.float32)
    rc = lib.oracle_group_norms(_ptr(w, _f32p), M, N, Ks, int(g_m), int(g_n), int(g), _ptr(out, _f32p))
    if rc != 0:
        raise ValueError("oracle_group_norms: bad arguments")
    return out


def reweight(norms, eps: float, threshold: float):
    """(penalty = 1/(norm^2 + eps) as float32, keep = norm > threshold as uint8), same shape as norms."""
    lib = _load()
    norms = _f32(norms)
    pen = np.empty_like(norms)
    keep = np.empty(norms.shape, dtype=np.uint8)
    lib.oracle_reweight(_ptr(norms, _f32p), ctypes.c_int64(norms.size), ctypes.c_float(eps), ctypes.c_float(threshold),
                        _ptr(pen, _f32p), _ptr(keep, _u8p))
    return pen, keep
