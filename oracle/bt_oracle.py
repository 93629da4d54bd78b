"""ctypes front end of the plain-C oracle (bt_oracle.c). TEST INFRASTRUCTURE ONLY.

The arithmetic lives in bt_oracle.c; this file only builds it with gcc, allocates
numpy output arrays and passes pointers.  It imports nothing from the CUDA
package.  Element kinds: "f32", "f16", "bf16", "f64" (2-byte kinds are carried
as uint16 arrays, since numpy has no bfloat16).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import NamedTuple, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bt_oracle.c")
_LIB = os.path.join(_HERE, "libbt_oracle.so")

CHUNK = 4096
KINDS = {"f32": 0, "f16": 1, "bf16": 2, "f64": 3}
ELEM_SIZE = {"f32": 4, "f16": 2, "bf16": 2, "f64": 8}
_UINT = {2: np.uint16, 4: np.uint32, 8: np.uint64}


def build(force: bool = False) -> str:
    """Compile bt_oracle.c into a shared object next to it (gcc, -O2)."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
             or os.path.getmtime(_LIB) < os.path.getmtime(os.path.join(_HERE, "bt_oracle.h")))
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, vp, i32 = ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int
        L.oracle_elem_size.restype = i32
        L.oracle_elem_size.argtypes = [i32]
        L.oracle_compress.restype = u64
        L.oracle_compress.argtypes = [vp, u64, i32, vp, vp, vp]
        L.oracle_decompress.restype = None
        L.oracle_decompress.argtypes = [vp, vp, u64, i32, vp]
        L.oracle_decompress_chunked.restype = None
        L.oracle_decompress_chunked.argtypes = [vp, vp, vp, u64, i32, vp]
        L.oracle_relu_fwd_compress.restype = u64
        L.oracle_relu_fwd_compress.argtypes = [vp, u64, i32, vp, vp, vp, vp]
        L.oracle_prune_fwd_compress.restype = u64
        L.oracle_prune_fwd_compress.argtypes = [vp, u64, i32, ctypes.c_float, vp, vp, vp, vp]
        L.oracle_mask_compress.restype = u64
        L.oracle_mask_compress.argtypes = [vp, u64, i32, vp, vp, vp]
        L.oracle_relu6_fwd_compress.restype = u64
        L.oracle_relu6_fwd_compress.argtypes = [vp, u64, i32, vp, vp, vp, vp]
        L.oracle_relu6_bwd_from_stash.restype = None
        L.oracle_relu6_bwd_from_stash.argtypes = [vp, vp, u64, i32, vp, vp]
        L.oracle_relu_bwd_from_bitmap.restype = None
        L.oracle_relu_bwd_from_bitmap.argtypes = [vp, vp, u64, i32, vp]
        L.oracle_compressed_bytes.restype = u64
        L.oracle_compressed_bytes.argtypes = [u64, u64, i32]
        L.oracle_narrow_compress.restype = u64
        L.oracle_narrow_compress.argtypes = [vp, u64, i32, i32, ctypes.c_float, vp, vp, vp, vp]
        L.oracle_maxpool2x2_fwd.restype = None
        L.oracle_maxpool2x2_fwd.argtypes = [vp, u64, u64, u64, i32, vp, vp]
        L.oracle_maxpool2x2_bwd.restype = None
        L.oracle_maxpool2x2_bwd.argtypes = [vp, vp, u64, u64, u64, i32, vp]
        L.oracle_widen_decompress.restype = None
        L.oracle_widen_decompress.argtypes = [vp, vp, u64, i32, vp]
        L.oracle_float_to_half.restype = ctypes.c_uint16
        L.oracle_float_to_half.argtypes = [ctypes.c_uint32]
        L.oracle_float_to_bfloat16.restype = ctypes.c_uint16
        L.oracle_float_to_bfloat16.argtypes = [ctypes.c_uint32]
        L.oracle_half_to_float.restype = ctypes.c_float
        L.oracle_half_to_float.argtypes = [ctypes.c_uint16]
        _lib = L
    return _lib


class Compressed(NamedTuple):
    bitmap: np.ndarray   # uint32[ceil(n/32)]
    values: np.ndarray   # raw unsigned patterns, length nnz
    prefix: np.ndarray   # uint64[ceil(n/4096)]
    nnz: int
    n: int


def _raw(a: np.ndarray) -> np.ndarray:
    """Flat, contiguous view of `a` as unsigned integers of the same width."""
    a = np.ascontiguousarray(a).reshape(-1)
    return a.view(_UINT[a.dtype.itemsize])


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def compress(dense: np.ndarray) -> Compressed:
    x = _raw(dense)
    n, es = x.size, x.dtype.itemsize
    bitmap = np.full((n + 31) // 32, 0xDEADBEEF, dtype=np.uint32)
    values = np.empty(n, dtype=x.dtype)
    prefix = np.full((n + CHUNK - 1) // CHUNK, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)
    nnz = int(lib().oracle_compress(_ptr(x), n, es, _ptr(bitmap), _ptr(values), _ptr(prefix)))
    return Compressed(bitmap, values[:nnz].copy(), prefix, nnz, n)


def decompress(c: Compressed, chunked: bool = False) -> np.ndarray:
    es = c.values.dtype.itemsize
    out = np.full(c.n, 0xA5, dtype=np.uint8).repeat(es).view(c.values.dtype)
    vals = np.ascontiguousarray(c.values)
    if chunked:
        lib().oracle_decompress_chunked(_ptr(c.bitmap), _ptr(vals), _ptr(c.prefix), c.n, es, _ptr(out))
    else:
        lib().oracle_decompress(_ptr(c.bitmap), _ptr(vals), c.n, es, _ptr(out))
    return out


def relu_fwd_compress(pre_act: np.ndarray, kind: str, want_y: bool = True):
    """Returns (y or None, Compressed).  `pre_act` holds raw patterns of `kind`."""
    x = _raw(pre_act)
    assert x.dtype.itemsize == ELEM_SIZE[kind]
    n = x.size
    y = np.empty(n, dtype=x.dtype) if want_y else None
    bitmap = np.full((n + 31) // 32, 0xDEADBEEF, dtype=np.uint32)
    values = np.empty(n, dtype=x.dtype)
    prefix = np.full((n + CHUNK - 1) // CHUNK, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)
    nnz = int(lib().oracle_relu_fwd_compress(_ptr(x), n, KINDS[kind], _ptr(y), _ptr(bitmap),
                                              _ptr(values), _ptr(prefix)))
    return y, Compressed(bitmap, values[:nnz].copy(), prefix, nnz, n)


def prune_fwd_compress(x: np.ndarray, kind: str, tau: float, want_y: bool = True):
    """Activation pruning with threshold `tau` (a binary32 value) joined to the stash.
    Returns (y or None, Compressed).  `x` holds raw patterns of `kind`."""
    xr = _raw(x)
    assert xr.dtype.itemsize == ELEM_SIZE[kind]
    n = xr.size
    y = np.empty(n, dtype=xr.dtype) if want_y else None
    bitmap = np.full((n + 31) // 32, 0xDEADBEEF, dtype=np.uint32)
    values = np.empty(n, dtype=xr.dtype)
    prefix = np.full((n + CHUNK - 1) // CHUNK, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)
    nnz = int(lib().oracle_prune_fwd_compress(_ptr(xr), n, KINDS[kind], ctypes.c_float(tau), _ptr(y), _ptr(bitmap),
                                               _ptr(values), _ptr(prefix)))
    return y, Compressed(bitmap, values[:nnz].copy(), prefix, nnz, n)


def mask_compress(x: np.ndarray, mask_bitmap: np.ndarray, want_y: bool = True):
    """Double-mask form: returns (y or None, values) for raw patterns `x` under `mask_bitmap`."""
    xr = _raw(x)
    n = xr.size
    bm = np.ascontiguousarray(mask_bitmap, dtype=np.uint32)
    assert bm.size >= (n + 31) // 32
    y = np.empty(n, dtype=xr.dtype) if want_y else None
    values = np.empty(n, dtype=xr.dtype)
    cnt = int(lib().oracle_mask_compress(_ptr(xr), n, xr.dtype.itemsize, _ptr(bm), _ptr(y), _ptr(values)))
    return y, values[:cnt].copy()


def relu6_fwd_compress(pre_act: np.ndarray, kind: str, want_y: bool = True):
    """ReLU6 joined to the stash.  Returns (y or None, Compressed)."""
    x = _raw(pre_act)
    assert x.dtype.itemsize == ELEM_SIZE[kind]
    n = x.size
    y = np.empty(n, dtype=x.dtype) if want_y else None
    bitmap = np.full((n + 31) // 32, 0xDEADBEEF, dtype=np.uint32)
    values = np.empty(n, dtype=x.dtype)
    prefix = np.full((n + CHUNK - 1) // CHUNK, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)
    nnz = int(lib().oracle_relu6_fwd_compress(_ptr(x), n, KINDS[kind], _ptr(y), _ptr(bitmap), _ptr(values),
                                               _ptr(prefix)))
    return y, Compressed(bitmap, values[:nnz].copy(), prefix, nnz, n)


def relu6_bwd_from_stash(c: Compressed, kind: str, grad_out: np.ndarray) -> np.ndarray:
    g = _raw(grad_out)
    assert g.size == c.n and g.dtype.itemsize == ELEM_SIZE[kind]
    out = np.empty_like(g)
    bm = np.ascontiguousarray(c.bitmap, dtype=np.uint32)
    vals = np.ascontiguousarray(c.values)
    lib().oracle_relu6_bwd_from_stash(_ptr(bm), _ptr(vals), c.n, KINDS[kind], _ptr(g), _ptr(out))
    return out


def relu_bwd_from_bitmap(bitmap: np.ndarray, grad_out: np.ndarray) -> np.ndarray:
    g = _raw(grad_out)
    out = np.empty_like(g)
    bm = np.ascontiguousarray(bitmap, dtype=np.uint32)
    lib().oracle_relu_bwd_from_bitmap(_ptr(bm), _ptr(g), g.size, g.dtype.itemsize, _ptr(out))
    return out


def narrow_compress(x: np.ndarray, to_kind: str, fused: bool = False, tau: float = 0.0, want_y: bool = False):
    """Down-cast on stash: `x` holds binary32 patterns; the stashed values are `to_kind` ("f16" / "bf16")
    patterns.  Returns (y or None, Compressed) with `values` of dtype uint16."""
    x = _raw(x)
    assert x.dtype.itemsize == 4 and to_kind in ("f16", "bf16")
    n = x.size
    y = np.empty(n, dtype=x.dtype) if want_y else None
    bitmap = np.full((n + 31) // 32, 0xDEADBEEF, dtype=np.uint32)
    values = np.empty(n, dtype=np.uint16)
    prefix = np.full((n + CHUNK - 1) // CHUNK, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)
    nnz = int(lib().oracle_narrow_compress(_ptr(x), n, KINDS[to_kind], int(fused), float(np.float32(tau)), _ptr(y),
                                            _ptr(bitmap), _ptr(values), _ptr(prefix)))
    return y, Compressed(bitmap, values[:nnz].copy(), prefix, nnz, n)


def maxpool2x2_fwd(x: np.ndarray, planes: int, height: int, width: int, kind: str):
    """Returns (y, codes): the pooled raw patterns (planes * height/2 * width/2) and the 2-bit winner codes."""
    x = _raw(x)
    assert x.size == planes * height * width and height % 2 == 0 and width % 2 == 0
    outputs = planes * (height // 2) * (width // 2)
    y = np.empty(outputs, dtype=x.dtype)
    codes = np.full((outputs + 15) // 16, 0xDEADBEEF, dtype=np.uint32)
    lib().oracle_maxpool2x2_fwd(_ptr(x), planes, height, width, KINDS[kind], _ptr(y), _ptr(codes))
    return y, codes


def maxpool2x2_bwd(codes: np.ndarray, grad_out: np.ndarray, planes: int, height: int, width: int) -> np.ndarray:
    g = _raw(grad_out)
    gin = np.empty(planes * height * width, dtype=g.dtype)
    lib().oracle_maxpool2x2_bwd(_ptr(codes), _ptr(g), planes, height, width, g.dtype.itemsize, _ptr(gin))
    return gin


def widen_decompress(c: Compressed, from_kind: str) -> np.ndarray:
    """The binary32 tensor (raw uint32 patterns) a narrowed stash restores to."""
    assert c.values.dtype == np.uint16 and from_kind in ("f16", "bf16")
    out = np.full(c.n, 0xDEADBEEF, dtype=np.uint32)
    vals = np.ascontiguousarray(c.values) if c.values.size else np.zeros(1, np.uint16)
    lib().oracle_widen_decompress(_ptr(c.bitmap), _ptr(vals), c.n, KINDS[from_kind], _ptr(out))
    return out


def float_to_half(bits: int) -> int:
    return int(lib().oracle_float_to_half(bits))


def float_to_bfloat16(bits: int) -> int:
    return int(lib().oracle_float_to_bfloat16(bits))


def compressed_bytes(n: int, nnz: int, elem_size: int) -> int:
    return int(lib().oracle_compressed_bytes(n, nnz, elem_size))


def half_to_float(h: int) -> float:
    return float(lib().oracle_half_to_float(h))
