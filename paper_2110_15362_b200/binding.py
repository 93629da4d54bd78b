"""Thin ctypes binding of libbittrain.so: same names as the C ABI, argument
marshalling only.  Every step of the codec runs in the library's CUDA kernels;
there is no fallback: if the shared object is missing this module raises.

Tensors are torch CUDA tensors (device memory and streams are torch's); the
functions pass their data pointers, the element count and the current stream.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

BT_F32, BT_F16, BT_BF16, BT_F64 = 0, 1, 2, 3
(BT_OK, BT_ERR_NULL, BT_ERR_DTYPE, BT_ERR_ALIGN, BT_ERR_WORKSPACE, BT_ERR_CAPACITY, BT_ERR_TIMEOUT, BT_ERR_CUDA,
 BT_ERR_TOO_LARGE, BT_ERR_SHAPE) = range(10)
STATUS_NAMES = ["BT_OK", "BT_ERR_NULL", "BT_ERR_DTYPE", "BT_ERR_ALIGN", "BT_ERR_WORKSPACE", "BT_ERR_CAPACITY",
                "BT_ERR_TIMEOUT", "BT_ERR_CUDA", "BT_ERR_TOO_LARGE", "BT_ERR_SHAPE"]
NOALLOC_MAX_ELEMS = 1 << 26
CHUNK = 4096

DTYPE_CODE = {torch.float32: BT_F32, torch.float16: BT_F16, torch.bfloat16: BT_BF16, torch.float64: BT_F64}
EXPORTS = ("bt_compressed_bytes", "bt_workspace_bytes", "bt_compress", "bt_decompress",
           "bt_relu_fwd_compress", "bt_relu_bwd_from_bitmap", "bt_host_staging_bytes", "bt_compress_host",
           "bt_decompress_host", "bt_relu_fwd_compress_host", "bt_relu_bwd_from_bitmap_host", "bt_compress_noalloc",
           "bt_prune_fwd_compress", "bt_mask_compress", "bt_compress_arena", "bt_prune_fwd_compress_arena",
           "bt_decompress_arena", "bt_relu6_fwd_compress", "bt_relu6_bwd_from_stash", "bt_compress_narrow",
           "bt_prune_fwd_compress_narrow", "bt_decompress_widen", "bt_maxpool2x2_fwd", "bt_maxpool2x2_bwd",
           "bt_compress_narrow_arena", "bt_prune_fwd_compress_narrow_arena", "bt_decompress_widen_arena",
           "bt_relu6_fwd_compress_arena", "bt_relu6_bwd_from_stash_arena", "bt_maxpool2x2_bwd_masked", "bt_set_max_ctas",
           "bt_batch_workspace_bytes", "bt_compress_batch", "bt_relu_fwd_compress_batch", "bt_decompress_batch",
           "bt_relu_bwd_from_bitmap_batch", "bt_compress_arena_batch", "bt_relu_fwd_compress_arena_batch",
           "bt_decompress_arena_batch")

MAX_BATCH_PER_LAUNCH = 32


class BatchItem(ctypes.Structure):
    """bt_batch_item of the C ABI: one tensor of a batched call (device pointers as integers)."""
    _fields_ = [("dense", ctypes.c_void_p), ("y_out", ctypes.c_void_p), ("bitmap", ctypes.c_void_p),
                ("values", ctypes.c_void_p), ("values_capacity", ctypes.c_uint64), ("chunk_prefix", ctypes.c_void_p),
                ("nnz_out", ctypes.c_void_p), ("dev_status", ctypes.c_void_p), ("n", ctypes.c_uint64)]


_lib: Optional[ctypes.CDLL] = None


class BitTrainError(RuntimeError):
    def __init__(self, call: str, status: int):
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{call} returned {name}")
        self.status = status


def library_path() -> str:
    return _build.LIB_PATH


def lib() -> ctypes.CDLL:
    """Load libbittrain.so (built in-tree by build.build_library()).  No fallback."""
    global _lib
    if _lib is None:
        _lib = load_library(library_path())
    return _lib


def load_library(path: str) -> ctypes.CDLL:
    """Open a build of the library and declare the C ABI's signatures on it."""
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with "
                          "`python -m paper_2110_15362_b200.build` (needs nvcc); there is no CPU fallback")
    L = ctypes.CDLL(path)
    u64, vp, i32, sz = ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.bt_compressed_bytes.restype = sz
    L.bt_compressed_bytes.argtypes = [u64, u64, i32]
    L.bt_set_max_ctas.restype = i32
    L.bt_set_max_ctas.argtypes = [i32]
    L.bt_workspace_bytes.restype = sz
    L.bt_workspace_bytes.argtypes = [u64]
    L.bt_compress.restype = i32
    L.bt_compress.argtypes = [vp, u64, i32, vp, vp, u64, vp, vp, vp, sz, vp, vp]
    L.bt_batch_workspace_bytes.restype = sz
    L.bt_batch_workspace_bytes.argtypes = [ctypes.POINTER(u64), ctypes.c_uint32]
    for name in ("bt_compress_batch", "bt_relu_fwd_compress_batch"):
        getattr(L, name).restype = i32
        getattr(L, name).argtypes = [ctypes.POINTER(BatchItem), ctypes.c_uint32, i32, vp, sz, vp]
    for name in ("bt_decompress_batch", "bt_relu_bwd_from_bitmap_batch"):
        getattr(L, name).restype = i32
        getattr(L, name).argtypes = [ctypes.POINTER(BatchItem), ctypes.c_uint32, i32, vp]
    for name in ("bt_compress_arena_batch", "bt_relu_fwd_compress_arena_batch"):
        getattr(L, name).restype = i32
        getattr(L, name).argtypes = [ctypes.POINTER(BatchItem), ctypes.c_uint32, i32, vp, u64, vp, vp, vp, sz, vp]
    L.bt_decompress_arena_batch.restype = i32
    L.bt_decompress_arena_batch.argtypes = [ctypes.POINTER(BatchItem), ctypes.c_uint32, i32, vp, vp, vp]
    L.bt_decompress.restype = i32
    L.bt_decompress.argtypes = [vp, vp, vp, u64, i32, vp, vp]
    L.bt_relu_fwd_compress.restype = i32
    L.bt_relu_fwd_compress.argtypes = [vp, u64, i32, vp, vp, vp, u64, vp, vp, vp, sz, vp, vp]
    L.bt_relu_bwd_from_bitmap.restype = i32
    L.bt_relu_bwd_from_bitmap.argtypes = [vp, vp, u64, i32, vp, vp]
    L.bt_prune_fwd_compress.argtypes = [vp, u64, i32, ctypes.c_float, vp, vp, vp, u64, vp, vp, vp, sz, vp, vp]
    L.bt_prune_fwd_compress.restype = i32
    L.bt_mask_compress.argtypes = [vp, u64, i32, vp, vp, vp, vp, u64, vp]
    L.bt_mask_compress.restype = i32
    L.bt_compress_arena.argtypes = [vp, u64, i32, vp, vp, u64, vp, vp, vp, vp, vp, sz, vp, vp]
    L.bt_compress_arena.restype = i32
    L.bt_prune_fwd_compress_arena.argtypes = [vp, u64, i32, ctypes.c_float, vp, vp, vp, u64, vp, vp, vp, vp, vp, sz, vp, vp]
    L.bt_prune_fwd_compress_arena.restype = i32
    L.bt_decompress_arena.argtypes = [vp, vp, vp, vp, u64, i32, vp, vp]
    L.bt_decompress_arena.restype = i32
    L.bt_relu6_fwd_compress.argtypes = [vp, u64, i32, vp, vp, vp, u64, vp, vp, vp, sz, vp, vp]
    L.bt_relu6_fwd_compress.restype = i32
    L.bt_relu6_bwd_from_stash.argtypes = [vp, vp, vp, vp, u64, i32, vp, vp]
    L.bt_relu6_bwd_from_stash.restype = i32
    L.bt_compress_narrow.argtypes = [vp, u64, i32, vp, vp, u64, vp, vp, vp, sz, vp, vp]
    L.bt_compress_narrow.restype = i32
    L.bt_prune_fwd_compress_narrow.argtypes = [vp, u64, i32, ctypes.c_float, vp, vp, vp, u64, vp, vp, vp, sz, vp, vp]
    L.bt_prune_fwd_compress_narrow.restype = i32
    L.bt_decompress_widen.argtypes = [vp, vp, vp, u64, i32, vp, vp]
    L.bt_decompress_widen.restype = i32
    L.bt_maxpool2x2_fwd.argtypes = [vp, u64, u64, u64, i32, vp, vp, vp]
    L.bt_maxpool2x2_fwd.restype = i32
    L.bt_maxpool2x2_bwd.argtypes = [vp, vp, u64, u64, u64, i32, vp, vp]
    L.bt_maxpool2x2_bwd.restype = i32
    L.bt_maxpool2x2_bwd_masked.argtypes = [vp, vp, vp, u64, u64, u64, i32, vp, vp]
    L.bt_maxpool2x2_bwd_masked.restype = i32
    L.bt_compress_narrow_arena.argtypes = [vp, u64, i32, vp, vp, u64, vp, vp, vp, vp, vp, sz, vp, vp]
    L.bt_compress_narrow_arena.restype = i32
    L.bt_prune_fwd_compress_narrow_arena.argtypes = [vp, u64, i32, ctypes.c_float, vp, vp, vp, u64, vp, vp, vp, vp, vp, sz,
                                                     vp, vp]
    L.bt_prune_fwd_compress_narrow_arena.restype = i32
    L.bt_decompress_widen_arena.argtypes = [vp, vp, vp, vp, u64, i32, vp, vp]
    L.bt_decompress_widen_arena.restype = i32
    L.bt_relu6_fwd_compress_arena.argtypes = [vp, u64, i32, vp, vp, vp, u64, vp, vp, vp, vp, vp, sz, vp, vp]
    L.bt_relu6_fwd_compress_arena.restype = i32
    L.bt_relu6_bwd_from_stash_arena.argtypes = [vp, vp, vp, vp, vp, u64, i32, vp, vp]
    L.bt_relu6_bwd_from_stash_arena.restype = i32
    L.bt_compress_noalloc.restype = i32
    L.bt_compress_noalloc.argtypes = [vp, u64, i32, vp, vp, u64, vp, vp, vp, vp]
    L.bt_host_staging_bytes.restype = sz
    L.bt_host_staging_bytes.argtypes = [u64, i32]
    L.bt_compress_host.restype = i32
    L.bt_compress_host.argtypes = [vp, u64, i32, vp, vp, u64, vp, vp, vp, sz, vp]
    L.bt_decompress_host.restype = i32
    L.bt_decompress_host.argtypes = [vp, vp, vp, u64, u64, i32, vp, vp, sz, vp]
    L.bt_relu_fwd_compress_host.restype = i32
    L.bt_relu_fwd_compress_host.argtypes = [vp, u64, i32, vp, vp, vp, u64, vp, vp, vp, sz, vp]
    L.bt_relu_bwd_from_bitmap_host.restype = i32
    L.bt_relu_bwd_from_bitmap_host.argtypes = [vp, vp, u64, i32, vp, vp, sz, vp]
    return L


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(call: str, status: int, check: bool) -> int:
    if check and status != BT_OK:
        raise BitTrainError(call, status)
    return status


def bt_compressed_bytes(n: int, nnz: int, dtype) -> int:
    code = DTYPE_CODE.get(dtype, dtype)
    return int(lib().bt_compressed_bytes(n, nnz, code))


def bt_workspace_bytes(n: int) -> int:
    return int(lib().bt_workspace_bytes(n))


def bt_compress(dense: torch.Tensor, bitmap: torch.Tensor, values: torch.Tensor, chunk_prefix: torch.Tensor,
                nnz_out: torch.Tensor, workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                *, n: Optional[int] = None, values_capacity: Optional[int] = None, stream=None,
                check: bool = True) -> int:
    n = dense.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    st = lib().bt_compress(_ptr(dense), n, DTYPE_CODE[dense.dtype], _ptr(bitmap), _ptr(values), cap,
                           _ptr(chunk_prefix), _ptr(nnz_out), _ptr(workspace),
                           workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream))
    return _check("bt_compress", st, check)


def bt_batch_workspace_bytes(ns) -> int:
    """Bytes of workspace a batched call over tensors of these element counts needs."""
    arr = (ctypes.c_uint64 * len(ns))(*[int(v) for v in ns])
    return int(lib().bt_batch_workspace_bytes(arr, len(ns)))


def batch_items(dense, stashes, y_out=None) -> "ctypes.Array":
    """The host array of bt_batch_item for tensors `dense[k]` stashed into `stashes[k]` (Stash objects), with the
    dense outputs `y_out[k]` if given.  Marshalling only: built once, it can be passed to many calls."""
    items = (BatchItem * len(dense))()
    for k, (x, st) in enumerate(zip(dense, stashes)):
        items[k] = BatchItem(_ptr(x), _ptr(y_out[k]) if y_out is not None else None, _ptr(st.bitmap), _ptr(st.values),
                             st.values.numel(), _ptr(st.chunk_prefix), _ptr(st.nnz_out), _ptr(st.dev_status), x.numel())
    return items


def bt_compress_batch(items, dtype: torch.dtype, workspace: torch.Tensor, *, stream=None, check: bool = True) -> int:
    """bt_compress of every tensor of `items` (from batch_items) in one pass."""
    st = lib().bt_compress_batch(items, len(items), DTYPE_CODE[dtype], _ptr(workspace), _nbytes(workspace), _stream(stream))
    return _check("bt_compress_batch", st, check)


def bt_relu_fwd_compress_batch(items, dtype: torch.dtype, workspace: torch.Tensor, *, stream=None,
                               check: bool = True) -> int:
    """bt_relu_fwd_compress of every tensor of `items` (from batch_items) in one pass."""
    st = lib().bt_relu_fwd_compress_batch(items, len(items), DTYPE_CODE[dtype], _ptr(workspace), _nbytes(workspace),
                                          _stream(stream))
    return _check("bt_relu_fwd_compress_batch", st, check)


def bt_compress_arena_batch(items, dtype: torch.dtype, arena: torch.Tensor, arena_cursor: torch.Tensor,
                            values_offsets_out: torch.Tensor, workspace: torch.Tensor, *, fused: bool = False, stream=None,
                            check: bool = True) -> int:
    """The tensors of `items` pushed into the arena back to back by one pass (fused: ReLU forward first);
    values_offsets_out is a device int64 tensor with one word per item."""
    fn = lib().bt_relu_fwd_compress_arena_batch if fused else lib().bt_compress_arena_batch
    st = fn(items, len(items), DTYPE_CODE[dtype], _ptr(arena), _nbytes(arena), _ptr(arena_cursor), _ptr(values_offsets_out),
            _ptr(workspace), _nbytes(workspace), _stream(stream))
    return _check("bt_compress_arena_batch", st, check)


def bt_decompress_arena_batch(items, dtype: torch.dtype, arena: torch.Tensor, values_offsets: torch.Tensor, *, stream=None,
                              check: bool = True) -> int:
    """Every item's y_out restored from (bitmap, arena + values_offsets[k], chunk_prefix) in one pass."""
    st = lib().bt_decompress_arena_batch(items, len(items), DTYPE_CODE[dtype], _ptr(arena), _ptr(values_offsets), _stream(stream))
    return _check("bt_decompress_arena_batch", st, check)


def bt_decompress_batch(items, dtype: torch.dtype, *, stream=None, check: bool = True) -> int:
    """bt_decompress of every stash of `items` into its y_out, in one pass."""
    st = lib().bt_decompress_batch(items, len(items), DTYPE_CODE[dtype], _stream(stream))
    return _check("bt_decompress_batch", st, check)


def bt_relu_bwd_from_bitmap_batch(items, dtype: torch.dtype, *, stream=None, check: bool = True) -> int:
    """bt_relu_bwd_from_bitmap of every item (dense: upstream gradient, y_out: input gradient), in one pass."""
    st = lib().bt_relu_bwd_from_bitmap_batch(items, len(items), DTYPE_CODE[dtype], _stream(stream))
    return _check("bt_relu_bwd_from_bitmap_batch", st, check)


def bt_compress_noalloc(dense: torch.Tensor, bitmap: torch.Tensor, values: torch.Tensor, chunk_prefix: torch.Tensor,
                        nnz_out: torch.Tensor, dev_status: Optional[torch.Tensor] = None, *, n: Optional[int] = None,
                        values_capacity: Optional[int] = None, stream=None, check: bool = True) -> int:
    """bt_compress without a workspace argument: the scratch is a fixed array inside the library, so the
    call allocates nothing (for callers that may not); n is limited to NOALLOC_MAX_ELEMS."""
    n = dense.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    st = lib().bt_compress_noalloc(_ptr(dense), n, DTYPE_CODE[dense.dtype], _ptr(bitmap), _ptr(values), cap,
                                   _ptr(chunk_prefix), _ptr(nnz_out), _ptr(dev_status), _stream(stream))
    return _check("bt_compress_noalloc", st, check)


def bt_relu_fwd_compress(pre_act: torch.Tensor, y_out: Optional[torch.Tensor], bitmap: torch.Tensor,
                         values: torch.Tensor, chunk_prefix: torch.Tensor, nnz_out: torch.Tensor,
                         workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                         *, n: Optional[int] = None, values_capacity: Optional[int] = None, stream=None,
                         check: bool = True) -> int:
    n = pre_act.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    st = lib().bt_relu_fwd_compress(_ptr(pre_act), n, DTYPE_CODE[pre_act.dtype], _ptr(y_out), _ptr(bitmap),
                                    _ptr(values), cap, _ptr(chunk_prefix), _ptr(nnz_out), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _ptr(dev_status),
                                    _stream(stream))
    return _check("bt_relu_fwd_compress", st, check)



def bt_prune_fwd_compress(x: torch.Tensor, tau: float, y_out: Optional[torch.Tensor], bitmap: torch.Tensor,
                          values: torch.Tensor, chunk_prefix: torch.Tensor, nnz_out: torch.Tensor,
                          workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                          *, n: Optional[int] = None, values_capacity: Optional[int] = None, stream=None,
                          check: bool = True) -> int:
    """Activation pruning fused with the stash: elements <= tau (a binary32 threshold) become +0."""
    n = x.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    st = lib().bt_prune_fwd_compress(_ptr(x), n, DTYPE_CODE[x.dtype], ctypes.c_float(tau), _ptr(y_out), _ptr(bitmap),
                                     _ptr(values), cap, _ptr(chunk_prefix), _ptr(nnz_out), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _ptr(dev_status),
                                     _stream(stream))
    return _check("bt_prune_fwd_compress", st, check)

def bt_set_max_ctas(max_ctas: int) -> int:
    """Limits the CTAs of every later compress-family launch of the calling thread (0: no limit); returns the limit
    it replaces."""
    prev = lib().bt_set_max_ctas(int(max_ctas))
    if prev < 0:
        raise ValueError("bt_set_max_ctas: the limit must not be negative")
    return prev


def bt_compress_narrow(dense: torch.Tensor, bitmap: torch.Tensor, values: torch.Tensor, chunk_prefix: torch.Tensor,
                       nnz_out: torch.Tensor, workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                       *, n: Optional[int] = None, values_capacity: Optional[int] = None, stream=None,
                       check: bool = True) -> int:
    """Down-cast on stash: a float32 tensor whose stashed values take the (16-bit) dtype of `values`."""
    n = dense.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    assert dense.dtype == torch.float32
    st = lib().bt_compress_narrow(_ptr(dense), n, DTYPE_CODE[values.dtype], _ptr(bitmap), _ptr(values), cap,
                                  _ptr(chunk_prefix), _ptr(nnz_out), _ptr(workspace), _nbytes(workspace),
                                  _ptr(dev_status), _stream(stream))
    return _check("bt_compress_narrow", st, check)


def bt_prune_fwd_compress_narrow(x: torch.Tensor, tau: float, y_out: Optional[torch.Tensor], bitmap: torch.Tensor,
                                 values: torch.Tensor, chunk_prefix: torch.Tensor, nnz_out: torch.Tensor,
                                 workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                                 *, n: Optional[int] = None, values_capacity: Optional[int] = None, stream=None,
                                 check: bool = True) -> int:
    """Fused forward (tau = 0: ReLU) of a float32 tensor whose stashed values take the 16-bit dtype of `values`."""
    n = x.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    assert x.dtype == torch.float32
    st = lib().bt_prune_fwd_compress_narrow(_ptr(x), n, DTYPE_CODE[values.dtype], ctypes.c_float(tau), _ptr(y_out),
                                            _ptr(bitmap), _ptr(values), cap, _ptr(chunk_prefix), _ptr(nnz_out),
                                            _ptr(workspace), _nbytes(workspace), _ptr(dev_status), _stream(stream))
    return _check("bt_prune_fwd_compress_narrow", st, check)


def bt_decompress_widen(bitmap: torch.Tensor, values: torch.Tensor, chunk_prefix: torch.Tensor, dense_out: torch.Tensor,
                        *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    """Restores a narrowed stash (16-bit `values`) into a float32 tensor."""
    n = dense_out.numel() if n is None else n
    assert dense_out.dtype == torch.float32
    st = lib().bt_decompress_widen(_ptr(bitmap), _ptr(values), _ptr(chunk_prefix), n, DTYPE_CODE[values.dtype],
                                   _ptr(dense_out), _stream(stream))
    return _check("bt_decompress_widen", st, check)


def bt_maxpool2x2_fwd(x: torch.Tensor, y: torch.Tensor, codes: Optional[torch.Tensor], *, planes: Optional[int] = None,
                      height: Optional[int] = None, width: Optional[int] = None, stream=None, check: bool = True) -> int:
    """2x2 / stride 2 max pooling of a contiguous (..., H, W) tensor into y, with 2-bit winner codes (int32 words,
    ceil(outputs / 16) of them) if `codes` is given."""
    height = x.shape[-2] if height is None else height
    width = x.shape[-1] if width is None else width
    planes = x.numel() // max(1, height * width) if planes is None else planes
    st = lib().bt_maxpool2x2_fwd(_ptr(x), planes, height, width, DTYPE_CODE[x.dtype], _ptr(y), _ptr(codes), _stream(stream))
    return _check("bt_maxpool2x2_fwd", st, check)


def bt_maxpool2x2_bwd(codes: torch.Tensor, grad_out: torch.Tensor, grad_in: torch.Tensor, *, planes: Optional[int] = None,
                      height: Optional[int] = None, width: Optional[int] = None, stream=None, check: bool = True) -> int:
    """The pooling's backward pass from the codes alone; grad_in has the (..., H, W) shape of the pooled tensor's input."""
    height = grad_in.shape[-2] if height is None else height
    width = grad_in.shape[-1] if width is None else width
    planes = grad_in.numel() // max(1, height * width) if planes is None else planes
    st = lib().bt_maxpool2x2_bwd(_ptr(codes), _ptr(grad_out), planes, height, width, DTYPE_CODE[grad_out.dtype],
                                 _ptr(grad_in), _stream(stream))
    return _check("bt_maxpool2x2_bwd", st, check)


def bt_maxpool2x2_bwd_masked(codes: torch.Tensor, pooled_bitmap: torch.Tensor, grad_out: torch.Tensor, grad_in: torch.Tensor,
                             *, planes: Optional[int] = None, height: Optional[int] = None, width: Optional[int] = None,
                             stream=None, check: bool = True) -> int:
    """Backward pass of ReLU + pooling done pooling first: the gradient of a pooled output whose bit in
    `pooled_bitmap` is clear counts as zero."""
    height = grad_in.shape[-2] if height is None else height
    width = grad_in.shape[-1] if width is None else width
    planes = grad_in.numel() // max(1, height * width) if planes is None else planes
    st = lib().bt_maxpool2x2_bwd_masked(_ptr(codes), _ptr(pooled_bitmap), _ptr(grad_out), planes, height, width,
                                        DTYPE_CODE[grad_out.dtype], _ptr(grad_in), _stream(stream))
    return _check("bt_maxpool2x2_bwd_masked", st, check)


def bt_mask_compress(x: torch.Tensor, mask_bitmap: torch.Tensor, mask_chunk_prefix: torch.Tensor,
                     y_out: Optional[torch.Tensor], values: torch.Tensor, *, n: Optional[int] = None,
                     values_capacity: Optional[int] = None, stream=None, check: bool = True) -> int:
    """Double-mask form: the values of x at the set bits of an existing stash's bitmap (and the masked dense y)."""
    n = x.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    st = lib().bt_mask_compress(_ptr(x), n, DTYPE_CODE[x.dtype], _ptr(mask_bitmap), _ptr(mask_chunk_prefix),
                                _ptr(y_out), _ptr(values), cap, _stream(stream))
    return _check("bt_mask_compress", st, check)


def bt_compress_arena(dense: torch.Tensor, bitmap: torch.Tensor, arena: torch.Tensor, arena_cursor: torch.Tensor,
                      values_offset_out: torch.Tensor, chunk_prefix: torch.Tensor, nnz_out: torch.Tensor,
                      workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None, *, n: Optional[int] = None,
                      stream=None, check: bool = True) -> int:
    """bt_compress whose values go behind the cursor of a caller-owned arena (a uint8 device tensor)."""
    n = dense.numel() if n is None else n
    st = lib().bt_compress_arena(_ptr(dense), n, DTYPE_CODE[dense.dtype], _ptr(bitmap), _ptr(arena), _nbytes(arena),
                                 _ptr(arena_cursor), _ptr(values_offset_out), _ptr(chunk_prefix), _ptr(nnz_out),
                                 _ptr(workspace), _nbytes(workspace), _ptr(dev_status), _stream(stream))
    return _check("bt_compress_arena", st, check)


def bt_prune_fwd_compress_arena(x: torch.Tensor, tau: float, y_out: Optional[torch.Tensor], bitmap: torch.Tensor,
                                arena: torch.Tensor, arena_cursor: torch.Tensor, values_offset_out: torch.Tensor,
                                chunk_prefix: torch.Tensor, nnz_out: torch.Tensor, workspace: torch.Tensor,
                                dev_status: Optional[torch.Tensor] = None, *, n: Optional[int] = None, stream=None,
                                check: bool = True) -> int:
    """Fused forward (tau = 0: ReLU) whose values go behind the cursor of a caller-owned arena."""
    n = x.numel() if n is None else n
    st = lib().bt_prune_fwd_compress_arena(_ptr(x), n, DTYPE_CODE[x.dtype], ctypes.c_float(tau), _ptr(y_out),
                                           _ptr(bitmap), _ptr(arena), _nbytes(arena), _ptr(arena_cursor),
                                           _ptr(values_offset_out), _ptr(chunk_prefix), _ptr(nnz_out),
                                           _ptr(workspace), _nbytes(workspace), _ptr(dev_status), _stream(stream))
    return _check("bt_prune_fwd_compress_arena", st, check)


def bt_decompress_arena(bitmap: torch.Tensor, arena: torch.Tensor, values_offset: torch.Tensor,
                        chunk_prefix: torch.Tensor, dense_out: torch.Tensor, *, n: Optional[int] = None, stream=None,
                        check: bool = True) -> int:
    n = dense_out.numel() if n is None else n
    st = lib().bt_decompress_arena(_ptr(bitmap), _ptr(arena), _ptr(values_offset), _ptr(chunk_prefix), n,
                                   DTYPE_CODE[dense_out.dtype], _ptr(dense_out), _stream(stream))
    return _check("bt_decompress_arena", st, check)


def bt_compress_narrow_arena(dense: torch.Tensor, to_dtype: torch.dtype, bitmap: torch.Tensor, arena: torch.Tensor,
                             arena_cursor: torch.Tensor, values_offset_out: torch.Tensor, chunk_prefix: torch.Tensor,
                             nnz_out: torch.Tensor, workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                             *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    """bt_compress_narrow whose 16-bit values (of `to_dtype`) go behind the cursor of a caller-owned arena."""
    n = dense.numel() if n is None else n
    assert dense.dtype == torch.float32
    st = lib().bt_compress_narrow_arena(_ptr(dense), n, DTYPE_CODE[to_dtype], _ptr(bitmap), _ptr(arena), _nbytes(arena),
                                        _ptr(arena_cursor), _ptr(values_offset_out), _ptr(chunk_prefix), _ptr(nnz_out),
                                        _ptr(workspace), _nbytes(workspace), _ptr(dev_status), _stream(stream))
    return _check("bt_compress_narrow_arena", st, check)


def bt_prune_fwd_compress_narrow_arena(x: torch.Tensor, to_dtype: torch.dtype, tau: float, y_out: Optional[torch.Tensor],
                                       bitmap: torch.Tensor, arena: torch.Tensor, arena_cursor: torch.Tensor,
                                       values_offset_out: torch.Tensor, chunk_prefix: torch.Tensor, nnz_out: torch.Tensor,
                                       workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                                       *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    """bt_prune_fwd_compress_narrow whose 16-bit values (of `to_dtype`) go behind the cursor of a caller-owned arena."""
    n = x.numel() if n is None else n
    assert x.dtype == torch.float32
    st = lib().bt_prune_fwd_compress_narrow_arena(_ptr(x), n, DTYPE_CODE[to_dtype], ctypes.c_float(tau), _ptr(y_out),
                                                  _ptr(bitmap), _ptr(arena), _nbytes(arena), _ptr(arena_cursor),
                                                  _ptr(values_offset_out), _ptr(chunk_prefix), _ptr(nnz_out),
                                                  _ptr(workspace), _nbytes(workspace), _ptr(dev_status), _stream(stream))
    return _check("bt_prune_fwd_compress_narrow_arena", st, check)


def bt_decompress_widen_arena(bitmap: torch.Tensor, arena: torch.Tensor, values_offset: torch.Tensor,
                              chunk_prefix: torch.Tensor, from_dtype: torch.dtype, dense_out: torch.Tensor,
                              *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    """Restores a narrowed stash whose 16-bit values (of `from_dtype`) sit in an arena into a float32 tensor."""
    n = dense_out.numel() if n is None else n
    assert dense_out.dtype == torch.float32
    st = lib().bt_decompress_widen_arena(_ptr(bitmap), _ptr(arena), _ptr(values_offset), _ptr(chunk_prefix), n,
                                         DTYPE_CODE[from_dtype], _ptr(dense_out), _stream(stream))
    return _check("bt_decompress_widen_arena", st, check)


def bt_relu6_fwd_compress_arena(pre_act: torch.Tensor, y_out: Optional[torch.Tensor], bitmap: torch.Tensor,
                                arena: torch.Tensor, arena_cursor: torch.Tensor, values_offset_out: torch.Tensor,
                                chunk_prefix: torch.Tensor, nnz_out: torch.Tensor, workspace: torch.Tensor,
                                dev_status: Optional[torch.Tensor] = None, *, n: Optional[int] = None, stream=None,
                                check: bool = True) -> int:
    """Fused ReLU6 forward whose values go behind the cursor of a caller-owned arena."""
    n = pre_act.numel() if n is None else n
    st = lib().bt_relu6_fwd_compress_arena(_ptr(pre_act), n, DTYPE_CODE[pre_act.dtype], _ptr(y_out), _ptr(bitmap),
                                           _ptr(arena), _nbytes(arena), _ptr(arena_cursor), _ptr(values_offset_out),
                                           _ptr(chunk_prefix), _ptr(nnz_out), _ptr(workspace), _nbytes(workspace),
                                           _ptr(dev_status), _stream(stream))
    return _check("bt_relu6_fwd_compress_arena", st, check)


def bt_relu6_bwd_from_stash_arena(bitmap: torch.Tensor, arena: torch.Tensor, values_offset: torch.Tensor,
                                  chunk_prefix: torch.Tensor, grad_out: torch.Tensor, grad_in: torch.Tensor,
                                  *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    """ReLU6 backward from a stash whose values sit in an arena."""
    n = grad_out.numel() if n is None else n
    st = lib().bt_relu6_bwd_from_stash_arena(_ptr(bitmap), _ptr(arena), _ptr(values_offset), _ptr(chunk_prefix),
                                             _ptr(grad_out), n, DTYPE_CODE[grad_out.dtype], _ptr(grad_in), _stream(stream))
    return _check("bt_relu6_bwd_from_stash_arena", st, check)


def bt_relu6_fwd_compress(pre_act: torch.Tensor, y_out: Optional[torch.Tensor], bitmap: torch.Tensor,
                          values: torch.Tensor, chunk_prefix: torch.Tensor, nnz_out: torch.Tensor,
                          workspace: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                          *, n: Optional[int] = None, values_capacity: Optional[int] = None, stream=None,
                          check: bool = True) -> int:
    n = pre_act.numel() if n is None else n
    cap = values.numel() if values_capacity is None else values_capacity
    st = lib().bt_relu6_fwd_compress(_ptr(pre_act), n, DTYPE_CODE[pre_act.dtype], _ptr(y_out), _ptr(bitmap),
                                     _ptr(values), cap, _ptr(chunk_prefix), _ptr(nnz_out), _ptr(workspace),
                                     _nbytes(workspace), _ptr(dev_status), _stream(stream))
    return _check("bt_relu6_fwd_compress", st, check)


def bt_relu6_bwd_from_stash(bitmap: torch.Tensor, values: torch.Tensor, chunk_prefix: torch.Tensor,
                            grad_out: torch.Tensor, grad_in: torch.Tensor, *, n: Optional[int] = None, stream=None,
                            check: bool = True) -> int:
    n = grad_out.numel() if n is None else n
    st = lib().bt_relu6_bwd_from_stash(_ptr(bitmap), _ptr(values), _ptr(chunk_prefix), _ptr(grad_out), n,
                                       DTYPE_CODE[grad_out.dtype], _ptr(grad_in), _stream(stream))
    return _check("bt_relu6_bwd_from_stash", st, check)


def bt_decompress(bitmap: torch.Tensor, values: torch.Tensor, chunk_prefix: torch.Tensor, dense_out: torch.Tensor,
                  *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    n = dense_out.numel() if n is None else n
    st = lib().bt_decompress(_ptr(bitmap), _ptr(values), _ptr(chunk_prefix), n, DTYPE_CODE[dense_out.dtype],
                             _ptr(dense_out), _stream(stream))
    return _check("bt_decompress", st, check)


def bt_relu_bwd_from_bitmap(bitmap: torch.Tensor, grad_out: torch.Tensor, grad_in: torch.Tensor,
                            *, n: Optional[int] = None, stream=None, check: bool = True) -> int:
    n = grad_out.numel() if n is None else n
    st = lib().bt_relu_bwd_from_bitmap(_ptr(bitmap), _ptr(grad_out), n, DTYPE_CODE[grad_out.dtype], _ptr(grad_in),
                                       _stream(stream))
    return _check("bt_relu_bwd_from_bitmap", st, check)


# ---- host-buffer forms: `host_*` are CPU tensors (pinned for speed), `staging` a CUDA uint8 tensor
def bt_host_staging_bytes(n: int, dtype) -> int:
    return int(lib().bt_host_staging_bytes(n, DTYPE_CODE.get(dtype, dtype)))


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


def bt_compress_host(host_dense: torch.Tensor, host_bitmap: torch.Tensor, host_values: torch.Tensor,
                     host_chunk_prefix: torch.Tensor, host_nnz: torch.Tensor, staging: torch.Tensor,
                     *, stream=None, check: bool = True) -> int:
    st = lib().bt_compress_host(_ptr(host_dense), host_dense.numel(), DTYPE_CODE[host_dense.dtype], _ptr(host_bitmap),
                                _ptr(host_values), host_values.numel(), _ptr(host_chunk_prefix), _ptr(host_nnz),
                                _ptr(staging), _nbytes(staging), _stream(stream))
    return _check("bt_compress_host", st, check)


def bt_relu_fwd_compress_host(host_pre_act: torch.Tensor, host_y_out: Optional[torch.Tensor],
                              host_bitmap: torch.Tensor, host_values: torch.Tensor, host_chunk_prefix: torch.Tensor,
                              host_nnz: torch.Tensor, staging: torch.Tensor, *, stream=None, check: bool = True) -> int:
    st = lib().bt_relu_fwd_compress_host(_ptr(host_pre_act), host_pre_act.numel(), DTYPE_CODE[host_pre_act.dtype],
                                         _ptr(host_y_out), _ptr(host_bitmap), _ptr(host_values), host_values.numel(),
                                         _ptr(host_chunk_prefix), _ptr(host_nnz), _ptr(staging), _nbytes(staging),
                                         _stream(stream))
    return _check("bt_relu_fwd_compress_host", st, check)


def bt_decompress_host(host_bitmap: torch.Tensor, host_values: torch.Tensor, host_chunk_prefix: torch.Tensor,
                       nnz: int, host_dense_out: torch.Tensor, staging: torch.Tensor, *, stream=None,
                       check: bool = True) -> int:
    st = lib().bt_decompress_host(_ptr(host_bitmap), _ptr(host_values), _ptr(host_chunk_prefix), nnz,
                                  host_dense_out.numel(), DTYPE_CODE[host_dense_out.dtype], _ptr(host_dense_out),
                                  _ptr(staging), _nbytes(staging), _stream(stream))
    return _check("bt_decompress_host", st, check)


def bt_relu_bwd_from_bitmap_host(host_bitmap: torch.Tensor, host_grad_out: torch.Tensor, host_grad_in: torch.Tensor,
                                 staging: torch.Tensor, *, stream=None, check: bool = True) -> int:
    st = lib().bt_relu_bwd_from_bitmap_host(_ptr(host_bitmap), _ptr(host_grad_out), host_grad_out.numel(),
                                            DTYPE_CODE[host_grad_out.dtype], _ptr(host_grad_in), _ptr(staging),
                                            _nbytes(staging), _stream(stream))
    return _check("bt_relu_bwd_from_bitmap_host", st, check)


class Stash:
    """Device buffers for one compressed tensor (allocation helper, no arithmetic)."""

    def __init__(self, n: int, dtype: torch.dtype, device="cuda", values_capacity: Optional[int] = None):
        self.n, self.dtype = n, dtype
        cap = n if values_capacity is None else values_capacity
        self.bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=device)
        self.values = torch.empty(cap, dtype=dtype, device=device)
        self.chunk_prefix = torch.empty((n + CHUNK - 1) // CHUNK, dtype=torch.int64, device=device)
        self.nnz_out = torch.empty(1, dtype=torch.int64, device=device)
        self.dev_status = torch.empty(1, dtype=torch.int32, device=device)

    @property
    def nnz(self) -> int:
        return int(self.nnz_out.item())

    @property
    def status(self) -> int:
        return int(self.dev_status.item())


def new_workspace(n: int, device="cuda") -> torch.Tensor:
    return torch.empty(bt_workspace_bytes(n), dtype=torch.uint8, device=device)
