"""Helpers of the GPU parity tests: guarded device buffers and one-call wrappers
that run a C-ABI entry point and bring every output back as numpy arrays."""
from __future__ import annotations

import numpy as np
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

GUARD = 64            # guard elements on each side of every output buffer
TDT = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16, "f64": torch.float64}
_INT = {2: torch.int16, 4: torch.int32, 8: torch.int64}


class Guarded:
    """A device buffer with canary regions before and after the part handed to the library."""

    def __init__(self, numel: int, dtype: torch.dtype, device="cuda", fill: int = 0x5A):
        self.numel = numel
        es = torch.empty((), dtype=dtype).element_size()
        # keep the inner pointer 16-byte aligned: guard is a multiple of 16 bytes for every width
        self.full = torch.empty(numel + 2 * GUARD, dtype=dtype, device=device)
        self.full.view(torch.uint8).fill_(fill)
        self.fill = fill
        self.inner = self.full[GUARD:GUARD + numel]
        assert self.inner.data_ptr() % 16 == 0 or numel == 0
        self.es = es

    def guards_intact(self) -> bool:
        raw = self.full.view(torch.uint8)
        g = GUARD * self.es
        return bool((raw[:g] == self.fill).all().item()) and bool((raw[raw.numel() - g:] == self.fill).all().item())

    def raw(self) -> np.ndarray:
        return W.raw_numpy(self.inner)


def from_raw(x: np.ndarray, kind: str, device="cuda") -> torch.Tensor:
    """Device tensor of torch dtype `kind` holding exactly the raw patterns in x."""
    es = x.dtype.itemsize
    t = torch.from_numpy(x.view({2: np.int16, 4: np.int32, 8: np.int64}[es]).copy()).to(device)
    return t.view(TDT[kind])


class GpuCompressed:
    def __init__(self, bitmap, values_all, prefix, nnz, status, y, guards_ok):
        self.bitmap, self.values_all, self.prefix = bitmap, values_all, prefix
        self.nnz, self.status, self.y, self.guards_ok = nnz, status, y, guards_ok

    @property
    def values(self):
        return self.values_all[:self.nnz]


def gpu_compress(x: torch.Tensor, relu: bool = False, want_y: bool = False, capacity=None,
                 in_place: bool = False, keep_device: bool = False, tau=None, narrow=None):
    """`tau` given: bt_prune_fwd_compress with that threshold (want_y / in_place as for the ReLU form).
    `narrow` ("f16" / "bf16"): the down-cast-on-stash entry points (float32 input, 16-bit values)."""
    n = x.numel()
    cap = n if capacity is None else capacity
    bitmap = Guarded((n + 31) // 32, torch.int32)
    values = Guarded(cap, TDT[narrow] if narrow else x.dtype)
    prefix = Guarded((n + 4095) // 4096, torch.int64)
    nnz = Guarded(1, torch.int64)
    status = Guarded(1, torch.int32)
    ws = B.new_workspace(n)
    y = None
    if relu or tau is not None:
        if in_place:
            y_t = x
        elif want_y:
            y = Guarded(n, x.dtype)
            y_t = y.inner
        else:
            y_t = None
        if narrow:
            B.bt_prune_fwd_compress_narrow(x, 0.0 if tau is None else tau, y_t, bitmap.inner, values.inner, prefix.inner,
                                           nnz.inner, ws, status.inner, n=n, values_capacity=cap)
        elif tau is not None:
            B.bt_prune_fwd_compress(x, tau, y_t, bitmap.inner, values.inner, prefix.inner, nnz.inner, ws,
                                    status.inner, n=n, values_capacity=cap)
        else:
            B.bt_relu_fwd_compress(x, y_t, bitmap.inner, values.inner, prefix.inner, nnz.inner, ws, status.inner,
                                   n=n, values_capacity=cap)
    elif narrow:
        B.bt_compress_narrow(x, bitmap.inner, values.inner, prefix.inner, nnz.inner, ws, status.inner,
                             n=n, values_capacity=cap)
    else:
        B.bt_compress(x, bitmap.inner, values.inner, prefix.inner, nnz.inner, ws, status.inner,
                      n=n, values_capacity=cap)
    torch.cuda.synchronize()
    ok = all(g.guards_intact() for g in (bitmap, values, prefix, nnz, status) + ((y,) if y is not None else ()))
    out = GpuCompressed(bitmap.raw().view(np.uint32), values.raw(), prefix.raw().view(np.uint64),
                        int(nnz.inner.item()), int(status.inner.item()),
                        (W.raw_numpy(x) if in_place else (y.raw() if y is not None else None)), ok)
    if keep_device:
        out.dev = (bitmap, values, prefix, nnz)
    return out


def gpu_decompress(bitmap: np.ndarray, values: np.ndarray, prefix: np.ndarray, n: int, kind: str):
    bm = torch.from_numpy(bitmap.view(np.int32).copy()).cuda()
    # at least one element so the pointer is never NULL-by-accident for empty value sets
    vals = from_raw(values if values.size else np.zeros(1, values.dtype), kind)
    pf = torch.from_numpy(prefix.view(np.int64).copy()).cuda()
    out = Guarded(n, TDT[kind])
    B.bt_decompress(bm, vals, pf, out.inner, n=n)
    torch.cuda.synchronize()
    return out.raw(), out.guards_intact()


def gpu_relu_bwd(bitmap: np.ndarray, g: torch.Tensor, in_place: bool = False):
    bm = torch.from_numpy(bitmap.view(np.int32).copy()).cuda()
    n = g.numel()
    if in_place:
        B.bt_relu_bwd_from_bitmap(bm, g, g, n=n)
        torch.cuda.synchronize()
        return W.raw_numpy(g), True
    out = Guarded(n, g.dtype)
    B.bt_relu_bwd_from_bitmap(bm, g, out.inner, n=n)
    torch.cuda.synchronize()
    return out.raw(), out.guards_intact()


def gpu_mask_compress(x: torch.Tensor, bitmap: np.ndarray, prefix: np.ndarray, nnz: int, mode: str = "with_y",
                      capacity=None):
    """bt_mask_compress under the given stash bitmap / prefix; returns (values[:nnz], y or None, guards intact).
    mode: "stash_only", "with_y" or "in_place" (y written over x)."""
    n = x.numel()
    cap = nnz if capacity is None else capacity
    bm = torch.from_numpy(bitmap.view(np.int32).copy()).cuda()
    pf = torch.from_numpy(prefix.view(np.int64).copy()).cuda()
    values = Guarded(max(cap, 1), x.dtype)
    y = None
    if mode == "with_y":
        y = Guarded(n, x.dtype)
        y_t = y.inner
    elif mode == "in_place":
        y_t = x
    else:
        y_t = None
    B.bt_mask_compress(x, bm, pf, y_t, values.inner, n=n, values_capacity=cap)
    torch.cuda.synchronize()
    ok = values.guards_intact() and (y is None or y.guards_intact())
    y_raw = y.raw() if y is not None else (W.raw_numpy(x) if mode == "in_place" else None)
    return values.raw()[:min(nnz, cap)], y_raw, ok
