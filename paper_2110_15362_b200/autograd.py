"""The stash wired into PyTorch's autograd: activations that a layer saves for its backward pass are kept
in the sparse-bitmap form and restored when the backward pass asks for them (the integration the paper
names as its first contribution and, for GPUs, as future work: section 1 and the conclusion).

Two pieces, both thin wrappers around the C-ABI calls (no arithmetic here):

* ``stash_saved_activations()`` -- a ``torch.autograd.graph.saved_tensors_hooks`` context.  Every eligible
  tensor saved inside it (CUDA, floating point, contiguous, large enough, not a parameter) is compressed
  with ``bt_compress``; only the bitmap, the chunk prefix array and exactly ``nnz`` values stay alive.  On
  the way back ``bt_decompress`` rebuilds the tensor bit for bit, so gradients are unchanged.  A tensor
  that would not shrink (too few zeros) is kept as it is.
* ``relu_stash(x)`` -- a ReLU whose forward pass writes the activation and its stash in one kernel
  (``bt_relu_fwd_compress``) and whose backward pass needs only the bitmap
  (``bt_relu_bwd_from_bitmap``).  Inside the context above its stash is shared with the next layer's saved
  input, so the activation is compressed once.

Getting the exact ``nnz`` to size the values costs one device-to-host read per packed tensor.  With
``stash_saved_activations(arena_bytes=...)`` the values go instead behind a device-side cursor into one
pre-allocated arena (the ``*_arena`` entry points): no host read in the forward pass; the device status
words are checked once, when the backward pass first asks for a tensor.  The cursor is reset on entering
the context, so one context entry covers one forward / backward pass.

``double_mask(out, like)`` is the double-mask form for normalisation layers: ``out`` (e.g. a batch-norm output)
is zeroed wherever ``like`` (the layer's input, a post-ReLU tensor) is zero, and its stash reuses the bitmap and
the prefix array of ``like``'s stash (``bt_mask_compress``); the backward pass masks the gradient with the same
bitmap.

``maxpool2x2_stash(x)`` is a 2x2 / stride 2 max pooling that keeps 2 bits per output for its backward pass
(``bt_maxpool2x2_fwd`` / ``bt_maxpool2x2_bwd``) instead of its input and an index tensor: behind a ``relu_stash``
the values of the pooled layer's input are then held by nothing, only its bitmap.  ``relu_maxpool2x2_stash(x)``
does both layers with the pooling first (the maximum commutes with the ReLU): the full-size activation is never
written and the fused ReLU + stash runs on the pooled quarter.

``relu6_stash(x)`` is the same for ReLU6 (``bt_relu6_fwd_compress`` / ``bt_relu6_bwd_from_stash``; its backward
pass reads the stashed values as well, which are the ones the next layer's saved input shares).  With
``stash_saved_activations(narrow=torch.float16)`` (or ``torch.bfloat16``) float32 activations are stashed with
16-bit values (``bt_compress_narrow`` / ``bt_decompress_widen``): lossy -- what the backward pass gets back is
the activation rounded to the narrow type.  Both work inside an arena context as well (the ``*_arena`` forms of
those calls); a ReLU6 stash is never narrowed.
"""
from __future__ import annotations

import weakref
from typing import Dict, Optional, Tuple

import torch

from . import binding as B

__all__ = ["PackedActivation", "stash_saved_activations", "relu_stash", "ReLUStash", "relu6_stash", "ReLU6Stash",
           "double_mask", "DoubleMask", "maxpool2x2_stash", "MaxPool2x2Stash", "relu_maxpool2x2_stash",
           "ReLUMaxPool2x2Stash"]


class PackedActivation:
    """What replaces a saved tensor: the stash and the metadata needed to rebuild it.  `values` is either the
    exact-size vector of values, or (arena mode) None with `arena`, `offset` (device word), `owner` and `stored`
    (the dtype of the values in the arena) set."""

    __slots__ = ("bitmap", "values", "chunk_prefix", "shape", "dtype", "device", "nnz", "arena", "offset", "owner",
                 "stored", "__weakref__")

    def __init__(self, bitmap, values, chunk_prefix, shape, dtype, device, nnz, arena=None, offset=None, owner=None,
                 stored=None):
        self.bitmap, self.values, self.chunk_prefix = bitmap, values, chunk_prefix
        self.shape, self.dtype, self.device, self.nnz = shape, dtype, device, nnz
        self.arena, self.offset, self.owner = arena, offset, owner
        self.stored = stored if stored is not None else (dtype if values is None else values.dtype)

    @property
    def numel(self) -> int:
        n = 1
        for s in self.shape:
            n *= s
        return n

    def nbytes(self) -> int:
        """Bytes of the stash (arena mode: reads nnz from the device)."""
        nnz = int(self.nnz.item()) if isinstance(self.nnz, torch.Tensor) else self.nnz
        return B.bt_compressed_bytes(self.numel, nnz, self.stored)

    def unpack(self) -> torch.Tensor:
        out = torch.empty(self.shape, dtype=self.dtype, device=self.device)
        if self.arena is not None:
            self.owner.check_statuses()
            if self.stored != self.dtype:              # a narrowed stash of a float32 tensor
                B.bt_decompress_widen_arena(self.bitmap, self.arena, self.offset, self.chunk_prefix, self.stored,
                                            out.view(-1))
            else:
                B.bt_decompress_arena(self.bitmap, self.arena, self.offset, self.chunk_prefix, out.view(-1))
        elif self.values.dtype != self.dtype:          # a narrowed stash of a float32 tensor
            B.bt_decompress_widen(self.bitmap, self.values, self.chunk_prefix, out.view(-1))
        else:
            B.bt_decompress(self.bitmap, self.values, self.chunk_prefix, out.view(-1))
        return out


def _usable(t: torch.Tensor) -> bool:
    """Can the library take this tensor as it is?  (contiguous and 16-byte aligned)"""
    return t.is_contiguous() and t.data_ptr() % 16 == 0


def _flat_input(t: torch.Tensor) -> torch.Tensor:
    """The tensor itself if the library can take it, else a contiguous, aligned copy."""
    return t if _usable(t) else t.clone(memory_format=torch.contiguous_format)


class _Scratch:
    """Per-device reusable buffers of the packing calls: workspace and a full-capacity values buffer."""

    def __init__(self, two_pass: bool = True):
        self.ws: Dict[torch.device, torch.Tensor] = {}
        self.values: Dict[Tuple[torch.device, torch.dtype], torch.Tensor] = {}
        self.two_pass = two_pass         # exact-size values without a full-capacity buffer (see _compress)

    def workspace(self, n: int, device) -> torch.Tensor:
        need = B.bt_workspace_bytes(n)
        ws = self.ws.get(device)
        if ws is None or ws.numel() < need:
            ws = self.ws[device] = torch.empty(need, dtype=torch.uint8, device=device)
        return ws

    def full_values(self, n: int, dtype, device) -> torch.Tensor:
        key = (device, dtype)
        v = self.values.get(key)
        if v is None or v.numel() < n:
            v = self.values[key] = torch.empty(n, dtype=dtype, device=device)
        return v


def _compress(flat: torch.Tensor, scratch: _Scratch, relu_into: Optional[torch.Tensor] = None,
              narrow: Optional[torch.dtype] = None, relu6: bool = False):
    """Runs the (fused) compressor on a flat tensor; returns bitmap, exact-size values, prefix, nnz.  `narrow`:
    16-bit dtype of the stashed values of a float32 tensor.  `relu6`: the fused form is ReLU6 (needs relu_into)."""
    n, dev = flat.numel(), flat.device
    if narrow is not None and flat.dtype != torch.float32:
        narrow = None
    bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
    prefix = torch.empty((n + B.CHUNK - 1) // B.CHUNK, dtype=torch.int64, device=dev)
    nnz_out = torch.empty(1, dtype=torch.int64, device=dev)
    status = torch.empty(1, dtype=torch.int32, device=dev)
    ws = scratch.workspace(n, dev)
    if scratch.two_pass and narrow is None:
        # Two passes instead of a values buffer of full capacity: the compressor with no room for values gives
        # bitmap, prefix and nnz (BT_ERR_CAPACITY is its expected answer), the host reads nnz, and the masked
        # gather fills a buffer of exactly that size from the activation.  Costs the gather (cheaper than a
        # compaction); saves a buffer as large as the largest activation for the whole step.
        if relu6:
            B.bt_relu6_fwd_compress(flat, relu_into, bitmap, None, prefix, nnz_out, ws, status, n=n, values_capacity=0)
        elif relu_into is None:
            B.bt_compress(flat, bitmap, None, prefix, nnz_out, ws, status, n=n, values_capacity=0)
        else:
            B.bt_relu_fwd_compress(flat, relu_into, bitmap, None, prefix, nnz_out, ws, status, n=n, values_capacity=0)
        nnz = int(nnz_out.item())
        st = int(status.item())
        if st not in (B.BT_OK, B.BT_ERR_CAPACITY):
            raise B.BitTrainError("bt_compress (autograd stash)", st)
        values = torch.empty(nnz, dtype=flat.dtype, device=dev)
        if nnz:
            B.bt_mask_compress(flat if relu_into is None else relu_into, bitmap, prefix, None, values, n=n)
        return bitmap, values, prefix, nnz
    full = scratch.full_values(n, narrow or flat.dtype, dev)
    if relu6:
        B.bt_relu6_fwd_compress(flat, relu_into, bitmap, full, prefix, nnz_out, ws, status, n=n, values_capacity=n)
    elif narrow is not None and relu_into is None:
        B.bt_compress_narrow(flat, bitmap, full, prefix, nnz_out, ws, status, n=n, values_capacity=n)
    elif narrow is not None:
        B.bt_prune_fwd_compress_narrow(flat, 0.0, relu_into, bitmap, full, prefix, nnz_out, ws, status, n=n,
                                       values_capacity=n)
    elif relu_into is None:
        B.bt_compress(flat, bitmap, full, prefix, nnz_out, ws, status, n=n, values_capacity=n)
    else:
        B.bt_relu_fwd_compress(flat, relu_into, bitmap, full, prefix, nnz_out, ws, status, n=n, values_capacity=n)
    nnz = int(nnz_out.item())                       # the one host read: sizes the values exactly
    st = int(status.item())
    if st != B.BT_OK:
        raise B.BitTrainError("bt_compress (autograd stash)", st)
    return bitmap, full[:nnz].clone(), prefix, nnz


def _compress_arena(flat: torch.Tensor, owner, relu_into: Optional[torch.Tensor] = None, relu6: bool = False):
    """Arena form of `_compress`: nothing is read back; returns bitmap, prefix, nnz word, offset word and the
    dtype of the values pushed (the owner's narrow type for a float32 tensor, except under ReLU6)."""
    n, dev = flat.numel(), flat.device
    narrow = owner.narrow if (flat.dtype == torch.float32 and not relu6) else None
    bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
    prefix = torch.empty((n + B.CHUNK - 1) // B.CHUNK, dtype=torch.int64, device=dev)
    words = torch.empty(2, dtype=torch.int64, device=dev)               # nnz, byte offset of the values
    status = torch.empty(1, dtype=torch.int32, device=dev)
    ws = owner.scratch.workspace(n, dev)
    if relu6:
        B.bt_relu6_fwd_compress_arena(flat, relu_into, bitmap, owner.arena, owner.cursor, words[1:], prefix, words[:1],
                                      ws, status, n=n)
    elif narrow is not None and relu_into is None:
        B.bt_compress_narrow_arena(flat, narrow, bitmap, owner.arena, owner.cursor, words[1:], prefix, words[:1], ws,
                                   status, n=n)
    elif narrow is not None:
        B.bt_prune_fwd_compress_narrow_arena(flat, narrow, 0.0, relu_into, bitmap, owner.arena, owner.cursor, words[1:],
                                             prefix, words[:1], ws, status, n=n)
    elif relu_into is None:
        B.bt_compress_arena(flat, bitmap, owner.arena, owner.cursor, words[1:], prefix, words[:1], ws, status, n=n)
    else:
        B.bt_prune_fwd_compress_arena(flat, 0.0, relu_into, bitmap, owner.arena, owner.cursor, words[1:], prefix,
                                      words[:1], ws, status, n=n)
    owner.statuses.append(status)
    return bitmap, prefix, words[:1], words[1:], narrow or flat.dtype


class stash_saved_activations(torch.autograd.graph.saved_tensors_hooks):
    """Context manager: saved activations are kept compressed between the forward and the backward pass.
    `arena_bytes`: keep all values in one pre-allocated arena of that size behind a device-side cursor (no
    host read per tensor; a RuntimeError at the first unpack if the arena was too small).  `narrow`
    (torch.float16 / torch.bfloat16): float32 activations are stashed with values of that type (lossy).
    `two_pass` (exact-size mode): size the values by a first pass without values and fill them with a masked
    gather, instead of compacting into a buffer of full capacity that stays allocated (default)."""

    def __init__(self, min_numel: int = 1 << 14, min_saving: float = 0.1, arena_bytes: Optional[int] = None,
                 device="cuda", narrow: Optional[torch.dtype] = None, two_pass: bool = True):
        if narrow not in (None, torch.float16, torch.bfloat16):
            raise ValueError("narrow must be torch.float16 or torch.bfloat16")
        self.min_numel, self.min_saving, self.narrow = min_numel, min_saving, narrow
        self.arena = self.cursor = None
        self.statuses: list = []
        self.loose_statuses: list = []   # status words of bitmap-only calls (BT_ERR_CAPACITY expected)
        if arena_bytes is not None:
            self.arena = torch.empty((arena_bytes + 15) // 16 * 16, dtype=torch.uint8, device=device)
            self.cursor = torch.zeros(1, dtype=torch.int64, device=device)
        self.scratch = _Scratch(two_pass)
        self.packed_bytes = 0            # bytes kept in compressed form so far
        self.dense_bytes = 0             # bytes the same tensors would have taken
        self._shared: Dict[int, Tuple[weakref.ref, weakref.ref]] = {}
        super().__init__(self._pack, self._unpack)

    # ---- sharing of one stash between several saves of the same tensor object
    # The table holds weak references only: a stash lives as long as the tensor object it belongs to (which
    # carries it as an attribute) or a saved-tensor slot of the graph, and is freed with them.
    def share(self, tensor: torch.Tensor, packed: PackedActivation) -> None:
        tensor._bt_packed = packed
        self._shared[id(tensor)] = (weakref.ref(tensor), weakref.ref(packed))

    def _lookup(self, tensor: torch.Tensor) -> Optional[PackedActivation]:
        hit = self._shared.get(id(tensor))
        if hit is None:
            return None
        ref, packed_ref = hit
        packed = packed_ref()
        if ref() is tensor and packed is not None:
            return packed
        del self._shared[id(tensor)]     # the id was recycled by another object
        return None

    def _eligible(self, t: torch.Tensor) -> bool:
        return (t.is_cuda and t.dtype in B.DTYPE_CODE and t.is_contiguous() and t.numel() >= self.min_numel
                and t.data_ptr() % 16 == 0               # the library wants 16-byte aligned tensors (a view may not be)
                and not isinstance(t, torch.nn.Parameter) and not (t.requires_grad and t.is_leaf))

    def check_statuses(self) -> None:
        """One host read for all status words collected so far; raises if an arena stash did not fit or a call
        failed."""
        if self.loose_statuses:
            words = torch.cat(self.loose_statuses)
            self.loose_statuses.clear()
            bad = words[(words != B.BT_OK) & (words != B.BT_ERR_CAPACITY)]
            if bad.numel():
                raise RuntimeError("a bitmap-only stash call failed: %s" % B.BitTrainError("bt_relu_fwd_compress", int(bad[0].item())))
        if self.statuses:
            worst = int(torch.cat(self.statuses).max().item())
            self.statuses.clear()
            if worst != B.BT_OK:
                raise RuntimeError("stash arena too small or a stash call failed: %s" %
                                   B.BitTrainError("bt_*_arena", worst))

    def _pack(self, t: torch.Tensor):
        if not self._eligible(t):
            return t
        shared = self._lookup(t)
        if shared is not None:
            return shared
        n, es = t.numel(), t.element_size()
        if self.arena is not None:
            bitmap, prefix, nnz_word, off_word, stored = _compress_arena(t.detach().view(-1), self)
            packed = PackedActivation(bitmap, None, prefix, tuple(t.shape), t.dtype, t.device, nnz_word,
                                      arena=self.arena, offset=off_word, owner=self, stored=stored)
            self.share(t, packed)
            self.dense_bytes += n * es
            return packed
        bitmap, values, prefix, nnz = _compress(t.detach().view(-1), self.scratch, narrow=self.narrow)
        if B.bt_compressed_bytes(n, nnz, values.dtype) > (1.0 - self.min_saving) * n * es:
            return t                                  # too few zeros: the stash would not be smaller
        packed = PackedActivation(bitmap, values, prefix, tuple(t.shape), t.dtype, t.device, nnz)
        self.share(t, packed)
        self.packed_bytes += packed.nbytes()
        self.dense_bytes += n * es
        return packed

    @staticmethod
    def _unpack(obj):
        return obj.unpack() if isinstance(obj, PackedActivation) else obj

    def __enter__(self):
        # status words the previous pass left unchecked (its backward pass may have run outside the context, or
        # asked for nothing): one host read here, where no launch of the new pass is waiting behind it
        self.check_statuses()
        if self.cursor is not None:
            self.cursor.zero_()                 # a new pass: the arena is empty again
        super().__enter__()
        return self

    def __exit__(self, *exc):
        self._shared.clear()
        return super().__exit__(*exc)


class ReLUStash(torch.autograd.Function):
    """ReLU with the stash fused into its forward pass; the backward pass reads only the bitmap."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, hooks: Optional[stash_saved_activations] = None, inplace: bool = False,
                keep_values: bool = True):
        if inplace and _usable(x):
            xc = y = x                   # the kernel may write the activation over its input
            ctx.mark_dirty(x)
        else:
            xc = _flat_input(x)
            y = torch.empty_like(xc)
        if not keep_values:
            # nobody will ask for the activation again (e.g. it only feeds a pooling layer that keeps winner codes):
            # the bitmap is all this ReLU's backward pass needs, so the values are not stored at all
            n, dev = xc.numel(), xc.device
            bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
            prefix = torch.empty((n + B.CHUNK - 1) // B.CHUNK, dtype=torch.int64, device=dev)
            nnz_out = torch.empty(1, dtype=torch.int64, device=dev)
            status = torch.empty(1, dtype=torch.int32, device=dev)
            scratch = hooks.scratch if hooks is not None else _Scratch()
            B.bt_relu_fwd_compress(xc.view(-1), y.view(-1), bitmap, None, prefix, nnz_out, scratch.workspace(n, dev), status,
                                   n=n, values_capacity=0)
            if hooks is not None:
                hooks.loose_statuses.append(status)     # BT_ERR_CAPACITY is the expected answer here
            elif int(status.item()) not in (B.BT_OK, B.BT_ERR_CAPACITY):
                raise B.BitTrainError("bt_relu_fwd_compress (bitmap only)", int(status.item()))
            ctx.save_for_backward(bitmap)
            return y
        if hooks is not None and hooks.arena is not None:
            bitmap, prefix, nnz_word, off_word, stored = _compress_arena(xc.view(-1), hooks, relu_into=y.view(-1))
            ctx.save_for_backward(bitmap)
            hooks.share(y, PackedActivation(bitmap, None, prefix, tuple(y.shape), y.dtype, y.device, nnz_word,
                                            arena=hooks.arena, offset=off_word, owner=hooks, stored=stored))
            hooks.dense_bytes += y.numel() * y.element_size()
            return y
        scratch = hooks.scratch if hooks is not None else _Scratch()
        bitmap, values, prefix, nnz = _compress(xc.view(-1), scratch, relu_into=y.view(-1),
                                                narrow=hooks.narrow if hooks is not None else None)
        ctx.save_for_backward(bitmap)     # released with the graph, like any saved tensor
        if hooks is not None:
            # the next layer will save y as its input: hand it this stash instead of compressing y again
            packed = PackedActivation(bitmap, values, prefix, tuple(y.shape), y.dtype, y.device, nnz)
            hooks.share(y, packed)
            hooks.packed_bytes += packed.nbytes()
            hooks.dense_bytes += y.numel() * y.element_size()
        return y

    @staticmethod
    def backward(ctx, grad: torch.Tensor):
        g = _flat_input(grad)
        gin = torch.empty_like(g)
        (bitmap,) = ctx.saved_tensors
        B.bt_relu_bwd_from_bitmap(bitmap, g.view(-1), gin.view(-1))
        return gin, None, None, None


def relu_stash(x: torch.Tensor, hooks: Optional[stash_saved_activations] = None, inplace: bool = False,
               keep_values: bool = True) -> torch.Tensor:
    """ReLU through the fused kernel.  Pass the active ``stash_saved_activations`` context as ``hooks`` to let
    the following layer reuse the stash for its saved input.  ``inplace=True`` writes the activation over ``x``
    (like ``torch.relu_``: only where ``x`` is not needed again, e.g. the output of a convolution).
    ``keep_values=False`` keeps the bitmap only: for an activation that no later layer saves (one that feeds
    ``maxpool2x2_stash``, say); a layer that does save it compresses it itself."""
    return ReLUStash.apply(x, hooks, inplace, keep_values)


class ReLU6Stash(torch.autograd.Function):
    """ReLU6 with the stash fused into its forward pass; the backward pass reads the bitmap and the stashed
    values (a stored 6 marks a saturated unit).  Exact-size values (one host read), or inside an arena context
    values in the arena; never narrowed (the backward pass compares the stored values with 6)."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, hooks: Optional[stash_saved_activations] = None, inplace: bool = False):
        if inplace and _usable(x):
            xc = y = x
            ctx.mark_dirty(x)
        else:
            xc = _flat_input(x)
            y = torch.empty_like(xc)
        ctx.owner = None
        if hooks is not None and hooks.arena is not None:
            bitmap, prefix, nnz_word, off_word, stored = _compress_arena(xc.view(-1), hooks, relu_into=y.view(-1),
                                                                         relu6=True)
            ctx.owner = hooks
            ctx.save_for_backward(bitmap, off_word, prefix)
            hooks.share(y, PackedActivation(bitmap, None, prefix, tuple(y.shape), y.dtype, y.device, nnz_word,
                                            arena=hooks.arena, offset=off_word, owner=hooks, stored=stored))
            hooks.dense_bytes += y.numel() * y.element_size()
            return y
        scratch = hooks.scratch if hooks is not None else _Scratch()
        bitmap, values, prefix, nnz = _compress(xc.view(-1), scratch, relu_into=y.view(-1), relu6=True)
        ctx.save_for_backward(bitmap, values, prefix)
        if hooks is not None:
            packed = PackedActivation(bitmap, values, prefix, tuple(y.shape), y.dtype, y.device, nnz)
            hooks.share(y, packed)
            hooks.packed_bytes += packed.nbytes()
            hooks.dense_bytes += y.numel() * y.element_size()
        return y

    @staticmethod
    def backward(ctx, grad: torch.Tensor):
        g = _flat_input(grad)
        gin = torch.empty_like(g)
        bitmap, values, prefix = ctx.saved_tensors
        if ctx.owner is not None:                      # arena mode: `values` is the offset word
            ctx.owner.check_statuses()
            B.bt_relu6_bwd_from_stash_arena(bitmap, ctx.owner.arena, values, prefix, g.view(-1), gin.view(-1))
        else:
            B.bt_relu6_bwd_from_stash(bitmap, values, prefix, g.view(-1), gin.view(-1))
        return gin, None, None


def relu6_stash(x: torch.Tensor, hooks: Optional[stash_saved_activations] = None, inplace: bool = False) -> torch.Tensor:
    """ReLU6 through the fused kernel; arguments as for ``relu_stash``."""
    return ReLU6Stash.apply(x, hooks, inplace)


class DoubleMask(torch.autograd.Function):
    """out masked by the zero pattern of `like` (double-mask batch normalisation): y = like != 0 ? out : +0.  The
    stash of y shares the bitmap and the prefix array of like's stash and gets its own values; the backward pass
    is the bitmap select.  `like` receives no gradient (the mask is a constant of the step)."""

    @staticmethod
    def forward(ctx, out: torch.Tensor, like: torch.Tensor, hooks: Optional[stash_saved_activations] = None,
                inplace: bool = False):
        if out.shape != like.shape or out.dtype != like.dtype:
            raise ValueError("double_mask: the two tensors must agree in shape and dtype")
        src = hooks._lookup(like) if hooks is not None else None
        if src is None or src.arena is not None or src.values.dtype != like.dtype:
            # no reusable stash of `like` (none yet, or one whose size only the device knows): make one
            scratch = hooks.scratch if hooks is not None else _Scratch()
            bitmap, values, prefix, nnz = _compress(_flat_input(like.detach()).view(-1), scratch)
            src = PackedActivation(bitmap, values, prefix, tuple(like.shape), like.dtype, like.device, nnz)
        if inplace and _usable(out):
            xc = y = out
            ctx.mark_dirty(out)
        else:
            xc = _flat_input(out)
            y = torch.empty_like(xc)
        values = torch.empty(max(src.nnz, 1), dtype=out.dtype, device=out.device)
        B.bt_mask_compress(xc.view(-1), src.bitmap, src.chunk_prefix, y.view(-1), values, values_capacity=src.nnz)
        ctx.save_for_backward(src.bitmap)
        if hooks is not None:
            packed = PackedActivation(src.bitmap, values[:src.nnz], src.chunk_prefix, tuple(y.shape), y.dtype, y.device,
                                      src.nnz)
            hooks.share(y, packed)
            hooks.packed_bytes += src.nnz * y.element_size()          # bitmap and prefix are the source's
            hooks.dense_bytes += y.numel() * y.element_size()
        return y

    @staticmethod
    def backward(ctx, grad: torch.Tensor):
        g = _flat_input(grad)
        gin = torch.empty_like(g)
        (bitmap,) = ctx.saved_tensors
        B.bt_relu_bwd_from_bitmap(bitmap, g.view(-1), gin.view(-1))
        return gin, None, None, None


def double_mask(out: torch.Tensor, like: torch.Tensor, hooks: Optional[stash_saved_activations] = None,
                inplace: bool = False) -> torch.Tensor:
    """``out`` with zeros wherever ``like`` is zero, stashed under ``like``'s bitmap (see ``DoubleMask``)."""
    return DoubleMask.apply(out, like, hooks, inplace)


class MaxPool2x2Stash(torch.autograd.Function):
    """2x2 / stride 2 max pooling of a (..., H, W) tensor (H and W even) whose backward pass needs only 2 bits per
    output.  The pooled output is an ordinary tensor: inside the hooks context the next layer's save compresses it."""

    @staticmethod
    def forward(ctx, x: torch.Tensor):
        if x.dim() < 2 or x.shape[-1] % 2 or x.shape[-2] % 2 or x.numel() == 0:
            raise ValueError("maxpool2x2_stash: the last two dimensions must be even and non-empty")
        xc = _flat_input(x)
        y = torch.empty(xc.shape[:-2] + (xc.shape[-2] // 2, xc.shape[-1] // 2), dtype=x.dtype, device=x.device)
        codes = torch.empty((y.numel() + 15) // 16, dtype=torch.int32, device=x.device)
        B.bt_maxpool2x2_fwd(xc, y, codes)
        ctx.save_for_backward(codes)
        ctx.in_shape = tuple(xc.shape)
        return y

    @staticmethod
    def backward(ctx, grad: torch.Tensor):
        (codes,) = ctx.saved_tensors
        g = _flat_input(grad)
        gin = torch.empty(ctx.in_shape, dtype=g.dtype, device=g.device)
        B.bt_maxpool2x2_bwd(codes, g, gin)
        return gin


def maxpool2x2_stash(x: torch.Tensor) -> torch.Tensor:
    """``torch.nn.functional.max_pool2d(x, 2)`` with a 2-bit-per-output backward record (see ``MaxPool2x2Stash``)."""
    return MaxPool2x2Stash.apply(x)


class ReLUMaxPool2x2Stash(torch.autograd.Function):
    """``max_pool2d(relu(x), 2)`` computed as ``relu(max_pool2d(x, 2))``: the maximum commutes with the ReLU, so the
    pooling runs first, on the pre-activation, and the fused ReLU + stash runs on a quarter of the elements.  The
    full-size activation is never written.  Kept for the backward pass: 2 bits per pooled output and the pooled
    activation's bitmap; the pooled activation's stash is shared with the next layer's save.  Output and input
    gradient are those of the two-step form: a window with a positive maximum has the same winner either way, and
    a window without one has a zero output and an all-zero gradient whichever position its code names."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, hooks: Optional[stash_saved_activations] = None):
        if x.dim() < 2 or x.shape[-1] % 2 or x.shape[-2] % 2 or x.numel() == 0:
            raise ValueError("relu_maxpool2x2_stash: the last two dimensions must be even and non-empty")
        xc = _flat_input(x)
        y = torch.empty(xc.shape[:-2] + (xc.shape[-2] // 2, xc.shape[-1] // 2), dtype=x.dtype, device=x.device)
        codes = torch.empty((y.numel() + 15) // 16, dtype=torch.int32, device=x.device)
        B.bt_maxpool2x2_fwd(xc, y, codes)
        flat = y.view(-1)
        if hooks is not None and hooks.arena is not None:
            bitmap, prefix, nnz_word, off_word, stored = _compress_arena(flat, hooks, relu_into=flat)
            hooks.share(y, PackedActivation(bitmap, None, prefix, tuple(y.shape), y.dtype, y.device, nnz_word,
                                            arena=hooks.arena, offset=off_word, owner=hooks, stored=stored))
            hooks.dense_bytes += y.numel() * y.element_size()
        else:
            scratch = hooks.scratch if hooks is not None else _Scratch()
            bitmap, values, prefix, nnz = _compress(flat, scratch, relu_into=flat,
                                                    narrow=hooks.narrow if hooks is not None else None)
            if hooks is not None:
                packed = PackedActivation(bitmap, values, prefix, tuple(y.shape), y.dtype, y.device, nnz)
                hooks.share(y, packed)
                hooks.packed_bytes += packed.nbytes()
                hooks.dense_bytes += y.numel() * y.element_size()
        ctx.save_for_backward(codes, bitmap)
        ctx.in_shape = tuple(xc.shape)
        return y

    @staticmethod
    def backward(ctx, grad: torch.Tensor):
        codes, bitmap = ctx.saved_tensors
        g = _flat_input(grad)
        gin = torch.empty(ctx.in_shape, dtype=g.dtype, device=g.device)
        B.bt_maxpool2x2_bwd_masked(codes, bitmap, g, gin)      # the ReLU's select and the pooling's scatter in one pass
        return gin, None


def relu_maxpool2x2_stash(x: torch.Tensor, hooks: Optional[stash_saved_activations] = None) -> torch.Tensor:
    """``max_pool2d(relu(x), 2)`` with the pooling moved in front of the ReLU (see ``ReLUMaxPool2x2Stash``)."""
    return ReLUMaxPool2x2Stash.apply(x, hooks)
