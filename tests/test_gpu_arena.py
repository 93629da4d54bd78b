"""Arena forms of the compressor: several tensors are stashed one after another behind a device-side cursor;
bitmap, prefix, nnz and the values found at the reported offsets match the CPU oracle bit for bit, the cursor
advances by exactly the (16-byte rounded) bytes pushed, an arena that is too small reports BT_ERR_CAPACITY and
leaves the cursor alone, and bt_decompress_arena restores every tensor."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

TDT = W.TORCH_DTYPES


def dev_tensor(raw, kind):
    iv = {2: np.int16, 4: np.int32, 8: np.int64}[raw.dtype.itemsize]
    return torch.from_numpy(raw.view(iv).copy()).cuda().view(TDT[kind])


def test_pushes_of_mixed_types_and_round_trip(oracle):
    B.lib()
    dev = "cuda"
    arena = torch.full((64 << 20,), 0x5A, dtype=torch.uint8, device=dev)
    cursor = torch.zeros(1, dtype=torch.int64, device=dev)
    ws = B.new_workspace(1 << 22, dev)
    plan = [("f32", 8192 * 37 + 5, None), ("bf16", 200704, 0.0), ("f64", 4097, None), ("f16", 0, None),
            ("f32", 1 << 20, 0.05), ("bf16", 33, None), ("f32", 16384 * 9 + 1, 0.0)]
    records, expect_cursor = [], 0
    for k, (kind, n, tau) in enumerate(plan):
        raw = (W.near_threshold_patterns(n, kind, seed=k) if tau else W.random_patterns(n, kind, 0.6, seed=100 + k))
        x = dev_tensor(raw, kind) if n else torch.empty(0, dtype=TDT[kind], device=dev)
        if tau is None:
            y_ref, c = None, oracle.compress(raw)
        else:
            y_ref, c = oracle.prune_fwd_compress(raw, kind, tau)
        bitmap = torch.empty(max((n + 31) // 32, 1), dtype=torch.int32, device=dev)
        prefix = torch.empty(max((n + 4095) // 4096, 1), dtype=torch.int64, device=dev)
        nnz = torch.full((1,), -1, dtype=torch.int64, device=dev)
        off = torch.full((1,), -1, dtype=torch.int64, device=dev)
        status = torch.full((1,), -1, dtype=torch.int32, device=dev)
        y = torch.empty_like(x) if tau is not None else None
        if tau is None:
            B.bt_compress_arena(x, bitmap, arena, cursor, off, prefix, nnz, ws, status, n=n)
        else:
            B.bt_prune_fwd_compress_arena(x, tau, y, bitmap, arena, cursor, off, prefix, nnz, ws, status, n=n)
        torch.cuda.synchronize()
        assert int(status.item()) == B.BT_OK and int(nnz.item()) == c.nnz
        assert int(off.item()) == expect_cursor
        es = raw.dtype.itemsize
        expect_cursor += (c.nnz * es + 15) // 16 * 16
        assert int(cursor.item()) == expect_cursor
        got = arena[int(off.item()):int(off.item()) + c.nnz * es].cpu().numpy().view(raw.dtype)
        assert np.array_equal(got, c.values)
        if n:
            assert np.array_equal(W.raw_numpy(bitmap[:(n + 31) // 32]).view(np.uint32), c.bitmap)
            assert np.array_equal(W.raw_numpy(prefix[:(n + 4095) // 4096]).view(np.uint64), c.prefix)
        if y_ref is not None:
            assert np.array_equal(W.raw_numpy(y), y_ref)
        records.append((kind, n, bitmap, prefix, off, raw if y_ref is None else y_ref))
    # nothing beyond the cursor was touched
    assert bool((arena[expect_cursor:] == 0x5A).all().item())
    # every stash decodes from the arena, in any order
    for kind, n, bitmap, prefix, off, ref in reversed(records):
        out = torch.empty(n, dtype=TDT[kind], device=dev)
        B.bt_decompress_arena(bitmap, arena, off, prefix, out, n=n)
        torch.cuda.synchronize()
        assert np.array_equal(W.raw_numpy(out), ref)
    # popping: a device write of an earlier offset makes the space reusable
    cursor.copy_(records[-1][4])
    kind, n = "f32", 8192 * 3
    raw = W.random_patterns(n, kind, 0.5, seed=999)
    c = oracle.compress(raw)
    bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
    prefix = torch.empty((n + 4095) // 4096, dtype=torch.int64, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    off = torch.zeros(1, dtype=torch.int64, device=dev)
    B.bt_compress_arena(dev_tensor(raw, kind), bitmap, arena, cursor, off, prefix, nnz, ws, None)
    torch.cuda.synchronize()
    assert int(off.item()) == int(records[-1][4].item())
    got = arena[int(off.item()):int(off.item()) + c.nnz * 4].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, c.values)


def test_arena_too_small_reports_and_keeps_the_cursor(oracle):
    B.lib()
    dev = "cuda"
    n = 8192 * 20 + 7
    raw = W.random_patterns(n, "f32", 0.5, seed=3)
    c = oracle.compress(raw)
    need = c.nnz * 4
    arena = torch.full((need - 64 + 256,), 0x5A, dtype=torch.uint8, device=dev)     # 256 bytes already in use below
    cursor = torch.full((1,), 256, dtype=torch.int64, device=dev)
    bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
    prefix = torch.empty((n + 4095) // 4096, dtype=torch.int64, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    off = torch.full((1,), 77, dtype=torch.int64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    guard = torch.full((4096,), 0x5A, dtype=torch.uint8, device=dev)                 # allocated right after, usually
    B.bt_compress_arena(dev_tensor(raw, "f32"), bitmap, arena, cursor, off, prefix, nnz, B.new_workspace(n, dev), status,
                        check=True)
    torch.cuda.synchronize()
    assert int(status.item()) == B.BT_ERR_CAPACITY
    assert int(cursor.item()) == 256 and int(off.item()) == 77                        # untouched
    assert int(nnz.item()) == c.nnz                                                   # still the true count
    assert np.array_equal(W.raw_numpy(bitmap).view(np.uint32), c.bitmap)
    assert np.array_equal(W.raw_numpy(prefix).view(np.uint64), c.prefix)
    assert bool((arena[:256] == 0x5A).all().item()) and bool((guard == 0x5A).all().item())
    # the values that did fit are the first ones
    fit = (arena.numel() - 256) // 4
    assert np.array_equal(arena[256:256 + 4 * fit].cpu().numpy().view(np.uint32), c.values[:fit])


def _around_zero_and_six(n, kind, seed):
    tdt = TDT[kind]
    t = (torch.randn(n, generator=torch.Generator().manual_seed(seed), dtype=torch.float64) * 4 + 3).to(tdt)
    x = W.raw_numpy(t).copy()
    rng = np.random.default_rng(seed)
    six = int(W.raw_numpy(torch.tensor([6.0], dtype=tdt))[0])
    pool = np.array([six, six + 1, six - 1, 0] + list(W.SPECIALS[kind]), dtype=x.dtype)
    where = rng.integers(0, n, size=max(1, n // 6))
    x[where] = pool[rng.integers(0, len(pool), size=where.size)]
    return x


def test_narrowed_and_relu6_pushes_share_one_arena(oracle):
    """The arena forms of the narrowing compressors and of the ReLU6 pair, mixed with plain pushes: 16-bit values
    advance the cursor by 2 * nnz (rounded to 16), everything found at the reported offsets is the oracle's, and
    the arena forms of the widening decompressor and of the ReLU6 backward read it back."""
    B.lib()
    dev = "cuda"
    arena = torch.full((48 << 20,), 0x5A, dtype=torch.uint8, device=dev)
    cursor = torch.zeros(1, dtype=torch.int64, device=dev)
    ws = B.new_workspace(1 << 22, dev)
    # (form, kind of the tensor, n, argument): narrow -> target type; narrow_fused -> (target type, tau); relu6 -> None
    plan = [("narrow", "f32", 8192 * 21 + 3, "f16"), ("relu6", "bf16", 200704, None), ("plain", "f32", 4097, None),
            ("narrow_fused", "f32", 16384 * 40 + 77, ("bf16", 0.0)), ("relu6", "f32", 8192 * 150 + 9, None),
            ("narrow_fused", "f32", 33, ("f16", 0.05)), ("narrow", "f32", 0, "bf16"), ("relu6", "f64", 5000, None),
            ("narrow", "f32", 1 << 20, "bf16"), ("relu6", "f16", 1, None)]
    records, expect_cursor = [], 0
    for k, (form, kind, n, arg) in enumerate(plan):
        if form == "relu6":
            raw = _around_zero_and_six(n, kind, seed=70 + k)
            y_ref, c = oracle.relu6_fwd_compress(raw, kind)
            stored = kind
        elif form == "plain":
            raw = W.random_patterns(n, kind, 0.6, seed=70 + k)
            y_ref, c, stored = None, oracle.compress(raw), kind
        elif form == "narrow":
            raw = W.random_patterns(n, kind, 0.6, seed=70 + k)
            (y_ref, c), stored = oracle.narrow_compress(raw, arg), arg
            y_ref = None
        else:
            raw = W.near_threshold_patterns(n, kind, seed=70 + k)
            y_ref, c = oracle.narrow_compress(raw, arg[0], fused=True, tau=arg[1], want_y=True)
            stored = arg[0]
        x = dev_tensor(raw, kind) if n else torch.empty(0, dtype=TDT[kind], device=dev)
        bitmap = torch.empty(max((n + 31) // 32, 1), dtype=torch.int32, device=dev)
        prefix = torch.empty(max((n + 4095) // 4096, 1), dtype=torch.int64, device=dev)
        nnz = torch.full((1,), -1, dtype=torch.int64, device=dev)
        off = torch.full((1,), -1, dtype=torch.int64, device=dev)
        status = torch.full((1,), -1, dtype=torch.int32, device=dev)
        y = torch.empty_like(x) if y_ref is not None else None
        if form == "relu6":
            B.bt_relu6_fwd_compress_arena(x, y, bitmap, arena, cursor, off, prefix, nnz, ws, status, n=n)
        elif form == "plain":
            B.bt_compress_arena(x, bitmap, arena, cursor, off, prefix, nnz, ws, status, n=n)
        elif form == "narrow":
            B.bt_compress_narrow_arena(x, TDT[arg], bitmap, arena, cursor, off, prefix, nnz, ws, status, n=n)
        else:
            B.bt_prune_fwd_compress_narrow_arena(x, TDT[arg[0]], arg[1], y, bitmap, arena, cursor, off, prefix, nnz, ws,
                                                 status, n=n)
        torch.cuda.synchronize()
        assert int(status.item()) == B.BT_OK and int(nnz.item()) == c.nnz
        assert int(off.item()) == expect_cursor
        es = c.values.dtype.itemsize
        assert es == {"f16": 2, "bf16": 2, "f32": 4, "f64": 8}[stored]
        expect_cursor += (c.nnz * es + 15) // 16 * 16
        assert int(cursor.item()) == expect_cursor
        got = arena[int(off.item()):int(off.item()) + c.nnz * es].cpu().numpy().view(c.values.dtype)
        assert np.array_equal(got, c.values)
        if n:
            assert np.array_equal(W.raw_numpy(bitmap[:(n + 31) // 32]).view(np.uint32), c.bitmap)
            assert np.array_equal(W.raw_numpy(prefix[:(n + 4095) // 4096]).view(np.uint64), c.prefix)
        if y_ref is not None:
            assert np.array_equal(W.raw_numpy(y), y_ref)
        records.append((form, kind, stored, n, bitmap, prefix, off, c))
    assert bool((arena[expect_cursor:] == 0x5A).all().item())
    for k, (form, kind, stored, n, bitmap, prefix, off, c) in enumerate(reversed(records)):
        if form in ("narrow", "narrow_fused"):
            out = torch.empty(n, dtype=torch.float32, device=dev)
            B.bt_decompress_widen_arena(bitmap, arena, off, prefix, TDT[stored], out, n=n)
            torch.cuda.synchronize()
            assert np.array_equal(W.raw_numpy(out).view(np.uint32), oracle.widen_decompress(c, stored))
            out16 = torch.empty(n, dtype=TDT[stored], device=dev)           # and through the 16-bit decompressor
            B.bt_decompress_arena(bitmap, arena, off, prefix, out16, n=n)
            torch.cuda.synchronize()
            assert np.array_equal(W.raw_numpy(out16).view(np.uint16), oracle.decompress(c))
        elif form == "relu6":
            g = W.random_patterns(n, kind, 0.05, seed=500 + k)
            ref = oracle.relu6_bwd_from_stash(c, kind, g)
            gt = dev_tensor(g, kind)
            gin = torch.empty_like(gt)
            B.bt_relu6_bwd_from_stash_arena(bitmap, arena, off, prefix, gt, gin, n=n)
            torch.cuda.synchronize()
            assert np.array_equal(W.raw_numpy(gin), ref)
            B.bt_relu6_bwd_from_stash_arena(bitmap, arena, off, prefix, gt, gt, n=n)      # over the gradient
            torch.cuda.synchronize()
            assert np.array_equal(W.raw_numpy(gt), ref)


def test_narrow_arena_capacity_counts_16_bit_elements(oracle):
    B.lib()
    dev = "cuda"
    n = 8192 * 9 + 5
    raw = W.random_patterns(n, "f32", 0.5, seed=13)
    _, c = oracle.narrow_compress(raw, "bf16")
    x = dev_tensor(raw, "f32")
    bitmap = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
    prefix = torch.empty((n + 4095) // 4096, dtype=torch.int64, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    ws = B.new_workspace(n, dev)
    for room, want in ((2 * c.nnz - 2, B.BT_ERR_CAPACITY), (2 * c.nnz, B.BT_OK)):
        room16 = (room + 15) // 16 * 16 if want == B.BT_OK else room // 16 * 16
        arena = torch.full((32 + room16,), 0x5A, dtype=torch.uint8, device=dev)
        cursor = torch.full((1,), 32, dtype=torch.int64, device=dev)
        off = torch.full((1,), 77, dtype=torch.int64, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.bt_compress_narrow_arena(x, torch.bfloat16, bitmap, arena, cursor, off, prefix, nnz, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == want and int(nnz.item()) == c.nnz
        assert bool((arena[:32] == 0x5A).all().item())
        if want == B.BT_OK:
            assert int(off.item()) == 32 and int(cursor.item()) == 32 + (2 * c.nnz + 15) // 16 * 16
            assert np.array_equal(arena[32:32 + 2 * c.nnz].cpu().numpy().view(np.uint16), c.values)
        else:
            assert int(off.item()) == 77 and int(cursor.item()) == 32
            fit = room16 // 2
            assert np.array_equal(arena[32:32 + 2 * fit].cpu().numpy().view(np.uint16), c.values[:fit])


def test_later_arena_forms_check_their_arguments():
    L = B.lib()
    n = 4096
    x = torch.zeros(n, device="cuda")
    arena = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    words = torch.zeros(4, dtype=torch.int64, device="cuda")
    bitmap = torch.zeros(n // 32, dtype=torch.int32, device="cuda")
    prefix = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = B.new_workspace(n)
    tail = (prefix.data_ptr(), words[2:].data_ptr(), ws.data_ptr(), ws.numel() * ws.element_size(), None, None)
    ar = (arena.data_ptr(), arena.numel(), words.data_ptr(), words[1:].data_ptr())
    assert L.bt_compress_narrow_arena(x.data_ptr(), n, B.BT_F32, bitmap.data_ptr(), *ar, *tail) == B.BT_ERR_DTYPE
    assert L.bt_compress_narrow_arena(x.data_ptr(), n, B.BT_F16, bitmap.data_ptr(), arena.data_ptr(), arena.numel(), None,
                                      words[1:].data_ptr(), *tail) == B.BT_ERR_NULL
    assert L.bt_relu6_fwd_compress_arena(x.data_ptr(), n, B.BT_F32, None, bitmap.data_ptr(), arena.data_ptr(), arena.numel(),
                                         words.data_ptr(), None, *tail) == B.BT_ERR_NULL
    assert L.bt_decompress_widen_arena(bitmap.data_ptr(), arena.data_ptr(), words[1:].data_ptr(), prefix.data_ptr(), n,
                                       B.BT_F32, x.data_ptr(), None) == B.BT_ERR_DTYPE
    assert L.bt_decompress_widen_arena(bitmap.data_ptr(), arena.data_ptr(), None, prefix.data_ptr(), n, B.BT_F16,
                                       x.data_ptr(), None) == B.BT_ERR_NULL
    assert L.bt_relu6_bwd_from_stash_arena(bitmap.data_ptr(), arena.data_ptr(), None, prefix.data_ptr(), x.data_ptr(), n,
                                           B.BT_F32, x.data_ptr(), None) == B.BT_ERR_NULL
    assert L.bt_relu6_bwd_from_stash_arena(bitmap.data_ptr(), arena.data_ptr(), words[1:].data_ptr() + 4, prefix.data_ptr(),
                                           x.data_ptr(), n, B.BT_F32, x.data_ptr(), None) == B.BT_ERR_ALIGN
