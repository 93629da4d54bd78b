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
