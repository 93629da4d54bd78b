"""A bounded wait that runs out: the kernel must return by itself, report BT_ERR_TIMEOUT in the status
word, write nothing outside its buffers, and leave the workspace and the context usable.

The failure is made without faulting or hanging anything: a build of the library with test hooks
(tests/checking_libs.py, -DBT_TEST_HOOKS; the product library has no such entry point) sets the bound of
every wait inside the compress kernels to a few nanoseconds, far less than the first bulk copy of a tile
takes, so the first wait of every CTA runs out although nothing is wrong.  The copies already in flight
are still awaited (with their own, fixed bound) before a CTA retires.
"""
import time

import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W
from tests import checking_libs as C
from tests.gpu_util import Guarded, from_raw

pytestmark = pytest.mark.gpu


@pytest.fixture()
def hooks(monkeypatch):
    L = C.hooks_lib()
    monkeypatch.setattr(B, "_lib", L)
    yield L
    L.bt_test_set_wait_ns(2_000_000_000)


def _buffers(n, dtype, cap=None):
    return (Guarded((n + 31) // 32, torch.int32), Guarded(n if cap is None else cap, dtype),
            Guarded((n + 4095) // 4096, torch.int64), Guarded(1, torch.int64), Guarded(1, torch.int32))


@pytest.mark.parametrize("kind,limit_ns", [("f32", 0), ("f32", 50), ("bf16", 100), ("f64", 50)])
def test_wait_runs_out_then_workspace_is_reusable(hooks, oracle, kind, limit_ns):
    n = 148 * 8192 * 5 + 4097 * 3 + 5          # several waves of tiles on every SM and a ragged tail
    raw_a = W.random_patterns(n, kind, 0.5, seed=41)
    raw_b = W.random_patterns(n, kind, 0.7, seed=42)
    x_a, x_b = from_raw(raw_a, kind), from_raw(raw_b, kind)
    ws = B.new_workspace(n)
    bitmap, values, prefix, nnz, status = _buffers(n, x_a.dtype)
    status.inner.fill_(-1)

    before = hooks.bt_test_set_wait_ns(limit_ns)
    assert before == 2_000_000_000              # the product's bound
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    rc = B.bt_compress(x_a, bitmap.inner, values.inner, prefix.inner, nnz.inner, ws, status.inner, check=False)
    torch.cuda.synchronize()
    took = time.perf_counter() - t0
    assert rc == B.BT_OK                        # the host saw nothing wrong: the launch itself succeeded
    assert int(status.inner.item()) == B.BT_ERR_TIMEOUT
    assert took < 1.0, f"the kernel took {took:.3f} s to give up"
    assert all(g.guards_intact() for g in (bitmap, values, prefix, nnz, status))

    # the next ordinary launch on the same workspace, other data: exactly the oracle's result
    assert hooks.bt_test_set_wait_ns(2_000_000_000) == limit_ns
    B.bt_compress(x_b, bitmap.inner, values.inner, prefix.inner, nnz.inner, ws, status.inner)
    torch.cuda.synchronize()
    c = oracle.compress(raw_b)
    assert int(status.inner.item()) == B.BT_OK and int(nnz.inner.item()) == c.nnz
    assert np.array_equal(bitmap.raw().view(np.uint32), c.bitmap)
    assert np.array_equal(prefix.raw().view(np.uint64), c.prefix)
    assert np.array_equal(values.raw()[:c.nnz], c.values)
    assert all(g.guards_intact() for g in (bitmap, values, prefix, nnz, status))


def test_fused_and_batched_forms_time_out_cleanly(hooks, oracle):
    sizes = [8192 * 300 + 77, 5, 8192 * 40, 4096 * 3 + 1]
    raws = [W.random_patterns(n, "f16", 0.5, seed=50 + i) for i, n in enumerate(sizes)]
    xs = [from_raw(r, "f16") for r in raws]
    stashes = [B.Stash(n, torch.float16, "cuda") for n in sizes]
    ys = [Guarded(n, torch.float16) for n in sizes]
    ws = torch.empty(B.bt_batch_workspace_bytes(sizes), dtype=torch.uint8, device="cuda")
    items = B.batch_items(xs, stashes, [y.inner for y in ys])

    hooks.bt_test_set_wait_ns(20)
    t0 = time.perf_counter()
    rc = B.bt_relu_fwd_compress_batch(items, torch.float16, ws, check=False)
    torch.cuda.synchronize()
    assert rc == B.BT_OK and time.perf_counter() - t0 < 1.0
    assert stashes[0].status == B.BT_ERR_TIMEOUT          # the tensor with tiles on every SM
    assert all(y.guards_intact() for y in ys)

    hooks.bt_test_set_wait_ns(2_000_000_000)
    B.bt_relu_fwd_compress_batch(items, torch.float16, ws)
    torch.cuda.synchronize()
    for raw, st, y in zip(raws, stashes, ys):
        y_ref, c = oracle.relu_fwd_compress(raw, "f16")
        assert st.status == B.BT_OK and st.nnz == c.nnz
        assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), c.bitmap)
        assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), c.prefix)
        assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values)
        assert np.array_equal(y.raw(), y_ref) and y.guards_intact()


def test_batched_arena_form_times_out_cleanly(hooks, oracle):
    """The batched arena form has one more wait (a tensor's place in the arena comes from the tensor before it):
    under a limit of a few nanoseconds the launch gives up by itself, and the next ordinary launch on the same
    workspace and arena is the oracle's."""
    sizes = [8192 * 200 + 5, 8192 * 150, 4097, 8192 * 170 + 1]
    raws = [W.random_patterns(n, "f32", 0.5, seed=90 + i) for i, n in enumerate(sizes)]
    xs = [from_raw(r, "f32") for r in raws]
    stashes = [B.Stash(n, torch.float32, "cuda", values_capacity=1) for n in sizes]
    items = B.batch_items(xs, stashes)
    arena = Guarded(sum(sizes), torch.float32)
    cursor = torch.zeros(1, dtype=torch.int64, device="cuda")
    offsets = torch.zeros(len(sizes), dtype=torch.int64, device="cuda")
    ws = torch.empty(B.bt_batch_workspace_bytes(sizes), dtype=torch.uint8, device="cuda")

    hooks.bt_test_set_wait_ns(30)
    t0 = time.perf_counter()
    rc = B.bt_compress_arena_batch(items, torch.float32, arena.inner.view(torch.uint8), cursor, offsets, ws, check=False)
    torch.cuda.synchronize()
    assert rc == B.BT_OK and time.perf_counter() - t0 < 1.0
    assert stashes[0].status == B.BT_ERR_TIMEOUT and arena.guards_intact()

    hooks.bt_test_set_wait_ns(2_000_000_000)
    cursor.zero_()
    B.bt_compress_arena_batch(items, torch.float32, arena.inner.view(torch.uint8), cursor, offsets, ws)
    torch.cuda.synchronize()
    at = 0
    raw_arena = arena.inner.view(torch.uint8)
    for k, raw in enumerate(raws):
        c = oracle.compress(raw)
        assert stashes[k].status == B.BT_OK and stashes[k].nnz == c.nnz and int(offsets[k].item()) == at
        assert np.array_equal(raw_arena[at:at + 4 * c.nnz].cpu().numpy().view(np.uint32), c.values)
        at += (4 * c.nnz + 15) // 16 * 16
    assert int(cursor.item()) == at and arena.guards_intact()
