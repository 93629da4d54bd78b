"""The batched forms (bt_compress_batch, bt_relu_fwd_compress_batch): every tensor of a batch must get exactly what
the oracle computes for that tensor alone -- the prefix restarts at each tensor -- whatever the mix of sizes (tensors
of a fraction of a tile, of several waves of tiles, ragged, empty), whatever the number of tensors (more than one
launch holds) and on a workspace that the batch before it left full of its own words."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W
from tests.gpu_util import TDT, from_raw

pytestmark = pytest.mark.gpu

SIZES = [5, 4096, 0, 8192 * 3 + 17, 33, 16384 * 9, 1, 8192 * 160 + 4097, 4095, 8192 * 40, 65536 + 31]


def run_batch(kind, sizes, seed, fused, want_y, ws=None, zeros=0.5):
    dt = TDT[kind]
    raws = [W.random_patterns(n, kind, zeros, seed=seed + 7 * k) for k, n in enumerate(sizes)]
    xs = [from_raw(r, kind) if r.size else torch.empty(0, dtype=dt, device="cuda") for r in raws]
    sts = [B.Stash(max(n, 1), dt)for n in sizes]
    ys = [torch.empty_like(x) for x in xs] if want_y else None
    items = B.batch_items(xs, sts, ys)
    for k, n in enumerate(sizes):                                   # Stash(max(n, 1)) keeps pointers non-NULL; the count is n
        items[k].n = n
    if ws is None:
        ws = torch.empty(B.bt_batch_workspace_bytes(sizes), dtype=torch.uint8, device="cuda")
        ws.random_(0, 255)
    (B.bt_relu_fwd_compress_batch if fused else B.bt_compress_batch)(items, dt, ws)
    torch.cuda.synchronize()
    return raws, sts, ys, ws


def check_batch(oracle, kind, raws, sts, ys, fused):
    for k, raw in enumerate(raws):
        n = raw.size
        st = sts[k]
        assert st.status == B.BT_OK, (k, n)
        if fused:
            y_ref, c = oracle.relu_fwd_compress(raw, kind)
        else:
            y_ref, c = None, oracle.compress(raw)
        assert st.nnz == c.nnz, (k, n)
        if n == 0:
            continue
        assert np.array_equal(W.raw_numpy(st.bitmap)[:(n + 31) // 32].view(np.uint32), c.bitmap), (k, n)
        assert np.array_equal(W.raw_numpy(st.chunk_prefix)[:(n + 4095) // 4096].view(np.uint64), c.prefix), (k, n)
        assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values), (k, n)
        if ys is not None:
            assert np.array_equal(W.raw_numpy(ys[k]), y_ref), (k, n)


@pytest.mark.parametrize("kind", ["f32", "bf16", "f16", "f64"])
@pytest.mark.parametrize("fused,want_y", [(False, False), (True, False), (True, True)])
def test_batch_equals_the_oracle_tensor_by_tensor(oracle, kind, fused, want_y):
    raws, sts, ys, ws = run_batch(kind, SIZES, 4100, fused, want_y)
    check_batch(oracle, kind, raws, sts, ys, fused)
    # the same workspace again, other data, other sizes: nothing of the first batch may be taken for the second's
    raws, sts, ys, _ = run_batch(kind, SIZES[::-1], 977, fused, want_y, ws=ws, zeros=0.8)
    check_batch(oracle, kind, raws, sts, ys, fused)


def test_more_tensors_than_one_launch_holds(oracle):
    sizes = [4096 * (1 + k % 5) + k for k in range(2 * B.MAX_BATCH_PER_LAUNCH + 3)]
    raws, sts, ys, _ = run_batch("f32", sizes, 31, False, False)
    check_batch(oracle, "f32", raws, sts, ys, False)


def test_batch_under_a_cta_limit(oracle):
    B.bt_set_max_ctas(3)
    try:
        raws, sts, ys, _ = run_batch("bf16", SIZES, 555, True, True)
    finally:
        B.bt_set_max_ctas(0)
    check_batch(oracle, "bf16", raws, sts, ys, True)


def test_batch_argument_checks():
    L = B.lib()
    x = torch.zeros(64, device="cuda")
    st = B.Stash(64, torch.float32)
    ws = torch.empty(B.bt_batch_workspace_bytes([64, 64]), dtype=torch.uint8, device="cuda")
    items = B.batch_items([x, x], [st, st], [x, x])
    assert B.bt_compress_batch(items, torch.float32, ws, check=False) == B.BT_ERR_SHAPE          # the plain form has no y
    items[1].y_out = None
    assert B.bt_relu_fwd_compress_batch(items, torch.float32, ws, check=False) == B.BT_ERR_SHAPE  # y for all or none
    items[0].y_out = None
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    assert B.bt_compress_batch(items, torch.float32, small, check=False) == B.BT_ERR_WORKSPACE
    items[1].bitmap = None
    assert B.bt_compress_batch(items, torch.float32, ws, check=False) == B.BT_ERR_NULL
    assert L.bt_compress_batch(None, 0, B.BT_F32, None, 0, None) == B.BT_OK


@pytest.mark.parametrize("kind", ["f32", "bf16", "f16", "f64"])
def test_batched_consumers_equal_the_oracle_tensor_by_tensor(oracle, kind):
    """bt_decompress_batch and bt_relu_bwd_from_bitmap_batch on the stashes a batched compressor wrote: per tensor
    the oracle's restored tensor and masked gradient, outputs between guard regions."""
    from tests.gpu_util import Guarded
    dt = TDT[kind]
    raws, sts, _, _ = run_batch(kind, SIZES, 8080, False, False)
    outs = [Guarded(max(r.size, 1), dt) for r in raws]
    items = B.batch_items([o.inner for o in outs], sts, [o.inner for o in outs])
    for k, r in enumerate(raws):
        items[k].n = r.size
        items[k].dense = None                                        # the restore reads no dense input
    B.bt_decompress_batch(items, dt)
    torch.cuda.synchronize()
    for k, (r, o) in enumerate(zip(raws, outs)):
        assert np.array_equal(o.raw()[:r.size], r), (k, r.size)
        assert o.guards_intact()
    # backward: gradients in, masked gradients out (one tensor in place)
    g_raws = [W.random_patterns(r.size, kind, 0.1, seed=9000 + k) for k, r in enumerate(raws)]
    gs = [from_raw(g, kind) if g.size else torch.empty(1, dtype=dt, device="cuda") for g in g_raws]
    gins = [Guarded(max(g.size, 1), dt) for g in g_raws]
    ys = [gi.inner for gi in gins]
    ys[3] = gs[3]                                                     # in place
    items = B.batch_items(gs, sts, ys)
    for k, r in enumerate(raws):
        items[k].n = r.size
    B.bt_relu_bwd_from_bitmap_batch(items, dt)
    torch.cuda.synchronize()
    for k, (r, g) in enumerate(zip(raws, g_raws)):
        if r.size == 0:
            continue
        want = oracle.relu_bwd_from_bitmap(oracle.compress(r).bitmap, g)
        got = W.raw_numpy(ys[k])[:r.size]
        assert np.array_equal(got, want), (k, r.size)
        assert gins[k].guards_intact()


def test_batched_consumers_over_more_tensors_than_one_launch_holds_and_argument_checks(oracle):
    sizes = [4096 * (1 + k % 5) + k for k in range(2 * B.MAX_BATCH_PER_LAUNCH + 3)]
    raws, sts, _, _ = run_batch("bf16", sizes, 61, False, False)
    outs = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for n in sizes]
    items = B.batch_items(outs, sts, outs)
    B.bt_decompress_batch(items, torch.bfloat16)
    torch.cuda.synchronize()
    for r, o in zip(raws, outs):
        assert np.array_equal(W.raw_numpy(o), r)
    items[5].y_out = None
    assert B.bt_decompress_batch(items, torch.bfloat16, check=False) == B.BT_ERR_NULL
    assert B.bt_relu_bwd_from_bitmap_batch(items, torch.bfloat16, check=False) == B.BT_ERR_NULL
    items[5].y_out = outs[5].data_ptr() + 2
    assert B.bt_decompress_batch(items, torch.bfloat16, check=False) == B.BT_ERR_ALIGN
    assert B.lib().bt_decompress_batch(None, 0, B.BT_F32, None) == B.BT_OK
    assert B.lib().bt_decompress_batch(items, 1, 11, None) == B.BT_ERR_DTYPE


def _arena_batch(kind, sizes, seed, fused, arena_bytes, cursor0=0, zeros=0.5):
    dt = TDT[kind]
    raws = [W.random_patterns(n, kind, zeros, seed=seed + 7 * k) for k, n in enumerate(sizes)]
    xs = [from_raw(r, kind) if r.size else torch.empty(0, dtype=dt, device="cuda") for r in raws]
    sts = [B.Stash(max(n, 1), dt, values_capacity=1) for n in sizes]          # the values go to the arena, not here
    items = B.batch_items(xs, sts)
    for k, n in enumerate(sizes):
        items[k].n = n
        items[k].values = None
        items[k].values_capacity = 0
    arena = torch.full((arena_bytes + 4096,), 0x5A, dtype=torch.uint8, device="cuda")
    cursor = torch.full((1,), cursor0, dtype=torch.int64, device="cuda")
    offsets = torch.full((len(sizes),), -7, dtype=torch.int64, device="cuda")
    ws = torch.empty(B.bt_batch_workspace_bytes(sizes), dtype=torch.uint8, device="cuda")
    ws.random_(0, 255)
    B.bt_compress_arena_batch(items, dt, arena[:arena_bytes], cursor, offsets, ws, fused=fused)
    torch.cuda.synchronize()
    return raws, sts, items, arena, cursor, offsets


@pytest.mark.parametrize("kind", ["f32", "bf16", "f16", "f64"])
@pytest.mark.parametrize("fused", [False, True])
def test_arena_batch_is_the_sequence_of_single_arena_pushes(oracle, kind, fused):
    """Values of all tensors back to back behind the cursor, 16-byte granules, exactly as one bt_compress_arena call
    per tensor would leave them; offsets, cursor, bitmaps, prefix arrays and counts against the oracle; nothing
    written beyond the final cursor; then the whole batch restored from the arena by one call."""
    es = np.dtype(W.random_patterns(1, kind, 0.0, seed=0).dtype).itemsize
    raws, sts, items, arena, cursor, offsets = _arena_batch(kind, SIZES, 321, fused, 64 << 20, cursor0=4096)
    at = 4096
    for k, raw in enumerate(raws):
        c = oracle.relu_fwd_compress(raw, kind)[1] if fused else oracle.compress(raw)
        assert sts[k].status == B.BT_OK and sts[k].nnz == c.nnz, k
        if raw.size == 0:
            assert int(offsets[k].item()) == 0
            continue
        assert int(offsets[k].item()) == at, k
        got = arena[at:at + c.nnz * es].cpu().numpy().view(raw.dtype)
        assert np.array_equal(got, c.values), k
        assert np.array_equal(W.raw_numpy(sts[k].bitmap)[:(raw.size + 31) // 32].view(np.uint32), c.bitmap), k
        assert np.array_equal(W.raw_numpy(sts[k].chunk_prefix)[:(raw.size + 4095) // 4096].view(np.uint64), c.prefix), k
        at += (c.nnz * es + 15) // 16 * 16
    assert int(cursor.item()) == at
    assert bool((arena[:4096] == 0x5A).all().item()) and bool((arena[at:] == 0x5A).all().item())
    # restore all of them with one call
    dt = TDT[kind]
    outs = [torch.empty(max(r.size, 1), dtype=dt, device="cuda") for r in raws]
    ritems = B.batch_items(outs, sts, outs)
    for k, r in enumerate(raws):
        ritems[k].n = r.size
        ritems[k].values = None
    B.bt_decompress_arena_batch(ritems, dt, arena, offsets)
    torch.cuda.synchronize()
    for k, raw in enumerate(raws):
        want = oracle.relu_fwd_compress(raw, kind)[0] if fused else raw
        assert np.array_equal(W.raw_numpy(outs[k])[:raw.size], want), k


def test_arena_batch_over_several_launches_and_an_arena_that_runs_full(oracle):
    sizes = [4096 * (1 + k % 5) + k for k in range(2 * B.MAX_BATCH_PER_LAUNCH + 3)]
    raws, sts, items, arena, cursor, offsets = _arena_batch("f32", sizes, 77, False, 16 << 20)
    at = 0
    for k, raw in enumerate(raws):                               # the cursor runs on from launch to launch
        c = oracle.compress(raw)
        assert sts[k].status == B.BT_OK and int(offsets[k].item()) == at
        assert np.array_equal(arena[at:at + 4 * c.nnz].cpu().numpy().view(np.uint32), c.values)
        at += (4 * c.nnz + 15) // 16 * 16
    assert int(cursor.item()) == at
    # an arena with room for the first two tensors only: the others report BT_ERR_CAPACITY, the cursor stays behind
    # the second, their counts, bitmaps and prefix arrays are still complete
    sizes = [8192 * 3 + 5, 4096, 8192 * 30 + 1, 100, 8192 * 2]
    counts = [oracle.compress(W.random_patterns(n, "f32", 0.5, seed=500 + 7 * k)).nnz for k, n in enumerate(sizes)]
    room = sum((4 * z + 15) // 16 * 16 for z in counts[:2]) + 16
    raws, sts, items, arena, cursor, offsets = _arena_batch("f32", sizes, 500, False, room)
    end2 = room - 16
    assert [st.status for st in sts] == [B.BT_OK, B.BT_OK, B.BT_ERR_CAPACITY, B.BT_ERR_CAPACITY, B.BT_ERR_CAPACITY]
    assert int(cursor.item()) == end2 and [int(o) for o in offsets[:2].tolist()] == [0, (4 * counts[0] + 15) // 16 * 16]
    assert [int(o) for o in offsets[2:].tolist()] == [-7, -7, -7]
    for k, raw in enumerate(raws):
        c = oracle.compress(raw)
        assert sts[k].nnz == c.nnz
        assert np.array_equal(W.raw_numpy(sts[k].bitmap)[:(raw.size + 31) // 32].view(np.uint32), c.bitmap)
        assert np.array_equal(W.raw_numpy(sts[k].chunk_prefix)[:(raw.size + 4095) // 4096].view(np.uint64), c.prefix)
    assert bool((arena[room:] == 0x5A).all().item())           # nothing beyond the arena, whatever did not fit


@pytest.mark.parametrize("kind", ["bf16", "f16"])
def test_batch_of_two_byte_runs_at_every_offset_from_a_16_byte_boundary(oracle, kind):
    """The batched kernel's copy-out of 2-byte runs (16-byte units, single values at the ragged ends) on tensors
    whose runs start at each of the eight positions relative to a unit."""
    from tests.test_gpu_parity import _runs_at_offset
    dt = TDT[kind]
    raws = [_runs_at_offset(kind, lead, 7100 + lead) for lead in range(8)]
    xs = [from_raw(r, kind) for r in raws]
    sts = [B.Stash(r.size, dt) for r in raws]
    ws = torch.empty(B.bt_batch_workspace_bytes([r.size for r in raws]), dtype=torch.uint8, device="cuda")
    B.bt_compress_batch(B.batch_items(xs, sts, None), dt, ws)
    torch.cuda.synchronize()
    check_batch(oracle, kind, raws, sts, None, False)


@pytest.mark.parametrize("kind", ["bf16", "f16"])
@pytest.mark.parametrize("want_y", [False, True])
def test_fused_batch_on_every_two_byte_pattern(oracle, kind, want_y):
    """The batched fused ReLU decides in the element's own type like the single-tensor kernel: all 65536 patterns of
    the type (shuffled, as two tensors of one batch) against the oracle."""
    rng = np.random.default_rng(4242)
    raws = [rng.permutation(np.arange(65536, dtype=np.uint16)), rng.permutation(np.arange(65536, dtype=np.uint16))[:40001]]
    dt = TDT[kind]
    xs = [from_raw(r, kind) for r in raws]
    sts = [B.Stash(r.size, dt) for r in raws]
    ys = [torch.empty_like(x) for x in xs] if want_y else None
    ws = torch.empty(B.bt_batch_workspace_bytes([r.size for r in raws]), dtype=torch.uint8, device="cuda")
    B.bt_relu_fwd_compress_batch(B.batch_items(xs, sts, ys), dt, ws)
    torch.cuda.synchronize()
    check_batch(oracle, kind, raws, sts, ys, True)
