"""GPU parity: every output of every C-ABI entry point, bit for bit, against the
CPU oracle on the same seeded inputs.  All calls go through the ctypes binding
of libbittrain.so."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

KINDS = ["f32", "f16", "bf16", "f64"]
SIZES = list(W.EDGE_SIZES) + [200704, 8192 * 37 + 5, 1 << 20]


@pytest.fixture(scope="module")
def G():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from tests import gpu_util
    B.lib()
    return gpu_util


def assert_same_compressed(g, c):
    assert g.guards_ok
    assert g.status == B.BT_OK
    assert g.nnz == c.nnz
    assert np.array_equal(g.bitmap, c.bitmap)
    assert np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values, c.values)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("n", SIZES)
def test_compress_decompress_edge_sizes(G, oracle, kind, n):
    x = W.random_patterns(n, kind, 0.5, seed=1000 + n)
    c = oracle.compress(x)
    g = G.gpu_compress(G.from_raw(x, kind))
    assert_same_compressed(g, c)
    out, ok = G.gpu_decompress(c.bitmap, c.values, c.prefix, n, kind)
    assert ok and np.array_equal(out, x)
    assert B.bt_compressed_bytes(n, g.nnz, G.TDT[kind]) == oracle.compressed_bytes(n, c.nnz, x.dtype.itemsize)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("zf", [0.0, 0.25, 0.9, 0.99, 1.0])
def test_compress_decompress_sparsity_levels(G, oracle, kind, zf):
    n = 8192 * 301 + 4097 + 13        # many tiles per CTA is not reached here, many CTAs are; ragged tail
    x = W.random_patterns(n, kind, zf, seed=int(zf * 100) + 5)
    c = oracle.compress(x)
    g = G.gpu_compress(G.from_raw(x, kind))
    assert_same_compressed(g, c)
    out, ok = G.gpu_decompress(g.bitmap, g.values, g.prefix, n, kind)
    assert ok and np.array_equal(out, x)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("n", [0, 1, 33, 4097, 8192 * 3 + 1000, 200704, 8192 * 150 + 77])
@pytest.mark.parametrize("mode", ["stash_only", "with_y", "in_place"])
def test_relu_fwd_compress(G, oracle, kind, n, mode):
    x = W.random_patterns(n, kind, 0.1, seed=2000 + n)
    y_ref, c = oracle.relu_fwd_compress(x, kind)
    xt = G.from_raw(x, kind)
    g = G.gpu_compress(xt, relu=True, want_y=(mode == "with_y"), in_place=(mode == "in_place"))
    assert_same_compressed(g, c)
    if mode == "stash_only":
        assert g.y is None
        assert np.array_equal(W.raw_numpy(xt), x)           # the input is left alone
    else:
        assert np.array_equal(g.y, y_ref)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("n", [0, 1, 7, 33, 4097, 8192 * 3 + 1003, 200704, (1 << 20) + 5])
@pytest.mark.parametrize("in_place", [False, True])
def test_relu_bwd_from_bitmap(G, oracle, kind, n, in_place):
    x = W.random_patterns(n, kind, 0.3, seed=3000 + n)
    gr = W.random_patterns(n, kind, 0.05, seed=4000 + n)    # gradients with NaN, inf, -0 patterns inside
    _, c = oracle.relu_fwd_compress(x, kind)
    ref = oracle.relu_bwd_from_bitmap(c.bitmap, gr)
    if n == 0:
        bm = np.zeros(1, np.uint32)
    else:
        bm = c.bitmap
    out, ok = G.gpu_relu_bwd(bm, G.from_raw(gr, kind) if n else torch.empty(0, dtype=G.TDT[kind], device="cuda"),
                             in_place=in_place)
    assert ok and np.array_equal(out, ref)


def test_cfg1_round_trip(G, oracle):
    x = W.cfg1("cuda")
    xr = W.raw_numpy(x)
    c = oracle.compress(xr)
    g = G.gpu_compress(x)
    assert_same_compressed(g, c)
    out, ok = G.gpu_decompress(g.bitmap, g.values, g.prefix, x.numel(), "f32")
    assert ok and np.array_equal(out, xr)
    assert B.bt_compressed_bytes(x.numel(), g.nnz, torch.float32) == x.numel() // 8 + 4 * g.nnz + 8 * 49


@pytest.mark.parametrize("variant", ["iid", "clustered"])
@pytest.mark.parametrize("s", W.SPARSITY_SWEEP)
def test_cfg3_reduced(G, oracle, variant, s):
    n = 1 << 22
    idx = W.SPARSITY_SWEEP.index(s)
    x = (W.cfg3_iid if variant == "iid" else W.cfg3_clustered)(n, s, idx, "cuda")
    xr = W.raw_numpy(x)
    c = oracle.compress(xr)
    g = G.gpu_compress(x)
    assert_same_compressed(g, c)
    out, ok = G.gpu_decompress(g.bitmap, g.values, g.prefix, n, "f32")
    assert ok and np.array_equal(out, xr)


def test_capacity_overflow_reports_and_stays_in_bounds(G, oracle):
    n = 8192 * 20 + 100
    x = W.random_patterns(n, "f32", 0.5, seed=77)
    c = oracle.compress(x)
    cap = c.nnz // 2
    g = G.gpu_compress(G.from_raw(x, "f32"), capacity=cap)
    assert g.guards_ok                                  # nothing written past the capacity
    assert g.status == B.BT_ERR_CAPACITY
    assert g.nnz == c.nnz                               # the true count is still reported
    assert np.array_equal(g.bitmap, c.bitmap) and np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values_all[:cap], c.values[:cap])


def test_workspace_is_reusable_without_clearing(G, oracle):
    n = 8192 * 40 + 1
    ws = B.new_workspace(n)
    ws.fill_(0xFF)                                      # garbage in: the call must not depend on it
    for seed in (1, 2, 3):
        x = W.random_patterns(n, "f16", 0.6, seed=seed)
        c = oracle.compress(x)
        st = B.Stash(n, torch.float16)
        B.bt_compress(G.from_raw(x, "f16"), st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
        torch.cuda.synchronize()
        assert st.nnz == c.nnz and st.status == B.BT_OK
        assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values)
        assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), c.prefix)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("offset_words", [1, 2, 3])
def test_bitmap_at_any_four_byte_boundary(G, oracle, kind, offset_words):
    """A bitmap that starts 4, 8 or 12 bytes off a 16-byte boundary (a slice of a larger buffer) goes through every
    kernel that writes or reads one: compress, fused forward, decompress, bitmap backward, masked gather, ReLU6
    backward, the batched form."""
    n = 8192 * 21 + 4097 + 9
    dt = G.TDT[kind]
    raw = W.random_patterns(n, kind, 0.5, seed=600 + offset_words)
    x = G.from_raw(raw, kind)
    c = oracle.compress(raw)
    words = (n + 31) // 32
    room = torch.full((words + 8,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    bitmap = room[offset_words:offset_words + words]
    assert bitmap.data_ptr() % 16 == 4 * offset_words
    st = B.Stash(n, dt)
    ws = B.new_workspace(n)
    B.bt_compress(x, bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
    torch.cuda.synchronize()
    assert st.status == B.BT_OK and st.nnz == c.nnz
    assert np.array_equal(W.raw_numpy(bitmap).view(np.uint32), c.bitmap)
    assert (room[:offset_words] == 0x5A5A5A5A).all() and (room[offset_words + words:] == 0x5A5A5A5A).all()
    assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values)
    # readers
    back = torch.empty_like(x)
    B.bt_decompress(bitmap, st.values, st.chunk_prefix, back)
    assert np.array_equal(W.raw_numpy(back), raw)
    g_raw = W.random_patterns(n, kind, 0.1, seed=601)
    g = G.from_raw(g_raw, kind)
    gin = torch.empty_like(g)
    B.bt_relu_bwd_from_bitmap(bitmap, g, gin)
    assert np.array_equal(W.raw_numpy(gin), oracle.relu_bwd_from_bitmap(c.bitmap, g_raw))
    vals2 = torch.empty(max(c.nnz, 1), dtype=dt, device="cuda")
    y2 = torch.empty_like(x)
    B.bt_mask_compress(g, bitmap, st.chunk_prefix, y2, vals2)
    y_ref, v_ref = oracle.mask_compress(g_raw, c.bitmap)
    assert np.array_equal(W.raw_numpy(vals2[:c.nnz]), v_ref) and np.array_equal(W.raw_numpy(y2), y_ref)
    B.bt_relu6_bwd_from_stash(bitmap, st.values, st.chunk_prefix, g, gin)
    assert np.array_equal(W.raw_numpy(gin), oracle.relu6_bwd_from_stash(c, kind, g_raw))
    # fused forward and the batched form writing the same unaligned bitmap
    y_ref, cr = oracle.relu_fwd_compress(raw, kind)
    B.bt_relu_fwd_compress(x, None, bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
    torch.cuda.synchronize()
    assert st.nnz == cr.nnz and np.array_equal(W.raw_numpy(bitmap).view(np.uint32), cr.bitmap)
    st.bitmap = bitmap
    items = B.batch_items([x], [st])
    B.bt_compress_batch(items, dt, torch.empty(B.bt_batch_workspace_bytes([n]), dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert st.nnz == c.nnz and np.array_equal(W.raw_numpy(bitmap).view(np.uint32), c.bitmap)
    assert (room[:offset_words] == 0x5A5A5A5A).all() and (room[offset_words + words:] == 0x5A5A5A5A).all()


def _runs_at_offset(kind, lead, seed):
    """2-byte patterns whose packed runs start `lead` values past a 16-byte boundary of values[]: segment 0
    (1024 elements) keeps exactly `lead` non-zeros, then come full segments (runs of 1024 values), segments
    with 1..15 survivors (runs shorter than one 16-byte unit, or one unit and ragged ends), an empty segment
    and a ragged tail."""
    n = 16384 * 5 + 1024 * 3 + 777
    x = W.random_patterns(n, kind, 0.0, seed=seed)
    rng = np.random.default_rng(seed)
    dense = x[:1024 * 6]
    dense[(dense & 0x7FFF) == 0] = 0x3F80                           # five runs of exactly 1024 values
    x[lead:1024] = 0
    for seg, keep in zip(range(20, 36), range(0, 16)):              # segments of the second tile: 0..15 survivors
        lo = 1024 * seg
        kill = np.ones(1024, dtype=bool)
        kill[rng.choice(1024, size=keep, replace=False)] = False
        x[lo:lo + 1024][kill] = 0
    return x


@pytest.mark.parametrize("kind", ["bf16", "f16"])
@pytest.mark.parametrize("lead", range(8))
def test_two_byte_runs_at_every_offset_from_a_16_byte_boundary(G, oracle, kind, lead):
    """The packed runs of 2-byte values leave in 16-byte units with single values at their ragged ends: every
    position of a run's start relative to the unit, full-length runs, runs of fewer values than a unit."""
    x = _runs_at_offset(kind, lead, 7000 + lead)
    c = oracle.compress(x)
    g = G.gpu_compress(G.from_raw(x, kind))
    assert_same_compressed(g, c)
    y_ref, cr = oracle.relu_fwd_compress(x, kind)
    g = G.gpu_compress(G.from_raw(x, kind), relu=True, want_y=True)
    assert_same_compressed(g, cr)
    assert np.array_equal(g.y, y_ref)
