"""GPU parity of the down-cast-on-stash entry points (bt_compress_narrow, bt_prune_fwd_compress_narrow) against
the CPU oracle, bit for bit: the structure of the binary32 stash, 16-bit values rounded to nearest even (every
rounding boundary, overflow, underflow, NaN), the unnarrowed dense output, capacity handling, and the backward
pass through the unchanged 16-bit decompressor and the bitmap-only ReLU backward."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

TO = ["f16", "bf16"]


@pytest.fixture(scope="module")
def G():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from tests import gpu_util
    B.lib()
    return gpu_util


def assert_same(g, c):
    assert g.guards_ok and g.status == B.BT_OK
    assert g.nnz == c.nnz
    assert np.array_equal(g.bitmap, c.bitmap)
    assert np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values.view(np.uint16), c.values)


def boundary_patterns(to_kind, seed):
    """binary32 patterns whose dropped bits sit at and around the rounding tie, over every exponent, with zeros,
    NaNs and infinities mixed in, shuffled."""
    dropped = 13 if to_kind == "f16" else 16
    rng = np.random.default_rng(seed)
    upper = rng.integers(0, 1 << (32 - dropped), size=120000, dtype=np.uint64) << dropped
    tie = 1 << (dropped - 1)
    lows = np.array([0, 1, tie - 1, tie, tie + 1, (1 << dropped) - 1], dtype=np.uint64)
    x = (upper[:, None] | lows[None, :]).reshape(-1).astype(np.uint32)
    x[rng.random(x.size) < 0.3] = 0
    special = np.array([0x80000000, 0x7F800000, 0xFF800000, 0x7FC00001, 0xFF800001, 0x33000000, 0x33000001, 0xB3000000,
                        0x477FEFFF, 0x477FF000, 0xC77FF000, 0x7F7FFFFF, 0x00000001, 0x387FFFFF, 0x38800000], dtype=np.uint32)
    x[: special.size] = special
    return x


def widen_on_gpu(G, g, n, to_kind):
    """bt_decompress_widen on a stash produced on the GPU; returns the raw binary32 patterns (guards checked)."""
    bm = torch.from_numpy(g.bitmap.view(np.int32).copy()).cuda()
    vals = G.from_raw(g.values if g.values.size else np.zeros(1, g.values.dtype), to_kind)
    pf = torch.from_numpy(g.prefix.view(np.int64).copy()).cuda()
    out = G.Guarded(n, torch.float32)
    B.bt_decompress_widen(bm, vals, pf, out.inner, n=n)
    torch.cuda.synchronize()
    assert out.guards_intact()
    return out.raw().view(np.uint32)


@pytest.mark.parametrize("to_kind", TO)
@pytest.mark.parametrize("n", [0, 1, 33, 1025, 4097, 16384 * 3 + 1001, 200704])
def test_plain_form(G, oracle, to_kind, n):
    x = W.random_patterns(n, "f32", 0.5, seed=900 + n)
    _, c = oracle.narrow_compress(x, to_kind)
    g = G.gpu_compress(G.from_raw(x, "f32"), narrow=to_kind)
    assert_same(g, c)
    if n:
        # the 16-bit stash goes through the unchanged decompressor
        out, ok = G.gpu_decompress(g.bitmap, g.values, g.prefix, n, to_kind)
        assert ok and np.array_equal(out.view(np.uint16), oracle.decompress(c))
        # and through the widening one, straight into binary32
        assert np.array_equal(widen_on_gpu(G, g, n, to_kind), oracle.widen_decompress(c, to_kind))


@pytest.mark.parametrize("to_kind", TO)
def test_every_rounding_boundary(G, oracle, to_kind):
    x = boundary_patterns(to_kind, 5)
    _, c = oracle.narrow_compress(x, to_kind)
    g = G.gpu_compress(G.from_raw(x, "f32"), narrow=to_kind)
    assert_same(g, c)
    full = oracle.compress(x)                                        # structure: that of the binary32 stash
    assert np.array_equal(g.bitmap, full.bitmap) and np.array_equal(g.prefix, full.prefix) and g.nnz == full.nnz
    assert np.array_equal(widen_on_gpu(G, g, x.size, to_kind), oracle.widen_decompress(c, to_kind))


@pytest.mark.parametrize("to_kind", TO)
@pytest.mark.parametrize("tau", [0.0, 0.05])
@pytest.mark.parametrize("n", [1, 4097, 16384 * 5 + 123, 802816])
@pytest.mark.parametrize("mode", ["stash_only", "with_y", "in_place"])
def test_fused_form(G, oracle, to_kind, tau, n, mode):
    x = W.near_threshold_patterns(n, "f32", seed=8100 + n)
    y_ref, c = oracle.narrow_compress(x, to_kind, fused=True, tau=tau, want_y=True)
    xt = G.from_raw(x, "f32")
    g = G.gpu_compress(xt, tau=tau, want_y=(mode == "with_y"), in_place=(mode == "in_place"), narrow=to_kind)
    assert_same(g, c)
    if mode == "stash_only":
        assert g.y is None and np.array_equal(W.raw_numpy(xt), x)
    else:
        assert np.array_equal(g.y, y_ref)                            # the dense output stays binary32
    # ReLU backward needs only the bitmap, which is the full-precision one
    grad = torch.randn(n, generator=torch.Generator().manual_seed(n)).cuda()
    gin, ok = G.gpu_relu_bwd(g.bitmap, grad)
    assert ok and np.array_equal(gin, oracle.relu_bwd_from_bitmap(c.bitmap, W.raw_numpy(grad)))


@pytest.mark.parametrize("to_kind", TO)
def test_every_pattern_class_many_tiles(G, oracle, to_kind):
    n = 8192 * 150 * 3 + 77                                          # several tiles per CTA, ragged tail
    x = W.random_patterns(n, "f32", 0.2, seed=12)
    y_ref, c = oracle.narrow_compress(x, to_kind, fused=True, tau=0.0, want_y=True)
    g = G.gpu_compress(G.from_raw(x, "f32"), relu=True, want_y=True, narrow=to_kind)
    assert_same(g, c)
    assert np.array_equal(g.y, y_ref)


@pytest.mark.parametrize("to_kind", TO)
def test_capacity_is_counted_in_16_bit_elements(G, oracle, to_kind):
    n = 8192 * 9 + 5
    x = W.random_patterns(n, "f32", 0.5, seed=13)
    _, c = oracle.narrow_compress(x, to_kind)
    cap = c.nnz - 1000
    g = G.gpu_compress(G.from_raw(x, "f32"), narrow=to_kind, capacity=cap)
    assert g.guards_ok and g.status == B.BT_ERR_CAPACITY and g.nnz == c.nnz
    assert np.array_equal(g.bitmap, c.bitmap) and np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values_all[:cap].view(np.uint16), c.values[:cap])
    g = G.gpu_compress(G.from_raw(x, "f32"), narrow=to_kind, capacity=c.nnz)
    assert_same(g, c)


def test_argument_checks(G):
    n = 4096
    x = torch.zeros(n, device="cuda")
    st = B.Stash(n, torch.float16)
    ws = B.new_workspace(n)
    L = B.lib()
    args = (st.bitmap.data_ptr(), st.values.data_ptr(), n, st.chunk_prefix.data_ptr(), st.nnz_out.data_ptr(), ws.data_ptr(),
            ws.numel() * ws.element_size(), st.dev_status.data_ptr(), None)
    assert L.bt_compress_narrow(x.data_ptr(), n, B.BT_F32, *args) == B.BT_ERR_DTYPE      # the target must be a 16-bit type
    assert L.bt_compress_narrow(x.data_ptr(), n, B.BT_F64, *args) == B.BT_ERR_DTYPE
    assert L.bt_compress_narrow(None, n, B.BT_F16, *args) == B.BT_ERR_NULL
    assert L.bt_compress_narrow(x.data_ptr(), n, B.BT_F16, *args) == B.BT_OK
    torch.cuda.synchronize()
    assert st.status == B.BT_OK and st.nnz == 0


@pytest.mark.parametrize("from_kind", TO)
def test_widen_every_nan_and_infinity_stash(G, oracle, from_kind):
    """bt_decompress_widen on stashes that hold every 16-bit NaN and infinity of the type, both signs, quiet and
    signalling, scattered among zeros and ordinary values over several chunks: the oracle's patterns bit for bit
    (a signalling NaN stays signalling; sign and payload are kept)."""
    if from_kind == "f16":
        mant = np.arange(0, 1024, dtype=np.uint16)
        specials = np.concatenate([0x7C00 | mant, 0xFC00 | mant]).astype(np.uint16)
    else:
        specials = np.concatenate([np.arange(0x7F80, 0x8000), np.arange(0xFF80, 0x10000)]).astype(np.uint16)
    n = 4096 * 5 + 777
    x = W.random_patterns(n, from_kind, 0.5, seed=7)
    rng = np.random.default_rng(11)
    where = rng.choice(n, size=specials.size, replace=False)
    x[where] = specials
    c = oracle.compress(x)                                   # the 16-bit stash, patterns untouched
    want = oracle.widen_decompress(c, from_kind)
    assert np.isnan(want.view(np.float32)).sum() >= specials.size - 2
    got = widen_on_gpu(G, c, n, from_kind)
    assert np.array_equal(got, want)
    # and the same stash restored in its own type, then cast by torch: NaN for NaN, equal elsewhere
    plain, ok = G.gpu_decompress(c.bitmap, c.values, c.prefix, n, from_kind)
    assert ok and np.array_equal(plain, x)
