"""GPU parity of the ReLU6 pair (bt_relu6_fwd_compress, bt_relu6_bwd_from_stash) against the CPU oracle, bit
for bit: values around 0 and 6, every bit-pattern class, edge sizes, in-place forms, and a full-size
MobileNetV2-shaped layer."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

KINDS = ["f32", "f16", "bf16", "f64"]


@pytest.fixture(scope="module")
def G():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from tests import gpu_util
    B.lib()
    return gpu_util


def around_zero_and_six(n, kind, seed):
    """Values spread over about [-8, 14] with exact 0, 6, their neighbours and the special patterns sprinkled in."""
    tdt = W.TORCH_DTYPES[kind]
    t = (torch.randn(n, generator=torch.Generator().manual_seed(seed), dtype=torch.float64) * 4 + 3).to(tdt)
    x = W.raw_numpy(t).copy()
    if n:
        rng = np.random.default_rng(seed)
        six = int(W.raw_numpy(torch.tensor([6.0], dtype=tdt))[0])
        pool = np.array([six, six + 1, six - 1, 0] + list(W.SPECIALS[kind]), dtype=x.dtype)
        where = rng.integers(0, n, size=max(1, n // 6))
        x[where] = pool[rng.integers(0, len(pool), size=where.size)]
    return x


def run_fwd(G, xt, mode):
    n = xt.numel()
    st = B.Stash(n, xt.dtype, "cuda")
    y = G.Guarded(n, xt.dtype) if mode == "with_y" else None
    y_t = y.inner if mode == "with_y" else (xt if mode == "in_place" else None)
    B.bt_relu6_fwd_compress(xt, y_t, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, B.new_workspace(n), st.dev_status,
                            n=n)
    torch.cuda.synchronize()
    return st, (y.raw() if y is not None else (W.raw_numpy(xt) if mode == "in_place" else None)), (y is None or y.guards_intact())


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("n", [0, 1, 33, 1025, 4097, 16384 * 3 + 1001, 200704])
@pytest.mark.parametrize("mode", ["stash_only", "with_y", "in_place"])
def test_relu6_pair(G, oracle, kind, n, mode):
    x = around_zero_and_six(n, kind, seed=300 + n)
    y_ref, c = oracle.relu6_fwd_compress(x, kind)
    xt = G.from_raw(x, kind) if n else torch.empty(0, dtype=G.TDT[kind], device="cuda")
    st, y, ok = run_fwd(G, xt, mode)
    assert ok and st.status == B.BT_OK and st.nnz == c.nnz
    if n:
        assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), c.bitmap)
        assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), c.prefix)
        assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values)
    if mode != "stash_only":
        assert np.array_equal(y, y_ref)
    # backward from the stash, out of place and over the gradient
    g = W.random_patterns(n, kind, 0.05, seed=400 + n)              # gradients with NaN, inf, -0 patterns inside
    ref = oracle.relu6_bwd_from_stash(c, kind, g)
    gt = G.from_raw(g, kind) if n else torch.empty(0, dtype=G.TDT[kind], device="cuda")
    gin = G.Guarded(n, gt.dtype)
    vals = st.values if c.nnz else torch.zeros(8, dtype=gt.dtype, device="cuda")
    B.bt_relu6_bwd_from_stash(st.bitmap, vals, st.chunk_prefix, gt, gin.inner, n=n)
    torch.cuda.synchronize()
    assert gin.guards_intact() and np.array_equal(gin.raw(), ref)
    B.bt_relu6_bwd_from_stash(st.bitmap, vals, st.chunk_prefix, gt, gt, n=n)
    torch.cuda.synchronize()
    assert np.array_equal(W.raw_numpy(gt), ref)


def test_full_size_mobilenet_layer_against_torch(G, oracle):
    """The largest ReLU6 site of the MobileNetV2-shaped set at batch 128: torch over the whole tensor, the oracle
    on sampled chunks."""
    shape = max(W.mobilenetv2_shapes(128), key=W.numel)
    n = W.numel(shape)
    pre = (torch.randn(n, device="cuda", generator=torch.Generator(device="cuda").manual_seed(5)) * 4 + 2)
    g = torch.randn(n, device="cuda", generator=torch.Generator(device="cuda").manual_seed(6))
    st = B.Stash(n, pre.dtype, "cuda")
    y = torch.empty_like(pre)
    B.bt_relu6_fwd_compress(pre, y, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, B.new_workspace(n), st.dev_status)
    gin = torch.empty_like(g)
    B.bt_relu6_bwd_from_stash(st.bitmap, st.values, st.chunk_prefix, g, gin)
    torch.cuda.synchronize()
    assert st.status == B.BT_OK
    assert torch.equal(y.view(torch.int32), (torch.nn.functional.relu6(pre) + 0.0).view(torch.int32))
    assert st.nnz == int(torch.count_nonzero(y))
    assert torch.equal(gin.view(torch.int32), torch.where((pre > 0) & (pre < 6), g, torch.zeros_like(g)).view(torch.int32))
    raw = W.raw_numpy(pre)
    bmp, pfx, vals = W.raw_numpy(st.bitmap).view(np.uint32), W.raw_numpy(st.chunk_prefix).view(np.uint64), W.raw_numpy(st.values)
    for ch in np.random.default_rng(2).integers(0, n // 4096, size=12):
        lo = int(ch) * 4096
        _, c = oracle.relu6_fwd_compress(raw[lo:lo + 4096], "f32")
        assert np.array_equal(bmp[lo // 32:lo // 32 + 128], c.bitmap)
        assert np.array_equal(vals[int(pfx[ch]):int(pfx[ch]) + c.nnz], c.values)


@pytest.mark.parametrize("kind", ["f16", "bf16"])
@pytest.mark.parametrize("mode", ["stash_only", "with_y"])
def test_every_two_byte_pattern_through_relu_and_relu6(G, oracle, kind, mode):
    """All 65536 patterns of a 2-byte type, shuffled, through the fused ReLU, the fused ReLU6 and the ReLU6
    backward: the decisions these take in the element's own type (kept iff greater than 0 or a NaN, saturated iff
    at least 6, the gradient passes iff the stashed value is below 6) must agree with the oracle's comparisons of
    the exactly widened values on every pattern -- both zeros, subnormals, 6 and its neighbours, the infinities
    and every NaN of either sign."""
    rng = np.random.default_rng(65536)
    x = rng.permutation(np.arange(65536, dtype=np.uint16))
    g = rng.permutation(np.arange(65536, dtype=np.uint16))
    xt = G.from_raw(x, kind)
    # ReLU
    y_ref, c = oracle.relu_fwd_compress(x, kind)
    r = G.gpu_compress(xt, relu=True, want_y=(mode == "with_y"))
    assert r.guards_ok and r.status == B.BT_OK and r.nnz == c.nnz
    assert np.array_equal(r.bitmap, c.bitmap) and np.array_equal(r.prefix, c.prefix) and np.array_equal(r.values, c.values)
    if mode == "with_y":
        assert np.array_equal(r.y, y_ref)
    # ReLU6 and its backward
    y6_ref, c6 = oracle.relu6_fwd_compress(x, kind)
    st, y6, ok = run_fwd(G, xt, mode)
    assert ok and st.status == B.BT_OK and st.nnz == c6.nnz
    assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), c6.bitmap)
    assert np.array_equal(W.raw_numpy(st.values[:c6.nnz]), c6.values)
    if mode == "with_y":
        assert np.array_equal(y6, y6_ref)
    gt = G.from_raw(g, kind)
    gin = G.Guarded(x.size, gt.dtype)
    B.bt_relu6_bwd_from_stash(st.bitmap, st.values, st.chunk_prefix, gt, gin.inner)
    torch.cuda.synchronize()
    assert np.array_equal(gin.raw(), oracle.relu6_bwd_from_stash(c6, kind, g)) and gin.guards_intact()
