"""GPU parity of the double-mask entry point (bt_mask_compress) against the CPU oracle, bit for bit: edge
sizes, mask densities from empty to full, masks that cover zero elements, a capacity below nnz, and the
round trip through bt_decompress with the shared bitmap and prefix array."""
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


def mask_stash(oracle, n, kind, density, seed):
    """A stash (bitmap, prefix, nnz) of a layer input with the given non-zero density."""
    src = W.random_patterns(n, kind, 1.0 - density, seed=seed, with_specials=False)
    return oracle.compress(src)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("n", list(W.EDGE_SIZES) + [200704, 8192 * 37 + 5])
@pytest.mark.parametrize("mode", ["stash_only", "with_y", "in_place"])
def test_mask_compress_edge_sizes(G, oracle, kind, n, mode):
    m = mask_stash(oracle, n, kind, 0.5, seed=50 + n)
    x = W.random_patterns(n, kind, 0.3, seed=60 + n)                    # zeros under set bits do occur
    y_ref, v_ref = oracle.mask_compress(x, m.bitmap if n else np.zeros(1, np.uint32))
    xt = G.from_raw(x, kind) if n else torch.empty(0, dtype=G.TDT[kind], device="cuda")
    bm = m.bitmap if n else np.zeros(1, np.uint32)
    pf = m.prefix if n else np.zeros(1, np.uint64)
    v, y, ok = G.gpu_mask_compress(xt, bm, pf, m.nnz, mode)
    assert ok
    assert np.array_equal(v, v_ref)
    if mode == "stash_only":
        assert y is None and np.array_equal(W.raw_numpy(xt), x)
    else:
        assert np.array_equal(y, y_ref)
    if n:
        out, ok2 = G.gpu_decompress(m.bitmap, v_ref, m.prefix, n, kind)   # the shared bitmap and prefix decode it
        assert ok2 and np.array_equal(out, y_ref)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("density", [0.0, 0.02, 0.5, 0.98, 1.0])
def test_mask_densities(G, oracle, kind, density):
    n = 4096 * 301 + 1029
    m = mask_stash(oracle, n, kind, density, seed=int(density * 100))
    x = W.random_patterns(n, kind, 0.1, seed=77)
    y_ref, v_ref = oracle.mask_compress(x, m.bitmap)
    v, y, ok = G.gpu_mask_compress(G.from_raw(x, kind), m.bitmap, m.prefix, m.nnz, "with_y")
    assert ok and np.array_equal(v, v_ref) and np.array_equal(y, y_ref)


def test_capacity_below_nnz_suppresses_stores(G, oracle):
    n = 50000
    m = mask_stash(oracle, n, "f32", 0.5, seed=5)
    x = W.random_patterns(n, "f32", 0.0, seed=6)
    _, v_ref = oracle.mask_compress(x, m.bitmap)
    cap = m.nnz // 2
    v, y, ok = G.gpu_mask_compress(G.from_raw(x, "f32"), m.bitmap, m.prefix, m.nnz, "with_y", capacity=cap)
    assert ok                                                        # nothing written past the capacity
    assert np.array_equal(v, v_ref[:cap])


def test_full_size_layer(G, oracle):
    """Largest layer of the ResNet-18-shaped set: the ReLU output's stash masks a second tensor of that shape."""
    shape = W.resnet18_shapes(32)[0]
    act = W.cfg2_layer(0, shape, "cuda").reshape(-1)
    bn_out = W.cfg2_grad(0, shape, "cuda").reshape(-1)               # any dense tensor of the same shape
    n = act.numel()
    st = B.Stash(n, act.dtype, "cuda")
    B.bt_compress(act, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, B.new_workspace(n, "cuda"), st.dev_status)
    nnz = st.nnz
    values = torch.empty(nnz, dtype=act.dtype, device="cuda")
    y = torch.empty_like(bn_out)
    B.bt_mask_compress(bn_out, st.bitmap, st.chunk_prefix, y, values)
    torch.cuda.synchronize()
    keep = act != 0
    assert torch.equal(y.view(torch.int32), torch.where(keep, bn_out, torch.zeros_like(bn_out)).view(torch.int32))
    assert torch.equal(values.view(torch.int32), bn_out[keep].view(torch.int32))
    back = torch.empty_like(bn_out)
    B.bt_decompress(st.bitmap, values, st.chunk_prefix, back)
    assert torch.equal(back.view(torch.int32), y.view(torch.int32))
    raw, bmp = W.raw_numpy(bn_out), W.raw_numpy(st.bitmap).view(np.uint32)
    pfx = W.raw_numpy(st.chunk_prefix).view(np.uint64)
    vals = W.raw_numpy(values)
    for ch in np.random.default_rng(1).integers(0, n // 4096, size=16):
        lo = int(ch) * 4096
        _, v = oracle.mask_compress(raw[lo:lo + 4096], bmp[lo // 32:lo // 32 + 128], want_y=False)
        assert np.array_equal(vals[int(pfx[ch]):int(pfx[ch]) + v.size], v)
