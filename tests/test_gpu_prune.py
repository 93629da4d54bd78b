"""GPU parity of the activation-pruning entry point (bt_prune_fwd_compress) against the CPU oracle: every
output bit for bit, for the paper's thresholds and a few others, on inputs crowded around the thresholds,
on every bit-pattern class, at sizes that span several tiles and a ragged tail, and at a full-size layer."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

KINDS = ["f32", "f16", "bf16", "f64"]
TAUS = list(W.PRUNE_THRESHOLDS) + [0.3, -0.02]


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
    assert np.array_equal(g.values, c.values)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("tau", TAUS)
@pytest.mark.parametrize("n", [0, 1, 33, 4097, 16384 * 3 + 1001, 200704])
@pytest.mark.parametrize("mode", ["stash_only", "with_y", "in_place"])
def test_prune_near_thresholds(G, oracle, kind, tau, n, mode):
    x = W.near_threshold_patterns(n, kind, seed=7000 + n)
    y_ref, c = oracle.prune_fwd_compress(x, kind, tau)
    xt = G.from_raw(x, kind)
    g = G.gpu_compress(xt, tau=tau, want_y=(mode == "with_y"), in_place=(mode == "in_place"))
    assert_same(g, c)
    if mode == "stash_only":
        assert g.y is None and np.array_equal(W.raw_numpy(xt), x)
    else:
        assert np.array_equal(g.y, y_ref)
    # the backward pass is the unchanged one: the stash decodes to the pruned activation
    if n:
        out, ok = G.gpu_decompress(g.bitmap, g.values, g.prefix, n, kind)
        assert ok and np.array_equal(out, y_ref)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("tau", [0.0, 0.05, float("inf"), float("-inf"), float("nan")])
def test_prune_every_pattern_class(G, oracle, kind, tau):
    n = 16384 * 150 + 77                                      # several tiles per CTA, ragged tail
    x = W.random_patterns(n, kind, 0.2, seed=11)              # NaNs, infinities, subnormals, signed zeros
    y_ref, c = oracle.prune_fwd_compress(x, kind, tau)
    g = G.gpu_compress(G.from_raw(x, kind), tau=tau, want_y=True)
    assert_same(g, c)
    assert np.array_equal(g.y, y_ref)


@pytest.mark.parametrize("kind", KINDS)
def test_threshold_zero_is_the_relu_entry_point(G, kind):
    n = 8192 * 40 + 5
    xt = G.from_raw(W.random_patterns(n, kind, 0.3, seed=3), kind)
    a = G.gpu_compress(xt, relu=True, want_y=True)
    b = G.gpu_compress(xt, tau=0.0, want_y=True)
    assert a.nnz == b.nnz and np.array_equal(a.bitmap, b.bitmap) and np.array_equal(a.values, b.values)
    assert np.array_equal(a.prefix, b.prefix) and np.array_equal(a.y, b.y)


def test_prune_full_size_layer_and_sparsity_gain(G, oracle):
    """The largest layer of the ResNet-18-shaped set (batch 32): oracle on sampled chunks, torch over the whole
    tensor, and the point of the exercise: a larger threshold stores fewer values."""
    shape = W.resnet18_shapes(32)[0]
    pre = W.cfg2_preact(0, shape, "cuda").reshape(-1)
    n = pre.numel()
    raw = W.raw_numpy(pre)
    prev = None
    for tau in W.PRUNE_THRESHOLDS:
        g = G.gpu_compress(pre, tau=tau, want_y=True)
        assert g.guards_ok and g.status == B.BT_OK
        y_t = torch.where(pre <= torch.tensor(tau, dtype=torch.float32, device="cuda"), torch.zeros_like(pre), pre)
        assert np.array_equal(g.y, W.raw_numpy(y_t))
        assert g.nnz == int(torch.count_nonzero(y_t.view(torch.int32)).item())
        rng = np.random.default_rng(int(tau * 1000))
        for ch in rng.integers(0, n // 4096, size=16):
            lo, hi = int(ch) * 4096, int(ch) * 4096 + 4096
            _, c = oracle.prune_fwd_compress(raw[lo:hi], "f32", tau)
            assert np.array_equal(g.bitmap[lo // 32:hi // 32], c.bitmap)
            start = int(g.prefix[ch])
            assert np.array_equal(g.values_all[start:start + c.nnz], c.values)
        if prev is not None:
            assert g.nnz < prev
        prev = g.nnz
