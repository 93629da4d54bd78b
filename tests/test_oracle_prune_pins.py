"""Pins the oracle's activation-pruning form (keep what exceeds a threshold, section 4 "Combining BitTrain
with Activation Pruning") to things other than itself: torch.where on exactly widened values, a closed-form
count, a worked example, and the properties that follow from the definition."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import workloads as W

UINT = {2: np.uint16, 4: np.uint32, 8: np.uint64}
NP2T = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}


def as_torch(x_raw: np.ndarray, kind: str) -> torch.Tensor:
    it = {2: torch.int16, 4: torch.int32}[x_raw.dtype.itemsize]
    return torch.from_numpy(x_raw.view({2: np.int16, 4: np.int32}[x_raw.dtype.itemsize]).copy()).view(NP2T[kind])


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("tau", W.PRUNE_THRESHOLDS + (0.3, -0.02))
@pytest.mark.parametrize("n", [0, 1, 31, 33, 4097, 20011])
def test_prune_matches_torch_where(oracle, kind, tau, n):
    x = W.near_threshold_patterns(n, kind, seed=n + 11)
    y, c = oracle.prune_fwd_compress(x, kind, tau)
    t = as_torch(x, kind)
    # widening to binary32 is exact for all three types; the threshold is a binary32 value
    pruned = t.float() <= torch.tensor(tau, dtype=torch.float32)
    y_ref = W.raw_numpy(torch.where(pruned, torch.zeros_like(t), t))
    assert np.array_equal(y, y_ref)
    # and the stash is Algorithm 1 of that tensor
    ref = oracle.compress(y_ref)
    assert c.nnz == ref.nnz
    assert np.array_equal(c.bitmap, ref.bitmap) and np.array_equal(c.values, ref.values)
    assert np.array_equal(c.prefix, ref.prefix)
    assert np.array_equal(oracle.decompress(c), y)


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
def test_threshold_zero_is_relu(oracle, kind):
    for seed in range(3):
        x = W.random_patterns(5000, kind, 0.3, seed=seed)          # every bit pattern class, NaNs included
        y0, c0 = oracle.prune_fwd_compress(x, kind, 0.0)
        y1, c1 = oracle.relu_fwd_compress(x, kind)
        assert np.array_equal(y0, y1) and c0.nnz == c1.nnz
        assert np.array_equal(c0.bitmap, c1.bitmap) and np.array_equal(c0.values, c1.values)


def test_closed_form_count_and_worked_example(oracle):
    # k/256, k = 0..255, is exact in binary32: exactly the k with k/256 > 1/16, i.e. k >= 17, survive
    x = (np.arange(256, dtype=np.float32) / 256).view(np.uint32)
    y, c = oracle.prune_fwd_compress(x, "f32", 0.0625)
    assert c.nnz == 256 - 17
    assert np.array_equal(y.view(np.float32)[:17], np.zeros(17, np.float32))
    assert np.array_equal(y[17:], x[17:])
    # worked by hand: threshold 0.01 as binary32; 0.01 itself does not exceed it, the next float does
    t = np.float32(0.01)
    vals = np.array([0.0, 0.005, t, np.nextafter(t, np.float32(1)), -1.0, np.nan, 0.2, -0.0, np.inf, -np.inf],
                    dtype=np.float32)
    y, c = oracle.prune_fwd_compress(vals.view(np.uint32), "f32", 0.01)
    yf = y.view(np.float32)
    assert c.nnz == 4 and int(c.bitmap[0]) == 0b0101101000
    assert yf[3] == vals[3] and np.isnan(yf[5]) and yf[6] == np.float32(0.2) and np.isinf(yf[8])
    assert not np.any(y[[0, 1, 2, 4, 7, 9]])                      # pruned entries are +0 bit patterns
    assert y[5] == vals.view(np.uint32)[5]                        # the NaN keeps its payload


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
def test_properties(oracle, kind):
    x = W.near_threshold_patterns(30000, kind, seed=5)
    prev = None
    for tau in (0.0, 0.01, 0.05, 0.1, 0.3):
        y, c = oracle.prune_fwd_compress(x, kind, tau)
        # pruning again with the same threshold changes nothing
        y2, c2 = oracle.prune_fwd_compress(y, kind, tau)
        assert np.array_equal(y2, y) and c2.nnz == c.nnz
        # whatever survives is an unchanged input element
        keep = y != 0
        assert np.array_equal(y[keep], x[keep])
        # a larger threshold keeps a subset (the compressed size can only shrink)
        if prev is not None:
            assert c.nnz <= prev[1] and not np.any(keep & ~prev[0])
        prev = (keep, c.nnz)
    # y is optional and does not change the stash
    _, c3 = oracle.prune_fwd_compress(x, kind, 0.05, want_y=False)
    _, c4 = oracle.prune_fwd_compress(x, kind, 0.05)
    assert c3.nnz == c4.nnz and np.array_equal(c3.values, c4.values) and np.array_equal(c3.bitmap, c4.bitmap)


def test_binary64_elements(oracle):
    rng = np.random.default_rng(3)
    x = rng.normal(0, 0.08, 10007)
    x[rng.random(x.size) < 0.2] = 0.0
    x[:4] = [np.float32(0.05), np.nextafter(np.float64(np.float32(0.05)), 1.0), np.nan, -0.0]
    for tau in (0.0, 0.05):
        y, c = oracle.prune_fwd_compress(x.view(np.uint64), "f64", tau)
        ref = np.where(x <= np.float64(np.float32(tau)), 0.0, x)          # NaN <= t is False: kept
        assert np.array_equal(y, ref.view(np.uint64))
        assert c.nnz == int(np.count_nonzero(ref.view(np.uint64)))
