"""Pins the oracle's double-mask form (the zero pattern of a normalisation layer's input applied to its
output, section 3.1) to numpy library routines, to the plain compressor in the case where both must agree,
and to a worked example."""
import numpy as np
import pytest

from paper_2110_15362_b200 import workloads as W


def bits_of(bitmap: np.ndarray, n: int) -> np.ndarray:
    return np.unpackbits(bitmap.view(np.uint8), bitorder="little")[:n].astype(bool)


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n", [0, 1, 31, 32, 33, 4095, 4097, 3 * 4096 + 17, 50021])
@pytest.mark.parametrize("density", [0.0, 0.3, 1.0])
def test_matches_numpy_indexing(oracle, kind, n, density):
    rng = np.random.default_rng(n + int(density * 10))
    x = W.random_patterns(n, kind, 0.2, seed=n + 1)                  # zeros and every pattern class inside
    mask = rng.random(n) < density
    packed = np.packbits(mask, bitorder="little")
    bitmap = np.concatenate([packed, np.zeros((-packed.size) % 4, np.uint8)]).view("<u4")
    y, values = oracle.mask_compress(x, bitmap)
    assert np.array_equal(values, x[mask])                           # pushed whatever the value, zeros included
    assert np.array_equal(y, np.where(mask, x, 0).astype(x.dtype))
    # the stash (mask bitmap, values, the mask's prefix) decodes to the masked tensor with Algorithm 2
    c_mask = oracle.compress(mask.astype(x.dtype))                   # only its bitmap and prefix are used
    assert np.array_equal(c_mask.bitmap, bitmap)
    stash = type(c_mask)(bitmap, values, c_mask.prefix, int(mask.sum()), n)
    assert np.array_equal(oracle.decompress(stash), y)
    assert np.array_equal(oracle.decompress(stash, chunked=True), y)
    _, v2 = oracle.mask_compress(x, bitmap, want_y=False)
    assert np.array_equal(v2, values)


@pytest.mark.parametrize("kind", ["f32", "bf16"])
def test_own_pattern_as_mask_is_the_plain_compressor(oracle, kind):
    x = W.random_patterns(20000, kind, 0.6, seed=4)
    c = oracle.compress(x)
    y, values = oracle.mask_compress(x, c.bitmap)
    assert np.array_equal(values, c.values) and np.array_equal(y, x)


def test_worked_example(oracle):
    x = np.array([1.5, 0.0, -2.0, 3.0, 0.0, 7.0], dtype=np.float32)
    bitmap = np.array([0b011010], dtype=np.uint32)                   # elements 1, 3, 4
    y, values = oracle.mask_compress(x.view(np.uint32), bitmap)
    assert values.view(np.float32).tolist() == [0.0, 3.0, 0.0]
    assert y.view(np.float32).tolist() == [0.0, 0.0, 0.0, 3.0, 0.0, 0.0]
