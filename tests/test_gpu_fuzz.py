"""Seeded random sweep over sizes, element types, zero fractions and entry points: every output of the GPU
library equals the CPU oracle's bit for bit.  Sizes cluster around the boundaries of the kernels' units
(32-element bitmap words, 1024-element warp quarters, 4096-element chunks, 8192 / 16384-element tiles, the
148-tile first wave) and also fall anywhere up to a few waves."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

UNITS = (32, 1024, 4096, 8192, 16384, 148 * 4096, 148 * 8192, 148 * 16384)


def cases(count=72, seed=2024):
    rng = np.random.default_rng(seed)
    out = []
    for k in range(count):
        kind = ("f32", "f16", "bf16", "f64")[k % 4]
        if k % 3 == 0:
            u = UNITS[int(rng.integers(0, len(UNITS)))]
            n = int(u * rng.integers(1, 4) + rng.integers(-3, 4))
        else:
            n = int(rng.integers(0, 3_000_000))
        n = max(n, 0)
        zf = float(rng.choice([0.0, 0.1, 0.5, 0.9, 0.999, 1.0]))
        op = ("compress", "relu", "prune", "mask")[int(rng.integers(0, 4))]
        out.append(pytest.param(kind, n, zf, op, k, id=f"{k}-{kind}-{n}-{zf}-{op}"))
    return out


@pytest.fixture(scope="module")
def G():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from tests import gpu_util
    B.lib()
    return gpu_util


@pytest.mark.parametrize("kind,n,zf,op,k", cases())
def test_random_case(G, oracle, kind, n, zf, op, k):
    x = W.random_patterns(n, kind, zf, seed=5000 + k)
    xt = G.from_raw(x, kind) if n else torch.empty(0, dtype=G.TDT[kind], device="cuda")
    if op == "mask":
        src = W.random_patterns(n, kind, 0.5, seed=6000 + k, with_specials=False)
        m = oracle.compress(src)
        y_ref, v_ref = oracle.mask_compress(x, m.bitmap if n else np.zeros(1, np.uint32))
        v, y, ok = G.gpu_mask_compress(xt, m.bitmap if n else np.zeros(1, np.uint32),
                                       m.prefix if n else np.zeros(1, np.uint64), m.nnz, "with_y")
        assert ok and np.array_equal(v, v_ref) and np.array_equal(y, y_ref)
        return
    if op == "compress":
        y_ref, c = None, oracle.compress(x)
        g = G.gpu_compress(xt)
    elif op == "relu":
        y_ref, c = oracle.relu_fwd_compress(x, kind)
        g = G.gpu_compress(xt, relu=True, want_y=True)
    else:
        tau = (0.0, 0.01, 0.05, 0.1)[k % 4]
        y_ref, c = oracle.prune_fwd_compress(x, kind, tau)
        g = G.gpu_compress(xt, tau=tau, want_y=True)
    assert g.guards_ok and g.status == B.BT_OK and g.nnz == c.nnz
    assert np.array_equal(g.bitmap, c.bitmap) and np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values, c.values)
    if y_ref is not None:
        assert np.array_equal(g.y, y_ref)
    if n:
        out, ok = G.gpu_decompress(c.bitmap, c.values, c.prefix, n, kind)
        assert ok and np.array_equal(out, x if y_ref is None else y_ref)
