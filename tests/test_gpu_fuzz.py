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


def later_cases(count=48, seed=2025):
    """The same kind of sweep over the entry points added after the hot path: the ReLU6 pair and the narrowing
    forms (binary32 tensors only) with their widening restore."""
    rng = np.random.default_rng(seed)
    out = []
    for k in range(count):
        op = ("relu6", "narrow_f16", "narrow_bf16")[k % 3]
        kind = ("f32", "f16", "bf16", "f64")[(k // 3) % 4] if op == "relu6" else "f32"
        if k % 2 == 0:
            u = UNITS[int(rng.integers(0, len(UNITS)))]
            n = int(u * rng.integers(1, 4) + rng.integers(-3, 4))
        else:
            n = int(rng.integers(0, 3_000_000))
        zf = float(rng.choice([0.0, 0.1, 0.5, 0.9, 0.999, 1.0]))
        out.append(pytest.param(kind, max(n, 0), zf, op, k, id=f"{k}-{kind}-{n}-{zf}-{op}"))
    return out


@pytest.mark.parametrize("kind,n,zf,op,k", later_cases())
def test_random_case_of_the_later_entry_points(G, oracle, kind, n, zf, op, k):
    x = W.random_patterns(n, kind, zf, seed=7000 + k)
    xt = G.from_raw(x, kind) if n else torch.empty(0, dtype=G.TDT[kind], device="cuda")
    if op == "relu6":
        x = x.copy()
        if n > 8:                                             # plant saturated units and the value just below 6
            six = {"f32": 0x40C00000, "f16": 0x4600, "bf16": 0x40C0, "f64": 0x4018000000000000}[kind]
            x[1::7] = six
            x[2::11] = six + 1
            x[3::13] = six - 1
            xt = G.from_raw(x, kind)
        y_ref, c = oracle.relu6_fwd_compress(x, kind)
        st = B.Stash(n, G.TDT[kind])
        y = torch.empty_like(xt)
        B.bt_relu6_fwd_compress(xt, y, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, B.new_workspace(n), st.dev_status)
        torch.cuda.synchronize()
        assert st.status == B.BT_OK and st.nnz == c.nnz
        if n:
            assert np.array_equal(W.raw_numpy(y), y_ref)
            assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), c.bitmap)
            assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), c.prefix)
            assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values)
            grad = G.from_raw(W.random_patterns(n, kind, 0.1, seed=8000 + k), kind)
            gin = torch.empty_like(grad)
            B.bt_relu6_bwd_from_stash(st.bitmap, st.values, st.chunk_prefix, grad, gin)
            torch.cuda.synchronize()
            assert np.array_equal(W.raw_numpy(gin), oracle.relu6_bwd_from_stash(c, kind, W.raw_numpy(grad)))
        return
    to_kind = op.split("_")[1]
    fused = k % 2 == 1
    y_ref, c = oracle.narrow_compress(x, to_kind, fused=fused, tau=0.0, want_y=fused)
    g = G.gpu_compress(xt, relu=fused, want_y=fused, narrow=to_kind)
    assert g.guards_ok and g.status == B.BT_OK and g.nnz == c.nnz
    assert np.array_equal(g.bitmap, c.bitmap) and np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values.view(np.uint16), c.values)
    if fused:
        assert np.array_equal(g.y, y_ref)
    if n:
        bm = torch.from_numpy(c.bitmap.view(np.int32).copy()).cuda()
        vals = G.from_raw(c.values if c.values.size else np.zeros(1, np.uint16), to_kind)
        pf = torch.from_numpy(c.prefix.view(np.int64).copy()).cuda()
        out = G.Guarded(n, torch.float32)
        B.bt_decompress_widen(bm, vals, pf, out.inner, n=n)
        torch.cuda.synchronize()
        assert out.guards_intact() and np.array_equal(out.raw().view(np.uint32), oracle.widen_decompress(c, to_kind))
