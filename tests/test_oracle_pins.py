"""Pins the CPU oracle to things other than itself: library routines (numpy
packbits / boolean indexing / cumsum, torch.relu, torch.where), closed forms,
the values Table 1 of the paper prints, invariants and brute force on tiny
inputs.  A dropped term, wrong bit order, off-by-one prefix or transposed
operand in bt_oracle.c fails at least one of these."""
import itertools
import os
from decimal import Decimal, ROUND_HALF_UP

import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_theoretical.txt")
UINT = {2: np.uint16, 4: np.uint32, 8: np.uint64}


def lib_compress(x_raw: np.ndarray):
    """The format written with numpy library routines only."""
    n = x_raw.size
    nz = x_raw != 0
    packed = np.packbits(nz, bitorder="little")                 # LSB-first bytes
    pad = (-packed.size) % 4
    bitmap = np.concatenate([packed, np.zeros(pad, np.uint8)]).view("<u4")
    values = x_raw[nz]
    chunks = (n + 4095) // 4096
    per_chunk = np.add.reduceat(nz.astype(np.uint64), np.arange(0, n, 4096)) if n else np.zeros(0, np.uint64)
    prefix = (np.concatenate([[0], np.cumsum(per_chunk)[:-1]]).astype(np.uint64)
              if chunks else np.zeros(0, np.uint64))
    return bitmap, values, prefix, int(nz.sum())


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n", W.EDGE_SIZES)
def test_compress_matches_numpy_routines(oracle, kind, n):
    x = W.random_patterns(n, kind, 0.5, seed=n + 7)
    c = oracle.compress(x)
    bitmap, values, prefix, nnz = lib_compress(x)
    assert c.nnz == nnz
    assert np.array_equal(c.bitmap, bitmap)
    assert np.array_equal(c.values, values)
    assert np.array_equal(c.prefix, prefix)
    assert c.bitmap.size == (n + 31) // 32 and c.prefix.size == (n + 4095) // 4096


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16", "f64"])
@pytest.mark.parametrize("n", W.EDGE_SIZES)
@pytest.mark.parametrize("zf", [0.0, 0.5, 0.97, 1.0])
def test_round_trip_and_invariants(oracle, kind, n, zf):
    if kind == "f64":
        rng = np.random.default_rng(n)
        x = rng.integers(0, 1 << 63, size=n, dtype=np.uint64)
        x[rng.random(n) < zf] = 0
    else:
        x = W.random_patterns(n, kind, zf, seed=3 * n + 1)
    c = oracle.compress(x)
    # lossless, bitwise, by both decoders (the chunked one only uses prefix[])
    assert np.array_equal(oracle.decompress(c), x)
    assert np.array_equal(oracle.decompress(c, chunked=True), x)
    # nnz == popcount(bitmap) == brute count
    pop = int(np.unpackbits(c.bitmap.view(np.uint8)).sum())
    assert c.nnz == pop == int(np.count_nonzero(x))
    # prefix: starts at 0, non-decreasing, increments are the chunk popcounts (<= 4096)
    if c.prefix.size:
        assert c.prefix[0] == 0
        words_per_chunk = 128
        cp = [int(np.unpackbits(c.bitmap[i:i + words_per_chunk].view(np.uint8)).sum())
              for i in range(0, c.bitmap.size, words_per_chunk)]
        assert len(cp) == c.prefix.size
        inc = np.diff(np.concatenate([c.prefix, [np.uint64(c.nnz)]]).astype(np.int64))
        assert np.array_equal(inc, np.array(cp)) and (inc <= 4096).all() and (inc >= 0).all()
    # padding bits are zero
    if n % 32:
        assert int(c.bitmap[-1]) >> (n % 32) == 0
    # closed form of the size
    es = x.dtype.itemsize
    assert oracle.compressed_bytes(n, c.nnz, es) == 4 * ((n + 31) // 32) + c.nnz * es + 8 * ((n + 4095) // 4096)
    if n % 32 == 0:
        assert oracle.compressed_bytes(n, c.nnz, es) == n // 8 + c.nnz * es + 8 * ((n + 4095) // 4096)


def test_all_zero_and_all_nonzero(oracle):
    n = 3 * 4096 + 100
    z = np.zeros(n, np.uint32)
    c = oracle.compress(z)
    assert c.nnz == 0 and not c.bitmap.any() and not c.prefix.any() and c.values.size == 0
    f = np.arange(1, n + 1, dtype=np.uint32)
    c = oracle.compress(f)
    assert c.nnz == n and np.array_equal(c.values, f)
    assert np.array_equal(c.prefix, np.arange(4) * 4096)
    assert (c.bitmap[:-1] == 0xFFFFFFFF).all() and c.bitmap[-1] == (1 << (n % 32)) - 1


def test_bit_order_is_lsb_first(oracle):
    # element 0 -> bit 0 of word 0; element 33 -> bit 1 of word 1; element 63 -> bit 31 of word 1
    x = np.zeros(64, np.uint32)
    x[[0, 33, 63]] = [5, 6, 7]
    c = oracle.compress(x)
    assert c.bitmap.tolist() == [1, (1 << 1) | (1 << 31)] and c.values.tolist() == [5, 6, 7]


def test_brute_force_all_zero_patterns(oracle):
    """Every one of the 2^n zero patterns for n = 1..12 with distinct payloads."""
    for n in range(1, 13):
        for mask in range(1 << n):
            x = np.array([(i + 1) * 0x01010101 if (mask >> i) & 1 else 0 for i in range(n)], np.uint32)
            c = oracle.compress(x)
            assert c.bitmap.tolist() == [mask]
            assert c.values.tolist() == [(i + 1) * 0x01010101 for i in range(n) if (mask >> i) & 1]
            assert c.nnz == bin(mask).count("1") and c.prefix.tolist() == [0]
            assert np.array_equal(oracle.decompress(c), x)


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
def test_brute_force_special_values(oracle, kind):
    """All combinations of special patterns for n = 1..3: only the all-zero pattern is dropped."""
    sp = W.SPECIALS[kind]
    es = 4 if kind == "f32" else 2
    for n in (1, 2, 3):
        for combo in itertools.product(sp[:9], repeat=n):
            x = np.array(combo, dtype=UINT[es])
            c = oracle.compress(x)
            assert c.values.tolist() == [v for v in combo if v != 0]
            assert c.bitmap[0] == sum(1 << i for i, v in enumerate(combo) if v != 0)
            assert np.array_equal(oracle.decompress(c), x)


def _round2(v: float) -> Decimal:
    return Decimal(repr(v)).quantize(Decimal("0.01"), rounding=ROUND_HALF_UP)


def test_table1_theoretical_columns(oracle):
    """compressed_bytes minus the prefix term reproduces every printed cell of Table 1."""
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 30
    for b, ch, w, h, n, pct, dense_mb, bitmap_mb, improv in rows:
        n, pct = int(n), int(pct)
        assert int(b) * int(ch) * int(w) * int(h) == n
        nnz = n * pct // 100
        assert nnz * 100 == n * pct
        mb = oracle.compressed_bytes(n, nnz, 4) - 8 * ((n + 4095) // 4096)
        dense = 4 * n
        assert _round2(dense / 2 ** 20) == Decimal(dense_mb) or abs(dense / 2 ** 20 - float(dense_mb)) <= 0.005 + 1e-12
        assert abs(mb / 2 ** 20 - float(bitmap_mb)) <= 0.005 + 1e-12, (n, pct)
        assert abs(100.0 * (1.0 - mb / dense) - float(improv)) <= 0.005 + 1e-12
        # the prefix array costs 8 bytes per 4096 elements on top of M_b
        assert oracle.compressed_bytes(n, nnz, 4) - mb == 8 * (n // 4096)


def test_half_widening_matches_numpy_for_every_pattern(oracle):
    allh = np.arange(65536, dtype=np.uint16)
    ref = allh.view(np.float16).astype(np.float32).view(np.uint32)
    got = np.array([np.float32(oracle.half_to_float(int(h))).view(np.uint32) for h in allh])
    nan = np.isnan(allh.view(np.float16))
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.isnan(got[nan].view(np.float32)).all()


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16", "f64"])
def test_relu_fwd_matches_torch_relu(oracle, kind):
    n = 2 * 4096 + 77
    t = (torch.randn(n, generator=torch.Generator().manual_seed(11), dtype=torch.float64) * 3).to(W.TORCH_DTYPES[kind])
    t[::97] = 0.0
    t[5::101] = -0.0
    t[7] = float("inf"); t[8] = float("-inf")
    x = W.raw_numpy(t)
    y, c = oracle.relu_fwd_compress(x, kind)
    # torch.relu keeps the sign of -0.0; adding +0.0 (exact in every precision) turns
    # that one case into +0.0, which is the reading taken here, and changes nothing else.
    y_ref = W.raw_numpy((torch.relu(t.double()) + 0.0).to(t.dtype))
    assert np.array_equal(y, y_ref)
    assert not (y == (1 << (8 * x.dtype.itemsize - 1))).any()                       # no -0.0 survives
    # bit i == (x[i] > 0), the ReLU derivative mask
    bits = np.unpackbits(c.bitmap.view(np.uint8), bitorder="little")[:n].astype(bool)
    assert np.array_equal(bits, (t.double() > 0).numpy())
    # and the compressed form is the plain compressor applied to y
    c2 = oracle.compress(y)
    assert c.nnz == c2.nnz and all(np.array_equal(a, b) for a, b in zip(c[:3], c2[:3]))
    y_none, c3 = oracle.relu_fwd_compress(x, kind, want_y=False)
    assert y_none is None and all(np.array_equal(a, b) for a, b in zip(c[:3], c3[:3]))


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16", "f64"])
def test_relu_fwd_special_patterns(oracle, kind):
    """+-0, negatives, -inf -> +0; positives incl. subnormals and +inf unchanged; NaN kept with payload."""
    es = W.ELEM_BYTES[kind]
    sp = np.array(W.SPECIALS[kind], dtype=UINT[es])
    y, c = oracle.relu_fwd_compress(sp, kind)
    sign = 1 << (8 * es - 1)
    expmask = {"f32": 0x7F800000, "f16": 0x7C00, "bf16": 0x7F80, "f64": 0x7FF0000000000000}[kind]
    for xin, yout in zip(sp.tolist(), y.tolist()):
        mag = xin & (sign - 1)
        is_nan = mag > expmask
        if is_nan or (mag != 0 and not xin & sign):
            assert yout == xin
        else:
            assert yout == 0


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16"])
def test_relu_bwd_matches_torch_where_and_autograd(oracle, kind):
    n = 4096 + 333
    gen = torch.Generator().manual_seed(5)
    x = torch.randn(n, generator=gen).to(W.TORCH_DTYPES[kind])
    g = torch.randn(n, generator=gen).to(W.TORCH_DTYPES[kind])
    g[3] = float("nan"); g[4] = float("inf"); g[9] = -0.0
    _, c = oracle.relu_fwd_compress(W.raw_numpy(x), kind)
    gin = oracle.relu_bwd_from_bitmap(c.bitmap, W.raw_numpy(g))
    bits = torch.from_numpy(np.unpackbits(c.bitmap.view(np.uint8), bitorder="little")[:n].astype(bool))
    ref = torch.where(bits, g, torch.zeros((), dtype=g.dtype))
    assert np.array_equal(gin, W.raw_numpy(ref))
    # autograd's ReLU gradient on NaN-free data (fp32 only: autograd multiplies nothing for relu)
    if kind == "f32":
        xg = x.clone().requires_grad_(True)
        gg = torch.randn(n, generator=gen)
        torch.relu(xg).backward(gg)
        mine = oracle.relu_bwd_from_bitmap(c.bitmap, W.raw_numpy(gg))
        assert np.array_equal(mine, W.raw_numpy(xg.grad))


def test_cfg1_statistics(oracle):
    x = W.cfg1()
    assert tuple(x.shape) == (1, 64, 56, 56) and x.numel() == 200704
    c = oracle.compress(W.raw_numpy(x))
    assert c.bitmap.size == 6272 and c.prefix.size == 49
    assert 0.48 < 1 - c.nnz / c.n < 0.52
    assert np.array_equal(oracle.decompress(c), W.raw_numpy(x))
