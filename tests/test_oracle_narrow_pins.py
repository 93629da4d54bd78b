"""Pins the oracle's down-cast-on-stash form (binary32 tensor, 16-bit stashed values) to library conversions
and to the plain compressor: numpy's float32 -> float16 cast and torch's float32 -> bfloat16 cast are both
IEEE round-to-nearest-even; the structure (bitmap, prefix, count) must be that of the binary32 stash."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import workloads as W


def boundary_patterns():
    """Every sign/exponent/upper-mantissa combination with the dropped low bits at and around the rounding
    tie: exhaustive over the kept bits, six settings of the dropped ones (float16 drops 13, bfloat16 16)."""
    out = {}
    for name, dropped in (("f16", 13), ("bf16", 16)):
        upper = np.arange(1 << (32 - dropped), dtype=np.uint64) << dropped
        tie = 1 << (dropped - 1)
        lows = np.array([0, 1, tie - 1, tie, tie + 1, (1 << dropped) - 1], dtype=np.uint64)
        out[name] = (upper[:, None] | lows[None, :]).reshape(-1).astype(np.uint32)
    return out


PATTERNS = boundary_patterns()


def oracle_convert(oracle, bits, to_kind):
    """The oracle's scalar conversion applied through its compress entry point (every non-zero element is
    pushed in order, so values[] of an all-non-zero input is the element-wise conversion)."""
    nz = bits[bits != 0]
    _, c = oracle.narrow_compress(nz, to_kind)
    assert c.nnz == nz.size
    return nz, c.values


def test_half_conversion_matches_numpy_on_every_rounding_boundary(oracle):
    bits, got = oracle_convert(oracle, PATTERNS["f16"], "f16")
    f = bits.view(np.float32)
    finite_or_inf = ~np.isnan(f)
    with np.errstate(over="ignore"):
        ref = f.astype(np.float16).view(np.uint16)
    assert np.array_equal(got[finite_or_inf], ref[finite_or_inf])
    assert (got[~finite_or_inf] == 0x7FFF).all() and (~finite_or_inf).sum() > 1000


def test_bfloat16_conversion_matches_torch_on_every_rounding_boundary(oracle):
    bits, got = oracle_convert(oracle, PATTERNS["bf16"], "bf16")
    t = torch.from_numpy(bits.view(np.int32)).view(torch.float32)
    nan = torch.isnan(t).numpy()
    ref = t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got[~nan], ref[~nan])
    assert (got[nan] == 0x7FFF).all() and nan.sum() > 100


def test_scalar_conversions_closed_forms(oracle):
    f2h, f2b = oracle.float_to_half, oracle.float_to_bfloat16
    b = lambda x: int(np.float32(x).view(np.uint32))
    assert f2h(b(1.0)) == 0x3C00 and f2h(b(-2.0)) == 0xC000 and f2h(b(65504.0)) == 0x7BFF
    assert f2h(b(65519.996)) == 0x7BFF and f2h(b(65520.0)) == 0x7C00              # the tie goes to the even side: inf
    assert f2h(b(2.0 ** -24)) == 0x0001 and f2h(b(2.0 ** -25)) == 0x0000          # tie between 0 and the smallest subnormal
    assert f2h(b(np.nextafter(np.float32(2.0 ** -25), np.float32(1)))) == 0x0001
    assert f2h(b(-(2.0 ** -26))) == 0x8000                                          # underflow keeps the sign
    assert f2h(b(2.0 ** -14)) == 0x0400 and f2h(b(np.nextafter(np.float32(2.0 ** -14), np.float32(0)))) == 0x0400
    assert f2h(b(1.0 + 2.0 ** -11)) == 0x3C00 and f2h(b(1.0 + 3 * 2.0 ** -11)) == 0x3C02   # ties to even, both ways
    assert f2h(0x7F800000) == 0x7C00 and f2h(0xFF800000) == 0xFC00
    assert f2h(0x7FC00001) == 0x7FFF and f2h(0xFF800001) == 0x7FFF                  # every NaN -> the one quiet NaN
    assert f2b(b(1.0)) == 0x3F80 and f2b(0x3F808000) == 0x3F80 and f2b(0x3F818000) == 0x3F82
    assert f2b(0x7F7FFFFF) == 0x7F80 and f2b(0xFF7FFFFF) == 0xFF80                  # rounds past the largest finite: inf
    assert f2b(0x00000001) == 0x0000 and f2b(0x80008001) == 0x8001
    assert f2b(0x7FC00000) == 0x7FFF and f2b(0xFFFFFFFF) == 0x7FFF


@pytest.mark.parametrize("to_kind", ["f16", "bf16"])
@pytest.mark.parametrize("n", [1, 31, 4096, 3 * 4096 + 77])
def test_structure_is_that_of_the_binary32_stash(oracle, to_kind, n):
    x = W.random_patterns(n, "f32", 0.5, seed=40 + n)
    x[: min(n, 8)] = np.array([0, 0x80000000, 1, 0x33000000, 0x7FC00001, 0x3F800000, 0, 0x00800000], dtype=np.uint32)[: min(n, 8)]
    full = oracle.compress(x)
    _, c = oracle.narrow_compress(x, to_kind)
    assert c.nnz == full.nnz and np.array_equal(c.bitmap, full.bitmap) and np.array_equal(c.prefix, full.prefix)
    assert c.values.dtype == np.uint16 and c.values.size == full.nnz
    # every stored value is the narrowed form of the corresponding full-precision value
    conv = oracle.float_to_half if to_kind == "f16" else oracle.float_to_bfloat16
    assert all(int(c.values[k]) == conv(int(full.values[k])) for k in range(0, full.nnz, max(1, full.nnz // 257)))
    # the 16-bit stash restores through the plain decompressor to the narrowed dense tensor
    dense16 = oracle.decompress(c)
    bits = np.unpackbits(c.bitmap.view(np.uint8), bitorder="little")[:n].astype(bool)
    assert not dense16[~bits].any() and np.array_equal(dense16[bits], c.values)
    assert oracle.compressed_bytes(n, c.nnz, 2) == 4 * ((n + 31) // 32) + 2 * c.nnz + 8 * ((n + 4095) // 4096)


@pytest.mark.parametrize("to_kind", ["f16", "bf16"])
@pytest.mark.parametrize("tau", [0.0, 0.05])
def test_fused_threshold_form(oracle, to_kind, tau):
    n = 2 * 4096 + 19
    t = torch.randn(n, generator=torch.Generator().manual_seed(77)) * 0.2
    t[3] = float("nan"); t[4] = float("inf"); t[5] = -0.0; t[6] = tau; t[7] = 1e-30
    x = W.raw_numpy(t)
    y, c = oracle.narrow_compress(x, to_kind, fused=True, tau=tau, want_y=True)
    y_ref, full = oracle.prune_fwd_compress(x, "f32", tau)
    assert np.array_equal(y, y_ref)                                  # the binary32 output is the pruning oracle's
    assert c.nnz == full.nnz and np.array_equal(c.bitmap, full.bitmap) and np.array_equal(c.prefix, full.prefix)
    keep = ~(t <= tau)
    tt = torch.where(keep, t, torch.zeros(()))[keep]
    ref = tt.to(torch.float16 if to_kind == "f16" else torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()
    ref[torch.isnan(tt).numpy()] = 0x7FFF
    assert np.array_equal(c.values, ref)
    if to_kind == "f16" and tau == 0.0:                              # 1e-30 underflows in binary16: a zero under a set bit
        assert c.values[np.flatnonzero(np.flatnonzero(keep.numpy()) == 7)[0]] == 0
    _, c2 = oracle.narrow_compress(x, to_kind, fused=True, tau=tau, want_y=False)
    assert np.array_equal(c2.values, c.values)


@pytest.mark.parametrize("to_kind", ["f16", "bf16"])
def test_widening_restore_matches_library_casts(oracle, to_kind):
    """Restoring a narrowed stash into binary32 = the narrowed dense tensor cast up by numpy / torch (exact
    casts), and narrowing the restored tensor again changes nothing."""
    n = 3 * 4096 + 55
    x = W.random_patterns(n, "f32", 0.4, seed=91)
    _, c = oracle.narrow_compress(x, to_kind)
    back = oracle.widen_decompress(c, to_kind)
    dense16 = oracle.decompress(c)
    if to_kind == "f16":
        ref = dense16.view(np.float16).astype(np.float32).view(np.uint32)
        nan = np.isnan(dense16.view(np.float16))
        assert np.array_equal(back[~nan], ref[~nan])
        assert (back[nan] == 0x7FFFE000).all() and nan.any()          # 0x7FFF widened: the payload moves up 13 bits
    else:
        ref = torch.from_numpy(dense16.view(np.int16)).view(torch.bfloat16).float().view(torch.int32).numpy().view(np.uint32)
        nan = torch.isnan(torch.from_numpy(dense16.view(np.int16)).view(torch.bfloat16)).numpy()
        assert np.array_equal(back[~nan], ref[~nan])
        assert (back[nan] == 0x7FFF0000).all() and nan.any()
    bits = np.unpackbits(c.bitmap.view(np.uint8), bitorder="little")[:n].astype(bool)
    assert not back[~bits].any()
    _, again = oracle.narrow_compress(back, to_kind)                 # idempotent on what survives as non-zero
    keep = c.values != 0                                             # an underflow to +0 drops out; -0 keeps its bit
    assert np.array_equal(again.values, c.values[keep])


def _hand_made_stash(oracle, values16):
    """A stash whose values are exactly `values16` (every bit set): what bt_compress gives for a 16-bit tensor
    without zeros, built with the plain compressor so that no narrowing step touches the patterns."""
    c = oracle.compress(values16)
    assert c.nnz == values16.size
    return c


def test_widening_every_half_nan_keeps_sign_and_payload(oracle):
    """All 2046 binary16 NaNs (both signs, quiet and signalling) through the widening restore.

    Reading pinned here: the restore moves the 10 mantissa bits into the top of the binary32 mantissa and
    the sign into bit 31, and does nothing else -- a signalling NaN stays signalling (quiet bit clear),
    where a hardware conversion would set the quiet bit.  Against numpy and against torch, whose casts may
    quiet: equal on sign and payload for every NaN, equal on every bit for the quiet ones, and for a
    signalling one the library result is the oracle's with at most the quiet bit added."""
    mant = np.arange(1, 1024, dtype=np.uint16)
    h = np.concatenate([0x7C00 | mant, 0xFC00 | mant]).astype(np.uint16)
    got = oracle.widen_decompress(_hand_made_stash(oracle, h), "f16")
    want = ((h.astype(np.uint32) & 0x8000) << 16) | 0x7F800000 | ((h.astype(np.uint32) & 0x3FF) << 13)
    assert np.array_equal(got, want)                                   # written out from the formats' layouts
    quiet = (h & 0x0200) != 0
    by_numpy = h.view(np.float16).astype(np.float32).view(np.uint32)
    by_torch = torch.from_numpy(h.view(np.int16).copy()).view(torch.float16).to(torch.float32).view(torch.int32).numpy().view(np.uint32)
    # numpy's cast keeps every NaN as it is; torch's sets the quiet bit, and gives the elements of an array's
    # unvectorised tail the one pattern 0x7FFFFFFF (those pin only that the result is a NaN)
    assert np.array_equal(by_numpy, got)
    kept = by_torch != 0x7FFFFFFF
    assert kept.sum() >= h.size - 16 and np.isnan(by_torch.view(np.float32)).all()
    for lib_bits, sel in ((by_numpy, np.ones(h.size, bool)), (by_torch, kept)):
        assert np.array_equal(lib_bits[quiet & sel], got[quiet & sel])
        assert np.array_equal(lib_bits[sel] | 0x00400000, got[sel] | 0x00400000)          # sign, exponent, payload
        assert np.isin(lib_bits[~quiet & sel] ^ got[~quiet & sel], (0, 0x00400000)).all()   # only the quiet bit may differ
    assert np.isnan(got.view(np.float32)).all()
    # a signalling NaN whose payload would vanish if the shift were wrong by one either way
    assert got[0] == 0x7F802000 and got[mant.size] == 0xFF802000
    # the scalar entry point agrees on the quiet ones (a float returned through Python is quieted on the way)
    for hh in (0x7E00, 0xFE00, 0x7FFF, 0xFE01):
        assert np.float32(oracle.half_to_float(hh)).view(np.uint32) == want[np.flatnonzero(h == hh)[0]]


def test_widening_every_bfloat16_nan_and_infinity(oracle):
    h = np.concatenate([np.arange(0x7F80, 0x8000), np.arange(0xFF80, 0x10000)]).astype(np.uint16)
    got = oracle.widen_decompress(_hand_made_stash(oracle, h), "bf16")
    assert np.array_equal(got, h.astype(np.uint32) << 16)
    by_torch = torch.from_numpy(h.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).view(torch.int32).numpy().view(np.uint32)
    assert np.array_equal(by_torch | 0x00400000, got | 0x00400000)
    quiet = (h & 0x0040) != 0
    assert np.array_equal(by_torch[quiet], got[quiet])
