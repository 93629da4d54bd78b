"""bt_compress_noalloc, the entry point for callers that may not allocate device memory (its scratch is
a fixed array inside the library): through the C ABI, two calls in a row, every output compared bit for
bit with what bt_compress writes for the same input and with the CPU oracle, up to the largest tensor the
built-in scratch serves and under the launch shape that needs the most of it.  Collected last on purpose:
a run that stops at the first failure has then already run every other test.  Works alone in a fresh
process as well as after the other tests (nothing here depends on state they leave behind)."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu


def outputs(st: B.Stash):
    torch.cuda.synchronize()
    nnz = st.nnz
    return (nnz, st.status, W.raw_numpy(st.bitmap), W.raw_numpy(st.chunk_prefix), W.raw_numpy(st.values[:nnz]))


@pytest.mark.parametrize("kind", ["f32", "bf16", "f64"])
def test_noalloc_matches_bt_compress_on_two_calls_in_a_row(oracle, kind):
    assert torch.cuda.is_available()
    L = B.lib()
    dt = W.TORCH_DTYPES[kind]
    sizes = (8192 * 37 + 4097 + 5, 200704)                    # second call smaller: stale scratch beyond it must not matter
    for call, n in enumerate(sizes):
        raw = W.random_patterns(n, kind, 0.5, seed=31337 + call)
        x = torch.from_numpy(raw.view({2: np.int16, 4: np.int32, 8: np.int64}[raw.dtype.itemsize]).copy()).cuda().view(dt)
        ref, got = B.Stash(n, dt), B.Stash(n, dt)
        B.bt_compress(x, ref.bitmap, ref.values, ref.chunk_prefix, ref.nnz_out, B.new_workspace(n), ref.dev_status)
        expect = outputs(ref)
        status = L.bt_compress_noalloc(x.data_ptr(), n, B.DTYPE_CODE[dt], got.bitmap.data_ptr(), got.values.data_ptr(),
                                       n, got.chunk_prefix.data_ptr(), got.nnz_out.data_ptr(),
                                       got.dev_status.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert status == B.BT_OK
        result = outputs(got)
        assert result[0] == expect[0] and result[1] == expect[1] == B.BT_OK
        for a, b in zip(result[2:], expect[2:]):
            assert np.array_equal(a, b)                        # bitmap, prefix, packed values: bit exact
        c = oracle.compress(raw)
        assert result[0] == c.nnz
        assert np.array_equal(result[2].view(np.uint32), c.bitmap) and np.array_equal(result[3].view(np.uint64), c.prefix)
        assert np.array_equal(result[4], c.values)


def _noalloc(L, x, st, n):
    return L.bt_compress_noalloc(x.data_ptr(), n, B.DTYPE_CODE[x.dtype], st.bitmap.data_ptr(), st.values.data_ptr(), n,
                                 st.chunk_prefix.data_ptr(), st.nnz_out.data_ptr(), st.dev_status.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream)


@pytest.mark.parametrize("kind,max_ctas", [("bf16", 0), ("f64", 1), ("f32", 3)])
def test_noalloc_at_its_largest_size_against_the_oracle(oracle, kind, max_ctas):
    """n == BT_NOALLOC_MAX_ELEMS exactly.  8-byte elements have the smallest tiles (one chunk each), and a launch
    limited to one CTA has one wave per tile: the shape that uses every word of the scratch."""
    L = B.lib()
    dt = W.TORCH_DTYPES[kind]
    n = B.NOALLOC_MAX_ELEMS
    raw = W.random_patterns(n, kind, 0.6, seed=2718)
    x = torch.from_numpy(raw.view({2: np.int16, 4: np.int32, 8: np.int64}[raw.dtype.itemsize])).cuda().view(dt)
    st = B.Stash(n, dt)
    before = B.bt_set_max_ctas(max_ctas)
    try:
        assert _noalloc(L, x, st, n) == B.BT_OK
        nnz, status, bitmap, prefix, values = outputs(st)
    finally:
        B.bt_set_max_ctas(before)
    c = oracle.compress(raw)
    assert status == B.BT_OK and nnz == c.nnz
    assert np.array_equal(bitmap.view(np.uint32), c.bitmap)
    assert np.array_equal(prefix.view(np.uint64), c.prefix)
    assert np.array_equal(values, c.values)
    # the next, small call on the scratch the large one filled
    m = 4096 * 3 + 17
    st2 = B.Stash(m, dt)
    assert _noalloc(L, x[:m], st2, m) == B.BT_OK
    nnz2, status2, bitmap2, prefix2, values2 = outputs(st2)
    c2 = oracle.compress(raw[:m])
    assert status2 == B.BT_OK and nnz2 == c2.nnz and np.array_equal(bitmap2.view(np.uint32), c2.bitmap)
    assert np.array_equal(prefix2.view(np.uint64), c2.prefix) and np.array_equal(values2, c2.values)


def test_noalloc_rejects_tensors_beyond_its_scratch():
    L = B.lib()
    A = 0x10000                                                # aligned fake addresses: the size check comes first
    assert L.bt_compress_noalloc(A, B.NOALLOC_MAX_ELEMS + 1, B.BT_F32, A, A, 1, A, A, A, None) == B.BT_ERR_TOO_LARGE
    assert L.bt_compress_noalloc(A, 16, 42, A, A, 1, A, A, A, None) == B.BT_ERR_DTYPE
    assert L.bt_compress_noalloc(None, 16, B.BT_F32, A, A, 1, A, A, A, None) == B.BT_ERR_NULL
