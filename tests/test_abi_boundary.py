"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, and its host arithmetic and argument checks
behave as documented (no kernel is launched on an argument error)."""
import ctypes
import os
import re

import pytest

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import build

HEADER = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "bittrain.h")


@pytest.fixture(scope="module")
def L():
    build.build_library()
    return B.lib()


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(bt_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert set(B.EXPORTS) <= set(names) and len(names) >= 6
    for name in names:
        assert hasattr(L, name), name


def test_compressed_bytes_closed_form(L, oracle):
    for dt, es in ((B.BT_F32, 4), (B.BT_F16, 2), (B.BT_BF16, 2)):
        for n, nnz in ((0, 0), (1, 1), (31, 7), (32, 32), (33, 0), (4096, 100), (4097, 4097), (200704, 100352),
                       (1 << 28, 1 << 27), (3 * 4096 + 17, 12)):
            got = L.bt_compressed_bytes(n, nnz, dt)
            assert got == 4 * ((n + 31) // 32) + nnz * es + 8 * ((n + 4095) // 4096)
            assert got == oracle.compressed_bytes(n, nnz, es)
            if n % 32 == 0:
                assert got == n // 8 + nnz * es + 8 * ((n + 4095) // 4096)
    assert L.bt_compressed_bytes(100, 10, 99) == 0
    assert L.bt_compressed_bytes(200704, 100352, B.BT_F32) == 426888


def test_workspace_bytes_grows_with_n(L):
    assert L.bt_workspace_bytes(0) > 0
    assert L.bt_workspace_bytes(1 << 28) >= 8 * ((1 << 28) // 8192)
    assert L.bt_workspace_bytes(1 << 20) <= L.bt_workspace_bytes(1 << 21)


def test_argument_errors_are_reported_before_any_launch(L):
    # 16-byte aligned fake addresses: never dereferenced, because every call below fails its checks first
    A = 0x10000
    ws = L.bt_workspace_bytes(8192)
    ok_args = dict(dense=A, n=8192, dt=B.BT_F32, bitmap=A, values=A, cap=8192, prefix=A, nnz=A, ws=A, wsb=ws,
                   status=A, stream=None)

    def call(**kw):
        a = dict(ok_args, **kw)
        return L.bt_compress(a["dense"], a["n"], a["dt"], a["bitmap"], a["values"], a["cap"], a["prefix"], a["nnz"],
                             a["ws"], a["wsb"], a["status"], a["stream"])

    assert call(dt=7) == B.BT_ERR_DTYPE
    assert call(dense=None) == B.BT_ERR_NULL
    assert call(bitmap=None) == B.BT_ERR_NULL
    assert call(prefix=None) == B.BT_ERR_NULL
    assert call(nnz=None) == B.BT_ERR_NULL
    assert call(ws=None) == B.BT_ERR_NULL
    assert call(values=None) == B.BT_ERR_NULL
    assert call(dense=A + 4) == B.BT_ERR_ALIGN
    assert call(values=A + 8) == B.BT_ERR_ALIGN
    assert call(prefix=A + 4) == B.BT_ERR_ALIGN
    assert call(nnz=A + 4) == B.BT_ERR_ALIGN
    assert call(wsb=ws - 1) == B.BT_ERR_WORKSPACE
    assert L.bt_decompress(A, A, A, 10, 9, A, None) == B.BT_ERR_DTYPE
    assert L.bt_decompress(None, A, A, 10, B.BT_F16, A, None) == B.BT_ERR_NULL
    assert L.bt_decompress(A, A, A, 10, B.BT_F16, A + 2, None) == B.BT_ERR_ALIGN
    assert L.bt_decompress(A, A, A, 0, B.BT_F16, None, None) == B.BT_OK          # n == 0 touches nothing
    assert L.bt_relu_bwd_from_bitmap(A, None, 10, B.BT_F32, A, None) == B.BT_ERR_NULL
    assert L.bt_relu_bwd_from_bitmap(A, A, 10, 5, A, None) == B.BT_ERR_DTYPE
    assert L.bt_relu_bwd_from_bitmap(A, A + 2, 10, B.BT_BF16, A, None) == B.BT_ERR_ALIGN
    assert L.bt_relu_bwd_from_bitmap(None, None, 0, B.BT_BF16, None, None) == B.BT_OK
    assert L.bt_relu_fwd_compress(A, 8192, B.BT_F32, A + 4, A, A, 8192, A, A, A, ws, A, None) == B.BT_ERR_ALIGN


def test_later_entry_points_check_their_arguments_before_any_launch(L):
    """The calls added after the hot path (narrowing, widening, ReLU6, pooling, masked gather, arena forms): every
    call below fails its host-side checks, so the fake addresses are never dereferenced."""
    A = 0x10000
    ws = L.bt_workspace_bytes(8192)
    tail = (A, A, A, ws, A, None)                                   # chunk_prefix, nnz_out, workspace, bytes, status, stream
    arena = (A, 1 << 20, A, A)                                      # arena, arena_bytes, cursor, values_offset_out
    assert L.bt_compress_narrow(A, 8192, B.BT_F32, A, A, 8192, *tail) == B.BT_ERR_DTYPE
    assert L.bt_compress_narrow(None, 8192, B.BT_F16, A, A, 8192, *tail) == B.BT_ERR_NULL
    assert L.bt_prune_fwd_compress_narrow(A, 8192, B.BT_F64, 0.0, None, A, A, 8192, *tail) == B.BT_ERR_DTYPE
    assert L.bt_prune_fwd_compress_narrow(A + 4, 8192, B.BT_BF16, 0.0, None, A, A, 8192, *tail) == B.BT_ERR_ALIGN
    assert L.bt_decompress_widen(A, A, A, 10, B.BT_F32, A, None) == B.BT_ERR_DTYPE
    assert L.bt_decompress_widen(A, A, None, 10, B.BT_F16, A, None) == B.BT_ERR_NULL
    assert L.bt_decompress_widen(None, None, None, 0, B.BT_F16, None, None) == B.BT_OK
    assert L.bt_relu6_fwd_compress(A, 8192, 11, None, A, A, 8192, *tail) == B.BT_ERR_DTYPE
    assert L.bt_relu6_fwd_compress(A, 8192, B.BT_F32, None, None, A, 8192, *tail) == B.BT_ERR_NULL
    assert L.bt_relu6_bwd_from_stash(A, A, A, None, 10, B.BT_F32, A, None) == B.BT_ERR_NULL
    assert L.bt_relu6_bwd_from_stash(A, A, A, A, 10, B.BT_F32, A + 8, None) == B.BT_ERR_ALIGN
    assert L.bt_mask_compress(None, 10, B.BT_F32, A, A, None, A, 10, None) == B.BT_ERR_NULL
    assert L.bt_mask_compress(A, 10, 9, A, A, None, A, 10, None) == B.BT_ERR_DTYPE
    assert L.bt_maxpool2x2_fwd(A, 4, 3, 8, B.BT_F32, A, A, None) == B.BT_ERR_SHAPE
    assert L.bt_maxpool2x2_fwd(A, 4, 8, 0, B.BT_F32, A, A, None) == B.BT_ERR_SHAPE
    assert L.bt_maxpool2x2_fwd(None, 4, 8, 8, B.BT_F32, A, A, None) == B.BT_ERR_NULL
    assert L.bt_maxpool2x2_fwd(None, 0, 8, 8, B.BT_F32, None, None, None) == B.BT_OK
    assert L.bt_maxpool2x2_bwd(A, A, 4, 8, 8, 13, A, None) == B.BT_ERR_DTYPE
    assert L.bt_maxpool2x2_bwd_masked(A, None, A, 4, 8, 8, B.BT_F32, A, None) == B.BT_ERR_NULL
    assert L.bt_maxpool2x2_bwd_masked(A, A + 2, A, 4, 8, 8, B.BT_F32, A, None) == B.BT_ERR_ALIGN
    assert L.bt_maxpool2x2_bwd_masked(A, A, A, 4, 8, 7, B.BT_F32, A, None) == B.BT_ERR_SHAPE
    # arena forms
    assert L.bt_compress_arena(A, 8192, B.BT_F32, A, A, 1 << 20, None, A, *tail) == B.BT_ERR_NULL      # no cursor
    assert L.bt_compress_arena(A, 8192, B.BT_F32, A, A, 1 << 20, A, None, *tail) == B.BT_ERR_NULL      # no offset word
    assert L.bt_compress_arena(A, 8192, B.BT_F32, A, A, 1 << 20, A + 4, A, *tail) == B.BT_ERR_ALIGN
    assert L.bt_prune_fwd_compress_arena(A, 8192, 9, 0.0, None, A, *arena, *tail) == B.BT_ERR_DTYPE
    assert L.bt_decompress_arena(A, A, None, A, 10, B.BT_F32, A, None) == B.BT_ERR_NULL
    assert L.bt_compress_narrow_arena(A, 8192, B.BT_F32, A, *arena, *tail) == B.BT_ERR_DTYPE
    assert L.bt_compress_narrow_arena(A, 8192, B.BT_F16, A, A, 1 << 20, None, A, *tail) == B.BT_ERR_NULL
    assert L.bt_prune_fwd_compress_narrow_arena(A, 8192, B.BT_F64, 0.0, None, A, *arena, *tail) == B.BT_ERR_DTYPE
    assert L.bt_prune_fwd_compress_narrow_arena(A, 8192, B.BT_BF16, 0.0, A + 2, A, *arena, *tail) == B.BT_ERR_ALIGN
    assert L.bt_relu6_fwd_compress_arena(A, 8192, B.BT_F32, None, A, A, 1 << 20, A, None, *tail) == B.BT_ERR_NULL
    assert L.bt_decompress_widen_arena(A, A, A, A, 10, B.BT_F64, A, None) == B.BT_ERR_DTYPE
    assert L.bt_decompress_widen_arena(A, A, None, A, 10, B.BT_F16, A, None) == B.BT_ERR_NULL
    assert L.bt_relu6_bwd_from_stash_arena(A, A, None, A, A, 10, B.BT_F32, A, None) == B.BT_ERR_NULL
    assert L.bt_relu6_bwd_from_stash_arena(A, A, A + 4, A, A, 10, B.BT_F32, A, None) == B.BT_ERR_ALIGN
    assert L.bt_relu6_bwd_from_stash_arena(None, None, None, None, None, 0, B.BT_F32, None, None) == B.BT_OK


def test_bitmap_needs_four_byte_alignment_only(L):
    """The bitmap is an array of 32-bit words: 4-byte alignment is all the format asks for, in the compressors and
    in every consumer.  A 2-byte offset is refused; a 4-byte offset passes the alignment check (shown here by the
    check that comes after it; the GPU tests run such bitmaps through every kernel)."""
    A = 0x10000
    ws = L.bt_workspace_bytes(8192)
    for off, expect in ((2, B.BT_ERR_ALIGN), (4, B.BT_ERR_WORKSPACE), (8, B.BT_ERR_WORKSPACE), (12, B.BT_ERR_WORKSPACE)):
        assert L.bt_compress(A, 8192, B.BT_F32, A + off, A, 8192, A, A, A, ws - 1, A, None) == expect
        assert L.bt_relu_fwd_compress(A, 8192, B.BT_BF16, None, A + off, A, 8192, A, A, A, ws - 1, A, None) == expect
    assert L.bt_compress_noalloc(A, 16, B.BT_F32, A + 2, A, 16, A, A, A, None) == B.BT_ERR_ALIGN
    assert L.bt_decompress(A + 2, A, A, 10, B.BT_F32, A, None) == B.BT_ERR_ALIGN
    assert L.bt_decompress_widen(A + 2, A, A, 10, B.BT_F16, A, None) == B.BT_ERR_ALIGN
    assert L.bt_relu_bwd_from_bitmap(A + 2, A, 10, B.BT_F32, A, None) == B.BT_ERR_ALIGN
    assert L.bt_relu6_bwd_from_stash(A + 2, A, A, A, 10, B.BT_F32, A, None) == B.BT_ERR_ALIGN
    assert L.bt_mask_compress(A, 10, B.BT_F32, A + 2, A, None, A, 10, None) == B.BT_ERR_ALIGN
    # a 4-byte offset and a second, real fault: the second one is what gets reported
    assert L.bt_decompress(A + 4, A, A, 10, B.BT_F32, A + 2, None) == B.BT_ERR_ALIGN
    assert L.bt_decompress(A + 4, A, A + 4, 10, B.BT_F32, A, None) == B.BT_ERR_ALIGN


def test_header_puts_the_codec_proper_first_and_states_what_the_library_keeps():
    import os
    import re
    text = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "bittrain.h")).read()
    names = re.findall(r"^(?:int|size_t|long long)\s+(bt_\w+)\s*\(", text, flags=re.M)
    assert names[:6] == ["bt_compressed_bytes", "bt_workspace_bytes", "bt_compress", "bt_decompress",
                         "bt_relu_fwd_compress", "bt_relu_bwd_from_bitmap"]
    head = text[:text.index("#ifndef BITTRAIN_H")]
    assert "bitmap 4-byte aligned" in head
    assert "bt_set_max_ctas" in head and "counter" in head          # the host-side state is named, not denied
    assert "keeps no" not in head


def test_cta_limit_is_per_thread_host_state(L):
    import threading
    assert L.bt_set_max_ctas(0) == 0
    assert L.bt_set_max_ctas(74) == 0 and L.bt_set_max_ctas(49) == 74
    assert L.bt_set_max_ctas(-1) == -1 and L.bt_set_max_ctas(49) == 49          # a negative limit changes nothing
    seen = []
    t = threading.Thread(target=lambda: seen.append((L.bt_set_max_ctas(5), L.bt_set_max_ctas(0))))
    t.start(), t.join()
    assert seen == [(0, 5)]                                                      # another thread starts without a limit
    assert L.bt_set_max_ctas(0) == 49


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "library_path", lambda: str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        B.lib()


def test_test_hooks_exist_only_in_the_checking_builds(L):
    """The product library exports no test hook; the two checking builds (tests/lib/, loaded by tests only) export
    every symbol of the header plus their hook."""
    import ctypes
    from tests import checking_libs as C
    for hook in ("bt_test_set_wait_ns", "bt_test_bounds_violations"):
        assert not hasattr(L, hook), hook
    for path, hook in ((C.HOOKS_PATH, "bt_test_set_wait_ns"), (C.BOUNDS_PATH, "bt_test_bounds_violations")):
        C._build.build_library(out=path, extra_flags=C._FLAGS[path])      # a no-op when up to date
        T = ctypes.CDLL(path)
        assert hasattr(T, hook)
        for name in B.EXPORTS:
            assert hasattr(T, name), (path, name)
