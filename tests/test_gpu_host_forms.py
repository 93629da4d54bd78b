"""GPU parity of the host-buffer entry points: inputs and outputs live in (pinned) host memory, the
staging area on the device; every output is compared bit for bit with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu
TDT = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16, "f64": torch.float64}


def host_tensor(raw: np.ndarray, kind: str) -> torch.Tensor:
    t = torch.from_numpy(raw.view({2: np.int16, 4: np.int32, 8: np.int64}[raw.dtype.itemsize]).copy()).view(TDT[kind])
    return t.pin_memory()


@pytest.mark.parametrize("kind", ["f32", "bf16", "f16", "f64"])
@pytest.mark.parametrize("n", [0, 1, 33, 4097, 8192 * 5 + 123, 200704])
def test_host_round_trip_and_relu_pair(oracle, kind, n):
    assert torch.cuda.is_available()
    dt = TDT[kind]
    x = W.random_patterns(n, kind, 0.5, seed=9000 + n)
    c = oracle.compress(x)
    staging = torch.empty(max(B.bt_host_staging_bytes(n, dt), 256), dtype=torch.uint8, device="cuda")
    h_x = host_tensor(x, kind)
    h_bitmap = torch.empty((n + 31) // 32, dtype=torch.int32).pin_memory()
    h_values = torch.empty(n, dtype=dt).pin_memory()
    h_prefix = torch.empty((n + 4095) // 4096, dtype=torch.int64).pin_memory()
    h_nnz = torch.full((1,), -1, dtype=torch.int64).pin_memory()

    B.bt_compress_host(h_x, h_bitmap, h_values, h_prefix, h_nnz, staging)
    nnz = int(h_nnz.item())
    assert nnz == c.nnz
    assert np.array_equal(W.raw_numpy(h_bitmap).view(np.uint32), c.bitmap)
    assert np.array_equal(W.raw_numpy(h_prefix).view(np.uint64), c.prefix)
    assert np.array_equal(W.raw_numpy(h_values[:nnz]), c.values)

    h_back = torch.empty(n, dtype=dt).pin_memory()
    B.bt_decompress_host(h_bitmap, h_values, h_prefix, nnz, h_back, staging)
    assert np.array_equal(W.raw_numpy(h_back), x)

    # fused forward (with dense y) and the bitmap backward
    y_ref, cr = oracle.relu_fwd_compress(x, kind)
    h_y = torch.empty(n, dtype=dt).pin_memory()
    B.bt_relu_fwd_compress_host(h_x, h_y, h_bitmap, h_values, h_prefix, h_nnz, staging)
    assert int(h_nnz.item()) == cr.nnz
    assert np.array_equal(W.raw_numpy(h_y), y_ref)
    assert np.array_equal(W.raw_numpy(h_bitmap).view(np.uint32), cr.bitmap)
    assert np.array_equal(W.raw_numpy(h_values[:cr.nnz]), cr.values)
    g = W.random_patterns(n, kind, 0.05, seed=9500 + n)
    h_g, h_gin = host_tensor(g, kind), torch.empty(n, dtype=dt).pin_memory()
    B.bt_relu_bwd_from_bitmap_host(h_bitmap, h_g, h_gin, staging)
    assert np.array_equal(W.raw_numpy(h_gin), oracle.relu_bwd_from_bitmap(cr.bitmap, g))


def test_host_capacity_and_argument_errors(oracle):
    n = 8192 * 3 + 5
    x = W.random_patterns(n, "f32", 0.2, seed=5)
    c = oracle.compress(x)
    staging = torch.empty(B.bt_host_staging_bytes(n, torch.float32), dtype=torch.uint8, device="cuda")
    h_x = host_tensor(x, "f32")
    h_bitmap = torch.empty((n + 31) // 32, dtype=torch.int32).pin_memory()
    h_prefix = torch.empty((n + 4095) // 4096, dtype=torch.int64).pin_memory()
    h_nnz = torch.zeros(1, dtype=torch.int64).pin_memory()
    small = torch.full((c.nnz // 2 + 16,), 7, dtype=torch.float32).pin_memory()
    cap = c.nnz // 2
    st = B.lib().bt_compress_host(h_x.data_ptr(), n, B.BT_F32, h_bitmap.data_ptr(), small.data_ptr(), cap,
                                  h_prefix.data_ptr(), h_nnz.data_ptr(), staging.data_ptr(), staging.numel(), None)
    assert st == B.BT_ERR_CAPACITY and int(h_nnz.item()) == c.nnz
    assert np.array_equal(W.raw_numpy(small[:cap]), c.values[:cap])
    assert (small[cap:] == 7).all()                                       # nothing past the capacity
    # too small a staging area, bad dtype: reported before anything is copied or launched
    assert B.lib().bt_compress_host(h_x.data_ptr(), n, B.BT_F32, h_bitmap.data_ptr(), small.data_ptr(), cap,
                                    h_prefix.data_ptr(), h_nnz.data_ptr(), staging.data_ptr(), 1024, None) == B.BT_ERR_WORKSPACE
    assert B.lib().bt_decompress_host(h_bitmap.data_ptr(), small.data_ptr(), h_prefix.data_ptr(), 1, n, 9,
                                      h_x.data_ptr(), staging.data_ptr(), staging.numel(), None) == B.BT_ERR_DTYPE


@pytest.mark.parametrize("where", ["pageable", "pinned_unaligned", "pinned_odd_capacity"])
def test_host_value_buffers_of_every_kind(oracle, where):
    """The packed values reach the host by two routes: a page-locked, 16-byte aligned buffer is written by the
    device itself (exactly nnz values, one synchronisation), any other buffer by a sized copy after a first
    synchronisation.  Same results either way; nothing behind the values is touched."""
    kind, dt, n = "bf16", torch.bfloat16, 8192 * 7 + 4097 + 3
    x = W.random_patterns(n, kind, 0.5, seed=77)
    c = oracle.compress(x)
    assert c.nnz % 8 != 0                                                  # the last 16-byte vector is partial
    staging = torch.empty(B.bt_host_staging_bytes(n, dt), dtype=torch.uint8, device="cuda")
    h_x = host_tensor(x, kind)
    h_bitmap = torch.empty((n + 31) // 32, dtype=torch.int32).pin_memory()
    h_prefix = torch.empty((n + 4095) // 4096, dtype=torch.int64).pin_memory()
    h_nnz = torch.zeros(1, dtype=torch.int64).pin_memory()
    room = torch.full((n + 64,), 3.0, dtype=dt)
    if where == "pageable":
        buf, cap = room[:n], n
    elif where == "pinned_unaligned":
        room = room.pin_memory()
        buf, cap = room[1:n + 1], n                                       # 2 bytes off a 16-byte boundary
    else:
        room = room.pin_memory()
        buf, cap = room[:n], c.nnz + 5                                    # capacity just above nnz
    st = B.lib().bt_compress_host(h_x.data_ptr(), n, B.BT_BF16, h_bitmap.data_ptr(), buf.data_ptr(), cap,
                                  h_prefix.data_ptr(), h_nnz.data_ptr(), staging.data_ptr(), staging.numel(), None)
    assert st == B.BT_OK and int(h_nnz.item()) == c.nnz
    assert np.array_equal(W.raw_numpy(buf[:c.nnz]), c.values)
    assert (buf[c.nnz:] == 3.0).all()                                      # exactly nnz values were written
    assert np.array_equal(W.raw_numpy(h_bitmap).view(np.uint32), c.bitmap)
    assert np.array_equal(W.raw_numpy(h_prefix).view(np.uint64), c.prefix)
