"""Calls that overlap on the GPU (different streams, a workspace each) do not disturb one another: every
output still matches the CPU oracle bit for bit."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [8192 * 40 + 5, 8192 * 400 + 77])
def test_two_streams_compress_concurrently(oracle, n):
    B.lib()
    dev = torch.device("cuda")
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    xs_raw = [W.random_patterns(n, "f32", 0.5, seed=91), W.random_patterns(n, "f32", 0.8, seed=92)]
    refs = [oracle.compress(xs_raw[0]), oracle.relu_fwd_compress(xs_raw[1], "f32")[1]]
    xs = [torch.from_numpy(x.view(np.int32).copy()).to(dev).view(torch.float32) for x in xs_raw]
    stashes = [B.Stash(n, torch.float32, dev) for _ in range(2)]
    wss = [B.new_workspace(n, dev) for _ in range(2)]
    torch.cuda.synchronize()
    for rep in range(20):
        for st in stashes:
            st.bitmap.zero_(); st.values.zero_(); st.chunk_prefix.zero_(); st.nnz_out.zero_()
        torch.cuda.synchronize()
        for k in range(8):                                   # several launches queued on each stream
            with torch.cuda.stream(streams[0]):
                B.bt_compress(xs[0], stashes[0].bitmap, stashes[0].values, stashes[0].chunk_prefix,
                              stashes[0].nnz_out, wss[0], stashes[0].dev_status, stream=streams[0])
            with torch.cuda.stream(streams[1]):
                B.bt_relu_fwd_compress(xs[1], None, stashes[1].bitmap, stashes[1].values, stashes[1].chunk_prefix,
                                       stashes[1].nnz_out, wss[1], stashes[1].dev_status, stream=streams[1])
        torch.cuda.synchronize()
        for st, c in zip(stashes, refs):
            assert st.status == B.BT_OK and st.nnz == c.nnz
            assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), c.bitmap)
            assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), c.prefix)
            assert np.array_equal(W.raw_numpy(st.values[:c.nnz]), c.values)
