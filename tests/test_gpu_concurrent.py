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


def test_graph_replays_share_one_workspace_across_sizes():
    """A captured graph of launches of different sizes and element types that share ONE workspace, replayed many
    times with the inputs changed in between: every replay's words in the workspace must be told from the
    previous replay's (same captured arguments) and from the other launches' (other sizes, same memory)."""
    B.lib()
    dev = torch.device("cuda")
    sizes = [(8192 * 300 + 11, torch.float32), (8192 * 3 + 5, torch.float32), (16384 * 200 + 3, torch.bfloat16),
             (8192 * 149, torch.float32), (77, torch.float32), (4096 * 148 * 3 + 1, torch.float64)]
    xs = [torch.zeros(n, dtype=dt, device=dev) for n, dt in sizes]
    stashes = [B.Stash(n, dt, dev) for n, dt in sizes]
    ws = B.new_workspace(max(n for n, _ in sizes), dev)
    ws.random_(0, 255)
    gen = torch.Generator(device=dev).manual_seed(5)

    def refill():
        for x in xs:
            t = torch.randn(x.numel(), device=dev, generator=gen)
            x.copy_(torch.where(torch.rand(x.numel(), device=dev, generator=gen) < 0.6, torch.zeros((), device=dev), t).to(x.dtype))

    def launch_all():
        for x, st in zip(xs, stashes):
            B.bt_compress(x, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)

    refill()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        launch_all()                                          # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        launch_all()
    iv = {2: torch.int16, 4: torch.int32, 8: torch.int64}
    for rep in range(40):
        refill()
        g.replay()
        if rep % 3 == 0:
            g.replay()                                        # the same inputs twice in a row as well
        torch.cuda.synchronize()
        for x, st in zip(xs, stashes):
            bits = x.view(iv[x.element_size()])
            mask = bits != 0
            nnz = int(mask.sum())
            assert st.status == B.BT_OK and st.nnz == nnz, (rep, x.numel())
            assert torch.equal(st.values[:nnz].view(bits.dtype), bits[mask]), (rep, x.numel())
            back = torch.empty_like(x)
            B.bt_decompress(st.bitmap, st.values, st.chunk_prefix, back)
            assert torch.equal(back.view(bits.dtype), bits), (rep, x.numel())
