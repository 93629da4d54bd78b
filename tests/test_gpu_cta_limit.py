"""bt_set_max_ctas: compress-family launches limited to a share of the SMs give the same results, bit for bit, as
unlimited ones -- a single CTA walking every tile, grids that leave a ragged last wave, limits above the SM count,
every element type and fused form -- and two limited launches on two streams agree with the oracle as well."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from tests import gpu_util
    B.lib()
    return gpu_util


@pytest.fixture(autouse=True)
def no_limit_afterwards():
    yield
    B.bt_set_max_ctas(0)


@pytest.mark.parametrize("limit", [1, 3, 49, 74, 100000])
@pytest.mark.parametrize("kind", ["f32", "bf16", "f64"])
@pytest.mark.parametrize("n", [1, 8192 * 5 + 3, 16384 * 83 + 17])
def test_limited_grids_match_the_oracle(G, oracle, limit, kind, n):
    x = W.random_patterns(n, kind, 0.5, seed=n % 1000 + limit)
    c = oracle.compress(x)
    assert B.bt_set_max_ctas(limit) == 0
    g = G.gpu_compress(G.from_raw(x, kind))
    assert B.bt_set_max_ctas(0) == limit
    assert g.guards_ok and g.status == B.BT_OK and g.nnz == c.nnz
    assert np.array_equal(g.bitmap, c.bitmap) and np.array_equal(g.prefix, c.prefix)
    assert np.array_equal(g.values.view(c.values.dtype), c.values)


@pytest.mark.parametrize("limit", [2, 37, 64])
def test_limited_fused_forms(G, oracle, limit):
    n = 8192 * 300 + 4099
    x = W.near_threshold_patterns(n, "f32", seed=limit)
    B.bt_set_max_ctas(limit)
    y_ref, c = oracle.prune_fwd_compress(x, "f32", 0.05)
    g = G.gpu_compress(G.from_raw(x, "f32"), tau=0.05, want_y=True)
    assert g.guards_ok and g.status == B.BT_OK and g.nnz == c.nnz and np.array_equal(g.y, y_ref)
    assert np.array_equal(g.bitmap, c.bitmap) and np.array_equal(g.prefix, c.prefix) and np.array_equal(g.values.view(np.uint32), c.values)
    _, cn = oracle.narrow_compress(x, "bf16", fused=True, tau=0.0)
    g = G.gpu_compress(G.from_raw(x, "f32"), relu=True, narrow="bf16")
    assert g.guards_ok and g.status == B.BT_OK and g.nnz == cn.nnz
    assert np.array_equal(g.bitmap, cn.bitmap) and np.array_equal(g.values.view(np.uint16), cn.values)


def test_two_limited_launches_side_by_side_and_in_a_graph(oracle):
    B.lib()
    dev = torch.device("cuda")
    n = 8192 * 400 + 11
    raws = [W.random_patterns(n, "f32", 0.5, seed=s) for s in (1, 2)]
    refs = [oracle.compress(r) for r in raws]
    xs = [torch.from_numpy(r.view(np.int32).copy()).to(dev).view(torch.float32) for r in raws]
    stashes = [B.Stash(n, torch.float32, dev) for _ in raws]
    wss = [B.new_workspace(n, dev) for _ in raws]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]

    def launch_both():
        for x, st, ws, s in zip(xs, stashes, wss, streams):
            B.bt_compress(x, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status, stream=s)

    B.bt_set_max_ctas(60)
    for _ in range(3):
        launch_both()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        main = torch.cuda.current_stream()
        for s in streams:
            s.wait_stream(main)
        launch_both()
        for s in streams:
            main.wait_stream(s)
    B.bt_set_max_ctas(0)                                    # the captured launches keep their 60 CTAs
    for st in stashes:
        st.values.zero_(), st.bitmap.zero_(), st.nnz_out.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for st, c in zip(stashes, refs):
        assert st.status == B.BT_OK and st.nnz == c.nnz
        assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), c.bitmap)
        assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), c.prefix)
        assert np.array_equal(W.raw_numpy(st.values[:c.nnz]).view(np.uint32), c.values)
