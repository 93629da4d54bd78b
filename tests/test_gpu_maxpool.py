"""GPU parity of the max pooling with winner codes (bt_maxpool2x2_fwd / bt_maxpool2x2_bwd) against the CPU oracle,
bit for bit, on every element type, on shapes that are ragged against the 16-output code words and the thread
blocks, with ties, signed zeros, NaNs and infinities; at full size against torch's own pooling on the GPU
(values, index tensor, autograd); and with element indices beyond 32 bits."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W

pytestmark = pytest.mark.gpu

KINDS = ["f32", "f16", "bf16", "f64"]
SHAPES = [(1, 2, 2), (3, 8, 8), (5, 14, 14), (2, 6, 38), (7, 2, 2), (64, 28, 28), (33, 112, 2), (3, 2, 1000), (131, 10, 6),
          (3, 6, 40), (1, 2, 8), (9, 4, 4), (37, 18, 24)]


@pytest.fixture(scope="module")
def G():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from tests import gpu_util
    B.lib()
    return gpu_util


def run_fwd(G, xt, planes, h, w, want_codes=True):
    outputs = planes * (h // 2) * (w // 2)
    y = G.Guarded(outputs, xt.dtype)
    codes = G.Guarded((outputs + 15) // 16, torch.int32) if want_codes else None
    B.bt_maxpool2x2_fwd(xt, y.inner, codes.inner if codes else None, planes=planes, height=h, width=w)
    torch.cuda.synchronize()
    assert y.guards_intact() and (codes is None or codes.guards_intact())
    return y.raw(), (codes.raw().view(np.uint32) if codes else None)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("shape", SHAPES)
def test_forward_and_backward_match_the_oracle(G, oracle, kind, shape):
    planes, h, w = shape
    n = planes * h * w
    x = W.random_patterns(n, kind, 0.4, seed=planes * 1000 + h * 10 + w)          # NaNs, infinities, many zero ties
    if n >= 64:
        x[8:16] = x[8]                                                             # runs of equal values
    y_ref, c_ref = oracle.maxpool2x2_fwd(x, planes, h, w, kind)
    xt = G.from_raw(x, kind)
    y, codes = run_fwd(G, xt, planes, h, w)
    assert np.array_equal(y, y_ref) and np.array_equal(codes, c_ref)
    y2, none = run_fwd(G, xt, planes, h, w, want_codes=False)
    assert none is None and np.array_equal(y2, y_ref)
    assert np.array_equal(W.raw_numpy(xt), x)                                      # the input is untouched
    g = W.random_patterns(y_ref.size, kind, 0.1, seed=77)
    gin = G.Guarded(n, G.TDT[kind])
    B.bt_maxpool2x2_bwd(torch.from_numpy(c_ref.view(np.int32).copy()).cuda(), G.from_raw(g, kind), gin.inner,
                        planes=planes, height=h, width=w)
    torch.cuda.synchronize()
    assert gin.guards_intact() and np.array_equal(gin.raw(), oracle.maxpool2x2_bwd(c_ref, g, planes, h, w))
    # masked form: the ReLU's select on the pooled gradient and the scatter in one pass
    mask = oracle.compress(W.random_patterns(y_ref.size, kind, 0.5, seed=78, with_specials=False)).bitmap
    gin2 = G.Guarded(n, G.TDT[kind])
    B.bt_maxpool2x2_bwd_masked(torch.from_numpy(c_ref.view(np.int32).copy()).cuda(),
                               torch.from_numpy(mask.view(np.int32).copy()).cuda(), G.from_raw(g, kind), gin2.inner,
                               planes=planes, height=h, width=w)
    torch.cuda.synchronize()
    masked_g = oracle.relu_bwd_from_bitmap(mask, g)
    assert gin2.guards_intact() and np.array_equal(gin2.raw(), oracle.maxpool2x2_bwd(c_ref, masked_g, planes, h, w))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_full_size_layer_against_torch(G, dtype):
    """A VGG-sized pooling input ([32,64,224,224]: 103 M elements) against torch's pooling on the GPU: pooled
    values, the positions its index tensor names, and autograd's gradient."""
    n_, c_, h, w = 32, 64, 224, 224
    x = torch.clamp_min(torch.randn(n_, c_, h, w, device="cuda", generator=torch.Generator(device="cuda").manual_seed(3)), 0).to(dtype)
    ref, idx = torch.nn.functional.max_pool2d(x, 2, return_indices=True)
    y = torch.empty_like(ref)
    codes = torch.empty((ref.numel() + 15) // 16, dtype=torch.int32, device="cuda")
    B.bt_maxpool2x2_fwd(x, y, codes)
    assert torch.equal(y, ref)
    ho, wo = h // 2, w // 2
    k = (2 * (idx // w - 2 * torch.arange(ho, device="cuda").view(1, 1, ho, 1)) +
         (idx % w - 2 * torch.arange(wo, device="cuda").view(1, 1, 1, wo))).reshape(-1)
    got = (codes.view(-1, 1).to(torch.int64) >> (2 * torch.arange(16, device="cuda"))) & 3
    assert torch.equal(got.reshape(-1)[:k.numel()], k)
    g = torch.randn(ref.shape, device="cuda", generator=torch.Generator(device="cuda").manual_seed(4)).to(dtype)
    xr = x.clone().requires_grad_()
    torch.nn.functional.max_pool2d(xr, 2).backward(g)
    gin = torch.empty_like(x)
    B.bt_maxpool2x2_bwd(codes, g, gin)
    assert torch.equal(gin, xr.grad)


@pytest.mark.parametrize("extra", [2, 8])                       # width 2^15 + 2: pair form; 2^15 + 8: vector form
def test_more_than_two_to_the_32_elements(G, extra):
    free, _ = torch.cuda.mem_get_info()
    if free < 40 << 30:
        pytest.skip("needs about 25 GB of free device memory")
    planes, h, w = 2, 1 << 16, (1 << 15) + extra                                  # 4.3 G elements of 2 bytes
    x = torch.empty(planes, h, w, dtype=torch.bfloat16, device="cuda")
    step = 1 << 13
    for k, lo in enumerate(range(0, h, step)):                                     # seeded, slab by slab
        x[:, lo:lo + step] = torch.randn(planes, step, w, device="cuda", dtype=torch.float32,
                                         generator=torch.Generator(device="cuda").manual_seed(40 + k)).clamp_min_(0).to(torch.bfloat16)
    ho, wo = h // 2, w // 2
    y = torch.empty(planes, ho, wo, dtype=x.dtype, device="cuda")
    codes = torch.empty((y.numel() + 15) // 16, dtype=torch.int32, device="cuda")
    B.bt_maxpool2x2_fwd(x, y, codes)
    # slab by slab against the plain statement of the pooling (max over the four strided views)
    for lo in range(0, ho, step):
        xs = x[:, 2 * lo:2 * (lo + step)]
        ref = torch.maximum(torch.maximum(xs[:, 0::2, 0::2], xs[:, 0::2, 1::2]), torch.maximum(xs[:, 1::2, 0::2], xs[:, 1::2, 1::2]))
        assert torch.equal(y[:, lo:lo + step], ref)
    # the backward pass puts every gradient where the forward pass found the maximum: pooling gin * (x == winner) again gives g
    g = torch.ones_like(y)
    gin = torch.empty_like(x)
    B.bt_maxpool2x2_bwd(codes, g, gin)
    for lo in range(0, ho, step):
        gs, xs = gin[:, 2 * lo:2 * (lo + step)], x[:, 2 * lo:2 * (lo + step)]
        cnt = gs[:, 0::2, 0::2] + gs[:, 0::2, 1::2] + gs[:, 1::2, 0::2] + gs[:, 1::2, 1::2]
        assert bool((cnt == 1).all())                                              # exactly one position per window
        assert bool((xs[gs == 1].numel() == y[:, lo:lo + step].numel()))
        picked = (xs * gs)
        again = torch.maximum(torch.maximum(picked[:, 0::2, 0::2], picked[:, 0::2, 1::2]),
                              torch.maximum(picked[:, 1::2, 0::2], picked[:, 1::2, 1::2]))
        assert torch.equal(again, y[:, lo:lo + step])                              # and it is a maximal one
    del x, y, codes, g, gin
    torch.cuda.empty_cache()


def test_argument_checks(G):
    x = torch.zeros(4, 6, 6, device="cuda")
    y = torch.zeros(4, 3, 3, device="cuda")
    L = B.lib()
    assert L.bt_maxpool2x2_fwd(x.data_ptr(), 4, 5, 6, B.BT_F32, y.data_ptr(), None, None) == B.BT_ERR_SHAPE
    assert L.bt_maxpool2x2_fwd(x.data_ptr(), 4, 6, 0, B.BT_F32, y.data_ptr(), None, None) == B.BT_ERR_SHAPE
    assert L.bt_maxpool2x2_fwd(x.data_ptr(), 4, 6, 6, 7, y.data_ptr(), None, None) == B.BT_ERR_DTYPE
    assert L.bt_maxpool2x2_fwd(None, 4, 6, 6, B.BT_F32, y.data_ptr(), None, None) == B.BT_ERR_NULL
    assert L.bt_maxpool2x2_fwd(x.data_ptr() + 4, 4, 6, 6, B.BT_F32, y.data_ptr(), None, None) == B.BT_ERR_ALIGN
    assert L.bt_maxpool2x2_fwd(x.data_ptr(), 0, 6, 6, B.BT_F32, y.data_ptr(), None, None) == B.BT_OK
    assert L.bt_maxpool2x2_bwd(None, y.data_ptr(), 4, 6, 6, B.BT_F32, x.data_ptr(), None) == B.BT_ERR_NULL
