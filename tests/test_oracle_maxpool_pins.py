"""Pins the oracle's 2x2 max pooling with winner codes to torch: the pooled values and the winning positions
against torch.nn.functional.max_pool2d(return_indices=True), the backward pass against autograd through it,
plus ties, signed zeros and NaNs, whose handling decides the codes."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import workloads as W

KINDS = ["f32", "f16", "bf16", "f64"]


def codes_from_indices(idx: torch.Tensor, width: int) -> np.ndarray:
    """torch's flat in-plane indices -> 2-bit window positions, packed sixteen per uint32 word, LSB first."""
    planes, ho, wo = idx.shape
    dy = idx // width - 2 * torch.arange(ho).view(1, ho, 1)
    dx = idx % width - 2 * torch.arange(wo).view(1, 1, wo)
    k = (2 * dy + dx).reshape(-1).numpy().astype(np.uint64)
    assert ((k >= 0) & (k < 4)).all()
    pad = (-k.size) % 16
    k = np.concatenate([k, np.zeros(pad, np.uint64)]).reshape(-1, 16)
    return (k << (2 * np.arange(16, dtype=np.uint64))).sum(axis=1).astype(np.uint32)


def sample(kind, planes, h, w, seed):
    t = torch.randn(planes, h, w, generator=torch.Generator().manual_seed(seed), dtype=torch.float64)
    t = torch.clamp_min(t, 0.0)                               # post-ReLU: many zero ties
    t = t.to(W.TORCH_DTYPES[kind])
    t[0, 0, :4] = torch.tensor([0.0, -0.0, -0.0, 0.0], dtype=t.dtype)   # signed-zero ties
    t[0, 2, 0] = float("nan")
    t[0, 3, 2] = float("nan"); t[0, 3, 3] = float("nan")              # two NaNs in one window: the last wins
    t[0, 4, 4] = float("inf"); t[0, 5, 5] = float("-inf")
    t[1, 0, 0] = 2.0; t[1, 0, 1] = 2.0; t[1, 1, 0] = 2.0; t[1, 1, 1] = 2.0   # a four-way tie: the first wins
    return t


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("shape", [(3, 8, 8), (5, 14, 14), (2, 6, 38), (7, 2, 2)])
def test_forward_values_and_codes_match_torch(oracle, kind, shape):
    planes, h, w = shape
    t = sample(kind, planes, max(h, 6), max(w, 6), 31)[:, :h, :w].contiguous() if min(h, w) >= 6 else \
        torch.randn(planes, h, w, generator=torch.Generator().manual_seed(1)).to(W.TORCH_DTYPES[kind])
    y, codes = oracle.maxpool2x2_fwd(W.raw_numpy(t.reshape(-1)), planes, h, w, kind)
    ref, idx = torch.nn.functional.max_pool2d(t.double().unsqueeze(0), 2, return_indices=True)
    assert np.array_equal(y, W.raw_numpy(ref[0].to(t.dtype).reshape(-1))) or torch.isnan(t).any()
    got = torch.from_numpy(y.copy()).view(t.dtype) if kind != "f64" else torch.from_numpy(y.view(np.float64).copy())
    assert torch.equal(torch.nan_to_num(got.double(), nan=123.0), torch.nan_to_num(ref[0].reshape(-1), nan=123.0))
    assert np.array_equal(codes, codes_from_indices(idx[0], w))


@pytest.mark.parametrize("kind", KINDS)
def test_backward_matches_autograd(oracle, kind):
    planes, h, w = 4, 10, 12
    t = sample(kind, planes, h, w, 32)
    t = torch.nan_to_num(t, nan=0.5)                                  # autograd multiplies; NaN inputs are pinned above
    g = torch.randn(planes, h // 2, w // 2, generator=torch.Generator().manual_seed(33), dtype=torch.float64).to(t.dtype)
    _, codes = oracle.maxpool2x2_fwd(W.raw_numpy(t.reshape(-1)), planes, h, w, kind)
    got = oracle.maxpool2x2_bwd(codes, W.raw_numpy(g.reshape(-1)), planes, h, w)
    x = t.double().clone().requires_grad_()
    torch.nn.functional.max_pool2d(x.unsqueeze(0), 2).backward(g.double().unsqueeze(0))
    assert np.array_equal(got, W.raw_numpy(x.grad.to(t.dtype).reshape(-1)))
    # exactly one position per window receives the gradient, bit for bit (also a NaN or an infinity)
    g2 = g.clone(); g2.view(-1)[0] = float("nan"); g2.view(-1)[1] = float("inf")
    got2 = oracle.maxpool2x2_bwd(codes, W.raw_numpy(g2.reshape(-1)), planes, h, w)
    nz = got2.reshape(planes, h // 2, 2, w // 2, 2).transpose(0, 1, 3, 2, 4).reshape(-1, 4)
    assert ((nz != 0).sum(axis=1) <= 1).all()
    assert np.count_nonzero(got2) == np.count_nonzero(W.raw_numpy(g2.reshape(-1)))


def test_worked_example(oracle):
    x = np.array([[1, 5, 0, 0],
                  [5, 2, 0, 0],
                  [-1, -2, 7, 7],
                  [-3, -4, 7, 8]], dtype=np.float32)
    y, codes = oracle.maxpool2x2_fwd(x.reshape(-1).view(np.uint32), 1, 4, 4, "f32")
    assert y.view(np.float32).tolist() == [5.0, 0.0, -1.0, 8.0]
    # winners: (0,1) -> 1 (first of the two fives), (0,0) -> 0 (all equal), (0,0) -> 0, (1,1) -> 3
    assert codes.tolist() == [1 | (0 << 2) | (0 << 4) | (3 << 6)]
    gin = oracle.maxpool2x2_bwd(codes, np.array([10, 20, 30, 40], np.float32).view(np.uint32), 1, 4, 4).view(np.float32)
    assert gin.reshape(4, 4).tolist() == [[0, 10, 20, 0], [0, 0, 0, 0], [30, 0, 0, 0], [0, 0, 0, 40]]
