"""Pins the oracle's ReLU6 pair (the activation of the MobileNetV2 family) to torch: the forward against
torch.nn.functional.relu6, the backward against autograd through it, plus the special patterns."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import workloads as W

KINDS = ["f32", "f16", "bf16", "f64"]


def sample(kind, n, seed):
    t = (torch.randn(n, generator=torch.Generator().manual_seed(seed), dtype=torch.float64) * 4).to(W.TORCH_DTYPES[kind])
    t[::53] = 0.0
    t[3::59] = 6.0
    t[5::61] = -0.0
    t[7] = float("inf"); t[8] = float("-inf")
    t[9] = torch.nextafter(torch.tensor(6.0, dtype=t.dtype), torch.tensor(0.0, dtype=t.dtype)) if t.dtype != torch.bfloat16 \
        else torch.tensor(5.96875, dtype=torch.bfloat16)             # the bf16 value just below 6
    return t


@pytest.mark.parametrize("kind", KINDS)
def test_forward_matches_torch_relu6(oracle, kind):
    n = 3 * 4096 + 91
    t = sample(kind, n, 21)
    y, c = oracle.relu6_fwd_compress(W.raw_numpy(t), kind)
    y_ref = W.raw_numpy((torch.nn.functional.relu6(t.double()) + 0.0).to(t.dtype))      # + 0.0: no -0.0 (as for ReLU)
    assert np.array_equal(y, y_ref)
    c2 = oracle.compress(y)                                          # and the stash is Algorithm 1 of y
    assert c.nnz == c2.nnz and all(np.array_equal(a, b) for a, b in zip(c[:3], c2[:3]))
    bits = np.unpackbits(c.bitmap.view(np.uint8), bitorder="little")[:n].astype(bool)
    assert np.array_equal(bits, (t.double() > 0).numpy())
    assert np.array_equal(oracle.decompress(c), y)
    _, c3 = oracle.relu6_fwd_compress(W.raw_numpy(t), kind, want_y=False)
    assert all(np.array_equal(a, b) for a, b in zip(c[:3], c3[:3]))


@pytest.mark.parametrize("kind", KINDS)
def test_backward_matches_autograd(oracle, kind):
    n = 2 * 4096 + 33
    t = sample(kind, n, 22)
    g = torch.randn(n, generator=torch.Generator().manual_seed(23), dtype=torch.float64).to(t.dtype)
    g[11] = float("nan"); g[12] = float("inf"); g[13] = -1.0
    _, c = oracle.relu6_fwd_compress(W.raw_numpy(t), kind)
    got = oracle.relu6_bwd_from_stash(c, kind, W.raw_numpy(g))
    x = t.double().clone().requires_grad_()
    finite_g = torch.nan_to_num(g.double(), nan=1.0, posinf=2.0, neginf=-2.0)     # autograd multiplies; keep it finite
    torch.nn.functional.relu6(x).backward(finite_g)
    passed = x.grad != 0
    passed |= (finite_g == 0) & (x.detach() > 0) & (x.detach() < 6)
    ref = torch.where(passed, g, torch.zeros((), dtype=g.dtype))
    assert np.array_equal(got, W.raw_numpy(ref))
    # saturated and non-positive units pass nothing, whatever the gradient holds
    tt = t.double()
    assert not got[((tt >= 6) | (tt <= 0)).numpy()].any()


@pytest.mark.parametrize("kind", ["f32", "f16", "bf16", "f64"])
def test_special_patterns(oracle, kind):
    es = W.ELEM_BYTES[kind]
    sp = np.array(W.SPECIALS[kind], dtype={2: np.uint16, 4: np.uint32, 8: np.uint64}[es])
    y, c = oracle.relu6_fwd_compress(sp, kind)
    six = {"f32": 0x40C00000, "f16": 0x4600, "bf16": 0x40C0, "f64": 0x4018000000000000}[kind]
    sign = 1 << (8 * es - 1)
    expmask = {"f32": 0x7F800000, "f16": 0x7C00, "bf16": 0x7F80, "f64": 0x7FF0000000000000}[kind]
    for xin, yout in zip(sp.tolist(), y.tolist()):
        mag = xin & (sign - 1)
        if mag > expmask:
            assert yout == xin                                       # NaN kept with its payload
        elif xin & sign or mag == 0:
            assert yout == 0
        elif xin >= six:
            assert yout == six                                       # +inf and everything from 6 up saturate
        else:
            assert yout == xin
