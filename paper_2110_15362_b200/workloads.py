"""Seeded synthetic inputs shaped like the paper's CNN training workloads.

This module only draws random tensors; it holds none of the codec's arithmetic
and is the one module both the CUDA tests/bench and the CPU oracle's callers
share.  The paper evaluates on ImageNet / CIFAR-10 activations of pre-trained
CNNs (section 4 "Setup"); those are not available offline, so tensors with the
same layer shapes and the sparsity regimes the paper reports (about 50 % zeros
after ReLU, above 70 % with pruning; sections 3.1 and 4) stand in for them.

Every generator takes a `device` and a seed and returns torch tensors; the same
bytes are then handed to the CUDA library and (via `raw_numpy`) to the oracle.
"""
from __future__ import annotations

import math
from typing import Dict, Iterator, List, Sequence, Tuple

import numpy as np
import torch

TORCH_DTYPES = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16, "f64": torch.float64}
_INT_VIEW = {1: torch.uint8, 2: torch.int16, 4: torch.int32, 8: torch.int64}
_NP_UINT = {2: np.uint16, 4: np.uint32, 8: np.uint64}

SPARSITY_SWEEP = (0.0, 0.25, 0.5, 0.7, 0.9, 0.99)
ELEM_BYTES = {"f32": 4, "f16": 2, "bf16": 2, "f64": 8}


def raw_numpy(t: torch.Tensor) -> np.ndarray:
    """Flat numpy array of the tensor's raw bit patterns (uint16/uint32/uint64)."""
    t = t.detach().contiguous().reshape(-1)
    es = t.element_size()
    return t.view(_INT_VIEW[es]).cpu().numpy().view(_NP_UINT[es])


def numel(shape: Sequence[int]) -> int:
    return int(math.prod(shape))


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, mu: float, seed: int, device) -> torch.Tensor:
    x = torch.randn(numel(shape), generator=_gen(seed, device), device=device, dtype=torch.float32)
    if mu != 0.0:
        x += mu
    return x.reshape(tuple(shape))


def mu_for_zero_fraction(s: float) -> float:
    """Mean of a unit-variance Gaussian pre-activation whose ReLU output has zero fraction s."""
    s = min(max(s, 1e-9), 1.0 - 1e-9)
    # inverse normal CDF through erfinv: Phi^-1(s) = sqrt(2) * erfinv(2s - 1)
    return -math.sqrt(2.0) * float(torch.erfinv(torch.tensor(2.0 * s - 1.0, dtype=torch.float64)))


# --------------------------------------------------------------------------- config 1
CFG1_SHAPE = (1, 64, 56, 56)


def cfg1(device="cpu", seed: int = 0) -> torch.Tensor:
    """One fp32 post-ReLU tensor [1,64,56,56]: max(0, N(0,1)), about half exact +0.0."""
    return torch.clamp_min_(_normal(CFG1_SHAPE, 0.0, seed, device), 0.0)


# --------------------------------------------------------------------------- config 2
def resnet18_shapes(batch: int = 32) -> List[Tuple[int, int, int, int]]:
    """Post-ReLU activation shapes of a ResNet-18 at 224x224 input (17 tensors)."""
    return ([(batch, 64, 112, 112)] + [(batch, 64, 56, 56)] * 4 + [(batch, 128, 28, 28)] * 4
            + [(batch, 256, 14, 14)] * 4 + [(batch, 512, 7, 7)] * 4)


def cfg2_layer(index: int, shape, device="cpu", target_zero_fraction: float = 0.5) -> torch.Tensor:
    mu = mu_for_zero_fraction(target_zero_fraction)
    return torch.clamp_min_(_normal(shape, mu, 100 + index, device), 0.0)


def cfg2_preact(index: int, shape, device="cpu", target_zero_fraction: float = 0.5) -> torch.Tensor:
    """The pre-activation whose ReLU is `cfg2_layer(index, ...)` (same seed, no clamp)."""
    return _normal(shape, mu_for_zero_fraction(target_zero_fraction), 100 + index, device)


def cfg2_grad(index: int, shape, device="cpu") -> torch.Tensor:
    return _normal(shape, 0.0, 150 + index, device)


# --------------------------------------------------------------------------- config 3
def cfg3_iid(n: int, s: float, index: int, device="cpu") -> torch.Tensor:
    """fp32, zeros at i.i.d. Bernoulli(s) positions, non-zeros |N(0,1)| + 1e-3."""
    g = _gen(300 + index, device)
    keep = torch.rand(n, generator=g, device=device) >= s
    v = torch.randn(n, generator=g, device=device).abs_().add_(1e-3)
    return torch.where(keep, v, torch.zeros((), device=device))


def _geometric(k: int, mean: float, g: torch.Generator, device) -> torch.Tensor:
    """k draws of a geometric length with support >= 1 and the given mean."""
    if mean <= 1.0:
        return torch.ones(k, dtype=torch.int64, device=device)
    return torch.empty(k, device=device, dtype=torch.float64).geometric_(1.0 / mean, generator=g).to(torch.int64)


def cfg3_clustered(n: int, s: float, index: int, device="cpu") -> torch.Tensor:
    """fp32, zeros and non-zeros in alternating runs of geometric length.

    Non-zero runs have mean m1 = max(1, 64(1-s)/s) and zero runs mean m0 = m1*s/(1-s),
    so zero runs have mean 64 wherever that leaves m1 >= 1; s = 0 is all non-zero."""
    g = _gen(400 + index, device)
    v = torch.randn(n, generator=g, device=device).abs_().add_(1e-3)
    if s <= 0.0:
        return v
    if s >= 1.0:
        return torch.zeros(n, device=device)
    m1 = max(1.0, 64.0 * (1.0 - s) / s)
    m0 = m1 * s / (1.0 - s)
    pairs = int(n / (m0 + m1) * 1.2) + 64
    first_is_zero = bool(torch.rand(1, generator=g, device=device).item() < 0.5)
    while True:
        z = _geometric(pairs, m0, g, device)
        o = _geometric(pairs, m1, g, device)
        lens = torch.stack((z, o) if first_is_zero else (o, z), dim=1).reshape(-1)
        if int(lens.sum().item()) >= n:
            break
        pairs *= 2
    flags = torch.zeros(2 * pairs, dtype=torch.bool, device=device)
    flags[(1 if first_is_zero else 0)::2] = True          # True marks a non-zero run
    keep = torch.repeat_interleave(flags, lens)[:n]
    return torch.where(keep, v, torch.zeros((), device=device))


# --------------------------------------------------------------------------- config 4
def vgg16_shapes(batch: int = 64) -> List[Tuple[int, int, int, int]]:
    """Conv outputs of a VGG-16 at 224x224 input (13 tensors)."""
    return ([(batch, 64, 224, 224)] * 2 + [(batch, 128, 112, 112)] * 2 + [(batch, 256, 56, 56)] * 3
            + [(batch, 512, 28, 28)] * 3 + [(batch, 512, 14, 14)] * 3)


def cfg4_preact(index: int, shape, kind: str, device="cpu") -> torch.Tensor:
    """N(0,1) pre-activations drawn in fp32 and rounded to `kind` by torch."""
    return _normal(shape, 0.0, 500 + index, device).to(TORCH_DTYPES[kind])


def cfg4_grad(index: int, shape, kind: str, device="cpu") -> torch.Tensor:
    return _normal(shape, 0.0, 600 + index, device).to(TORCH_DTYPES[kind])


# --------------------------------------------------------------------------- config 5
def mobilenetv2_shapes(batch: int = 128) -> List[Tuple[int, int, int, int]]:
    """ReLU6 sites of a MobileNetV2 at 224x224: after the stem, after every expand
    1x1 (when the expansion factor is above 1), after every depthwise 3x3, and
    after the last 1x1 convolution (35 tensors)."""
    shapes = [(batch, 32, 112, 112)]
    c_in, res = 32, 112
    for t, c, reps, stride in ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                               (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)):
        for r in range(reps):
            st = stride if r == 0 else 1
            hidden = c_in * t
            if t != 1:
                shapes.append((batch, hidden, res, res))      # after the expand 1x1
            res = res // st
            shapes.append((batch, hidden, res, res))          # after the depthwise 3x3
            c_in = c
    shapes.append((batch, 1280, res, res))
    return shapes


def cfg5_zero_fractions(count: int) -> List[float]:
    g = _gen(700, "cpu")
    return (0.7 + 0.15 * torch.rand(count, generator=g, dtype=torch.float64)).tolist()


def cfg5_layer(index: int, shape, zero_fraction: float, device="cpu") -> torch.Tensor:
    x = _normal(shape, mu_for_zero_fraction(zero_fraction), 710 + index, device)
    return x.clamp_(0.0, 6.0)


# --------------------------------------------------------------------------- edge cases
EDGE_SIZES = (0, 1, 31, 32, 33, 63, 64, 4095, 4096, 4097, 8191, 8192, 8193, 3 * 4096 + 17,
              16384, 16385, 40000, 5 * 8192 + 4095)

SPECIAL_F32 = (0x00000000, 0x80000000, 0x3F800000, 0xBF800000, 0x00000001, 0x80000001,
               0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00001, 0x7F800001, 0xFF800001)
SPECIAL_F16 = (0x0000, 0x8000, 0x3C00, 0xBC00, 0x0001, 0x8001, 0x7C00, 0xFC00, 0x7E00, 0xFE01,
               0x7C01, 0xFC01)
SPECIAL_BF16 = (0x0000, 0x8000, 0x3F80, 0xBF80, 0x0001, 0x8001, 0x7F80, 0xFF80, 0x7FC0, 0xFFC1,
                0x7F81, 0xFF81)
SPECIAL_F64 = (0x0000000000000000, 0x8000000000000000, 0x3FF0000000000000, 0xBFF0000000000000,
               0x0000000000000001, 0x8000000000000001, 0x7FF0000000000000, 0xFFF0000000000000,
               0x7FF8000000000000, 0xFFF8000000000001, 0x7FF0000000000001, 0xFFF0000000000001,
               0x0000000100000000, 0x00000000FFFFFFFF)          # the last two: non-zero in one 32-bit half only
SPECIALS = {"f32": SPECIAL_F32, "f16": SPECIAL_F16, "bf16": SPECIAL_BF16, "f64": SPECIAL_F64}


def random_patterns(n: int, kind: str, zero_fraction: float, seed: int, with_specials: bool = True
                    ) -> np.ndarray:
    """Raw unsigned patterns of `kind`: uniformly random bits (so NaNs, infinities,
    subnormals and negative values all occur), zeroed at Bernoulli(zero_fraction)
    positions, with the special patterns (signed zeros, infinities, NaNs, smallest
    subnormals) sprinkled in."""
    es = ELEM_BYTES[kind]
    rng = np.random.default_rng(seed)
    if es == 8:
        x = rng.integers(0, 1 << 63, size=n, dtype=np.uint64) | (rng.integers(0, 2, size=n, dtype=np.uint64) << np.uint64(63))
    else:
        x = rng.integers(0, 1 << (8 * es), size=n, dtype=np.uint64).astype(_NP_UINT[es])
    x[rng.random(n) < zero_fraction] = 0
    if with_specials and n:
        sp = np.array(SPECIALS[kind], dtype=_NP_UINT[es])
        where = rng.integers(0, n, size=max(1, n // 7))
        x[where] = sp[rng.integers(0, len(sp), size=where.size)]
    return x


def prune_preact(n: int, device="cpu", seed: int = 0) -> torch.Tensor:
    """fp32 pre-activations for the pruning measurement: N(0, 0.15), so that half are not positive and
    about three quarters do not exceed 0.1 -- the paper's observation that more than 70 % of a network's
    activations are close to zero (section 3.1, activation histogram)."""
    g = _gen(900 + seed, device)
    return torch.randn(n, generator=g, device=device) * 0.15


# pruning thresholds of the paper's activation-pruning study (section 4, Figure 9)
PRUNE_THRESHOLDS = (0.0, 0.01, 0.05, 0.1)


def near_threshold_patterns(n: int, kind: str, taus=PRUNE_THRESHOLDS, seed: int = 0) -> np.ndarray:
    """Raw patterns of `kind` for the pruning tests: close-to-zero activations of both signs (the bulk of
    a network's activations), and, sprinkled in, each threshold as the element type rounds it, its two
    neighbours in that type, the special patterns and exact zeros.  Draws only; no comparison is made here."""
    es = ELEM_BYTES[kind]
    tdt = TORCH_DTYPES[kind]
    g = torch.Generator().manual_seed(seed)
    body = (torch.randn(n, generator=g) * 0.08).to(tdt)
    x = raw_numpy(body).copy()
    if n:
        rng = np.random.default_rng(seed + 1)
        edge = []
        for t in taus:
            r = int(raw_numpy(torch.tensor([t], dtype=torch.float32).to(tdt))[0])
            edge += [r, r + 1, max(r - 1, 0), r | (1 << (8 * es - 1))]
        pool = np.array(edge + list(SPECIALS[kind]) + [0, 0, 0], dtype=_NP_UINT[es])
        where = rng.integers(0, n, size=max(1, n // 5))
        x[where] = pool[rng.integers(0, len(pool), size=where.size)]
    return x


def iter_layers(shapes) -> Iterator[Tuple[int, Tuple[int, ...], int]]:
    for i, s in enumerate(shapes):
        yield i, tuple(s), numel(s)
