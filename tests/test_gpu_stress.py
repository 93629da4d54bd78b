"""Randomised stress of the single-pass compaction protocol: random sizes (one element to tens of millions), zero
fractions, element types and CTA limits; two fused launches at a time on two streams, each with its own workspace filled
with garbage and reused back to back for two different tensors in turn; every output compared with torch routines on the GPU.  Runs for
BT_STRESS_SECONDS (default 5; a 300-second run covers some 200 000 cases)."""
import os
import time

import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from tests.test_gpu_full_size import bits_of, torch_bitmap, torch_prefix

pytestmark = pytest.mark.gpu


def test_random_concurrent_launches_match_torch():
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    B.lib()
    dev = torch.device("cuda")
    budget = float(os.environ.get("BT_STRESS_SECONDS", "5"))
    rng = np.random.default_rng(int(os.environ.get("BT_STRESS_SEED", "1")))
    t_end = time.time() + budget
    dts = [torch.float32, torch.bfloat16, torch.float16]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    cases = 0
    while time.time() < t_end or cases < 20:
        n = int(rng.choice([rng.integers(1, 100_000), rng.integers(100_000, 3_000_000), rng.integers(3_000_000, 60_000_000)]))
        s = float(rng.choice([0.0, 0.3, 0.5, 0.9, 0.999, 1.0]))
        dt = dts[int(rng.integers(0, 3))]
        refs = []                                                    # two different tensors of the same size
        for which in range(2):
            g = torch.Generator(device=dev).manual_seed(int(rng.integers(0, 1 << 30)))
            pre = torch.randn(n, device=dev, generator=g, dtype=torch.float32)
            sw = s if which == 0 else float(rng.choice([0.0, 0.5, 0.97]))
            thr = float(torch.quantile(pre[:min(n, 1_000_000)], sw)) if 0.0 < sw < 1.0 else (-1e9 if sw == 0.0 else 1e9)
            pre = (pre - thr).to(dt)
            y_ref = torch.where(pre > 0, pre, torch.zeros((), device=dev, dtype=dt))
            mask = bits_of(y_ref) != 0
            refs.append((pre, y_ref, int(mask.sum()), torch_bitmap(mask), torch_prefix(mask), bits_of(y_ref)[mask]))
        outs = []
        B.bt_set_max_ctas(int(rng.choice([0, 0, 0, 2, 7, 24, 49, 74, 111])))       # a share of the SMs per launch, or none
        for k, st_ in enumerate(streams):
            st_.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(st_):
                stash = B.Stash(n, dt, dev)
                ws = B.new_workspace(n, dev)
                ws.random_(0, 255)                                   # the workspace needs no initialisation
                y = torch.empty(n, device=dev, dtype=dt) if k == 0 else None
                reps = int(rng.integers(1, 5))
                for r in range(reps):                                # the same workspace back to back, the two tensors in turn:
                    pre = refs[(r + k) % 2][0]                       # words the launch before left there belong to other data
                    B.bt_relu_fwd_compress(pre, y, stash.bitmap, stash.values, stash.chunk_prefix, stash.nnz_out, ws,
                                           stash.dev_status, stream=st_)
                back = torch.empty(n, device=dev, dtype=dt)
                B.bt_decompress(stash.bitmap, stash.values, stash.chunk_prefix, back, stream=st_)
                outs.append((stash, y, back, refs[(reps - 1 + k) % 2]))
        limit = B.bt_set_max_ctas(0)
        torch.cuda.synchronize()
        for stash, y, back, (_, y_ref, nnz, bm_ref, pf_ref, v_ref) in outs:
            where = f"case {cases}: n={n} zeros={s} {dt} max_ctas={limit}"
            assert stash.status == B.BT_OK and stash.nnz == nnz, where
            assert torch.equal(stash.bitmap, bm_ref) and torch.equal(stash.chunk_prefix, pf_ref), where
            assert torch.equal(bits_of(stash.values[:nnz]), v_ref), where
            assert torch.equal(bits_of(back), bits_of(y_ref)), where
            assert y is None or torch.equal(bits_of(y), bits_of(y_ref)), where
        cases += 1
    print("stress cases:", cases)
