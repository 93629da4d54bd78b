"""A VGG-16-shaped training step with and without the stash (random weights, random images).

    python -m paper_2110_15362_b200.demo_vgg_step [--batch 32] [--size 224] [--dtype f32|bf16] [--arena-gib 8]

Builds the thirteen 3x3 convolutions and five 2x2 max-pools of VGG-16 (no batch normalisation, a small
linear head), runs forward + backward several ways -- plain PyTorch (in-place ReLU), saved activations
stashed (exact-size values, one host read per tensor), the same with the pooling layers keeping 2-bit winner
codes instead of their input and an index tensor, that with the values in an arena (no host read), the arena with
each ReLU + pooling pair done pooling first (the full-size activation in front of a pooling layer is never
written), and (fp32 only) the arena with the values down-cast to bfloat16 on stash, which is lossy in the gradients -- and prints one
JSON line with the bytes kept for the saved ReLU outputs relative to their dense size, the device memory held between the forward and the backward pass, the peak above the model's own tensors
and the step time of each.  The peak also
holds what no stash touches: the transients of the widest layer (its pre-activation, its gradients, the
restored activation) and the max-pool indices, so it drops by less than the saved activations do.  The paper
measures the training-memory footprint of such models on ImageNet / CIFAR-10 with pre-trained weights; with
random weights and inputs about half of every ReLU output is zero, which is the sparsity level the paper
reports for ReLU layers, so the activation-memory ratio is comparable while accuracy is not touched here.
"""
from __future__ import annotations

import argparse
import gc
import json
import sys

import torch
import torch.nn.functional as F

from . import autograd as A
from . import binding as B

HELD = []          # device bytes allocated at the end of each forward pass (read by measure())
CFG = (64, 64, "M", 128, 128, "M", 256, 256, 256, "M", 512, 512, 512, "M", 512, 512, 512, "M")


def make_weights(dtype, device, seed=0):
    g = torch.Generator(device=device).manual_seed(seed)
    ws, c_in = [], 3
    for c in CFG:
        if c == "M":
            continue
        w = torch.randn(c, c_in, 3, 3, generator=g, device=device, dtype=torch.float32) * (2.0 / (9 * c_in)) ** 0.5
        ws.append(w.to(dtype).requires_grad_())
        c_in = c
    head = (torch.randn(1000, 512, generator=g, device=device) * 0.02).to(dtype).requires_grad_()
    return ws, head


def step(x, ws, head, relu, pool=lambda t: F.max_pool2d(t, 2), relu_before_pool=None, relu_pool=None):
    """`relu_before_pool`: the activation used where a pooling layer follows (default: `relu`).  `relu_pool`: one
    call that does the activation and the pooling layer behind it (replaces both there)."""
    h, k = x, 0
    for i, c in enumerate(CFG):
        if c == "M":
            if relu_pool is None:
                h = pool(h)
        else:
            h = F.conv2d(h, ws[k], padding=1)
            if CFG[i + 1] == "M" and relu_pool is not None:
                h = relu_pool(h)
            else:
                h = (relu_before_pool if relu_before_pool is not None and CFG[i + 1] == "M" else relu)(h)
            k += 1
    logits = F.linear(h.mean(dim=(2, 3)), head)
    loss = logits.float().square().mean()
    del h, logits
    HELD.append(torch.cuda.memory_allocated())                # what the graph holds between the two passes
    loss.backward()
    for w in ws + [head]:
        w.grad = None
    return float(loss.detach())


def measure(fn, reps=3):
    fn()                                                      # warm-up (cuDNN algorithm choice, allocator)
    torch.cuda.synchronize()
    gc.collect()                                              # tensors kept alive only by reference cycles (a caller's
    torch.cuda.empty_cache()                                  # earlier work) must not be freed in mid-measurement
    best, peak, loss = None, 0, None
    for _ in range(reps):
        torch.cuda.reset_peak_memory_stats()
        base = torch.cuda.memory_allocated()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        loss = fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        best = ms if best is None else min(best, ms)
        peak = max(peak, torch.cuda.max_memory_allocated() - base)
        held = HELD[-1] - base
    return {"held_after_forward_mib": round(held / 2 ** 20, 1), "peak_mib": round(peak / 2 ** 20, 1),
            "step_ms": round(best, 2), "loss": loss}


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--size", type=int, default=224)
    ap.add_argument("--dtype", choices=["f32", "bf16"], default="f32")
    ap.add_argument("--arena-gib", type=float, default=8.0)
    args = ap.parse_args(argv)

    B.lib()
    dev = torch.device("cuda")
    dtype = {"f32": torch.float32, "bf16": torch.bfloat16}[args.dtype]
    ws, head = make_weights(dtype, dev)
    x = torch.randn(args.batch, 3, args.size, args.size, device=dev, dtype=dtype,
                    generator=torch.Generator(device=dev).manual_seed(1))

    out = {"model": "VGG-16 shaped (13 conv, 5 max-pool, no BN), random weights and inputs", "batch": args.batch,
           "size": args.size, "dtype": args.dtype}
    out["plain"] = measure(lambda: step(x, ws, head, torch.relu_))

    def scratch_mib(hooks):
        t = list(hooks.scratch.ws.values()) + list(hooks.scratch.values.values())
        return round(sum(b.numel() * b.element_size() for b in t) / 2 ** 20, 1)

    # one context object per variant, entered once per step: its scratch (workspace and a full-capacity values
    # buffer) is allocated by the warm-up step and reported on its own
    hooks1 = A.stash_saved_activations()

    def stashed():
        with hooks1:
            before = hooks1.packed_bytes, hooks1.dense_bytes
            loss = step(x, ws, head, lambda t: A.relu_stash(t, hooks1, inplace=True))
            out["saved_activation_bytes_over_dense"] = round((hooks1.packed_bytes - before[0]) /
                                                             max(1, hooks1.dense_bytes - before[1]), 4)
        return loss

    out["stashed"] = measure(stashed)
    out["stashed"]["scratch_mib"] = scratch_mib(hooks1)
    del hooks1
    torch.cuda.empty_cache()
    hooks2 = A.stash_saved_activations()

    def stashed_pool():
        with hooks2:
            return step(x, ws, head, lambda t: A.relu_stash(t, hooks2, inplace=True), A.maxpool2x2_stash,
                        lambda t: A.relu_stash(t, hooks2, inplace=True, keep_values=False))

    out["stashed_pool_codes"] = measure(stashed_pool)
    out["stashed_pool_codes"]["scratch_mib"] = scratch_mib(hooks2)
    del hooks2
    torch.cuda.empty_cache()

    arena_hooks = A.stash_saved_activations(arena_bytes=int(args.arena_gib * 2 ** 30))

    def arena():
        with arena_hooks:
            return step(x, ws, head, lambda t: A.relu_stash(t, arena_hooks, inplace=True), A.maxpool2x2_stash,
                        lambda t: A.relu_stash(t, arena_hooks, inplace=True, keep_values=False))

    out["stashed_arena"] = measure(arena)
    out["stashed_arena"]["arena_used_mib"] = round(int(arena_hooks.cursor.item()) / 2 ** 20, 1)
    out["stashed_arena"]["peak_mib_with_arena_used"] = round(out["stashed_arena"]["peak_mib"] +
                                                            out["stashed_arena"]["arena_used_mib"], 1)
    del arena_hooks
    torch.cuda.empty_cache()
    first_hooks = A.stash_saved_activations(arena_bytes=int(args.arena_gib * 2 ** 30))

    def arena_pool_first():
        with first_hooks:
            return step(x, ws, head, lambda t: A.relu_stash(t, first_hooks, inplace=True),
                        relu_pool=lambda t: A.relu_maxpool2x2_stash(t, first_hooks))

    out["stashed_arena_pool_first"] = measure(arena_pool_first)
    out["stashed_arena_pool_first"]["arena_used_mib"] = round(int(first_hooks.cursor.item()) / 2 ** 20, 1)
    if dtype == torch.float32:
        del first_hooks
        torch.cuda.empty_cache()
        narrow_hooks = A.stash_saved_activations(arena_bytes=int(args.arena_gib * 2 ** 30), narrow=torch.bfloat16)

        def arena_narrow():
            with narrow_hooks:
                return step(x, ws, head, lambda t: A.relu_stash(t, narrow_hooks, inplace=True), A.maxpool2x2_stash,
                            lambda t: A.relu_stash(t, narrow_hooks, inplace=True, keep_values=False))

        out["stashed_arena_bf16_values"] = measure(arena_narrow)
        out["stashed_arena_bf16_values"]["arena_used_mib"] = round(int(narrow_hooks.cursor.item()) / 2 ** 20, 1)
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
