"""Parity at the full sizes of the five workload configurations, in the launch configuration the
benchmark times (the library's own launch shapes, one stream).

Whole tensors against the CPU oracle, every output compared element by element, outputs in guarded
buffers: the 1 GiB tensor of configuration 3 (i.i.d. at half zeros, clustered at 90 % zeros), the largest
tensor of configuration 4 in bfloat16 and binary16 (fused forward with the dense output, and the backward
pass), one layer of configuration 5, and every layer of configuration 2.

The rest of the sweep (every sparsity, every distinct shape, the forward-then-reverse trace) is checked
three ways per tensor: (1) the oracle on randomly sampled 4096-element chunks (bitmap words, packed values,
prefix entry, restored elements), (2) torch routines on the GPU over the whole tensor (boolean indexing,
packed bits, chunk counts, relu, where) as an independent full-size check, (3) properties that hold at any
size (nnz == popcount(bitmap), the round trip is the identity bit for bit, bytes formula)."""
import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import workloads as W
from tests.gpu_util import Guarded

pytestmark = pytest.mark.gpu
DEV = "cuda"
IV = {2: torch.int16, 4: torch.int32}


def bits_of(t):
    return t.view(IV[t.element_size()])


def torch_bitmap(mask: torch.Tensor) -> torch.Tensor:
    """LSB-first uint32 words of a boolean vector, built with torch on the GPU in slices."""
    n = mask.numel()
    out = torch.empty((n + 31) // 32, dtype=torch.int32, device=mask.device)
    shifts = torch.arange(32, device=mask.device, dtype=torch.int64)
    step = 1 << 24
    for lo in range(0, n, step):
        m = mask[lo:lo + step]
        pad = (-m.numel()) % 32
        if pad:
            m = torch.nn.functional.pad(m, (0, pad))
        w = (m.view(-1, 32).to(torch.int64) << shifts).sum(dim=1)
        out[lo // 32: lo // 32 + w.numel()] = w.to(torch.int32)
    return out


def torch_prefix(mask: torch.Tensor) -> torch.Tensor:
    n = mask.numel()
    pad = (-n) % 4096
    m = torch.nn.functional.pad(mask, (0, pad)) if pad else mask
    per_chunk = m.view(-1, 4096).sum(dim=1, dtype=torch.int64)
    return torch.cumsum(per_chunk, 0) - per_chunk


def check_against_torch(st: B.Stash, y: torch.Tensor):
    """Whole-tensor check of a stash of y (y already post-ReLU where that applies)."""
    mask = bits_of(y) != 0
    nnz = int(mask.sum().item())
    assert st.status == B.BT_OK and st.nnz == nnz
    assert not hasattr(st, "intact") or st.intact()          # nothing written outside the stash's buffers
    assert torch.equal(st.bitmap, torch_bitmap(mask))
    assert torch.equal(st.chunk_prefix, torch_prefix(mask))
    assert torch.equal(bits_of(st.values[:nnz]), bits_of(y)[mask])
    # nnz == popcount(bitmap), by a different route than the packing above
    b = st.bitmap.view(torch.uint8)
    pop = sum(int(((b >> k) & 1).sum(dtype=torch.int64).item()) for k in range(8))
    assert pop == nnz
    n = y.numel()
    assert B.bt_compressed_bytes(n, nnz, y.dtype) == 4 * ((n + 31) // 32) + nnz * y.element_size() + 8 * ((n + 4095) // 4096)
    return nnz


def check_sampled_chunks(oracle, st: B.Stash, y: torch.Tensor, restored, seed: int, samples: int = 24):
    n = y.numel()
    chunks = (n + 4095) // 4096
    rng = np.random.default_rng(seed)
    picks = sorted(set(rng.integers(0, chunks, size=samples).tolist()) | {0, chunks - 1})
    prefix = st.chunk_prefix
    nnz = st.nnz
    for c in picks:
        lo, hi = c * 4096, min(n, (c + 1) * 4096)
        ref = oracle.compress(W.raw_numpy(y[lo:hi]))
        words = W.raw_numpy(st.bitmap[lo // 32:(hi + 31) // 32]).view(np.uint32)
        assert np.array_equal(words, ref.bitmap), c
        start = int(prefix[c].item())
        end = int(prefix[c + 1].item()) if c + 1 < chunks else nnz
        assert end - start == ref.nnz, c
        assert np.array_equal(W.raw_numpy(st.values[start:end]), ref.values), c
        if restored is not None:
            assert np.array_equal(W.raw_numpy(restored[lo:hi]), W.raw_numpy(y[lo:hi])), c


def compress(x, ws=None):
    n = x.numel()
    st = GStash(n, x.dtype, DEV)
    B.bt_compress(x, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws if ws is not None else B.new_workspace(n, DEV),
                  st.dev_status)
    return st


def decompress(st, like):
    out = torch.empty_like(like)
    B.bt_decompress(st.bitmap, st.values, st.chunk_prefix, out)
    return out


class GStash(B.Stash):
    """B.Stash with every buffer between canary regions (same attributes, plus intact())."""

    def __init__(self, n, dtype, device=DEV, values_capacity=None):
        self.n, self.dtype = n, dtype
        cap = n if values_capacity is None else values_capacity
        self._g = [Guarded((n + 31) // 32, torch.int32), Guarded(cap, dtype), Guarded((n + 4095) // 4096, torch.int64),
                   Guarded(1, torch.int64), Guarded(1, torch.int32)]
        self.bitmap, self.values, self.chunk_prefix, self.nnz_out, self.dev_status = (g.inner for g in self._g)

    def intact(self):
        return all(g.guards_intact() for g in self._g)


class GuardedStash:
    """The buffers of one stash, each between canary regions."""

    def __init__(self, n, dtype):
        self.bitmap = Guarded((n + 31) // 32, torch.int32)
        self.values = Guarded(n, dtype)
        self.prefix = Guarded((n + 4095) // 4096, torch.int64)
        self.nnz = Guarded(1, torch.int64)
        self.status = Guarded(1, torch.int32)

    def args(self):
        return self.bitmap.inner, self.values.inner, self.prefix.inner, self.nnz.inner

    def intact(self):
        return all(g.guards_intact() for g in (self.bitmap, self.values, self.prefix, self.nnz, self.status))

    def equals(self, c):
        nnz = int(self.nnz.inner.item())
        assert int(self.status.inner.item()) == B.BT_OK and nnz == c.nnz
        assert np.array_equal(self.bitmap.raw().view(np.uint32), c.bitmap)
        assert np.array_equal(self.prefix.raw().view(np.uint64), c.prefix)
        assert np.array_equal(W.raw_numpy(self.values.inner[:nnz]), c.values)
        assert self.intact()


def whole_tensor_round_trip(oracle, x):
    """bt_compress, bt_decompress and bt_relu_bwd_from_bitmap of one tensor, every output against the oracle."""
    n = x.numel()
    raw = W.raw_numpy(x)
    st = GuardedStash(n, x.dtype)
    B.bt_compress(x, *st.args(), B.new_workspace(n, DEV), st.status.inner)
    c = oracle.compress(raw)
    st.equals(c)
    back = Guarded(n, x.dtype)
    B.bt_decompress(st.bitmap.inner, st.values.inner, st.prefix.inner, back.inner)
    assert np.array_equal(back.raw(), oracle.decompress(c)) and back.guards_intact()
    assert np.array_equal(back.raw(), raw)
    del back
    g = torch.randn(n, generator=torch.Generator(device=DEV).manual_seed(n % 1000003), device=DEV, dtype=torch.float32).to(x.dtype)
    gin = Guarded(n, x.dtype)
    B.bt_relu_bwd_from_bitmap(st.bitmap.inner, g, gin.inner)
    assert np.array_equal(gin.raw(), oracle.relu_bwd_from_bitmap(c.bitmap, W.raw_numpy(g))) and gin.guards_intact()
    return c


def test_cfg3_one_gibibyte_iid_half_zeros_whole_tensor_against_the_oracle(oracle):
    x = W.cfg3_iid(1 << 28, 0.5, W.SPARSITY_SWEEP.index(0.5), DEV)
    c = whole_tensor_round_trip(oracle, x)
    assert abs(c.nnz / x.numel() - 0.5) < 0.01


def test_cfg3_one_gibibyte_clustered_ninety_percent_zeros_whole_tensor_against_the_oracle(oracle):
    x = W.cfg3_clustered(1 << 28, 0.9, W.SPARSITY_SWEEP.index(0.9), DEV)
    c = whole_tensor_round_trip(oracle, x)
    assert abs(c.nnz / x.numel() - 0.1) < 0.02


@pytest.mark.parametrize("kind", ["bf16", "f16"])
def test_cfg4_largest_tensor_fused_pair_whole_tensor_against_the_oracle(oracle, kind):
    shapes = W.vgg16_shapes(64)
    i = max(range(len(shapes)), key=lambda k: W.numel(shapes[k]))
    n = W.numel(shapes[i])
    assert n == 205520896
    pre = W.cfg4_preact(i, shapes[i], kind, DEV).reshape(-1)
    g = W.cfg4_grad(i, shapes[i], kind, DEV).reshape(-1)
    y_ref, c = oracle.relu_fwd_compress(W.raw_numpy(pre), kind)
    ws = B.new_workspace(n, DEV)
    st = GuardedStash(n, pre.dtype)
    y = Guarded(n, pre.dtype)
    B.bt_relu_fwd_compress(pre, y.inner, *st.args(), ws, st.status.inner)
    st.equals(c)
    assert np.array_equal(y.raw(), y_ref) and y.guards_intact()
    st2 = GuardedStash(n, pre.dtype)                         # the form without the dense output
    B.bt_relu_fwd_compress(pre, None, *st2.args(), ws, st2.status.inner)
    st2.equals(c)
    del st2, y
    gin = Guarded(n, pre.dtype)
    B.bt_relu_bwd_from_bitmap(st.bitmap.inner, g, gin.inner)
    assert np.array_equal(gin.raw(), oracle.relu_bwd_from_bitmap(c.bitmap, W.raw_numpy(g))) and gin.guards_intact()
    back = Guarded(n, pre.dtype)
    B.bt_decompress(st.bitmap.inner, st.values.inner, st.prefix.inner, back.inner)
    assert np.array_equal(back.raw(), y_ref) and back.guards_intact()


def test_cfg5_one_layer_whole_tensor_against_the_oracle(oracle):
    shapes = W.mobilenetv2_shapes(128)
    fractions = W.cfg5_zero_fractions(len(shapes))
    i = max(range(len(shapes)), key=lambda k: W.numel(shapes[k]))       # the largest layer of the trace
    x = W.cfg5_layer(i, shapes[i], fractions[i], DEV).reshape(-1)
    c = whole_tensor_round_trip(oracle, x)
    assert abs((1 - c.nnz / x.numel()) - fractions[i]) < 0.02


def test_cfg2_resnet18_batch32_every_layer_against_the_oracle(oracle):
    for i, shape, n in W.iter_layers(W.resnet18_shapes(32)):
        x = W.cfg2_layer(i, shape, DEV).reshape(-1)
        st = GuardedStash(n, x.dtype)
        B.bt_compress(x, *st.args(), B.new_workspace(n, DEV), st.status.inner)
        back = Guarded(n, x.dtype)
        B.bt_decompress(st.bitmap.inner, st.values.inner, st.prefix.inner, back.inner)
        torch.cuda.synchronize()
        st.equals(oracle.compress(W.raw_numpy(x)))            # every layer whole
        assert np.array_equal(back.raw(), W.raw_numpy(x)) and back.guards_intact()


@pytest.mark.parametrize("variant", ["iid", "clustered"])
@pytest.mark.parametrize("s", W.SPARSITY_SWEEP)
def test_cfg3_one_gibibyte_sparsity_sweep(oracle, variant, s):
    n = 1 << 28
    idx = W.SPARSITY_SWEEP.index(s)
    x = (W.cfg3_iid if variant == "iid" else W.cfg3_clustered)(n, s, idx, DEV)
    st = compress(x)
    back = decompress(st, x)
    nnz = check_against_torch(st, x)
    assert abs((1 - nnz / n) - s) < 0.02
    assert torch.equal(bits_of(back), bits_of(x))
    check_sampled_chunks(oracle, st, x, back, seed=17 + idx)
    # the bitmap-masked gradient at the same size
    g = W.cfg2_grad(idx, (n,), DEV)
    gin = torch.empty_like(g)
    B.bt_relu_bwd_from_bitmap(st.bitmap, g, gin)
    assert torch.equal(bits_of(gin), bits_of(torch.where(bits_of(x) != 0, g, torch.zeros((), device=DEV))))
    del x, st, back, g, gin
    torch.cuda.empty_cache()


@pytest.mark.parametrize("kind", ["bf16", "f16"])
def test_cfg4_vgg16_batch64_fused_relu_pair(oracle, kind):
    shapes = W.vgg16_shapes(64)
    seen = set()
    for i, shape, n in W.iter_layers(shapes):
        if shape in seen and i not in (0, len(shapes) - 1):
            continue                                         # one tensor per distinct shape (plus first and last)
        seen.add(shape)
        pre = W.cfg4_preact(i, shape, kind, DEV).reshape(-1)
        g = W.cfg4_grad(i, shape, kind, DEV).reshape(-1)
        y_ref = (torch.relu(pre) + 0.0).to(pre.dtype)        # +0.0: torch.relu keeps the sign of -0.0
        ws = B.new_workspace(n, DEV)
        # stash only
        st = GStash(n, pre.dtype, DEV)
        B.bt_relu_fwd_compress(pre, None, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
        check_against_torch(st, y_ref)
        check_sampled_chunks(oracle, st, y_ref, None, seed=40 + i, samples=12)
        # with the dense output
        st2 = GStash(n, pre.dtype, DEV)
        y = torch.empty_like(pre)
        B.bt_relu_fwd_compress(pre, y, st2.bitmap, st2.values, st2.chunk_prefix, st2.nnz_out, ws, st2.dev_status)
        assert torch.equal(bits_of(y), bits_of(y_ref))
        assert torch.equal(st2.bitmap, st.bitmap) and st2.nnz == st.nnz
        assert torch.equal(bits_of(st2.values[:st.nnz]), bits_of(st.values[:st.nnz]))
        # backward from the bitmap
        gin = torch.empty_like(g)
        B.bt_relu_bwd_from_bitmap(st.bitmap, g, gin)
        assert torch.equal(bits_of(gin), bits_of(torch.where(pre > 0, g, torch.zeros((), device=DEV, dtype=g.dtype))))
        del pre, g, y, y_ref, st, st2, gin
        torch.cuda.empty_cache()


def test_cfg5_mobilenetv2_batch128_forward_then_reverse(oracle):
    shapes = W.mobilenetv2_shapes(128)
    fractions = W.cfg5_zero_fractions(len(shapes))
    assert len(shapes) == 35 and sum(W.numel(s) for s in shapes) == 781541376
    n_max = max(W.numel(s) for s in shapes)
    ws = B.new_workspace(n_max, DEV)
    stashes, nnzs, total_bytes = [], [], 0
    for i, shape, n in W.iter_layers(shapes):                 # forward order, one stream
        x = W.cfg5_layer(i, shape, fractions[i], DEV).reshape(-1)
        st = GStash(n, x.dtype, DEV, values_capacity=n)
        B.bt_compress(x, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
        nnz = int((bits_of(x) != 0).sum().item())
        assert st.nnz == nnz and st.status == B.BT_OK and st.intact()
        assert abs((1 - nnz / n) - fractions[i]) < 0.02
        if i % 6 == 0:
            check_sampled_chunks(oracle, st, x, None, seed=70 + i, samples=8)
        # keep the exact-size stash, as a training step would (values trimmed to nnz)
        st.values = st.values[:nnz].clone()
        stashes.append((i, shape, n, st))
        nnzs.append(nnz)
        total_bytes += B.bt_compressed_bytes(n, nnz, torch.float32)
        del x
    dense_bytes = 4 * sum(n for _, _, n, _ in stashes)
    assert total_bytes == sum(n // 8 + 4 * z + 8 * (n // 4096) for (_, _, n, _), z in zip(stashes, nnzs))
    assert 0.15 * dense_bytes < total_bytes < 0.36 * dense_bytes      # 70-85 % zeros: about 18-33 % of dense
    for i, shape, n, st in reversed(stashes):                # restore in reverse order
        back = torch.empty(n, dtype=torch.float32, device=DEV)
        B.bt_decompress(st.bitmap, st.values, st.chunk_prefix, back)
        x = W.cfg5_layer(i, shape, fractions[i], DEV).reshape(-1)
        assert torch.equal(bits_of(back), bits_of(x))
        del back, x


def test_more_than_two_to_the_32_elements(oracle):
    """Element indices, bitmap word indices and packed offsets beyond 32 bits: a bf16 tensor of 2^32 + 70001
    elements (8.6 GB dense, ragged against words, chunks and tiles).  Checked in slices with torch, on sampled
    chunks with the oracle (the last chunks lie beyond element 2^32), and through every kernel of the path."""
    n = (1 << 32) + 70001
    free, _ = torch.cuda.mem_get_info()
    if free < 60 << 30:
        pytest.skip("needs about 45 GB of free device memory")
    step = 1 << 28
    pre = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    for k, lo in enumerate(range(0, n, step)):                # seeded, slice by slice
        m = min(step, n - lo)
        pre[lo:lo + m] = torch.randn(m, generator=torch.Generator(device=DEV).manual_seed(9000 + k), device=DEV,
                                     dtype=torch.float32).to(torch.bfloat16)
    st = GStash(n, pre.dtype, DEV)
    ws = B.new_workspace(n, DEV)
    y = torch.empty_like(pre)
    B.bt_relu_fwd_compress(pre, y, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
    torch.cuda.synchronize()
    assert st.status == B.BT_OK and st.intact()
    nnz = st.nnz
    # whole tensor, slice by slice: the dense output, the bitmap, the prefix array and the packed values
    total = 0
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        y_ref = torch.clamp_min(pre[lo:hi].float(), 0.0).to(torch.bfloat16)
        y_ref = torch.where(y_ref == 0, torch.zeros_like(y_ref), y_ref)                 # +0 for -0.0
        assert torch.equal(bits_of(y[lo:hi]), bits_of(y_ref))
        mask = bits_of(y_ref) != 0
        assert torch.equal(st.bitmap[lo // 32:(hi + 31) // 32], torch_bitmap(mask))       # slices start on word boundaries
        c0, c1 = lo // 4096, (hi + 4095) // 4096
        assert torch.equal(st.chunk_prefix[c0:c1], torch_prefix(mask) + total)
        cnt = int(mask.sum().item())
        assert torch.equal(bits_of(st.values[total:total + cnt]), bits_of(y_ref)[mask])
        total += cnt
        del y_ref, mask
    assert total == nnz and nnz > (1 << 31)                  # packed offsets pass 2^31 as well
    check_sampled_chunks(oracle, st, y, None, seed=5, samples=16)
    chunks = (n + 4095) // 4096
    for c in (chunks - 1, chunks - 2, (1 << 32) // 4096, (1 << 32) // 4096 - 1):          # around element 2^32 and the ragged end
        lo, hi = c * 4096, min(n, (c + 1) * 4096)
        ref = oracle.compress(W.raw_numpy(y[lo:hi]))
        start = int(st.chunk_prefix[c].item())
        assert np.array_equal(W.raw_numpy(st.bitmap[lo // 32:(hi + 31) // 32]).view(np.uint32), ref.bitmap)
        assert np.array_equal(W.raw_numpy(st.values[start:start + ref.nnz]), ref.values)
    # the plain compressor on y gives the same stash
    st2 = GStash(n, pre.dtype, DEV)
    B.bt_compress(y, st2.bitmap, st2.values, st2.chunk_prefix, st2.nnz_out, ws, st2.dev_status)
    assert st2.status == B.BT_OK and st2.nnz == nnz
    assert torch.equal(st2.bitmap, st.bitmap) and torch.equal(st2.chunk_prefix, st.chunk_prefix)
    assert torch.equal(bits_of(st2.values[:nnz]), bits_of(st.values[:nnz]))
    del st2
    # restore, masked gradient (in place), masked gather
    back = torch.empty_like(y)
    B.bt_decompress(st.bitmap, st.values, st.chunk_prefix, back)
    assert torch.equal(bits_of(back), bits_of(y))
    B.bt_relu_bwd_from_bitmap(st.bitmap, pre, back)           # the pre-activation doubles as the gradient
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        assert torch.equal(bits_of(back[lo:hi]), bits_of(torch.where(bits_of(y[lo:hi]) != 0, pre[lo:hi],
                                                                     torch.zeros((), device=DEV, dtype=pre.dtype))))
    vals = torch.empty(nnz, dtype=pre.dtype, device=DEV)
    B.bt_mask_compress(pre, st.bitmap, st.chunk_prefix, None, vals)
    torch.cuda.synchronize()
    assert torch.equal(bits_of(vals), bits_of(st.values[:nnz]))   # where a bit is set, pre == y
    del pre, y, back, vals, st, ws
    torch.cuda.empty_cache()


def test_the_benchmarks_own_step_against_the_oracle(oracle):
    """The benchmark's batch object in the configuration it is timed in (one stream, four launches per tensor, no
    graph, no CTA limit): after two steps over a batch of two tensors, the batch's own check, and both stashes of
    the last tensor, the restored tensor and the masked gradient whole against the oracle."""
    import bench
    batch = bench.Batch(torch.device(DEV), 2)
    assert batch.count == 2 and batch.n == 1 << 28
    batch.step()
    batch.step()
    nnz = batch.check()
    x, pre = batch.x[-1], batch.pre[-1]
    c = oracle.compress(W.raw_numpy(x))
    y_ref, cr = oracle.relu_fwd_compress(W.raw_numpy(pre), "f32")
    assert np.array_equal(y_ref, W.raw_numpy(x))                        # the pre-activation's ReLU is the activation
    for st, ref in ((batch.sa, c), (batch.sb, cr)):
        assert st.status == B.BT_OK and st.nnz == ref.nnz == nnz
        assert np.array_equal(W.raw_numpy(st.bitmap).view(np.uint32), ref.bitmap)
        assert np.array_equal(W.raw_numpy(st.chunk_prefix).view(np.uint64), ref.prefix)
        assert np.array_equal(W.raw_numpy(st.values[:ref.nnz]), ref.values)
    # the step's last launch left the masked gradient in the output buffer; the restore is repeated here
    assert np.array_equal(W.raw_numpy(batch.out), oracle.relu_bwd_from_bitmap(cr.bitmap, W.raw_numpy(batch.g)))
    B.bt_decompress(batch.sa.bitmap, batch.sa.values, batch.sa.chunk_prefix, batch.out)
    assert np.array_equal(W.raw_numpy(batch.out), oracle.decompress(c))
    assert B.bt_set_max_ctas(0) == 0                                    # the benchmark sets no CTA limit


@pytest.mark.parametrize("kind,op", [("f32", "compress"), ("bf16", "relu"), ("bf16", "relu_y"), ("f16", "decompress"), ("f32", "relu_bwd"),
                                     ("f32", "prune"), ("f32", "narrow"), ("f32", "widen"), ("bf16", "relu6_bwd"), ("f32", "mask_y"),
                                     ("bf16", "maxpool_bwd"), ("f64", "compress"), ("f32", "batch_restore")])
def test_the_profiling_cases_of_the_benchmark_run(kind, op):
    """`python bench.py --case <dtype> <op>` is the command every summary under profiles/ names: each case runs to
    the end and reports BT_OK (here on 2^20 elements)."""
    import bench
    args = bench.parse_args(["--case", kind, op, "--log2n", "20", "--reps", "2"])
    assert bench.run_case(args) == 0
