"""The stash inside PyTorch's autograd: saved activations are compressed between the passes, gradients are
bit-identical to plain PyTorch (the codec is lossless), and the peak memory of a ReLU network drops."""
import pytest
import torch

from paper_2110_15362_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def A():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    B.lib()
    from paper_2110_15362_b200 import autograd
    return autograd


def mlp(width, depth, seed, dtype=torch.float32):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return [(torch.randn(width, width, generator=g, device="cuda", dtype=dtype) / width ** 0.5).requires_grad_()
            for _ in range(depth)]


def run(weights, x, relu, hooks=None):
    h = x
    for w in weights:
        h = relu(h @ w)
    loss = (h * h).sum()
    loss.backward()
    grads = [w.grad.clone() for w in weights]
    for w in weights:
        w.grad = None
    return loss.detach().clone(), grads


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16, torch.float64])
def test_gradients_are_bit_identical(A, dtype):
    weights = mlp(512, 4, seed=1, dtype=dtype)
    x = torch.randn(2048, 512, device="cuda", dtype=dtype, generator=torch.Generator(device="cuda").manual_seed(2))
    ref_loss, ref = run(weights, x, torch.relu)
    with A.stash_saved_activations(min_numel=1024) as hooks:
        loss1, g1 = run(weights, x, torch.relu)
        assert hooks.dense_bytes > 0 and hooks.packed_bytes < 0.7 * hooks.dense_bytes
    with A.stash_saved_activations(min_numel=1024) as hooks:
        loss2, g2 = run(weights, x, lambda t: A.relu_stash(t, hooks))
    loss3, g3 = run(weights, x, A.relu_stash)                       # the fused ReLU alone, no hooks
    for loss, grads in ((loss1, g1), (loss2, g2), (loss3, g3)):
        assert torch.equal(loss, ref_loss)
        for a, b in zip(grads, ref):
            assert torch.equal(a, b)


def test_pack_unpack_round_trip_and_skips(A):
    hooks = A.stash_saved_activations(min_numel=1024)
    t = torch.relu(torch.randn(64, 4096, device="cuda"))
    p = hooks._pack(t)
    assert isinstance(p, A.PackedActivation) and p.nnz == int(torch.count_nonzero(t))
    assert p.values.numel() == p.nnz                                # exact-size storage
    assert torch.equal(hooks._unpack(p).view(torch.int32), t.view(torch.int32))
    assert hooks._pack(t) is p                                      # the same tensor object is packed once
    dense = torch.randn(64, 4096, device="cuda")                   # no zeros: not worth a stash
    assert hooks._pack(dense) is dense
    small = torch.zeros(10, device="cuda")
    assert hooks._pack(small) is small
    param = torch.nn.Parameter(torch.zeros(1 << 16, device="cuda"))
    assert hooks._pack(param) is param
    cpu = torch.zeros(1 << 16)
    assert hooks._pack(cpu) is cpu
    view = torch.zeros(256, 512, device="cuda").t()                # not contiguous
    assert hooks._pack(view) is view
    odd = torch.zeros((1 << 16) + 1, device="cuda")[1:]            # contiguous but not 16-byte aligned
    assert odd.data_ptr() % 16 != 0 and hooks._pack(odd) is odd


def test_conv_network_trains_and_matches(A):
    torch.backends.cudnn.deterministic = True
    g = torch.Generator(device="cuda").manual_seed(3)
    w1 = (torch.randn(32, 3, 3, 3, generator=g, device="cuda") * 0.2).requires_grad_()
    w2 = (torch.randn(64, 32, 3, 3, generator=g, device="cuda") * 0.05).requires_grad_()
    x = torch.randn(16, 3, 64, 64, generator=g, device="cuda")

    def step(relu):
        h = relu(torch.nn.functional.conv2d(x, w1, padding=1))
        h = torch.nn.functional.max_pool2d(h, 2)
        h = relu(torch.nn.functional.conv2d(h, w2, padding=1))
        h.square().mean().backward()
        out = (w1.grad.clone(), w2.grad.clone())
        w1.grad = w2.grad = None
        return out

    ref = step(torch.relu)
    with A.stash_saved_activations(min_numel=1024) as hooks:
        got = step(lambda t: A.relu_stash(t, hooks))
        assert hooks.packed_bytes > 0
    for a, b in zip(got, ref):
        assert torch.equal(a, b)


def test_peak_memory_drops(A):
    width, depth, batch = 1024, 32, 16384                             # 64 MiB per fp32 activation, 2 GiB saved by plain PyTorch
    weights = mlp(width, depth, seed=5)
    x = torch.randn(batch, width, device="cuda", generator=torch.Generator(device="cuda").manual_seed(6))

    def peak(fn):
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        torch.cuda.reset_peak_memory_stats()
        base = torch.cuda.memory_allocated()
        fn()
        torch.cuda.synchronize()
        return torch.cuda.max_memory_allocated() - base

    def plain():
        run(weights, x, torch.relu)

    def stashed():
        with A.stash_saved_activations() as hooks:
            run(weights, x, lambda t: A.relu_stash(t, hooks))

    plain(); stashed()                                                # warm up allocator and cuBLAS workspaces
    p0, p1 = peak(plain), peak(stashed)
    assert p1 < 0.75 * p0, (p0, p1)


@pytest.mark.parametrize("fused", [False, True])
def test_arena_mode_matches_and_reports_overflow(A, fused):
    weights = mlp(512, 4, seed=7)
    x = torch.randn(4096, 512, device="cuda", generator=torch.Generator(device="cuda").manual_seed(8))
    ref_loss, ref = run(weights, x, torch.relu)
    hooks = A.stash_saved_activations(min_numel=1024, arena_bytes=64 << 20)
    for _ in range(2):                                               # the arena is reused pass after pass
        with hooks:
            loss, grads = run(weights, x, (lambda t: A.relu_stash(t, hooks)) if fused else torch.relu)
        assert torch.equal(loss, ref_loss)
        for a, b in zip(grads, ref):
            assert torch.equal(a, b)
        used = int(hooks.cursor.item())
        assert 0 < used < 0.7 * hooks.dense_bytes / 2 + (1 << 20) or used < hooks.dense_bytes
    small = A.stash_saved_activations(min_numel=1024, arena_bytes=1 << 20)        # far too small
    with pytest.raises(RuntimeError, match="arena too small"):
        with small:
            run(weights, x, torch.relu)
    for w in weights:
        w.grad = None


def test_inplace_relu_stash_matches(A):
    weights = mlp(256, 3, seed=9)
    x = torch.randn(1024, 256, device="cuda", generator=torch.Generator(device="cuda").manual_seed(10))
    ref_loss, ref = run(weights, x, torch.relu)
    with A.stash_saved_activations(min_numel=1024) as hooks:
        loss, grads = run(weights, x, lambda t: A.relu_stash(t, hooks, inplace=True))
    assert torch.equal(loss, ref_loss)
    for a, b in zip(grads, ref):
        assert torch.equal(a, b)


def test_vgg_demo_runs_and_losses_agree(A, capsys):
    import json
    from paper_2110_15362_b200 import demo_vgg_step
    assert demo_vgg_step.main(["--batch", "2", "--size", "64", "--arena-gib", "0.25"]) == 0
    out = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert out["plain"]["loss"] == pytest.approx(out["stashed"]["loss"], rel=1e-3)
    assert out["plain"]["loss"] == pytest.approx(out["stashed_arena"]["loss"], rel=1e-3)
    assert out["plain"]["loss"] == pytest.approx(out["stashed_pool_codes"]["loss"], rel=1e-3)
    assert out["plain"]["loss"] == pytest.approx(out["stashed_arena_pool_first"]["loss"], rel=1e-3)
    assert out["stashed_arena_pool_first"]["held_after_forward_mib"] <= out["stashed_arena"]["held_after_forward_mib"]
    assert out["plain"]["loss"] == pytest.approx(out["stashed_arena_bf16_values"]["loss"], rel=1e-3)   # forward not narrowed
    assert out["stashed_arena_bf16_values"]["arena_used_mib"] < 0.6 * out["stashed_arena"]["arena_used_mib"]
    assert 0.3 < out["saved_activation_bytes_over_dense"] < 0.8
    # what the graph holds between the two passes shrinks, most with the pooling layers on winner codes
    assert out["stashed_pool_codes"]["held_after_forward_mib"] < out["stashed"]["held_after_forward_mib"] \
        < out["plain"]["held_after_forward_mib"]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_relu6_stash_gradients_are_bit_identical(A, dtype):
    weights = mlp(512, 4, seed=5, dtype=dtype)
    x = 3 * torch.randn(2048, 512, device="cuda", dtype=dtype, generator=torch.Generator(device="cuda").manual_seed(6))
    relu6 = torch.nn.functional.relu6
    ref_loss, ref = run(weights, x, relu6)
    assert int((relu6(x @ weights[0]) == 6).sum()) > 1000           # the clamp is exercised
    with A.stash_saved_activations(min_numel=1024) as hooks:
        loss1, g1 = run(weights, x, lambda t: A.relu6_stash(t, hooks))
        assert hooks.packed_bytes < 0.7 * hooks.dense_bytes
    loss2, g2 = run(weights, x, A.relu6_stash)                      # without the hooks
    with A.stash_saved_activations(min_numel=1024, arena_bytes=64 << 20) as hooks:
        loss3, g3 = run(weights, x, lambda t: A.relu6_stash(t, hooks))      # inside an arena context: values in the arena
        assert 0 < int(hooks.cursor.item()) < 0.7 * hooks.dense_bytes and hooks.packed_bytes == 0
    for loss, grads in ((loss1, g1), (loss2, g2), (loss3, g3)):
        assert torch.equal(loss, ref_loss)
        for a, b in zip(grads, ref):
            assert torch.equal(a, b)


@pytest.mark.parametrize("narrow", [torch.float16, torch.bfloat16])
def test_narrowed_stash_is_the_rounded_activation(A, narrow):
    """Lossy by design: what the backward pass sees is the activation rounded to the narrow type, so the
    gradients equal those of a plain step whose saved activations are rounded the same way."""
    weights = mlp(512, 3, seed=7)
    x = torch.randn(2048, 512, device="cuda", generator=torch.Generator(device="cuda").manual_seed(8))
    hooks = A.stash_saved_activations(min_numel=1024, narrow=narrow)
    t = torch.relu(torch.randn(64, 4096, device="cuda"))
    p = hooks._pack(t)
    assert p.values.dtype == narrow and p.nnz == int(torch.count_nonzero(t))
    assert torch.equal(hooks._unpack(p), t.to(narrow).float())
    assert p.nbytes() == B.bt_compressed_bytes(t.numel(), p.nnz, narrow)

    class RoundSaved(torch.autograd.graph.saved_tensors_hooks):     # the plain-PyTorch statement of the same thing
        def __init__(self):
            super().__init__(lambda s: s.to(narrow).float() if s.dtype == torch.float32 and s.numel() >= 1024
                             and not (s.requires_grad and s.is_leaf) else s, lambda s: s)

    def relu_by_mask(t):                                            # saves a boolean mask, which no hook rounds
        return torch.where(t > 0, t, torch.zeros((), device=t.device))

    with RoundSaved():
        ref_loss, ref = run(weights, x, relu_by_mask)
    with A.stash_saved_activations(min_numel=1024, narrow=narrow) as hooks:
        loss1, g1 = run(weights, x, lambda t: A.relu_stash(t, hooks))
        assert hooks.packed_bytes < 0.4 * hooks.dense_bytes         # half the zeros gone, the rest at half width
    assert torch.equal(loss1, ref_loss)                             # the forward pass is not narrowed
    for a, b in zip(g1, ref):
        assert torch.equal(a, b)                                    # same rounded activations into the same GEMMs
    _, exact = run(weights, x, torch.relu)
    assert not torch.equal(g1[-1], exact[-1]) and torch.allclose(g1[-1], exact[-1], rtol=0.05, atol=0.5)
    # the same inside an arena: 16-bit values behind the cursor, no host read in the forward pass
    with A.stash_saved_activations(min_numel=1024, narrow=narrow, arena_bytes=32 << 20) as hooks:
        loss2, g2 = run(weights, x, lambda t: A.relu_stash(t, hooks))
        assert 0 < int(hooks.cursor.item()) < 0.4 * hooks.dense_bytes
    with A.stash_saved_activations(min_numel=1024, narrow=narrow, arena_bytes=32 << 20) as hooks:
        loss3, g3 = run(weights, x, relu_by_mask)                   # the hooks alone (plain narrowing compressor)
    assert torch.equal(loss2, ref_loss) and torch.equal(loss3, ref_loss)
    for a, b, c in zip(g2, g3, ref):
        assert torch.equal(a, c) and torch.equal(b, c)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_double_mask_batch_norm_block(A, dtype):
    """conv-free residual-style block: relu -> batch norm -> double mask -> linear.  Output, gradients and the
    stash (shared bitmap, own values) equal the plain PyTorch statement y = where(h != 0, bn(h), 0)."""
    g = torch.Generator(device="cuda").manual_seed(11)
    x = torch.randn(4096, 256, device="cuda", dtype=dtype, generator=g)
    w1 = (torch.randn(256, 256, device="cuda", dtype=dtype, generator=g) / 16).requires_grad_()
    w2 = (torch.randn(256, 256, device="cuda", dtype=dtype, generator=g) / 16).requires_grad_()
    gamma = torch.rand(256, device="cuda", dtype=dtype, generator=g).add_(0.5).requires_grad_()
    beta = torch.randn(256, device="cuda", dtype=dtype, generator=g).requires_grad_()

    def block(relu, mask):
        h = relu(x @ w1)
        b = torch.nn.functional.batch_norm(h, None, None, gamma, beta, training=True)
        y = mask(b, h)
        loss = ((y @ w2).float() ** 2).mean()
        loss.backward()
        grads = [p.grad.clone() for p in (w1, w2, gamma, beta)]
        for p in (w1, w2, gamma, beta):
            p.grad = None
        return loss.detach().clone(), y.detach().clone(), grads

    ref_loss, ref_y, ref = block(torch.relu, lambda b, h: torch.where(h != 0, b, torch.zeros((), device="cuda", dtype=dtype)))
    with A.stash_saved_activations(min_numel=1024) as hooks:
        loss, y, grads = block(lambda t: A.relu_stash(t, hooks), lambda b, h: A.double_mask(b, h, hooks))
        assert hooks.packed_bytes < 0.7 * hooks.dense_bytes
    loss2, y2, grads2 = block(torch.relu, A.double_mask)             # without hooks: the mask is derived on the spot
    for l, yy, gg in ((loss, y, grads), (loss2, y2, grads2)):
        assert torch.equal(l, ref_loss) and torch.equal(yy, ref_y)
        for a, b in zip(gg, ref):
            assert torch.equal(a, b)
    # the stash of the masked output shares the source's bitmap and holds exactly its count of values
    hooks = A.stash_saved_activations(min_numel=1024)
    h = A.relu_stash(torch.randn(64, 4096, device="cuda", dtype=dtype), hooks)
    b = torch.randn(64, 4096, device="cuda", dtype=dtype)
    m = A.double_mask(b, h, hooks)
    ph, pm = hooks._lookup(h), hooks._lookup(m)
    assert pm.bitmap is ph.bitmap and pm.chunk_prefix is ph.chunk_prefix and pm.values.numel() == ph.nnz
    assert torch.equal(hooks._unpack(pm), torch.where(h != 0, b, torch.zeros((), device="cuda", dtype=dtype)))


def test_views_that_the_library_cannot_take_are_copied(A):
    """A contiguous but misaligned view and a transposed view go through the fused functions via a copy."""
    base = torch.randn((1 << 16) + 1, device="cuda")
    for x in (base[1:], torch.randn(256, 512, device="cuda").t()):
        x = x.detach().requires_grad_()
        ref = torch.relu(x)
        ref.backward(torch.ones_like(ref))
        gref, x.grad = x.grad.clone(), None
        for fn, tref in ((A.relu_stash, ref), (A.relu6_stash, torch.nn.functional.relu6(x.detach()))):
            y = fn(x)
            assert torch.equal(y, tref)
            y.backward(torch.ones_like(y))
            assert torch.equal(x.grad, gref if fn is A.relu_stash else ((x.detach() > 0) & (x.detach() < 6)).float())
            x.grad = None
        m = A.double_mask(x.detach() + 1, x.detach().clamp_min(0))
        assert torch.equal(m, torch.where(x.detach() > 0, x.detach() + 1, torch.zeros((), device="cuda")))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_maxpool_stash_matches_torch(A, dtype):
    x = torch.randn(8, 16, 28, 36, device="cuda", generator=torch.Generator(device="cuda").manual_seed(21)).clamp_min_(0).to(dtype)
    w = (torch.randn(16, 16, 3, 3, device="cuda", generator=torch.Generator(device="cuda").manual_seed(22)) / 12).to(dtype).requires_grad_()

    def run_net(relu, pool, hooks=None):
        xx = x.clone().requires_grad_()
        h = pool(relu(torch.nn.functional.conv2d(xx, w, padding=1)))
        h = pool(relu(torch.nn.functional.conv2d(h, w, padding=1)))
        loss = h.float().square().mean()
        loss.backward()
        out = (loss.detach().clone(), xx.grad.clone(), w.grad.clone())
        w.grad = None
        return out

    torch.backends.cudnn.deterministic = True
    ref = run_net(torch.relu, lambda t: torch.nn.functional.max_pool2d(t, 2))
    got = run_net(torch.relu, A.maxpool2x2_stash)
    with A.stash_saved_activations(min_numel=1024) as hooks:
        got2 = run_net(lambda t: A.relu_stash(t, hooks), A.maxpool2x2_stash)
    with A.stash_saved_activations(min_numel=1024) as hooks:             # bitmap-only ReLU in front of the pooling
        got3 = run_net(lambda t: A.relu_stash(t, hooks, keep_values=False), A.maxpool2x2_stash)
        assert hooks.loose_statuses and hooks._lookup(torch.zeros(1)) is None
    hooks.check_statuses()                                                # also done on entering the next pass
    assert not hooks.loose_statuses
    with A.stash_saved_activations(min_numel=1024, arena_bytes=32 << 20) as hooks:
        got4 = run_net(lambda t: A.relu_stash(t, hooks, keep_values=False), A.maxpool2x2_stash)
        used = int(hooks.cursor.item())
    got5 = run_net(lambda t: A.relu_stash(t, keep_values=False), A.maxpool2x2_stash)
    assert used < 32 << 20
    # the two layers as one call, pooling first (the maximum commutes with the ReLU)
    got6 = run_net(lambda t: t, A.relu_maxpool2x2_stash)
    with A.stash_saved_activations(min_numel=1024) as hooks:
        got7 = run_net(lambda t: t, lambda t: A.relu_maxpool2x2_stash(t, hooks))
        assert hooks.packed_bytes > 0
    with A.stash_saved_activations(min_numel=1024, arena_bytes=32 << 20) as hooks:
        got8 = run_net(lambda t: t, lambda t: A.relu_maxpool2x2_stash(t, hooks))
        assert 0 < int(hooks.cursor.item()) < 32 << 20
    for g in (got, got2, got3, got4, got5, got6, got7, got8):
        for a, b in zip(g, ref):
            assert torch.equal(a, b)
    with pytest.raises(ValueError):
        A.maxpool2x2_stash(torch.zeros(2, 3, 5, 4, device="cuda"))
    # a non-contiguous input is taken through a copy
    xt = torch.randn(4, 6, 8, 10, device="cuda").transpose(0, 1)
    assert torch.equal(A.maxpool2x2_stash(xt), torch.nn.functional.max_pool2d(xt, 2))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16, torch.float64])
def test_relu_and_pooling_commuted_is_bit_identical(A, dtype):
    """relu_maxpool2x2_stash against max_pool2d(relu(x), 2) on inputs full of ties, windows without a positive
    element, exact zeros and NaNs: output and input gradient agree bit for bit (no -0 among the inputs: the
    framework's ReLU keeps that sign, the library's gives +0)."""
    g = torch.Generator(device="cuda").manual_seed(31)
    x = (torch.randint(-3, 4, (6, 5, 30, 44), device="cuda", generator=g).to(torch.float64) / 2).to(dtype)   # many ties
    x[0, 0, :6] = -1.0                                                   # whole windows without a positive element
    x[1, 1, 2:8, 4:12] = 0.0
    pick = torch.rand(x.shape, device="cuda", generator=g) < 0.01
    x[pick] = float("nan")
    x[2, 2, 4, 4] = x[2, 2, 4, 5] = x[2, 2, 5, 4] = float("nan")          # several NaNs in one window
    grad = torch.randn(6, 5, 15, 22, device="cuda", generator=g).to(dtype)
    iv = {torch.float32: torch.int32, torch.bfloat16: torch.int16, torch.float64: torch.int64}[dtype]
    xr = x.clone().requires_grad_()
    ref = torch.nn.functional.max_pool2d(torch.relu(xr), 2)
    ref.backward(grad)
    for hooks in (None, A.stash_saved_activations(min_numel=64), A.stash_saved_activations(min_numel=64, arena_bytes=1 << 20)):
        xs = x.clone().requires_grad_()
        if hooks is None:
            y = A.relu_maxpool2x2_stash(xs)
            y.backward(grad)
        else:
            with hooks:
                y = A.relu_maxpool2x2_stash(xs, hooks)
                packed = hooks._lookup(y)
                assert packed is not None and torch.equal(packed.unpack().view(iv), y.detach().view(iv))
                y.backward(grad)
        assert torch.equal(y.detach().view(iv), ref.detach().view(iv))
        assert torch.equal(xs.grad.view(iv), xr.grad.view(iv))
    with pytest.raises(ValueError):
        A.relu_maxpool2x2_stash(torch.zeros(2, 3, 5, 4, device="cuda"))
