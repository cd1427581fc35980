"""GPU: saved activations go through daf_compress / daf_decompress between forward and backward
(the end-to-end flow of Sec. 3.1 / Fig. 3(a)).  What the backward pass reads is checked against
the CPU oracle; a small CNN is trained with and without compression."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _ctx(**kw):
    from paper_2507_07149_b200.autograd import saved_activation_compression
    return saved_activation_compression(**kw)


@pytest.mark.parametrize("dtype,name", [(torch.float32, "f32"), (torch.float16, "f16")])
def test_backward_reads_what_the_oracle_decodes(dtype, name):
    """d/dx sum(x^2) = 2 * (the saved x): with the hooks on, the saved x is the decoded one."""
    daf.lib()
    rng = np.random.default_rng(11)
    n, G, beta, seed = 5 * 16384 + 4096, 256, 4.0, 77
    a = (rng.laplace(size=n) * np.repeat(rng.choice([0.5, 1.0, 6.0], n // G), G)).astype(np.float32)
    a = a.astype(np.float16) if name == "f16" else a
    x = torch.from_numpy(a).cuda().requires_grad_(True)
    ctx = _ctx(group_size=G, widths=(1, 2, 4, 8), bit_budget=beta, seed=seed, min_numel=1024)
    with ctx:
        y = x.pow(2).sum()
    y.backward()
    assert ctx.stats["tensors"] == 1 and ctx.stats["bytes_in"] == a.nbytes
    ref = oracle.compress(a, G, (1, 2, 4, 8), beta, dtype=name, seed=seed)
    assert len(np.unique(ref.bits)) >= 2
    dec = oracle.decompress(ref)
    got = x.grad.cpu().numpy()
    if name == "f16":
        want = (torch.from_numpy(dec) * 2).numpy()            # doubling is exact in fp16 (no overflow here)
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    else:
        want = dec.astype(np.float32) * np.float32(2)
        ulp = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert ulp.max() <= 1
    ctx.check_status()
    # stored form: the packed capacity the budget guarantees + 9 bytes per group + the window offsets, each part
    # padded to 16 bytes; no value was read back from the device to size it
    n_win, up16 = -(-n // 16384), lambda v: (v + 15) & ~15
    cap = daf.daf_sizes(daf.make_params(daf.dtype_code(x), n, G, (1, 2, 4, 8), beta)).packed_capacity
    assert int(ref.window_offsets[-1]) <= cap == n * 4 // 8
    assert ctx.stats["bytes_kept"] == up16(cap) + 2 * up16(4 * (n // G)) + up16(n // G) + up16(8 * (n_win + 1))
    assert ctx.stats["launches"] == 1


def test_two_saved_tensors_draw_from_disjoint_counters():
    daf.lib()
    rng = np.random.default_rng(5)
    n, G = 32768, 256
    a = rng.standard_normal(n).astype(np.float32)
    b = rng.standard_normal(n).astype(np.float32)
    xa = torch.from_numpy(a).cuda().requires_grad_(True)
    xb = torch.from_numpy(b).cuda().requires_grad_(True)
    ctx = _ctx(group_size=G, bit_budget=2.0, seed=3, min_numel=1024)
    with ctx:
        y = xa.pow(2).sum() + xb.pow(2).sum()
    y.backward()
    for arr, grad, base in ((a, xa.grad, 0), (b, xb.grad, n)):
        ref = oracle.compress(arr, G, (1, 2, 4, 8), 2.0, dtype="f32", seed=3, base=base)
        want = oracle.decompress(ref).astype(np.float32) * np.float32(2)
        got = grad.cpu().numpy()
        ulp = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert ulp.max() <= 1


def test_ineligible_tensors_pass_through():
    daf.lib()
    w = torch.nn.Parameter(torch.randn(1 << 16, device="cuda"))
    small = torch.randn(512, device="cuda", requires_grad=True)
    ragged = torch.randn((1 << 16) + 8, device="cuda", requires_grad=True)
    ctx = _ctx(min_numel=1024)
    with ctx:
        y = w.pow(2).sum() + small.pow(2).sum() + ragged.pow(2).sum()
    y.backward()
    assert ctx.stats["tensors"] == 0 and ctx.stats["passed_through"] >= 3
    assert torch.equal(w.grad, 2 * w.detach()) and torch.equal(small.grad, 2 * small.detach())


def _train(ctx_factory, steps=100, relu=torch.nn.ReLU):
    import contextlib
    torch.manual_seed(0)
    net = torch.nn.Sequential(
        torch.nn.Conv2d(3, 16, 3, padding=1), relu(),
        torch.nn.Conv2d(16, 32, 3, padding=1), relu(),
        torch.nn.AdaptiveAvgPool2d(4), torch.nn.Flatten(), torch.nn.Linear(512, 10)).cuda()
    opt = torch.optim.SGD(net.parameters(), lr=0.05, momentum=0.9)
    g = torch.Generator(device="cuda").manual_seed(1)
    proto = torch.randn(10, 3, 32, 32, device="cuda", generator=g)
    losses, ctx = [], None
    for step in range(steps):
        labels = torch.randint(0, 10, (32,), device="cuda", generator=g)
        xb = proto[labels] + 0.5 * torch.randn(32, 3, 32, 32, device="cuda", generator=g)
        ctx = ctx_factory(step) if ctx_factory else contextlib.nullcontext()
        with ctx:
            loss = torch.nn.functional.cross_entropy(net(xb), labels)
        opt.zero_grad()
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    return losses, ctx


def test_small_cnn_trains_on_compressed_activations():
    daf.lib()
    base, _ = _train(None)
    comp, ctx = _train(lambda step: _ctx(group_size=256, bit_budget=4.0, seed=step))
    assert ctx.stats["tensors"] >= 3                           # conv inputs / relu outputs of 2^19 and 2^20 elements
    assert ctx.stats["bytes_kept"] < 0.2 * ctx.stats["bytes_in"]   # about 4.3 of 32 bits per element
    assert np.mean(base[-5:]) < 0.3 * base[0]
    assert np.mean(comp[-5:]) < 0.3 * comp[0]                  # trains as well, within noise
    assert abs(np.mean(comp[-5:]) - np.mean(base[-5:])) < 0.25 * base[0]


def test_compressed_relu_layer_masks_with_the_restored_output():
    """CompressedReLU: forward = relu(x) exactly; backward = grad * (restored output > 0), the restored
    output being what the oracle decodes from the compression of relu(x)."""
    from paper_2507_07149_b200.autograd import CompressedReLU
    daf.lib()
    rng = np.random.default_rng(23)
    n, G, beta, seed = 16384 * 9 + 512, 256, 2.0, 41
    a = rng.standard_normal(n).astype(np.float32)
    gw = rng.standard_normal(n).astype(np.float32)
    x = torch.from_numpy(a).cuda().requires_grad_(True)
    layer = CompressedReLU(group_size=G, bit_budget=beta, seed=seed, min_numel=1024)
    y = layer(x)
    assert np.array_equal(y.detach().cpu().numpy().view(np.uint32), oracle.relu(a).view(np.uint32))
    (y * torch.from_numpy(gw).cuda()).sum().backward()
    ref = oracle.compress(oracle.relu(a), G, (1, 2, 4, 8), beta, seed=seed)
    restored = oracle.decompress(ref)
    want = gw * (restored > 0)
    assert np.array_equal(x.grad.cpu().numpy(), want.astype(np.float32))
    assert 0 < int((restored > 0).sum()) < int((a > 0).sum())     # at 2 bits some small positives are restored as 0
    # a small or ragged input takes the plain path
    small = torch.randn(100, device="cuda", requires_grad=True)
    layer(small).sum().backward()
    assert torch.equal(small.grad, (small.detach() > 0).float())


def test_small_cnn_trains_with_compressed_relu_layers():
    """The same network with its ReLUs replaced by CompressedReLU (fused producer forward, fused consumer backward)."""
    from paper_2507_07149_b200.autograd import CompressedReLU
    daf.lib()
    base, _ = _train(None)
    comp, _ = _train(None, relu=lambda: CompressedReLU(group_size=256, bit_budget=4.0, seed=7))
    assert np.mean(base[-5:]) < 0.3 * base[0]
    assert np.mean(comp[-5:]) < 0.3 * comp[0]
    assert abs(np.mean(comp[-5:]) - np.mean(base[-5:])) < 0.25 * base[0]


def test_saved_tensors_are_compressed_in_batches_and_offset_views_are_copied():
    """Seven saved tensors, queue of four: two launches.  Two of them are views that start 4 bytes into their storage
    (not on the 32-byte boundary the kernels need): they are copied, not rejected and not read misaligned.  Every
    gradient is what the oracle decodes, each tensor at its own counter base."""
    daf.lib()
    rng = np.random.default_rng(8)
    G, beta, seed = 128, 4.0, 19
    sizes = [16384 * 3, 16384 + 2048, 4096, 16384 * 2, 8192, 16384 * 5 + 128, 2048]
    arrays = [rng.standard_normal(n).astype(np.float32) * (1 + i) for i, n in enumerate(sizes)]
    leaves = []
    for i, a in enumerate(arrays):
        if i in (1, 4):
            store = torch.zeros(a.size + 1, device="cuda")
            store[1:] = torch.from_numpy(a).cuda()
            leaf = store[1:].detach().requires_grad_(True)
            assert leaf.data_ptr() % 32 == 4
        else:
            leaf = torch.from_numpy(a).cuda().requires_grad_(True)
        leaves.append(leaf)
    ctx = _ctx(group_size=G, bit_budget=beta, seed=seed, min_numel=1024, batch=4)
    with ctx:
        y = sum(v.pow(2).sum() for v in leaves)
    assert ctx.stats["launches"] == 2 and ctx.stats["tensors"] == 7
    y.backward()
    ctx.check_status()
    base = 0
    for a, leaf in zip(arrays, leaves):
        ref = oracle.compress(a, G, (1, 2, 4, 8), beta, dtype="f32", seed=seed, base=base)
        want = oracle.decompress(ref).astype(np.float32) * np.float32(2)
        got = leaf.grad.cpu().numpy()
        ulp = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert ulp.max() <= 1
        base += (a.size + 7) & ~7


def test_exclusion_predicate_and_views_of_parameters():
    daf.lib()
    w = torch.nn.Parameter(torch.randn(256, 256, device="cuda"))
    x = torch.randn(1 << 16, device="cuda", requires_grad=True)
    z = torch.randn(1 << 15, device="cuda", requires_grad=True)
    ctx = _ctx(min_numel=1024, exclude=lambda t: t.numel() == 1 << 15)
    with ctx:
        y = x.pow(2).sum() + z.pow(2).sum() + w.t().pow(2).sum()      # w.t() is a view of a parameter
    y.backward()
    assert ctx.stats["tensors"] == 1 and ctx.stats["passed_through"] >= 2
    assert torch.equal(z.grad, 2 * z.detach()) and torch.equal(w.grad, 2 * w.detach())
    assert not torch.equal(x.grad, 2 * x.detach())


def test_store_chooses_widths_under_the_memory_budget_and_drops_what_does_not_fit():
    """Three activations of 2^20 elements with importances 16, 2, 1 and a budget that holds one at 8 bits, one at 2 bits
    and nothing more: what the backward pass reads is the oracle's decoding at those widths, and zeros for the
    one that was dropped."""
    daf.lib()
    n, G, seed = 1 << 20, 256, 5
    rng = np.random.default_rng(21)
    arrays = [rng.standard_normal(n).astype(np.float32) for _ in range(3)]
    leaves = [torch.from_numpy(a).cuda().requires_grad_(True) for a in arrays]
    page = 65536
    pages = lambda b: -(-daf.store_bytes(n, G, b) // page)
    budget = (pages(8) + pages(2)) * page
    imp = {0: 16.0, 1: 2.0, 2: 1.0}
    ctx = _ctx(group_size=G, bit_budget=8.0, seed=seed, min_numel=1024, mem_budget=budget, importance=lambda i, t: imp[i],
               step_bytes=1 << 20)
    with ctx:
        y = sum(v.pow(2).sum() for v in leaves)
    widths = [ctx._store.width(ctx._base + i)[0] for i in range(3)]
    # tensor 0 alone: 8 bits.  Tensor 1 arrives: over budget; it is the less valuable per byte and goes 8 -> 4 -> 2.
    # Tensor 2 arrives at 8 bits, is the least valuable and shrinks to 1 bit, where it is worth 1 / 3 pages against
    # 2 / 5 pages for tensor 1 and 16 / 17 for tensor 0; still over budget, it is dropped.
    assert widths == [8, 2, 0]
    assert ctx.stats["dropped"] == 1 and ctx._store.stats()["used_bytes"] <= budget
    y.backward()
    ctx.check_status()
    base = 0
    for a, leaf, b in zip(arrays, leaves, widths):
        got = leaf.grad.cpu().numpy()
        if b == 0:
            assert not got.any()
        else:
            ref = oracle.compress(a, G, (1, 2, 4, 8), float(b), dtype="f32", seed=seed, base=base)
            want = oracle.decompress(ref).astype(np.float32) * np.float32(2)
            ulp = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
            assert ulp.max() <= 1
            base += n
    del y, leaves
    assert ctx._store.stats()["used_bytes"] == 0                      # every handle gave its pages back


def test_lowering_the_budget_moves_packed_activations_without_changing_them():
    daf.lib()
    n, G, seed = 1 << 20, 256, 9
    rng = np.random.default_rng(22)
    arrays = [rng.standard_normal(n).astype(np.float32) for _ in range(4)]
    leaves = [torch.from_numpy(a).cuda().requires_grad_(True) for a in arrays]
    one = -(-daf.store_bytes(n, G, 4) // 65536) * 65536
    step = 2 * one
    ctx = _ctx(group_size=G, bit_budget=4.0, seed=seed, min_numel=1024, mem_budget=2 * step, step_bytes=step, batch=1,
               importance=lambda i, t: float(1 + i))
    with ctx:
        parts = [v.pow(2).sum() for v in leaves]
    assert ctx._store.stats()["arena_bytes"] == 2 * step
    # the first two are consumed; the budget then halves: tensors 2 and 3 lie in the second step and move down
    (parts[0] + parts[1]).backward()
    del parts[0:2]
    ctx.set_budget(step)
    st = ctx._store.stats()
    assert st["arena_bytes"] == step and st["moves"] == 2 and st["evictions"] == 0
    (parts[0] + parts[1]).backward()
    base = 0
    for a, leaf in zip(arrays, leaves):
        ref = oracle.compress(a, G, (1, 2, 4, 8), 4.0, dtype="f32", seed=seed, base=base)
        want = oracle.decompress(ref).astype(np.float32) * np.float32(2)
        got = leaf.grad.cpu().numpy()
        ulp = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert ulp.max() <= 1
        base += n


def test_compressed_relu_accepts_offset_views_and_misaligned_gradients():
    from paper_2507_07149_b200.autograd import CompressedReLU
    daf.lib()
    rng = np.random.default_rng(29)
    n, G, beta, seed = 16384 * 3, 256, 4.0, 2
    a = rng.standard_normal(n).astype(np.float32)
    gw = rng.standard_normal(n).astype(np.float32)
    store = torch.zeros(n + 1, device="cuda")
    store[1:] = torch.from_numpy(a).cuda()
    x = store[1:].detach().requires_grad_(True)
    assert x.data_ptr() % 32 == 4
    layer = CompressedReLU(group_size=G, bit_budget=beta, seed=seed, min_numel=1024)
    y = layer(x)
    assert np.array_equal(y.detach().cpu().numpy().view(np.uint32), oracle.relu(a).view(np.uint32))
    gstore = torch.zeros(n + 1, device="cuda")
    gstore[1:] = torch.from_numpy(gw).cuda()
    y.backward(gstore[1:])                                           # a gradient that starts 4 bytes off the boundary
    restored = oracle.decompress(oracle.compress(oracle.relu(a), G, (1, 2, 4, 8), beta, seed=seed))
    assert np.array_equal(x.grad.cpu().numpy(), (gw * (restored > 0)).astype(np.float32))


def _resnet18(num_classes=10):
    """ResNet-18 (basic blocks 2-2-2-2, widths 64-128-256-512) with a 3x3 stem for small images."""
    nn = torch.nn

    class Block(nn.Module):
        def __init__(self, cin, cout, stride):
            super().__init__()
            self.c1 = nn.Conv2d(cin, cout, 3, stride, 1, bias=False)
            self.b1 = nn.BatchNorm2d(cout)
            self.c2 = nn.Conv2d(cout, cout, 3, 1, 1, bias=False)
            self.b2 = nn.BatchNorm2d(cout)
            self.down = None
            if stride != 1 or cin != cout:
                self.down = nn.Sequential(nn.Conv2d(cin, cout, 1, stride, bias=False), nn.BatchNorm2d(cout))

        def forward(self, x):
            y = torch.relu(self.b1(self.c1(x)))
            y = self.b2(self.c2(y))
            return torch.relu(y + (x if self.down is None else self.down(x)))

    layers, cin = [nn.Conv2d(3, 64, 3, 1, 1, bias=False), nn.BatchNorm2d(64), nn.ReLU()], 64
    for cout, stride in ((64, 1), (128, 2), (256, 2), (512, 2)):
        layers += [Block(cin, cout, stride), Block(cout, cout, 1)]
        cin = cout
    layers += [nn.AdaptiveAvgPool2d(1), nn.Flatten(), nn.Linear(512, num_classes)]
    return nn.Sequential(*layers)


def test_resnet18_trains_on_compressed_activations():
    """Twenty SGD steps of ResNet-18 on synthetic 32x32 images (batch 64), once as usual and once with every saved
    activation held compressed at 4 bits: the loss curves stay together, a fifth of the activation bytes is kept,
    one launch serves up to 16 saved tensors and no step waits for the device in its forward pass (step time on this
    launch-bound toy size: 4.2 ms plain, 6.9 ms with the hooks)."""
    import contextlib
    import time
    daf.lib()

    def run(make_ctx, steps=20):
        torch.manual_seed(0)
        net = _resnet18().cuda()
        opt = torch.optim.SGD(net.parameters(), lr=0.05, momentum=0.9)
        g = torch.Generator(device="cuda").manual_seed(1)
        proto = torch.randn(10, 3, 32, 32, device="cuda", generator=g)
        ctx = make_ctx()
        losses = []
        for step in range(steps):
            if step == 5:                                             # the first steps pay for algorithm selection
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            labels = torch.randint(0, 10, (64,), device="cuda", generator=g)
            xb = proto[labels] + 0.5 * torch.randn(64, 3, 32, 32, device="cuda", generator=g)
            if hasattr(ctx, "reseed"):
                ctx.reseed(step)
            with ctx:
                loss = torch.nn.functional.cross_entropy(net(xb), labels)
            opt.zero_grad()
            loss.backward()
            opt.step()
            losses.append(loss.detach())
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / (steps - 5)
        return [float(v) for v in losses], ctx, dt

    base, _, t_base = run(contextlib.nullcontext)
    comp, ctx, t_comp = run(lambda: _ctx(group_size=256, bit_budget=4.0, min_numel=16384))
    ctx.check_status()
    s = ctx.stats
    assert s["tensors"] >= 20 * 20                                    # some forty saved activations per step
    assert s["launches"] * 5 <= s["tensors"]                           # batched: far fewer launches than tensors
    assert s["bytes_kept"] < 0.16 * s["bytes_in"]                      # 4.3 of 32 bits
    assert np.mean(base[-5:]) < 0.5 * base[0] and np.mean(comp[-5:]) < 0.5 * comp[0]
    assert abs(np.mean(comp[-5:]) - np.mean(base[-5:])) < 0.25 * base[0]
    print(f"resnet18 b64: {t_base * 1e3:.1f} ms/step plain, {t_comp * 1e3:.1f} ms/step compressed; "
          f"kept {s['bytes_kept'] / s['bytes_in']:.3f} of the saved bytes in {s['launches'] / 20:.1f} launches/step "
          f"for {s['tensors'] / 20:.0f} tensors/step")


def test_resnet18_under_a_memory_budget_that_binds():
    """The same model with a store whose budget holds about a third of the 8-bit forms: widths go down, some
    activations are dropped, training still makes progress, and the arena is never overrun."""
    daf.lib()
    torch.manual_seed(0)
    net = _resnet18().cuda()
    opt = torch.optim.SGD(net.parameters(), lr=0.05, momentum=0.9)
    g = torch.Generator(device="cuda").manual_seed(1)
    proto = torch.randn(10, 3, 32, 32, device="cuda", generator=g)
    budget = 24 << 20
    ctx = _ctx(group_size=256, bit_budget=8.0, min_numel=16384, mem_budget=budget, step_bytes=8 << 20,
               importance=lambda i, t: 1.0 + (i % 5))
    losses = []
    for step in range(12):
        labels = torch.randint(0, 10, (64,), device="cuda", generator=g)
        xb = proto[labels] + 0.5 * torch.randn(64, 3, 32, 32, device="cuda", generator=g)
        ctx.reseed(step)
        with ctx:
            loss = torch.nn.functional.cross_entropy(net(xb), labels)
        st = ctx._store.stats()
        assert st["used_bytes"] <= budget and st["arena_bytes"] <= budget
        opt.zero_grad()
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    ctx.check_status()
    st = ctx._store.stats()
    assert st["resizes"] > 0 and st["used_bytes"] == 0
    assert all(np.isfinite(losses)) and np.mean(losses[-3:]) < losses[0]


def test_compressed_gelu_and_relu6_layers_follow_torch_within_the_quantization_step():
    """The layers against torch's own: forward equal (ReLU6) or within float rounding (GELU); backward equal to torch's
    derivative taken at the restored tensor, which differs from the true one by at most a quantization step."""
    from paper_2507_07149_b200.autograd import CompressedGELU, CompressedReLU6
    daf.lib()
    n, G = 16384 * 6, 256
    xs = torch.randn(n, device="cuda") * 3
    gw = torch.randn(n, device="cuda")
    for layer, plain in ((CompressedReLU6(group_size=G, bit_budget=8.0, min_numel=1024), torch.nn.functional.relu6),
                         (CompressedGELU(group_size=G, bit_budget=8.0, min_numel=1024), torch.nn.functional.gelu)):
        x = xs.clone().requires_grad_(True)
        y = layer(x)
        (y * gw).sum().backward()
        x2 = xs.clone().requires_grad_(True)
        y2 = plain(x2)
        (y2 * gw).sum().backward()
        assert torch.allclose(y, y2, rtol=1e-5, atol=1e-6)
        # at 8 bits a group of 256 normal values spans about 17 units: step 0.07; GELU' has slope <= 1.13
        bad = (x.grad - x2.grad).abs() > 0.1 * gw.abs() + 1e-6
        if isinstance(layer, CompressedReLU6):
            near = (xs.abs() < 0.08) | ((xs - 6).abs() < 0.08)        # the mask may flip only next to the kinks
            assert not (bad & ~near).any()
        else:
            assert not bad.any()
