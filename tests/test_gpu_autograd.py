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
    # stored form: packed bytes + 9 bytes per group + the window offsets
    n_win = -(-n // 16384)
    assert ctx.stats["bytes_kept"] == max(int(ref.window_offsets[-1]), 16) + 9 * (n // G) + 8 * (n_win + 1)


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
