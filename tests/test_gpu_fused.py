"""GPU: the fused producer daf_relu_compress (Sec. 3.2.3, kernel fusion) against the oracle --
the activation written out is relu(x) bit for bit, everything else is the compression of it."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

from gpu_util import to_device, to_host

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _input(rng, n, G, dtype, mixed):
    a = rng.standard_normal(n).astype(np.float32)
    if mixed:                                                     # a stretch of groups with very different ranges
        k = n // G
        s = np.ones(k, np.float32)
        s[k // 3: 2 * k // 3] = (10.0 ** rng.uniform(-2, 2, 2 * k // 3 - k // 3)).astype(np.float32)
        a *= np.repeat(s, G)
    a[::7] = -0.0                                                 # negative zeros must come out as +0
    if dtype == "f32":
        return a
    return a.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a)


def _check(a, dtype, G, beta, inplace, seed=3, act_code=daf.ACT_RELU):
    x = to_device(a, dtype)
    x0 = x.clone()
    act, c = daf.relu_compress(x, G, (1, 2, 4, 8), beta, seed=seed, inplace=inplace, check=True, act=act_code)
    y = daf.decompress(c)
    torch.cuda.synchronize()
    want_act = (oracle.relu if act_code == daf.ACT_RELU else oracle.relu6)(a, dtype)
    got_act = to_host(act, dtype)
    assert np.array_equal(got_act.view(np.uint32 if dtype == "f32" else np.uint16),
                          want_act.view(np.uint32 if dtype == "f32" else np.uint16))
    if inplace:
        assert act.data_ptr() == x.data_ptr()
    else:
        assert torch.equal(x.view(torch.int16 if dtype != "f32" else torch.int32),
                           x0.view(torch.int16 if dtype != "f32" else torch.int32))      # the input is left alone
    ref = oracle.compress(want_act, G, (1, 2, 4, 8), beta, dtype="bf16" if dtype == "bf16" else None, seed=seed)
    assert np.array_equal(c.bits.cpu().numpy(), ref.bits)
    assert np.array_equal(c.window_offsets.cpu().numpy().view(np.uint64), ref.window_offsets)
    assert np.array_equal(c.min.cpu().numpy().view(np.uint32), ref.mn.view(np.uint32))
    assert np.array_equal(c.scale.cpu().numpy().view(np.uint32), ref.scale.view(np.uint32))
    assert np.array_equal(c.packed[: ref.packed.size].cpu().numpy(), ref.packed)
    want = oracle.decompress(ref)
    got = to_host(y.reshape(-1), dtype)
    if dtype == "f32":
        d = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert d.max() <= 1
    else:
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    return ref


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G,beta,mixed", [(256, 4.0, False), (256, 3.0, False), (256, 4.0, True), (64, 2.0, True), (1024, 8.0, False)])
def test_relu_compress_matches_relu_then_compress(dtype, G, beta, mixed):
    rng = np.random.default_rng(G + int(beta * 10) + mixed)
    n = 16384 * 37 + G * 5                                        # several windows per CTA wave is not needed: ragged end
    ref = _check(_input(rng, n, G, dtype, mixed), dtype, G, beta, inplace=False)
    if mixed or beta == 3.0:
        assert len(np.unique(ref.bits)) >= 2


@pytest.mark.parametrize("mixed", [False, True])
def test_relu_compress_in_place(mixed):
    rng = np.random.default_rng(17 + mixed)
    n = 16384 * 700 + 256 * 9                                     # more windows than CTAs: every CTA stages several windows
    _check(_input(rng, n, 256, "f32", mixed), "f32", 256, 4.0, inplace=True)


def test_relu_compress_rejects_other_windows():
    x = torch.zeros(1 << 16, device="cuda")
    p = daf.make_params(daf.F32, x.numel(), 256, (1, 2, 4, 8), 4.0, window_elems=4096)
    c = daf.alloc_outputs(p, "cuda")
    with pytest.raises(daf.DafError) as e:
        daf.daf_relu_compress(p, x, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                              c.workspace, c.sizes.workspace)
    assert e.value.status == daf.ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G,beta,mixed,We", [(256, 2.0, False, 16384), (128, 3.0, True, 16384), (64, 1.0, True, 4096)])
def test_relu_grad_from_the_packed_output(dtype, G, beta, mixed, We):
    """daf_decompress_relu_grad = grad where the restored activation (in its own type) is > 0."""
    rng = np.random.default_rng(G + int(beta))
    n = We * 11 + G * 3
    a = oracle.relu(_input(rng, n, G, dtype, mixed), dtype)
    if dtype != "bf16":
        a[G * 5: G * 6] *= a.dtype.type(1e-7 if dtype == "f16" else 1e-40)     # a group that restores to (sub)normal dust
    g32 = rng.standard_normal(n).astype(np.float32)
    g = g32 if dtype == "f32" else (g32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(g32))
    x = to_device(a, dtype)
    code = {"f32": daf.F32, "f16": daf.F16, "bf16": daf.BF16}[dtype]
    p = daf.make_params(code, n, G, (1, 2, 4, 8), beta, window_elems=We, seed=9)
    c = daf.alloc_outputs(p, "cuda")
    daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace,
                     c.sizes.workspace)
    gd = to_device(g, dtype)
    out = daf.relu_grad(c, gd)
    torch.cuda.synchronize()
    ref = oracle.compress(a, G, (1, 2, 4, 8), beta, dtype="bf16" if dtype == "bf16" else None, window_elems=We, seed=9)
    restored = oracle.decompress(ref)
    if dtype == "bf16":
        positive = (restored != 0) & ((restored & 0x8000) == 0)
        want = np.where(positive, g, np.uint16(0)).astype(np.uint16)
    else:
        want = np.where(restored > 0, g, g.dtype.type(0)).astype(g.dtype)
    got = to_host(out, dtype)
    view = np.uint32 if dtype == "f32" else np.uint16
    assert np.array_equal(got.view(view), want.view(view))
    assert 0 < int((want.view(view) != 0).sum()) < n
    # in place
    daf.daf_decompress_relu_grad(p, c.packed, c.bits, c.min, c.scale, c.window_offsets, gd, gd)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(gd, dtype).view(view), want.view(view))


def test_fp32_outputs_must_be_32_byte_aligned():
    x = torch.randn(1 << 16, device="cuda")
    c = daf.compress(x, 256, (1, 2, 4, 8), 4.0)
    buf = torch.empty((1 << 16) + 8, device="cuda")
    with pytest.raises(daf.DafError) as e:
        daf.daf_decompress(c.params, c.packed, c.bits, c.min, c.scale, c.window_offsets, buf[4:4 + (1 << 16)])
    assert e.value.status == daf.ERR_INVALID_ARG
    daf.daf_decompress(c.params, c.packed, c.bits, c.min, c.scale, c.window_offsets, buf[8:8 + (1 << 16)])
    torch.cuda.synchronize()


def _scaled(a, dtype, k):
    """The input times k (so that part of it passes 6), in its own type."""
    if dtype == "bf16":
        return wl.f32_to_bf16_bits(oracle.widen(a, "bf16") * np.float32(k))
    return (a * a.dtype.type(k)).astype(a.dtype)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G,beta,mixed,inplace", [(256, 4.0, False, False), (256, 3.0, False, True), (64, 2.0, True, False)])
def test_relu6_compress_matches_relu6_then_compress(dtype, G, beta, mixed, inplace):
    rng = np.random.default_rng(G + int(beta * 10) + mixed + 100)
    n = 16384 * 23 + G * 5
    a = _scaled(_input(rng, n, G, dtype, mixed), dtype, 4.0)
    want = oracle.widen(oracle.relu6(a, dtype), dtype if dtype == "bf16" else None)
    assert (want == 6).sum() > n // 50 and (want == 0).sum() > n // 4
    _check(a, dtype, G, beta, inplace=inplace, act_code=daf.ACT_RELU6)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_relu6_grad_masks_both_ends(dtype):
    """grad where the restored activation lies strictly between 0 and 6: saturated elements restore to exactly 6 (the
    group maximum decodes as min + L * scale; where that rounds below 6 the gradient passes, as the oracle says)."""
    rng = np.random.default_rng(77)
    G, beta, n = 256, 4.0, 16384 * 5 + 256 * 3
    a = oracle.relu6(_scaled(_input(rng, n, G, dtype, False), dtype, 4.0), dtype)
    g32 = rng.standard_normal(n).astype(np.float32)
    g = g32 if dtype == "f32" else (g32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(g32))
    x = to_device(a, dtype)
    c = daf.compress(x, G, (1, 2, 4, 8), beta, seed=4)
    out = daf.relu_grad(c, to_device(g, dtype), act=daf.ACT_RELU6)
    torch.cuda.synchronize()
    ref = oracle.compress(a, G, (1, 2, 4, 8), beta, dtype="bf16" if dtype == "bf16" else None, seed=4)
    r = oracle.widen(oracle.decompress(ref), "bf16" if dtype == "bf16" else None)
    keep = (r > 0) & (r < 6)
    view = np.uint32 if dtype == "f32" else np.uint16
    want = np.where(keep, g.view(view), view(0)).astype(view)
    assert np.array_equal(to_host(out, dtype).view(view), want)
    assert int((r >= 6).sum()) > 0 and int((r <= 0).sum()) > 0 and int(keep.sum()) > 0


def _ulp32(v):
    return np.spacing(np.abs(v).astype(np.float32)).astype(np.float64)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G,beta,mixed", [(256, 4.0, False), (128, 3.0, True)])
def test_gelu_compress_writes_gelu_and_compresses_the_input(dtype, G, beta, mixed):
    """daf_act_compress(GELU): the activation written is GELU(x) to within 8 binary32 ulps plus 2^-24 |x| (the erf
    form: the far negative tail is rounding noise around 0) before the rounding to the output type; the compressed
    form is that of x itself, bit for bit."""
    rng = np.random.default_rng(G + 5)
    n = 16384 * 19 + G * 7
    a = _scaled(_input(rng, n, G, dtype, mixed), dtype, 3.0)
    x = to_device(a, dtype)
    x0 = x.clone()
    y, c = daf.relu_compress(x, G, (1, 2, 4, 8), beta, seed=6, check=True, act=daf.ACT_GELU)
    torch.cuda.synchronize()
    assert torch.equal(x.view(torch.int32 if dtype == "f32" else torch.int16), x0.view(torch.int32 if dtype == "f32" else torch.int16))
    x32 = oracle.widen(a, "bf16" if dtype == "bf16" else None)
    exact = oracle.gelu(x32)
    got = oracle.widen(to_host(y, dtype), "bf16" if dtype == "bf16" else None).astype(np.float64)
    tol = 8 * _ulp32(exact) + 2.0 ** -24 * np.abs(x32.astype(np.float64)) + 2.0 ** -40
    if dtype != "f32":                                            # plus the rounding to the 16-bit type (half an ulp of it)
        mant = 11 if dtype == "f16" else 8
        tol = tol + np.maximum(np.abs(exact) * 2.0 ** -mant, 2.0 ** -25 if dtype == "f16" else 0.0)
    assert np.all(np.abs(got - exact) <= tol), float(np.max(np.abs(got - exact) / tol))
    ref = oracle.compress(a, G, (1, 2, 4, 8), beta, dtype="bf16" if dtype == "bf16" else None, seed=6)
    assert np.array_equal(c.bits.cpu().numpy(), ref.bits)
    assert np.array_equal(c.window_offsets.cpu().numpy().view(np.uint64), ref.window_offsets)
    assert np.array_equal(c.min.cpu().numpy().view(np.uint32), ref.mn.view(np.uint32))
    assert np.array_equal(c.scale.cpu().numpy().view(np.uint32), ref.scale.view(np.uint32))
    assert np.array_equal(c.packed[: ref.packed.size].cpu().numpy(), ref.packed)
    if mixed:
        assert len(np.unique(ref.bits)) >= 2
    # the consumer: gradient times GELU'(restored input)
    g32 = rng.standard_normal(n).astype(np.float32)
    g = g32 if dtype == "f32" else (g32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(g32))
    out = daf.relu_grad(c, to_device(g, dtype), act=daf.ACT_GELU)
    torch.cuda.synchronize()
    r = oracle.widen(oracle.decompress(ref), "bf16" if dtype == "bf16" else None)
    gw = oracle.widen(g, "bf16" if dtype == "bf16" else None).astype(np.float64)
    want = gw * oracle.gelu_grad(r)
    got = oracle.widen(to_host(out, dtype), "bf16" if dtype == "bf16" else None).astype(np.float64)
    # factor within 2^-20; a restored binary32 value may differ from the oracle's by one ulp (|GELU''| <= 1.13)
    tol = np.abs(gw) * (2.0 ** -20 + 1.13 * _ulp32(r)) + _ulp32(want)
    if dtype != "f32":
        mant = 11 if dtype == "f16" else 8
        tol = tol + np.maximum(np.abs(want) * 2.0 ** -mant, 2.0 ** -25 if dtype == "f16" else 0.0)
    assert np.all(np.abs(got - want) <= tol), float(np.max(np.abs(got - want) / tol))


def test_gelu_compress_rejects_in_place_and_unknown_activations():
    x = torch.randn(1 << 16, device="cuda")
    with pytest.raises(daf.DafError) as e:
        daf.relu_compress(x, 256, (1, 2, 4, 8), 4.0, inplace=True, act=daf.ACT_GELU)
    assert e.value.status == daf.ERR_INVALID_ARG
    with pytest.raises(daf.DafError) as e:
        daf.relu_compress(x, 256, (1, 2, 4, 8), 4.0, act=7)
    assert e.value.status == daf.ERR_INVALID_ARG
    c = daf.compress(x, 256, (1, 2, 4, 8), 4.0)
    with pytest.raises(daf.DafError) as e:
        daf.relu_grad(c, x, act=0)
    assert e.value.status == daf.ERR_INVALID_ARG
