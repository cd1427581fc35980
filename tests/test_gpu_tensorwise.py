"""GPU: the per-tensor path (Eq. 1 with one min / max / width per activation tensor, behind it the collective
reduction of Sec. 3.2.1-3.2.2) against the oracle's staged functions run with the whole tensor as the one group."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

from gpu_util import to_device, to_host

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _as(a32, dtype):
    return a32 if dtype == "f32" else (a32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a32))


def _stats_words(stats):
    return stats[:3].cpu().numpy().view(np.float32)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n", [8, 8 * 33, 16384 * 5 + 8 * 77, (1 << 22) + 8])
def test_minmax_is_numpy_min_max(dtype, n):
    rng = np.random.default_rng(n)
    a32 = (rng.standard_normal(n) * 10.0 ** rng.uniform(-3, 3, n)).astype(np.float32)
    if dtype == "f16":
        a32 = np.clip(a32, -6e4, 6e4)
    a = _as(a32, dtype)
    x = to_device(a, dtype)
    stats = torch.full((8,), -1, dtype=torch.int32, device="cuda")      # stale contents must not matter
    daf.daf_tensor_minmax(x, stats)
    torch.cuda.synchronize()
    w = oracle.widen(a, "bf16" if dtype == "bf16" else None)
    got = _stats_words(stats)
    assert got[0] == w.min() and got[1] == w.max()
    mn, mx, R = oracle.stats(w, n)                                   # the oracle with the tensor as one group
    assert got[0].view(np.uint32) == mn.view(np.uint32)[0] and got[1].view(np.uint32) == mx.view(np.uint32)[0]
    assert got[2].view(np.uint32) == R.view(np.uint32)[0]


def test_minmax_orders_negative_zero_below_positive_zero_and_treats_tiny_ranges_as_constant():
    a = np.zeros(4096, np.float32)
    a[5] = -0.0
    x = to_device(a, "f32")
    stats = torch.zeros(8, dtype=torch.int32, device="cuda")
    daf.daf_tensor_minmax(x, stats)
    got = stats[:3].cpu().numpy().view(np.uint32)
    assert got[0] == 0x80000000 and got[1] == 0 and got[2] == 0        # min -0, max +0, range 0
    b = np.full(4096, 1.0, np.float32)
    b[7] = np.float32(1.0) + np.float32(2.0 ** -23)
    b *= np.float32(2.0 ** -100)                                     # range 2^-123 < 2^-118: constant
    daf.daf_tensor_minmax(to_device(b, "f32"), stats)
    got = _stats_words(stats)
    assert got[0] == b.min() and got[1] == b.max() and got[2] == 0.0


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("width", [1, 2, 4, 8])
@pytest.mark.parametrize("rounding", [daf.ROUND_STOCHASTIC, daf.ROUND_NEAREST])
def test_tensor_compress_and_decompress_match_the_oracle_with_one_group(dtype, width, rounding):
    rng = np.random.default_rng(width * 10 + rounding)
    n = 16384 * 3 + 8 * 123                                          # several chunks per warp and a ragged last chunk
    a = _as(rng.laplace(size=n).astype(np.float32), dtype)
    x = to_device(a, dtype)
    seed, base = 77, 8 * 1000
    packed, min_scale, stats = daf.tensor_compress(x, width, rounding=rounding, seed=seed, elem_index_base=base)
    y = daf.tensor_decompress(packed, width, min_scale, x.shape, x.dtype)
    torch.cuda.synchronize()
    w = oracle.widen(a, "bf16" if dtype == "bf16" else None)
    mn, mx, R = oracle.stats(w, n)
    bits = np.array([width], np.uint8)
    scale, inv = oracle.group_params(R, bits)
    codes = oracle.codes(w, n, mn, inv, bits, rounding=rounding, seed=seed, base=base)
    ref_packed = oracle.pack(codes, n, bits)
    ms = min_scale.cpu().numpy()
    assert ms[0].view(np.uint32) == mn.view(np.uint32)[0] and ms[1].view(np.uint32) == scale.view(np.uint32)[0]
    got_packed = packed[: n * width // 8].cpu().numpy()
    assert np.array_equal(oracle.unpack(got_packed, n, n, bits), codes)
    assert np.array_equal(got_packed, ref_packed)
    code = {"f32": oracle.F32, "f16": oracle.F16, "bf16": oracle.BF16}[dtype]
    want = oracle.decode(codes, n, mn, scale, code)
    got = to_host(y, dtype)
    if dtype == "f32":
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    else:
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))


def test_huge_range_and_constant_tensor():
    # a range above 2^126: 1/scale is subnormal, the clamp of the quantizer is what keeps the codes in range
    a = np.zeros(8192, np.float32)
    a[0], a[1] = np.float32(-1.5e38), np.float32(1.5e38)
    a[2:] = np.random.default_rng(0).uniform(-1.5e38, 1.5e38, a.size - 2).astype(np.float32)
    x = to_device(a, "f32")
    packed, min_scale, _ = daf.tensor_compress(x, 8, seed=1)
    mn, mx, R = oracle.stats(a, a.size)
    bits = np.array([8], np.uint8)
    scale, inv = oracle.group_params(R, bits)
    codes = oracle.codes(a, a.size, mn, inv, bits, seed=1)
    assert np.array_equal(packed[: a.size].cpu().numpy(), codes.astype(np.uint8))
    c = to_device(np.full(4096, 3.25, np.float32), "f32")
    packed, min_scale, _ = daf.tensor_compress(c, 4)
    y = daf.tensor_decompress(packed, 4, min_scale, c.shape, c.dtype)
    assert not packed[: 2048].any() and min_scale.cpu().tolist() == [3.25, 0.0] and bool((y == 3.25).all())


def test_argument_errors():
    x = torch.zeros(4096, device="cuda")
    stats = torch.zeros(8, dtype=torch.int32, device="cuda")
    packed = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    ms = torch.zeros(2, device="cuda")
    with pytest.raises(daf.DafError) as e:
        daf.daf_tensor_minmax(x[:4092], stats)                      # not a multiple of 8
    assert e.value.status == daf.ERR_SHAPE
    with pytest.raises(daf.DafError) as e:
        daf.daf_tensor_minmax(x[8:], stats[1:])                     # stats not 16-byte aligned
    assert e.value.status == daf.ERR_INVALID_ARG
    with pytest.raises(daf.DafError) as e:
        daf.daf_tensor_minmax(x[4:4092], stats)                     # fp32 input 16 bytes off the 32-byte boundary
    assert e.value.status == daf.ERR_INVALID_ARG
    daf.daf_tensor_minmax(x, stats)
    for kw, width in ((dict(), 3), (dict(rounding=7), 4), (dict(elem_index_base=4), 4)):
        with pytest.raises(daf.DafError) as e:
            daf.daf_tensor_compress(x, width, stats, packed, ms, **kw)
        assert e.value.status == daf.ERR_INVALID_ARG
