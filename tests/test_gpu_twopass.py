"""GPU parity of the two-pass compress route (widths kernel -> offsets kernel -> pack kernel; Sec. 3.4.1's greedy on
one warp per window, Eq. 1 with the chosen widths in a second pass) against the CPU oracle.  The library takes this
route by itself only for large calls on 16-bit elements; here DAF_FLAG_TWO_PASS forces it on calls the oracle finishes
in seconds, for every element type.  Cases of the general parity suite are re-run under that flag, then the route's own
corners: which kernels it stands in for, its capacity check, batched calls, rounding to nearest, the clamped quantizer."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

import test_gpu_parity as base
from gpu_util import assert_compress_parity, assert_decompress_parity, to_device

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(params=["behind the streaming kernel", "alone"])
def two_pass(request, monkeypatch):
    """Every parameter block made without explicit flags asks for the two-pass route: after a try of the streaming
    kernel whatever the call's size, or directly."""
    first = daf.FLAG_STREAM_ALWAYS if request.param == "behind the streaming kernel" else daf.FLAG_STREAM_NEVER
    monkeypatch.setattr(daf, "DEFAULT_FLAGS", first | daf.FLAG_TWO_PASS)


def _as(a32, dtype):
    return a32 if dtype == "f32" else (a32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a32))


@pytest.mark.parametrize("case", range(48))
def test_seeded_random_configurations(case, two_pass):
    base._random_configuration(case)                             # (group or window sizes the route does not take fall through to the general kernel)


@pytest.mark.parametrize("case", range(0, 36, 2))
def test_seeded_tie_heavy_configurations(case, two_pass):
    base.test_seeded_tie_heavy_configurations(case)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G", [128, 256, 512, 1024])
def test_mixed_widths_in_one_window(dtype, G, two_pass):
    base.test_mixed_widths_in_one_window(dtype, G)


@pytest.mark.parametrize("dtype,G", [("f32", 256), ("bf16", 128), ("f16", 1024)])
def test_a_few_mixed_windows_among_many_uniform_ones(dtype, G, two_pass):
    if dtype == "f16":                                           # the base case has no f16 variant: same recipe, smaller values
        rng = np.random.default_rng(5)
        n = 16384 * 300 + G * 3
        a32 = rng.standard_normal(n).astype(np.float32)
        for wdw in (17, 150, 299):
            scale = 10.0 ** rng.uniform(-2, 2, 16384 // G)
            a32[wdw * 16384:(wdw + 1) * 16384] *= np.repeat(scale, G).astype(np.float32)
        a = _as(a32, dtype)
        x, c, ref = assert_compress_parity(a, dtype, G, (1, 2, 4, 8), 4.0, seed=21, label="few-mixed/f16/two-pass")
        assert len(np.unique(ref.bits)) >= 2
        assert_decompress_parity(c, ref, dtype, "few-mixed/f16/two-pass")
    else:
        base.test_a_few_mixed_windows_among_many_uniform_ones(dtype, G)   # includes a range that needs the clamp (f32)


@pytest.mark.parametrize("G,n_last", [(128, 100), (128, 1), (256, 63), (512, 1), (512, 31), (1024, 15)])
def test_ragged_last_window(G, n_last, two_pass):
    base.test_ragged_last_window_takes_the_general_choice(G, n_last)


@pytest.mark.parametrize("G", [128, 256, 1024])
def test_huge_ranges_where_the_inverse_scale_is_subnormal(G, two_pass):
    """Ranges above 2^126: 1/scale is subnormal and the codes need the clamp (the pack kernel's careful quantizer)."""
    rng = np.random.default_rng(G)
    n = 16384 * 2 + G * 5
    a = rng.uniform(-1.6e38, 1.6e38, n).astype(np.float32)
    a[: n // 2] = rng.standard_normal(n // 2).astype(np.float32)   # ordinary groups in the same call
    for widths, beta in (((1, 2, 4, 8), 3.0), ((8,), 8.0)):
        x, c, ref = assert_compress_parity(a, "f32", G, widths, beta, seed=9, label=f"huge/G{G}/{widths}")
        assert_decompress_parity(c, ref, "f32", f"huge/G{G}")


@pytest.mark.parametrize("rounding", [daf.ROUND_STOCHASTIC, daf.ROUND_NEAREST])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rounding_modes_and_a_shard_offset(rounding, dtype, two_pass):
    rng = np.random.default_rng(31)
    n = 16384 * 5 + 128 * 77
    a32 = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // 128), 128)).astype(np.float32)
    a = _as(a32, dtype)
    x, c, ref = assert_compress_parity(a, dtype, 128, (2, 4, 8), 4.0, rounding=rounding, seed=77, base=8 * 12345,
                                        label=f"rounding {rounding}/{dtype}")
    assert_decompress_parity(c, ref, dtype, f"rounding {rounding}/{dtype}")


def test_the_flag_changes_no_result_and_needs_no_streaming_kernel():
    """One tensor through every launch policy: the outputs are the same bytes."""
    rng = np.random.default_rng(8)
    n, G = 16384 * 40 + 256 * 9, 256
    a = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-1, 1, n // G), G)).astype(np.float32)
    x = to_device(a, "f32")
    got = []
    for flags in (daf.FLAG_STREAM_NEVER | daf.FLAG_ONE_PASS, daf.FLAG_STREAM_NEVER | daf.FLAG_TWO_PASS,
                  daf.FLAG_STREAM_ALWAYS | daf.FLAG_ONE_PASS, daf.FLAG_STREAM_ALWAYS | daf.FLAG_TWO_PASS, 0):
        p = daf.make_params(daf.F32, n, G, (1, 2, 4, 8), 3.0, seed=4, flags=flags)
        c = daf.alloc_outputs(p, x.device)
        c.packed.zero_()
        daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace,
                         c.sizes.workspace)
        assert daf.daf_poll_status(c.workspace) == daf.OK
        got.append([t.cpu().numpy().copy() for t in (c.packed, c.bits, c.min, c.scale, c.window_offsets)])
    for other in got[1:]:
        for u, v in zip(got[0], other):
            assert np.array_equal(u.view(np.uint8), v.view(np.uint8))
    with pytest.raises(daf.DafError) as e:                       # both at once is an error
        daf.daf_sizes(daf.make_params(daf.F32, n, G, (1, 2, 4, 8), 3.0, flags=daf.FLAG_ONE_PASS | daf.FLAG_TWO_PASS))
    assert e.value.status == daf.ERR_INVALID_ARG


def test_capacity_error_is_reported_and_nothing_is_written_out_of_bounds():
    """Mixed widths, a packed buffer with room for about half of the windows: the offsets kernel reports the first
    window that does not fit, the windows that do fit are stored, nothing lands behind the capacity."""
    rng = np.random.default_rng(3)
    n, G = 16384 * 12, 128
    a32 = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // G), G)).astype(np.float32)
    a = wl.f32_to_bf16_bits(a32)
    x = to_device(a, "bf16")
    p = daf.make_params(daf.BF16, n, G, (2, 4, 8), 4.0, seed=6, flags=daf.FLAG_STREAM_NEVER | daf.FLAG_TWO_PASS)
    ref = oracle.compress(a, G, (2, 4, 8), 4.0, seed=6, dtype="bf16")
    woff = ref.window_offsets
    cap = int(woff[6]) + 40                                      # six windows fit; the seventh would end beyond
    cap -= cap % 16
    assert woff[6] <= cap < woff[7]
    c = daf.alloc_outputs(p, x.device)
    c.packed.fill_(0xA5)
    daf.daf_compress(p, x, c.packed, cap, c.bits, c.min, c.scale, c.window_offsets, c.workspace, c.sizes.workspace)
    assert daf.daf_poll_status(c.workspace) == daf.ERR_CAPACITY
    hdr = c.workspace[:16].cpu().numpy().view(np.uint32)
    assert hdr[2] == 6                                           # fail_window: the first one that does not fit
    assert bool((c.packed[cap:] == 0xA5).all())
    assert np.array_equal(c.packed[: int(woff[6])].cpu().numpy(), ref.packed[: int(woff[6])])
    assert bool((c.packed[int(woff[6]):cap] == 0xA5).all())      # window 6 itself is not stored either
    assert np.array_equal(c.window_offsets.cpu().numpy().astype(np.uint64), woff.astype(np.uint64))
    # the same buffers with enough room work again
    daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace,
                     c.sizes.workspace)
    assert daf.daf_poll_status(c.workspace) == daf.OK
    assert np.array_equal(c.packed[: ref.packed.size].cpu().numpy(), ref.packed)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_batched_calls_equal_single_calls(dtype, two_pass):
    base.test_batched_calls_equal_single_calls(dtype)


@pytest.mark.parametrize("G,beta,mixed", [(256, 4.0, 3), (1024, 4.0, 4), (128, 4.0, 0)])
def test_batched_calls_through_the_quick_and_the_full_kernel(G, beta, mixed, two_pass):
    base.test_batched_calls_through_the_quick_and_the_full_kernel(G, beta, mixed)


def test_large_16_bit_calls_take_the_route_by_default():
    """What the library does by itself: more than 4096 windows of bf16 with mixed widths.  The general kernel is not
    involved: its ticket counter (word 5 of the workspace header) stays zero; with DAF_FLAG_ONE_PASS it does not."""
    rng = np.random.default_rng(10)
    n, G = 16384 * 4200, 128
    scale = 10.0 ** rng.uniform(-1.5, 1.5, n // G)
    a = wl.f32_to_bf16_bits((rng.standard_normal(n, dtype=np.float32) * np.repeat(scale, G).astype(np.float32)))
    x = to_device(a, "bf16")
    outs = {}
    for flags in (0, daf.FLAG_ONE_PASS):
        p = daf.make_params(daf.BF16, n, G, (2, 4, 8), 4.0, seed=2, flags=flags)
        c = daf.alloc_outputs(p, x.device)
        daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace,
                         c.sizes.workspace)
        assert daf.daf_poll_status(c.workspace) == daf.OK
        ticket2 = int(c.workspace[20:24].cpu().numpy().view(np.uint32)[0])
        assert (ticket2 == 0) == (flags == 0)
        outs[flags] = c
    u, v = outs[0], outs[daf.FLAG_ONE_PASS]
    total = int(u.window_offsets[-1])
    assert total == int(v.window_offsets[-1]) and len(torch.unique(u.bits)) >= 2
    assert torch.equal(u.packed[:total], v.packed[:total]) and torch.equal(u.bits, v.bits)
    assert torch.equal(u.min.view(torch.int32), v.min.view(torch.int32)) and torch.equal(u.scale.view(torch.int32), v.scale.view(torch.int32))
    assert torch.equal(u.window_offsets, v.window_offsets)
    # sampled windows against the oracle, one by one (the oracle on 69 M elements would take too long)
    for wdw in (0, 2517, 4199):
        lo, hi = wdw * 16384, (wdw + 1) * 16384
        ref = oracle.compress(a[lo:hi], G, (2, 4, 8), 4.0, seed=2, dtype="bf16", base=lo)
        o = int(u.window_offsets[wdw])
        assert np.array_equal(u.packed[o:o + ref.packed.size].cpu().numpy(), ref.packed)
        assert np.array_equal(u.bits[wdw * 128:(wdw + 1) * 128].cpu().numpy(), ref.bits)
