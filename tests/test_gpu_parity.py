"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs -- group min / scale, widths, offsets, codes and packed bytes bit-exact;
dequantized values 0 ulp (fp16 / bf16) and within 1 ulp (fp32)."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

from gpu_util import (assert_compress_parity, assert_decompress_parity, gpu_compress, to_device, to_host)

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _gen(cfg, ti, spec):
    return wl.generate(cfg, ti, spec)


# ------------------------------------------------------------------ the five workloads (small enough for the oracle)
def test_cfg1_full():
    w = wl.workload(1)
    a = _gen(1, 0, w.tensors[0])
    x, c, ref = assert_compress_parity(a, "f32", w.group_size, w.widths, w.bit_budget, seed=0, label="cfg1")
    assert set(np.unique(ref.bits)) == {4}                    # ranges differ by far less than the 4 -> 8 threshold
    assert_decompress_parity(c, ref, "f32", "cfg1")


@pytest.mark.parametrize("ti", [3, 20, 56])                   # relu 64x56x56 block, a 28x28 conv, the last 7x7 relu
def test_cfg2_tensors_at_batch_4(ti):
    w = wl.workload(2, batch=4)
    spec = w.tensors[ti]
    a = _gen(2, ti, spec)
    x, c, ref = assert_compress_parity(a, "f32", w.group_size, w.widths, w.bit_budget, seed=spec.philox_seed,
                                       label=f"cfg2/{spec.name}")
    assert sorted(np.unique(ref.bits)) == [2, 4]              # half the groups at 2 bits, half at 4
    assert_decompress_parity(c, ref, "f32", f"cfg2/{spec.name}")


@pytest.mark.parametrize("ti", [1, 12, 31])                   # includes 960x7x7 (ragged last window)
def test_cfg3_tensors_at_batch_4(ti):
    w = wl.workload(3, batch=4)
    spec = w.tensors[ti]
    a = _gen(3, ti, spec)
    x, c, ref = assert_compress_parity(a, "f16", w.group_size, w.widths, w.bit_budget, seed=spec.philox_seed,
                                       label=f"cfg3/{spec.name}")
    assert_decompress_parity(c, ref, "f16", f"cfg3/{spec.name}")


@pytest.mark.parametrize("ti", [0, 1])
def test_cfg4_tensors_at_batch_2(ti):
    w = wl.workload(4, batch=2, layers=1)
    spec = w.tensors[ti]
    a = _gen(4, ti, spec)
    x, c, ref = assert_compress_parity(a, "bf16", w.group_size, w.widths, w.bit_budget, seed=spec.philox_seed,
                                       label=f"cfg4/{spec.name}")
    assert len(np.unique(ref.bits)) == 3                      # outlier groups force all three widths
    assert_decompress_parity(c, ref, "bf16", f"cfg4/{spec.name}")


@pytest.mark.parametrize("G", wl.SWEEP_GROUPS)
@pytest.mark.parametrize("beta", wl.SWEEP_BUDGETS)
def test_cfg5_sweep_point_on_a_slice(G, beta):
    w = wl.workload(5, numel=1 << 21, group_size=G, bit_budget=beta)
    a = _gen(5, 0, w.tensors[0])
    x, c, ref = assert_compress_parity(a, "f32", G, w.widths, beta, label=f"cfg5/G{G}/b{beta}")
    assert_decompress_parity(c, ref, "f32", f"cfg5/G{G}/b{beta}")


# ------------------------------------------------------------------ stress inputs
@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G", [32, 64, 128, 256, 512, 1024, 4096, 16384])
def test_mixed_widths_in_one_window(dtype, G):
    """Per-group scales spread over four decades: every width appears inside single windows."""
    rng = np.random.default_rng(G)
    n = 16384 * 3 + G * (3 if G < 16384 else 0)               # ragged last window unless G is the window
    scale = 10.0 ** rng.uniform(-2, 2, n // G)
    a32 = (rng.standard_normal(n) * np.repeat(scale, G)).astype(np.float32)
    a = a32 if dtype == "f32" else (a32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a32))
    for widths, beta in (((1, 2, 4, 8), 3.0), ((1, 2, 4, 8), 2.5), ((2, 4, 8), 4.0)):
        x, c, ref = assert_compress_parity(a, dtype, G, widths, beta, seed=G + 1, label=f"mixed/{dtype}/G{G}/{widths}/{beta}")
        if G <= 4096:
            assert len(np.unique(ref.bits)) >= 2
        assert_decompress_parity(c, ref, dtype, f"mixed/{dtype}/G{G}")


@pytest.mark.parametrize("widths", [(1,), (2,), (4,), (8,), (1, 2), (1, 4), (1, 8), (2, 4), (2, 8), (4, 8), (1, 2, 4), (1, 2, 8),
                                    (1, 4, 8), (2, 4, 8), (1, 2, 4, 8)])
def test_every_width_subset(widths):
    rng = np.random.default_rng(len(widths) * 100 + sum(widths))
    G, n = 64, 16384 * 2 + 64 * 5
    a = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-1, 1, n // G), G)).astype(np.float32)
    for beta in (float(min(widths)), min(widths) + 0.8, 3.3, 8.0):
        if beta < min(widths):
            continue
        x, c, ref = assert_compress_parity(a, "f32", G, widths, beta, seed=3, label=f"subset/{widths}/{beta}")
        assert_decompress_parity(c, ref, "f32", f"subset/{widths}/{beta}")


def test_degenerate_groups_zero_constant_and_signed_zero():
    G = 128
    vals = np.float32([0.0, -0.0, 1.0, -3.5, 6.0, 1e-30, 3e38, -3e38])
    a = np.repeat(vals, G).astype(np.float32)
    a = np.concatenate([a, np.tile(np.float32([0.0, -0.0]), G // 2), np.tile(np.float32([-0.0, 1.0]), G // 2),
                        np.random.default_rng(0).standard_normal(16384).astype(np.float32)])
    # subnormal-range group: range below 2^-118 is treated as constant
    tiny = np.zeros(G, np.float32)
    tiny[5] = np.float32(2.0 ** -120)
    a = np.concatenate([a, tiny]).astype(np.float32)
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, label="degenerate")
    assert np.all(ref.scale[:8] == 0)
    assert ref.mn.view(np.uint32)[8] == 0x80000000            # -0.0 orders below +0.0
    assert_decompress_parity(c, ref, "f32", "degenerate")


@pytest.mark.parametrize("G", [256, 1024, 16384])
def test_signed_zero_minimum_in_full_warp_groups(G):
    """Groups of 256 and more are reduced by the warp-wide redux path: -0.0 must still order below +0.0."""
    rng = np.random.default_rng(G)
    n = 16384 * 2
    a = np.abs(rng.standard_normal(n)).astype(np.float32)
    a[rng.integers(0, n, n // 8)] = 0.0
    a[rng.integers(0, n, n // 8)] = -0.0                      # smallest values are a mix of +0.0 and -0.0
    a[:G] = np.where(np.arange(G) % 2 == 0, np.float32(0.0), np.float32(-0.0))   # max must be +0.0, min -0.0
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, label=f"signed-zero/G{G}")
    assert ref.mn.view(np.uint32)[0] == 0x80000000
    assert_decompress_parity(c, ref, "f32", f"signed-zero/G{G}")


@pytest.mark.parametrize("G", [64, 256, 2048])
def test_huge_ranges_where_the_inverse_scale_is_subnormal(G):
    """Ranges beyond 2^126: 1/scale is a subnormal number and the code clamp can become active."""
    rng = np.random.default_rng(G + 7)
    n = 16384 * 3
    a = rng.random(n).astype(np.float32)
    big = rng.integers(0, n // G, 8)
    for g in big:
        a[g * G:(g + 1) * G] = (rng.random(G) * 1.6e38).astype(np.float32)     # range up to about 2^127
        a[g * G] = np.float32(1.6e38)
        a[g * G + 1] = np.float32(0.0)
    for widths, beta in (((1, 2, 4, 8), 8.0), ((1,), 1.0), ((1, 2, 4, 8), 3.0)):
        x, c, ref = assert_compress_parity(a, "f32", G, widths, beta, seed=11, label=f"huge/G{G}/{widths}/{beta}")
        assert_decompress_parity(c, ref, "f32", f"huge/G{G}")


def test_heavy_ties_relu6_saturation():
    """Most groups share the same range (clip at 0 and 6): the tie order by group index decides."""
    rng = np.random.default_rng(4)
    G, n = 128, 16384 * 4
    a = np.clip(rng.standard_normal(n) * 2, 0, 6).astype(np.float16)
    for beta in (1.5, 2.0, 2.75, 3.0):
        x, c, ref = assert_compress_parity(a, "f16", G, (1, 2, 4, 8), beta, seed=9, label=f"ties/{beta}")
        assert_decompress_parity(c, ref, "f16", f"ties/{beta}")


@pytest.mark.parametrize("G", [64, 256, 1024])
def test_different_ranges_with_equal_keys(G):
    """Ranges that are neighbouring floats: several of them round to the same importance key, so
    the order among those raises is by group index, not by range, and the budget's cut falls
    inside such runs for some of the budgets."""
    rng = np.random.default_rng(G + 17)
    W, n_win = 16384 // G, 3
    n_groups = W * n_win + 3                                     # ragged last window
    base = np.float32(3.99)                                      # R v stays in (or one above) the binade of R: keys coarser than ranges
    steps = rng.integers(0, 6, n_groups)                         # ranges base * (1 + j ulp), j = 0..5, in random order
    R = (np.full(n_groups, base, np.float32).view(np.uint32) + steps.astype(np.uint32)).view(np.float32)
    far = rng.random(n_groups) < 0.15                            # some groups far away, so that levels mix
    R = np.where(far, R * np.float32(2.0) ** rng.integers(-6, 7, n_groups).astype(np.float32), R).astype(np.float32)
    a = np.zeros((n_groups, G), np.float32)
    a[:, 1] = R                                                  # min 0, max R: the range is R exactly
    a[:, 2:] = rng.random((n_groups, G - 2), dtype=np.float32) * R[:, None] * np.float32(0.999)
    collided = False
    for b_lo, b_hi in ((1, 2), (2, 4), (4, 8)):
        v = oracle.raise_factor(b_lo, b_hi)
        keys = (R * v).astype(np.float32)
        for w in range(n_win):
            k, r = keys[w * W:(w + 1) * W], R[w * W:(w + 1) * W]
            order = np.argsort(k, kind="stable")
            same_key = k[order][1:] == k[order][:-1]
            collided |= bool(np.any(same_key & (r[order][1:] != r[order][:-1])))
    assert collided, "the construction no longer produces equal keys from different ranges"
    for beta in (1.25, 1.5, 2.5, 3.0, 3.5, 5.0, 6.0):
        x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), beta, seed=5, label=f"collide/G{G}/{beta}")
        assert_decompress_parity(c, ref, "f32", f"collide/G{G}/{beta}")


@pytest.mark.parametrize("dtype,G", [("f32", 256), ("f32", 64), ("bf16", 128), ("f32", 4096)])
def test_a_few_mixed_windows_among_many_uniform_ones(dtype, G):
    """Most windows end with one width for all groups (the quick kernel's case); a few windows far
    into the tensor have groups of very different ranges, one has a range that needs the clamp, and
    the last window is ragged: the call must come out the same whichever kernel finishes it."""
    rng = np.random.default_rng(G + len(dtype))
    n_win = 600                                                  # more windows than resident CTAs
    n = 16384 * n_win + G * 3
    a32 = rng.standard_normal(n).astype(np.float32)
    for wdw in (301, 302, 577):                                  # mixed ranges: the general bit choice
        lo = wdw * 16384
        scale = 10.0 ** rng.uniform(-3, 3, 16384 // G)
        a32[lo:lo + 16384] *= np.repeat(scale, G).astype(np.float32)
    if dtype == "f32":
        a32[450 * 16384] = np.float32(1.5e38)                      # 1/scale is not a normal number there
        a32[450 * 16384 + 1] = np.float32(-1.5e38)
    a = a32 if dtype == "f32" else wl.f32_to_bf16_bits(a32)
    for beta in (4.0, 2.0):
        x, c, ref = assert_compress_parity(a, dtype, G, (1, 2, 4, 8), beta, seed=21, label=f"few-mixed/{dtype}/G{G}/{beta}")
        assert len(np.unique(ref.bits)) >= 2
        assert_decompress_parity(c, ref, dtype, f"few-mixed/{dtype}/G{G}/{beta}")
    # and a tensor that never leaves the quick kernel, right after one that did, on fresh outputs
    u = rng.standard_normal(16384 * 40).astype(np.float32)
    u = u if dtype == "f32" else wl.f32_to_bf16_bits(u)
    x, c, ref = assert_compress_parity(u, dtype, G, (1, 2, 4, 8), 4.0, seed=22, label=f"all-uniform/{dtype}/G{G}")
    assert_decompress_parity(c, ref, dtype, f"all-uniform/{dtype}/G{G}")


@pytest.mark.parametrize("G,n_last", [(32, 5), (64, 37), (128, 100), (256, 63), (512, 1), (2048, 3)])
def test_ragged_last_window_takes_the_general_choice(G, n_last):
    """A last window with a group count that is not a power of two, with mixed widths."""
    rng = np.random.default_rng(G * 7 + n_last)
    n = 16384 * 2 + G * n_last
    a = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // G), G)).astype(np.float32)
    for widths, beta in (((1, 2, 4, 8), 3.0), ((2, 4, 8), 4.0), ((1, 2, 4, 8), 4.0)):
        x, c, ref = assert_compress_parity(a, "f32", G, widths, beta, seed=11, label=f"ragged/G{G}/{widths}/{beta}")
        assert_decompress_parity(c, ref, "f32", f"ragged/G{G}")


@pytest.mark.parametrize("We", [4096, 8192, 16384])
@pytest.mark.parametrize("rounding", [daf.ROUND_STOCHASTIC, daf.ROUND_NEAREST])
def test_window_sizes_rounding_modes_and_shards(We, rounding):
    rng = np.random.default_rng(We + rounding)
    G, n = 256, We * 7 + 256 * 9
    a = (rng.laplace(size=n) * np.repeat(10.0 ** rng.uniform(-1, 1, n // G), G)).astype(np.float32)
    seed = 0xDEADBEEF12345678
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, window_elems=We, rounding=rounding, seed=seed,
                                       label=f"We{We}/r{rounding}")
    assert_decompress_parity(c, ref, "f32", f"We{We}/r{rounding}")
    # a window-aligned shard compressed with its element base reproduces the same bytes
    lo, hi = 2 * We, 5 * We
    xs, cs, refs = assert_compress_parity(a[lo:hi], "f32", G, (1, 2, 4, 8), 3.0, window_elems=We, rounding=rounding,
                                          seed=seed, base=lo, label="shard")
    full = c.packed[: c.packed_bytes()].cpu().numpy()
    woff = c.window_offsets.cpu().numpy()
    assert np.array_equal(cs.packed[: cs.packed_bytes()].cpu().numpy(), full[int(woff[2]):int(woff[5])])


def test_large_element_index_base_uses_the_high_counter_word():
    rng = np.random.default_rng(8)
    a = rng.standard_normal(16384 * 2).astype(np.float32)
    base = (1 << 35) + 16384 * 3
    x, c, ref = assert_compress_parity(a, "f32", 256, (2, 4), 3.0, seed=77, base=base, label="bigbase")


def test_single_group_and_single_window():
    rng = np.random.default_rng(2)
    for n, G in ((32, 32), (256, 256), (16384, 16384), (16384, 64), (4096, 128)):
        a = rng.standard_normal(n).astype(np.float32)
        x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 4.0, label=f"tiny/{n}/{G}")
        assert_decompress_parity(c, ref, "f32", f"tiny/{n}/{G}")


# ------------------------------------------------------------------ decompress fed with oracle buffers
@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_decompress_of_oracle_buffers(dtype):
    rng = np.random.default_rng(12)
    G, n = 64, 16384 * 2 + 64 * 7
    a32 = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // G), G)).astype(np.float32)
    a = a32 if dtype == "f32" else (a32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a32))
    ref = oracle.compress(a, G, (1, 2, 4, 8), 3.0, dtype="bf16" if dtype == "bf16" else None, seed=5)
    p = daf.make_params({"f32": daf.F32, "f16": daf.F16, "bf16": daf.BF16}[dtype], n, G, (1, 2, 4, 8), 3.0, seed=5)
    packed = torch.zeros(ref.packed.size + 16, dtype=torch.uint8, device="cuda")
    packed[: ref.packed.size] = torch.from_numpy(ref.packed).cuda()
    out = torch.empty(n, dtype={"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[dtype], device="cuda")
    daf.daf_decompress(p, packed, torch.from_numpy(ref.bits).cuda(), torch.from_numpy(ref.mn).cuda(),
                       torch.from_numpy(ref.scale).cuda(), torch.from_numpy(ref.window_offsets.view(np.int64)).cuda(), out)
    torch.cuda.synchronize()
    got, want = to_host(out, dtype), oracle.decompress(ref)
    assert np.array_equal(got.view(np.uint32 if dtype == "f32" else np.uint16),
                          want.view(np.uint32 if dtype == "f32" else np.uint16))


# ------------------------------------------------------------------ standalone scan
@pytest.mark.parametrize("n_groups", [1, 31, 8192, 8193, 100_003, 3_000_000])
def test_group_offsets_against_oracle(n_groups):
    rng = np.random.default_rng(n_groups)
    bits = rng.choice(np.uint8([1, 2, 4, 8]), n_groups)
    for G, misalign in ((64, 0), (4096, 0), (256, 3)):
        buf = torch.zeros(n_groups + 16, dtype=torch.uint8, device="cuda")
        d_bits = buf[misalign: misalign + n_groups]
        d_bits.copy_(torch.from_numpy(bits))
        off = torch.empty(n_groups + 1, dtype=torch.int64, device="cuda")
        ws_bytes = daf.daf_group_offsets_workspace(n_groups)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        daf.daf_group_offsets(d_bits, n_groups, G, off, ws, ws_bytes)
        assert daf.daf_poll_status(ws) == daf.OK
        assert np.array_equal(off.cpu().numpy().view(np.uint64), oracle.offsets(bits, G))


def test_budget_above_the_largest_width():
    """Budget 12 with widths {1,2,4}: every group ends at 4 bits, the capacity is that of 4 bits, parity as usual."""
    rng = np.random.default_rng(12)
    n = 16384 * 9 + 256 * 5
    a = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // 256), 256)).astype(np.float32)
    xd, c, ref = assert_compress_parity(a, "f32", 256, (1, 2, 4), 12.0, seed=3, label="budget 12")
    assert set(np.unique(ref.bits)) == {4} and c.sizes.packed_capacity == n * 4 // 8
    assert_decompress_parity(c, ref, "f32", "budget 12")


# ------------------------------------------------------------------ device-detected errors, guard bands
def test_capacity_error_is_reported_and_nothing_is_written_out_of_bounds():
    rng = np.random.default_rng(3)
    n, G = 16384 * 6, 256
    a = rng.standard_normal(n).astype(np.float32)
    x = to_device(a, "f32")
    p = daf.make_params(daf.F32, n, G, (4,), 4.0)
    c = daf.alloc_outputs(p, x.device)
    cap = 16384 * 4 // 8 * 3                                   # room for three of the six windows
    c.packed.fill_(0xA5)
    daf.daf_compress(p, x, c.packed, cap, c.bits, c.min, c.scale, c.window_offsets, c.workspace, c.sizes.workspace)
    assert daf.daf_poll_status(c.workspace) == daf.ERR_CAPACITY
    assert bool((c.packed[cap:] == 0xA5).all())
    ref = oracle.compress(a, G, (4,), 4.0)
    assert np.array_equal(c.packed[:cap].cpu().numpy(), ref.packed[:cap])
    # the same buffers with enough room work again (the workspace is reset by every call)
    daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace,
                     c.sizes.workspace)
    assert daf.daf_poll_status(c.workspace) == daf.OK
    assert np.array_equal(c.packed[: ref.packed.size].cpu().numpy(), ref.packed)


def test_outputs_have_intact_guard_bands():
    rng = np.random.default_rng(6)
    n, G = 16384 * 3 + 128 * 5, 128
    a = rng.standard_normal(n).astype(np.float16)
    x = to_device(a, "f16")
    p = daf.make_params(daf.F16, n, G, (1, 2, 4, 8), 2.5, seed=1)
    sz = daf.daf_sizes(p)
    pad = 256

    def guarded(nbytes):
        t = torch.full((nbytes + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
        return t, t[pad: pad + nbytes]

    bufs = {k: guarded(nb) for k, nb in (("packed", sz.packed_capacity), ("bits", sz.n_groups), ("mn", 4 * sz.n_groups),
                                         ("scale", 4 * sz.n_groups), ("woff", 8 * (sz.n_windows + 1)), ("out", 2 * n))}
    ws = torch.empty(sz.workspace, dtype=torch.uint8, device="cuda")
    daf.daf_compress(p, x, bufs["packed"][1], sz.packed_capacity, bufs["bits"][1], bufs["mn"][1], bufs["scale"][1],
                     bufs["woff"][1], ws, sz.workspace)
    assert daf.daf_poll_status(ws) == daf.OK
    daf.daf_decompress(p, bufs["packed"][1], bufs["bits"][1], bufs["mn"][1], bufs["scale"][1], bufs["woff"][1],
                       bufs["out"][1])
    torch.cuda.synchronize()
    for name, (full, inner) in bufs.items():
        assert bool((full[:pad] == 0xA5).all()) and bool((full[pad + inner.numel():] == 0xA5).all()), name
    ref = oracle.compress(a, G, (1, 2, 4, 8), 2.5, seed=1)
    assert np.array_equal(bufs["out"][1].cpu().numpy().view(np.uint16), oracle.decompress(ref).view(np.uint16))


@pytest.mark.parametrize("case", range(48))
def test_seeded_random_configurations(case):
    """Group size, window size, widths, budget, type, rounding, length and value mix drawn from a
    seed: uniform stretches, stretches of mixed ranges, constant groups and a ragged end in one tensor."""
    _random_configuration(case)


@pytest.mark.parametrize("case", range(0, 48, 2))
def test_seeded_random_configurations_full_kernel_alone(case, default_quick_limit):
    """The same with the library's default limit: calls this small skip the quick kernel."""
    _random_configuration(case)


def test_small_uniform_call_full_kernel_alone(default_quick_limit):
    a = _gen(1, 0, wl.workload(1).tensors[0])[: 16384 * 9 + 2048]
    x, c, ref = assert_compress_parity(a, "f32", 256, (1, 2, 4, 8), 4.0, seed=5, label="small/full-only")
    assert set(np.unique(ref.bits)) == {4}
    assert_decompress_parity(c, ref, "f32", "small/full-only")


def _random_configuration(case):
    rng = np.random.default_rng(1000 + case)
    dtype = ("f32", "f16", "bf16")[case % 3]
    We = int(rng.choice([4096, 8192, 16384]))
    G = int(rng.choice([g for g in (32, 64, 128, 256, 512, 1024, 2048, 4096) if g <= We]))
    widths = tuple(sorted(rng.choice([1, 2, 4, 8], size=int(rng.integers(1, 5)), replace=False).tolist()))
    beta = float(rng.choice([min(widths), min(widths) + 0.5, 2.0, 3.0, 4.0, 8.0]))
    beta = max(beta, float(min(widths)))
    n_groups = int(rng.integers(1, 40 * We // G + 2))
    x = rng.standard_normal((n_groups, G)).astype(np.float32)
    kind = rng.random(n_groups)
    scale = np.where(kind < 0.25, 10.0 ** rng.uniform(-3, 3, n_groups), 1.0).astype(np.float32)   # mixed ranges
    x *= scale[:, None]
    x[kind > 0.95] = np.float32(rng.standard_normal())                                            # constant groups
    if case % 5 == 0:
        x = np.abs(x)                                                                                # one-sided (ReLU-like)
    a = x.reshape(-1)
    a = a if dtype == "f32" else (a.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a))
    rounding = daf.ROUND_NEAREST if case % 7 == 3 else daf.ROUND_STOCHASTIC
    label = f"random/{case}/{dtype}/G{G}/We{We}/{widths}/{beta}"
    xd, c, ref = assert_compress_parity(a, dtype, G, widths, beta, window_elems=We, rounding=rounding,
                                        seed=case * 7919 + 1, label=label)
    assert_decompress_parity(c, ref, dtype, label)


def test_shards_cut_by_daf_shard_reproduce_the_unsharded_result():
    """Three ranks' slices (daf_shard: window-aligned, bases moved) compressed one by one equal the pieces of the oracle's
    result for the whole tensor: widths, minima, scales, packed bytes; window offsets restart in every slice."""
    rng = np.random.default_rng(77)
    G, widths, beta, seed = 128, (1, 2, 4, 8), 3.0, 5
    n = 16384 * 10 + 128 * 9
    a = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-1, 1, n // G), G)).astype(np.float32)
    ref = oracle.compress(a, G, widths, beta, seed=seed)
    x = to_device(a, "f32")
    whole = daf.make_params(daf.F32, n, G, widths, beta, seed=seed)
    for rank in range(3):
        p, first = daf.daf_shard(whole, rank, 3)
        m = int(p.numel)
        c = daf.alloc_outputs(p, "cuda")
        daf.daf_compress(p, x[first:first + m], c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                         c.workspace, c.sizes.workspace)
        assert daf.daf_poll_status(c.workspace) == daf.OK
        g0, g1 = first // G, (first + m) // G
        w0 = first // 16384
        assert np.array_equal(c.bits.cpu().numpy(), ref.bits[g0:g1])
        assert np.array_equal(c.min.cpu().numpy().view(np.uint32), ref.mn[g0:g1].view(np.uint32))
        assert np.array_equal(c.scale.cpu().numpy().view(np.uint32), ref.scale[g0:g1].view(np.uint32))
        woff = c.window_offsets.cpu().numpy().view(np.uint64)
        base = int(ref.window_offsets[w0])
        assert np.array_equal(woff + np.uint64(base), ref.window_offsets[w0:w0 + woff.size])
        assert np.array_equal(c.packed[: int(woff[-1])].cpu().numpy(), ref.packed[base: base + int(woff[-1])])


def test_streamed_host_round_trip_equals_the_oracle_on_the_whole_tensor():
    """HostRoundTrip: pinned host tensor in, restored values out, through chunks that overlap copies and kernels; the
    result is what the oracle decodes for the whole tensor (the chunks are shards with the counter base moved)."""
    rng = np.random.default_rng(91)
    G, widths, beta, seed = 256, (1, 2, 4, 8), 4.0, 12
    n = 16384 * 9 + 256 * 3                                         # two whole chunks of four windows and a ragged one
    a = rng.laplace(size=n).astype(np.float32)
    h_in = torch.from_numpy(a).pin_memory()
    h_out = torch.empty_like(h_in).pin_memory()
    rt = daf.HostRoundTrip(torch.float32, G, widths, beta, seed=seed, chunk_elems=16384 * 4)
    for _ in range(2):                                              # twice: the slots are reused
        h_out.zero_()
        rt(h_in, h_out)
        torch.cuda.synchronize()
        want = oracle.decompress(oracle.compress(a, G, widths, beta, seed=seed))
        assert np.array_equal(h_out.numpy().view(np.uint32), want.view(np.uint32))


# ------------------------------------------------------------------ batched calls
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_batched_calls_equal_single_calls(dtype):
    rng = np.random.default_rng(30)
    G, widths, beta = 128, (1, 2, 4, 8), 3.0
    sizes = [16384 * 2 + 128, 128, 16384, 16384 * 5 + 128 * 77, 4096]
    arrays = []
    for n in sizes:
        a32 = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-1, 1, n // G), G)).astype(np.float32)
        arrays.append(a32 if dtype == "f32" else wl.f32_to_bf16_bits(a32))
    xs = [to_device(a, dtype) for a in arrays]
    code = {"f32": daf.F32, "bf16": daf.BF16}[dtype]
    params = [daf.make_params(code, a.size, G, widths, beta, seed=100 + i) for i, a in enumerate(arrays)]
    outs = [daf.alloc_outputs(p, "cuda") for p in params]
    ws_bytes = daf.daf_batch_workspace(params)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    daf.daf_compress_batch(params, xs, [o.packed for o in outs], [o.sizes.packed_capacity for o in outs],
                           [o.bits for o in outs], [o.min for o in outs], [o.scale for o in outs],
                           [o.window_offsets for o in outs], ws, ws_bytes)
    assert daf.daf_poll_status(ws) == daf.OK
    ys = [torch.empty_like(x) for x in xs]
    daf.daf_decompress_batch(params, [o.packed for o in outs], [o.bits for o in outs], [o.min for o in outs],
                             [o.scale for o in outs], [o.window_offsets for o in outs], ys)
    torch.cuda.synchronize()
    for i, a in enumerate(arrays):
        ref = oracle.compress(a, G, widths, beta, dtype="bf16" if dtype == "bf16" else None, seed=100 + i)
        o = outs[i]
        assert np.array_equal(o.bits.cpu().numpy(), ref.bits), i
        assert np.array_equal(o.window_offsets.cpu().numpy().view(np.uint64), ref.window_offsets), i
        assert np.array_equal(o.packed[: ref.packed.size].cpu().numpy(), ref.packed), i
        assert np.array_equal(o.min.cpu().numpy().view(np.uint32), ref.mn.view(np.uint32)), i
        assert np.array_equal(o.scale.cpu().numpy().view(np.uint32), ref.scale.view(np.uint32)), i
        want = oracle.decompress(ref)
        got = to_host(ys[i], dtype)
        assert np.array_equal(got.view(np.uint32 if dtype == "f32" else np.uint16),
                              want.view(np.uint32 if dtype == "f32" else np.uint16)), i


@pytest.mark.parametrize("G,beta,mixed", [(256, 4.0, None), (256, 4.0, 3), (64, 2.0, 1), (1024, 4.0, 4), (4096, 8.0, None), (128, 4.0, 0)])
def test_batched_calls_through_the_quick_and_the_full_kernel(G, beta, mixed):
    """A set of tensors with ragged ends in one batched call; `mixed` names a tensor with groups of very
    different ranges (the quick kernel gives up there and the full kernel redoes the whole set)."""
    rng = np.random.default_rng(G + (mixed or 0))
    widths = (1, 2, 4, 8)
    sizes = [16384 * 7 + G, 16384 * 3, G * 2, 16384 * 21 + G * 5, 16384 * 2]
    arrays = []
    for i, n in enumerate(sizes):
        a32 = rng.standard_normal(n).astype(np.float32)
        if mixed == i:
            a32 *= np.repeat(10.0 ** rng.uniform(-3, 3, n // G), G).astype(np.float32)
        arrays.append(a32)
    xs = [to_device(a, "f32") for a in arrays]
    params = [daf.make_params(daf.F32, a.size, G, widths, beta, seed=500 + i) for i, a in enumerate(arrays)]
    outs = [daf.alloc_outputs(p, "cuda") for p in params]
    ws_bytes = daf.daf_batch_workspace(params)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    for _ in range(2):                                           # the second call reuses the workspace as it was left
        daf.daf_compress_batch(params, xs, [o.packed for o in outs], [o.sizes.packed_capacity for o in outs],
                               [o.bits for o in outs], [o.min for o in outs], [o.scale for o in outs],
                               [o.window_offsets for o in outs], ws, ws_bytes)
        assert daf.daf_poll_status(ws) == daf.OK
    ys = [torch.empty_like(x) for x in xs]
    daf.daf_decompress_batch(params, [o.packed for o in outs], [o.bits for o in outs], [o.min for o in outs],
                             [o.scale for o in outs], [o.window_offsets for o in outs], ys)
    torch.cuda.synchronize()
    for i, a in enumerate(arrays):
        ref = oracle.compress(a, G, widths, beta, seed=500 + i)
        o = outs[i]
        assert np.array_equal(o.bits.cpu().numpy(), ref.bits), i
        assert np.array_equal(o.window_offsets.cpu().numpy().view(np.uint64), ref.window_offsets), i
        assert np.array_equal(o.packed[: ref.packed.size].cpu().numpy(), ref.packed), i
        assert np.array_equal(o.min.cpu().numpy().view(np.uint32), ref.mn.view(np.uint32)), i
        assert np.array_equal(o.scale.cpu().numpy().view(np.uint32), ref.scale.view(np.uint32)), i
        d = np.abs(ys[i].cpu().numpy().view(np.int32).astype(np.int64) - oracle.decompress(ref).view(np.int32).astype(np.int64))
        assert d.max() <= 1, (i, int(d.max()))
    if mixed is not None:
        assert len(np.unique(oracle.compress(arrays[mixed], G, widths, beta, seed=500 + mixed).bits)) >= 2


def test_batched_calls_replayed_from_a_cuda_graph():
    """The calls only enqueue work (a memset and kernels), so a layer list can be captured once and
    replayed: compress + decompress of three tensors captured in a CUDA graph, replayed on new contents."""
    rng = np.random.default_rng(77)
    G, widths, beta = 256, (1, 2, 4, 8), 4.0
    sizes = [16384 * 40 + G * 3, 16384 * 6, 16384 * 13 + G]
    xs = [torch.empty(n, dtype=torch.float32, device="cuda") for n in sizes]
    params = [daf.make_params(daf.F32, n, G, widths, beta, seed=900 + i) for i, n in enumerate(sizes)]
    outs = [daf.alloc_outputs(p, "cuda") for p in params]
    ys = [torch.empty_like(x) for x in xs]
    ws_bytes = daf.daf_batch_workspace(params)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")

    def step():
        daf.daf_compress_batch(params, xs, [o.packed for o in outs], [o.sizes.packed_capacity for o in outs],
                               [o.bits for o in outs], [o.min for o in outs], [o.scale for o in outs],
                               [o.window_offsets for o in outs], ws, ws_bytes)
        daf.daf_decompress_batch(params, [o.packed for o in outs], [o.bits for o in outs], [o.min for o in outs],
                                 [o.scale for o in outs], [o.window_offsets for o in outs], ys)

    def fill(mixed):
        arrays = []
        for i, (x, n) in enumerate(zip(xs, sizes)):
            a = rng.standard_normal(n).astype(np.float32)
            if i == mixed:
                a *= np.repeat(10.0 ** rng.uniform(-2, 2, n // G), G).astype(np.float32)
            x.copy_(torch.from_numpy(a))
            arrays.append(a)
        return arrays

    fill(None)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                                   # first call outside the capture (one-time set-up)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for mixed in (None, 1):                                      # uniform windows only, then a tensor the quick kernel gives up on
        arrays = fill(mixed)
        graph.replay()
        torch.cuda.synchronize()
        assert daf.daf_poll_status(ws) == daf.OK
        for i, a in enumerate(arrays):
            ref = oracle.compress(a, G, widths, beta, seed=900 + i)
            o = outs[i]
            assert np.array_equal(o.bits.cpu().numpy(), ref.bits), (mixed, i)
            assert np.array_equal(o.window_offsets.cpu().numpy().view(np.uint64), ref.window_offsets), (mixed, i)
            assert np.array_equal(o.packed[: ref.packed.size].cpu().numpy(), ref.packed), (mixed, i)
            d = np.abs(ys[i].cpu().numpy().view(np.int32).astype(np.int64)
                       - oracle.decompress(ref).view(np.int32).astype(np.int64))
            assert d.max() <= 1, (mixed, i, int(d.max()))
        if mixed is not None:
            assert len(np.unique(oracle.compress(arrays[mixed], G, widths, beta, seed=900 + mixed).bits)) >= 2


@pytest.mark.parametrize("G", [64, 256])
def test_non_finite_inputs_stay_inside_the_buffers(G):
    """NaN / Inf inputs: results unspecified, but nothing may be written outside the caller's buffers and
    the calls must complete (widths come from integer budget arithmetic whatever the keys are)."""
    rng = np.random.default_rng(G)
    n = 16384 * 6 + G * 3
    a = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // G), G)).astype(np.float32)
    bad = rng.integers(0, n, 400)
    a[bad[:150]] = np.nan
    a[bad[150:250]] = np.inf
    a[bad[250:350]] = -np.inf
    a[G * 40: G * 41] = np.nan                                   # a whole group of NaN
    a[G * 50: G * 51] = np.inf                                   # ... and of +Inf
    x = to_device(a, "f32")
    pad = 512
    for beta in (2.0, 3.0, 4.0):
        p = daf.make_params(daf.F32, n, G, (1, 2, 4, 8), beta, seed=2)
        sz = daf.daf_sizes(p)

        def guarded(nbytes):
            t = torch.full((nbytes + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
            return t, t[pad: pad + nbytes]

        bufs = {k: guarded(nb) for k, nb in (("packed", sz.packed_capacity), ("bits", sz.n_groups), ("mn", 4 * sz.n_groups),
                                             ("scale", 4 * sz.n_groups), ("woff", 8 * (sz.n_windows + 1)), ("out", 4 * n))}
        ws = torch.empty(sz.workspace, dtype=torch.uint8, device="cuda")
        daf.daf_compress(p, x, bufs["packed"][1], sz.packed_capacity, bufs["bits"][1], bufs["mn"][1], bufs["scale"][1],
                         bufs["woff"][1], ws, sz.workspace)
        assert daf.daf_poll_status(ws) == daf.OK
        bits = bufs["bits"][1].cpu().numpy()
        assert set(np.unique(bits)) <= {1, 2, 4, 8}
        woff = bufs["woff"][1].cpu().numpy().view(np.uint64)
        assert int(woff[-1]) == int(bits.astype(np.int64).sum()) * G // 8 <= sz.packed_capacity
        daf.daf_decompress(p, bufs["packed"][1], bufs["bits"][1], bufs["mn"][1], bufs["scale"][1], bufs["woff"][1],
                           bufs["out"][1])
        torch.cuda.synchronize()
        for name, (full, inner) in bufs.items():
            assert bool((full[:pad] == 0xA5).all()) and bool((full[pad + inner.numel():] == 0xA5).all()), (beta, name)


@pytest.mark.parametrize("case", range(36))
def test_seeded_tie_heavy_configurations(case):
    """Few distinct ranges per window (integer-valued data): candidate raises collide on the same key all the
    time, so the order among equal keys (level, then group) decides most widths."""
    rng = np.random.default_rng(50000 + case)
    dtype = ("f32", "f16", "bf16")[case % 3]
    We = int(rng.choice([4096, 8192, 16384]))
    G = int(rng.choice([g for g in (32, 64, 128, 256, 512, 1024) if g <= We]))
    widths = tuple(sorted(rng.choice([1, 2, 4, 8], size=int(rng.integers(2, 5)), replace=False).tolist()))
    beta = min(float(min(widths) + rng.choice([0.25, 0.5, 1.0, 1.5, 2.0, 3.0])), 8.0)
    n_groups = int(rng.integers(1, 8 * We // G + 2))
    x = rng.integers(0, int(rng.integers(2, 7)), size=(n_groups, G)).astype(np.float32)
    x *= rng.choice([1.0, 2.0, 0.5, 3.0], size=(n_groups, 1)).astype(np.float32)
    if case % 4 == 0:
        x[rng.random(n_groups) < 0.3] = 1.0                       # constant groups
    a = x.reshape(-1)
    a = a if dtype == "f32" else (a.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a))
    label = f"ties/{case}/{dtype}/G{G}/We{We}/{widths}/{beta}"
    xd, c, ref = assert_compress_parity(a, dtype, G, widths, beta, window_elems=We, seed=case, label=label)
    assert_decompress_parity(c, ref, dtype, label)


# ---------------------------------------------------------------------------------------------------------------
# Bounded waits.  Nothing here faults, traps or spins without limit: a window (tile) that is never produced leaves
# its look-back descriptor empty, the kernels behind it poll a few thousand times, give up, record DAF_ERR_TIMEOUT,
# poison their own descriptors and return; the context stays usable.
# ---------------------------------------------------------------------------------------------------------------
HEADER_BYTES = 256                                                   # status, ticket, fail_window, fail_site, retry, ticket2, ...
_POISON = np.uint64(3) << np.uint64(62)


def _prepared_workspace(nbytes, ticket_word, first_ticket, poison_at=None, descriptors_at=HEADER_BYTES):
    """An all-zero workspace whose ticket counter starts at `first_ticket` (window / tile 0 is then never handed out),
    optionally with one pre-poisoned descriptor."""
    ws = np.zeros(nbytes, np.uint8)
    ws[4 * ticket_word:4 * ticket_word + 4] = np.array([first_ticket], np.uint32).view(np.uint8)
    if poison_at is not None:
        o = descriptors_at + 8 * poison_at
        ws[o:o + 8] = np.array([_POISON], np.uint64).view(np.uint8)
    return torch.from_numpy(ws).cuda()


@pytest.mark.parametrize("poisoned", [False, True])
def test_compress_look_back_gives_up_when_a_window_is_never_produced(poisoned):
    """The general kernel with its ticket counter started at 1: window 0 is never taken, so window 1's look-back
    finds an empty descriptor (and runs out), or a poisoned one (and stops at once, without a report of its own).
    Either way nothing is stored, the guard bands stay intact, and the next ordinary call succeeds."""
    n_windows, G, widths, beta = 8, 256, (1, 2, 4, 8), 3.0
    a = wl.generate(77, 0, wl.TensorSpec("t", (n_windows * 16384,), "f32", "logscale", 3))
    x = torch.from_numpy(a).cuda()
    flags = daf.FLAG_STREAM_NEVER | daf.FLAG_ONE_PASS | daf.FLAG_KEEP_WORKSPACE | daf.flag_poll_limit(3000)
    p = daf.make_params(daf.F32, x.numel(), G, widths, beta, seed=3, flags=flags)
    sz = daf.daf_sizes(p)
    guard = 4096
    packed = torch.full((sz.packed_capacity + guard,), 0xA5, dtype=torch.uint8, device="cuda")
    woff = torch.full((sz.n_windows + 1 + 8,), -1, dtype=torch.int64, device="cuda")
    c = daf.alloc_outputs(p, "cuda")
    # descriptors of the general kernel: the second array behind the header; ticket2 is 32-bit word 5 of the header
    ws = _prepared_workspace(sz.workspace, 5, 1, poison_at=0 if poisoned else None,
                             descriptors_at=HEADER_BYTES + 8 * sz.n_windows)
    daf.daf_compress(p, x, packed, sz.packed_capacity, c.bits, c.min, c.scale, woff, ws, sz.workspace)
    status = daf.daf_poll_status(ws)
    assert status == (daf.OK if poisoned else daf.ERR_TIMEOUT)
    torch.cuda.synchronize()
    assert bool((packed == 0xA5).all()), "a window behind the missing one was stored"
    assert bool((woff == -1).all()), "a window behind the missing one got an offset"
    d = ws[HEADER_BYTES + 8 * sz.n_windows:HEADER_BYTES + 16 * sz.n_windows].cpu().numpy().view(np.uint64)
    assert all(int(v) >> 62 == 3 for v in d[1:]), "every window behind the missing one must end up poisoned"
    # the context is fine: the same tensor through an ordinary call
    assert_compress_parity(a, "f32", G, widths, beta, seed=3, label="after a timed-out call")


@pytest.mark.parametrize("poisoned", [False, True])
def test_group_offsets_look_back_gives_up_when_a_tile_is_never_produced(poisoned):
    n_groups = 8192 * 6 + 100                                        # 7 tiles
    rng = np.random.default_rng(11)
    bits = rng.choice(np.array([1, 2, 4, 8], np.uint8), n_groups)
    d_bits = torch.from_numpy(bits).cuda()
    off = torch.full((n_groups + 1 + 8,), -1, dtype=torch.int64, device="cuda")
    nbytes = daf.daf_group_offsets_workspace(n_groups)
    ws = _prepared_workspace(nbytes, 1, 1, poison_at=0 if poisoned else None)   # the tile counter is word 1 of the header
    daf.daf_group_offsets_diag(d_bits, n_groups, 64, off, ws, nbytes, daf.FLAG_KEEP_WORKSPACE | daf.flag_poll_limit(3000))
    assert daf.daf_poll_status(ws) == (daf.OK if poisoned else daf.ERR_TIMEOUT)
    torch.cuda.synchronize()
    assert bool((off == -1).all()), "a tile behind the missing one wrote offsets"
    d = ws[HEADER_BYTES:HEADER_BYTES + 8 * 7].cpu().numpy().view(np.uint64)
    assert all(int(v) >> 62 == 3 for v in d[1:])
    # and the ordinary call on the same workspace is right
    daf.daf_group_offsets(d_bits, n_groups, 64, off, ws, nbytes)
    assert daf.daf_poll_status(ws) == daf.OK
    want = np.concatenate([[0], np.cumsum(bits.astype(np.uint64) * 8)])
    assert np.array_equal(off[:n_groups + 1].cpu().numpy().view(np.uint64), want)
