"""GPU parity of the two-width streaming kernel (a budget between two allowed widths, Sec. 3.4.1's greedy in closed
form: the k groups of a window with the largest ranges are raised once more) against the CPU oracle.  The general parity
suite already sends every such call through it (the tests ask for the streaming kernels whatever the call's size);
here: calls it must FINISH (the fallback is not asked for: word 4 of the workspace header, `retry`, stays 0), calls it
must give up on, ties, constant groups, ragged last windows, batched calls."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

from gpu_util import assert_compress_parity, assert_decompress_parity, to_device

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _as(a32, dtype):
    return a32 if dtype == "f32" else (a32.astype(np.float16) if dtype == "f16" else wl.f32_to_bf16_bits(a32))


def _retry_word(c):
    return int(c.workspace[16:20].cpu().numpy().view(np.uint32)[0])


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("G", [256, 512, 1024])
@pytest.mark.parametrize("widths,beta", [((1, 2, 4, 8), 3.0), ((1, 2, 4, 8), 2.5), ((1, 2, 4, 8), 1.25), ((2, 4, 8), 5.0),
                                         ((2, 4, 8), 3.0), ((1, 8), 4.0), ((1, 2, 4, 8), 7.5)])
def test_windows_of_two_widths_are_finished_by_the_streaming_kernel(dtype, G, widths, beta):
    """Ranges within a factor of two of each other: the levels never interleave.  Several whole windows and a ragged
    last one whose group count leaves a different remainder of the budget."""
    rng = np.random.default_rng(G + len(widths) + int(beta * 4))
    n = 16384 * 5 + G * (3 if G < 1024 else 5)
    scale = rng.uniform(1.0, 2.0, n // G)
    a = _as((rng.uniform(-1, 1, n) * np.repeat(scale, G)).astype(np.float32), dtype)
    label = f"two-width/{dtype}/G{G}/{widths}/{beta}"
    # (a shard of a larger tensor: the Philox counters start at a large element index)
    x, c, ref = assert_compress_parity(a, dtype, G, widths, beta, seed=G + 7, base=8 * ((1 << 33) + 4099), label=label)
    assert _retry_word(c) == 0, "the two-width kernel gave up on windows it should finish"
    assert len(np.unique(ref.bits)) == 2
    assert_decompress_parity(c, ref, dtype, label)


@pytest.mark.parametrize("G", [256, 1024])
def test_equal_ranges_are_raised_in_index_order(G):
    """Every group holds the same values: all keys tie, and the groups raised are the first k of each window."""
    n = 16384 * 3 + G * 2
    block = np.linspace(-1.0, 1.0, G, dtype=np.float32)
    a = np.tile(block, n // G)
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, seed=1, label=f"ties/G{G}")
    assert _retry_word(c) == 0
    per = 16384 // G
    first = ref.bits[:per]
    assert list(first) == [4] * (per // 2) + [2] * (per - per // 2)
    # two distinct ranges, interleaved: the larger ones first, then the smaller ones in index order
    b = a.copy().reshape(-1, G)
    b[::3] *= np.float32(1.5)
    x, c, ref = assert_compress_parity(b.reshape(-1), "f32", G, (1, 2, 4, 8), 3.0, seed=2, label=f"two ranges/G{G}")
    assert _retry_word(c) == 0
    assert_decompress_parity(c, ref, "f32", f"two ranges/G{G}")


def test_constant_groups():
    """Groups of range zero have key zero and are raised last.  With two allowed widths (no level below the budget's
    own, none above the next) the streaming kernel finishes such windows; with more levels it hands the call over: a
    raise of key zero sorts behind every raise of the level above."""
    rng = np.random.default_rng(4)
    G, n = 256, 16384 * 4
    a = (rng.uniform(-1, 1, n) * np.repeat(rng.uniform(1.0, 1.5, n // G), G)).astype(np.float32).reshape(-1, G)
    a[5::7] = np.float32(0.25)                                    # constant groups: 9 or 10 of a window's 64
    a = a.reshape(-1)
    # 60 of 64 groups are raised: all that have a range and some that have none (no level below, none above)
    x, c, ref = assert_compress_parity(a, "f32", G, (2, 4), 3.9, seed=5, label="constant groups, bottom level")
    assert _retry_word(c) == 0 and set(np.unique(ref.bits)) == {2, 4}
    assert int((ref.bits.reshape(-1, 64)[0] == 4).sum()) == 60 and bool((ref.scale[ref.bits == 4] == 0).any())
    assert_decompress_parity(c, ref, "f32", "constant groups, bottom level")
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, seed=5, label="constant groups, a level below")
    assert _retry_word(c) == 1
    assert_decompress_parity(c, ref, "f32", "constant groups, a level below")


@pytest.mark.parametrize("where", ["first window", "a window far into the tensor", "the ragged last window"])
def test_one_window_of_interleaving_levels_sends_the_call_to_the_fallback(where):
    rng = np.random.default_rng(6)
    G, n_win = 256, 700                                           # more windows than the device holds CTAs
    n = 16384 * n_win + G * 9
    a = rng.uniform(-1, 1, n).astype(np.float32)
    lo = {"first window": 0, "a window far into the tensor": 431 * 16384, "the ragged last window": n_win * 16384}[where]
    hi = min(lo + 16384, n)
    a[lo:hi] *= np.repeat(10.0 ** rng.uniform(-3, 3, (hi - lo) // G), G).astype(np.float32)
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, seed=8, label=f"give up/{where}")
    assert _retry_word(c) == 1 and len(np.unique(ref.bits)) >= 3
    assert_decompress_parity(c, ref, "f32", f"give up/{where}")
    # right afterwards, on fresh outputs, a call the kernel finishes
    u = rng.uniform(-1, 1, 16384 * 20).astype(np.float32)
    x, c, ref = assert_compress_parity(u, "f32", G, (1, 2, 4, 8), 3.0, seed=9, label="after a given-up call")
    assert _retry_word(c) == 0


def test_a_range_that_needs_the_clamp_sends_the_call_to_the_fallback():
    rng = np.random.default_rng(7)
    G, n = 512, 16384 * 6
    a = rng.uniform(-1.6e38, 1.6e38, n).astype(np.float32)       # every range above 2^126, all within a factor of two
    a.reshape(-1, G)[:, 0] = np.float32(-1.6e38)
    a.reshape(-1, G)[:, 1] = np.float32(1.6e38)
    x, c, ref = assert_compress_parity(a, "f32", G, (1, 2, 4, 8), 3.0, seed=3, label="clamp")
    assert _retry_word(c) == 1
    assert_decompress_parity(c, ref, "f32", "clamp")


def test_batched_call_and_policy_flags():
    """Tensors of different lengths in one batched call; the same tensor with the streaming kernels switched off."""
    rng = np.random.default_rng(12)
    G = 256
    sizes = [16384 * 3 + G * 5, 16384, 16384 * 7, G * 9]
    arrays = [(rng.uniform(-1, 1, n) * np.repeat(rng.uniform(1, 2, n // G), G)).astype(np.float32) for n in sizes]
    xs = [to_device(a, "f32") for a in arrays]
    params = [daf.make_params(daf.F32, x.numel(), G, (1, 2, 4, 8), 3.0, seed=100 + i) for i, x in enumerate(xs)]
    outs = [daf.alloc_outputs(p, "cuda") for p in params]
    ws_bytes = daf.daf_batch_workspace(params)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    daf.daf_compress_batch(params, xs, [o.packed for o in outs], [o.sizes.packed_capacity for o in outs], [o.bits for o in outs],
                           [o.min for o in outs], [o.scale for o in outs], [o.window_offsets for o in outs], ws, ws_bytes)
    assert daf.daf_poll_status(ws) == daf.OK
    assert int(ws[16:20].cpu().numpy().view(np.uint32)[0]) == 0
    for i, (a, o) in enumerate(zip(arrays, outs)):
        ref = oracle.compress(a, G, (1, 2, 4, 8), 3.0, seed=100 + i)
        total = int(o.window_offsets[-1])
        assert total == ref.packed.size and np.array_equal(o.packed[:total].cpu().numpy(), ref.packed), f"tensor {i}"
        assert np.array_equal(o.bits.cpu().numpy(), ref.bits) and np.array_equal(o.window_offsets.cpu().numpy().astype(np.uint64), ref.window_offsets.astype(np.uint64))
        assert np.array_equal(o.min.cpu().numpy().view(np.uint32), ref.mn.view(np.uint32))
        assert np.array_equal(o.scale.cpu().numpy().view(np.uint32), ref.scale.view(np.uint32))
    # the first tensor alone, streaming kernels off: the same bytes from the general kernel
    p = daf.make_params(daf.F32, xs[0].numel(), G, (1, 2, 4, 8), 3.0, seed=100, flags=daf.FLAG_STREAM_NEVER)
    c = daf.alloc_outputs(p, "cuda")
    daf.daf_compress(p, xs[0], c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace, c.sizes.workspace)
    total = int(c.window_offsets[-1])
    assert torch.equal(c.packed[:total], outs[0].packed[:total]) and torch.equal(c.bits, outs[0].bits)
