"""GPU parity at the benchmark's full sizes, in the launch configuration that is timed (one batched
call per set for workloads 2-4, single-tensor calls for the 2^30-element sweep): windows are
independent and the random stream is indexed by element, so the oracle checks sampled windows one by
one -- widths, min, scale, window offsets' differences, packed bytes and decoded values."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

WE = 16384


def _device_tensor(cfg, ti, spec):
    tdt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.int16}[spec.dtype]
    h = torch.empty(spec.numel, dtype=tdt, pin_memory=True)
    wl.generate(cfg, ti, spec, out=h.numpy().view(wl.np_dtype(spec.dtype)))
    d = h.cuda()
    return d.view(torch.bfloat16) if spec.dtype == "bf16" else d


def _host_slice(x, lo, hi, dtype):
    s = x[lo:hi]
    if dtype == "bf16":
        return s.view(torch.int16).cpu().numpy().view(np.uint16)
    return s.cpu().numpy()


def _check_window(x, y, o, w, wi, seed, label):
    """Window wi of one tensor: x input, y decoded output, o the compress outputs."""
    n, G = x.numel(), w.group_size
    lo, hi = wi * WE, min(n, (wi + 1) * WE)
    dtype = w.tensors[0].dtype
    a = _host_slice(x, lo, hi, dtype)
    ref = oracle.compress(a, G, w.widths, w.bit_budget, dtype=None if dtype != "bf16" else "bf16", seed=seed, base=lo)
    g0, g1 = lo // G, hi // G
    woff = o.window_offsets[wi:wi + 2].cpu().numpy().view(np.uint64)
    assert int(woff[1] - woff[0]) == ref.packed.size, label
    assert np.array_equal(o.bits[g0:g1].cpu().numpy(), ref.bits), label
    assert np.array_equal(o.min[g0:g1].cpu().numpy().view(np.uint32), ref.mn.view(np.uint32)), label
    assert np.array_equal(o.scale[g0:g1].cpu().numpy().view(np.uint32), ref.scale.view(np.uint32)), label
    assert np.array_equal(o.packed[int(woff[0]):int(woff[1])].cpu().numpy(), ref.packed), label
    want = oracle.decompress(ref)
    got = _host_slice(y, lo, hi, dtype)
    if dtype == "f32":
        d = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert d.max() <= 1, (label, int(d.max()))
    else:
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16)), label
    return ref


@pytest.mark.parametrize("cfg", [2, 3, 4])
def test_full_size_sets_through_one_batched_call(cfg):
    daf.lib()
    w = wl.workload(cfg)
    xs = [_device_tensor(cfg, i, t) for i, t in enumerate(w.tensors)]
    params = [daf.make_params(daf.dtype_code(x), x.numel(), w.group_size, w.widths, w.bit_budget, seed=t.philox_seed)
              for x, t in zip(xs, w.tensors)]
    outs = [daf.alloc_outputs(p, "cuda") for p in params]
    ys = [torch.empty_like(x) for x in xs]
    ws_bytes = daf.daf_batch_workspace(params)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    daf.daf_compress_batch(params, xs, [o.packed for o in outs], [o.sizes.packed_capacity for o in outs],
                           [o.bits for o in outs], [o.min for o in outs], [o.scale for o in outs],
                           [o.window_offsets for o in outs], ws, ws_bytes)
    assert daf.daf_poll_status(ws) == daf.OK
    daf.daf_decompress_batch(params, [o.packed for o in outs], [o.bits for o in outs], [o.min for o in outs],
                             [o.scale for o in outs], [o.window_offsets for o in outs], ys)
    torch.cuda.synchronize()
    rng = np.random.default_rng(cfg)
    picks = [(0, 0), (len(xs) - 1, outs[-1].sizes.n_windows - 1)]      # very first and very last window of the set
    for ti in range(len(xs)):                                          # the last (possibly ragged) window of every tensor
        picks.append((ti, outs[ti].sizes.n_windows - 1))
    for _ in range(64):                                                # and 64 at random
        ti = int(rng.integers(0, len(xs)))
        picks.append((ti, int(rng.integers(0, outs[ti].sizes.n_windows))))
    widths_seen = set()
    for ti, wi in sorted(set(picks)):
        ref = _check_window(xs[ti], ys[ti], outs[ti], w, wi, w.tensors[ti].philox_seed, f"cfg{cfg}/{w.tensors[ti].name}/w{wi}")
        widths_seen |= set(np.unique(ref.bits).tolist())
    if cfg == 2:
        assert widths_seen == {2, 4}                                   # half the groups of every window at 2 bits, half at 4
    # the whole set respects the budget
    total_bits = sum(int(o.window_offsets[-1].item()) for o in outs) * 8
    assert total_bits <= w.bit_budget * sum(x.numel() for x in xs)


def test_full_size_sweep_points():
    """All 16 (group size, budget) points on the 2^30-element tensor, 2 + 24 windows each."""
    daf.lib()
    w0 = wl.workload(5)
    x = _device_tensor(5, 0, w0.tensors[0])
    y = torch.empty_like(x)
    rng = np.random.default_rng(5)
    out = None
    for G in wl.SWEEP_GROUPS:
        for beta in wl.SWEEP_BUDGETS:
            w = wl.workload(5, group_size=G, bit_budget=beta)
            p = daf.make_params(daf.F32, x.numel(), G, w.widths, beta, seed=w.tensors[0].philox_seed)
            if out is None:                                            # sized for the largest outputs: G = 64, 8 bits
                out = daf.alloc_outputs(daf.make_params(daf.F32, x.numel(), 64, w.widths, 8.0), "cuda")
            sz = daf.daf_sizes(p)
            daf.daf_compress(p, x, out.packed, out.sizes.packed_capacity, out.bits, out.min, out.scale,
                             out.window_offsets, out.workspace, out.sizes.workspace)
            assert daf.daf_poll_status(out.workspace) == daf.OK
            daf.daf_decompress(p, out.packed, out.bits, out.min, out.scale, out.window_offsets, y)
            torch.cuda.synchronize()
            picks = {0, sz.n_windows - 1} | {int(v) for v in rng.integers(0, sz.n_windows, 24)}
            for wi in sorted(picks):
                _check_window(x, y, out, w, wi, w.tensors[0].philox_seed, f"cfg5/G{G}/b{beta}/w{wi}")
            assert int(out.window_offsets[sz.n_windows].item()) * 8 <= beta * x.numel()


def _host_threads():
    import os
    return max(1, min(32, os.cpu_count() or 1))


def test_full_tensor_headline_point():
    """The headline point (2^30 fp32 elements, groups of 256, 4 bits) compared with the oracle over the WHOLE tensor:
    every width, minimum, scale and window offset, the packed stream byte for byte, every decoded value.  The oracle
    runs over window-aligned shards on all host threads (windows are independent, the random stream is indexed by
    element)."""
    from concurrent.futures import ThreadPoolExecutor
    daf.lib()
    G, beta = 256, 4.0
    w = wl.workload(5, group_size=G, bit_budget=beta)
    x = _device_tensor(5, 0, w.tensors[0])
    n = x.numel()
    p = daf.make_params(daf.F32, n, G, w.widths, beta, seed=w.tensors[0].philox_seed)
    out = daf.alloc_outputs(p, "cuda")
    daf.daf_compress(p, x, out.packed, out.sizes.packed_capacity, out.bits, out.min, out.scale, out.window_offsets,
                     out.workspace, out.sizes.workspace)
    assert daf.daf_poll_status(out.workspace) == daf.OK
    y = torch.empty_like(x)
    daf.daf_decompress(p, out.packed, out.bits, out.min, out.scale, out.window_offsets, y)
    torch.cuda.synchronize()
    hx, hy = x.cpu().numpy(), y.cpu().numpy()
    bits, mn, sc = out.bits.cpu().numpy(), out.min.cpu().numpy(), out.scale.cpu().numpy()
    woff = out.window_offsets.cpu().numpy().view(np.uint64)
    packed = out.packed[:int(woff[-1])].cpu().numpy()
    del x, y
    shard = 1 << 22                                                   # 256 windows per shard

    def check(lo):
        hi = min(n, lo + shard)
        ref = oracle.compress(hx[lo:hi], G, w.widths, beta, seed=w.tensors[0].philox_seed, base=lo, want_codes=False)
        g0, g1, w0, w1 = lo // G, hi // G, lo // WE, (hi + WE - 1) // WE
        if not np.array_equal(bits[g0:g1], ref.bits):
            return f"widths differ in [{lo}, {hi})"
        if not np.array_equal(mn[g0:g1].view(np.uint32), ref.mn.view(np.uint32)):
            return f"minima differ in [{lo}, {hi})"
        if not np.array_equal(sc[g0:g1].view(np.uint32), ref.scale.view(np.uint32)):
            return f"scales differ in [{lo}, {hi})"
        if not np.array_equal(woff[w0:w1 + 1] - woff[w0], ref.window_offsets):
            return f"window offsets differ in [{lo}, {hi})"
        if not np.array_equal(packed[int(woff[w0]):int(woff[w1])], ref.packed):
            return f"packed bytes differ in [{lo}, {hi})"
        if not np.array_equal(hy[lo:hi].view(np.uint32), oracle.decompress(ref).view(np.uint32)):
            return f"decoded values differ in [{lo}, {hi})"
        return None

    with ThreadPoolExecutor(_host_threads()) as ex:
        bad = [r for r in ex.map(check, range(0, n, shard)) if r]
    assert not bad, bad[:3]
    assert int(woff[0]) == 0 and int(woff[-1]) * 8 <= beta * n


def test_full_tensor_widths_and_offsets_of_all_sweep_points():
    """The other sweep points: the oracle's statistics and bit choice over the FULL tensor (every width, minimum, scale
    and window offset); their packed bytes and decoded values are covered on sampled windows by
    test_full_size_sweep_points."""
    from concurrent.futures import ThreadPoolExecutor
    daf.lib()
    w0 = wl.workload(5)
    x = _device_tensor(5, 0, w0.tensors[0])
    n = x.numel()
    hx = x.cpu().numpy()
    out = None
    shard = 1 << 24
    for G in wl.SWEEP_GROUPS:
        # statistics do not depend on the budget: once per group size, on all host threads
        def ranges(lo):
            m, _, R = oracle.stats(hx[lo:lo + shard], G)
            return m, R
        with ThreadPoolExecutor(_host_threads()) as ex:
            parts = list(ex.map(ranges, range(0, n, shard)))
        ref_mn = np.concatenate([m for m, _ in parts])
        ref_R = np.concatenate([r for _, r in parts])
        for beta in wl.SWEEP_BUDGETS:
            if (G, beta) == (256, 4):
                continue                                              # compared in full above
            w = wl.workload(5, group_size=G, bit_budget=beta)
            p = daf.make_params(daf.F32, n, G, w.widths, beta, seed=w.tensors[0].philox_seed)
            if out is None:                                           # sized for the largest outputs: G = 64, 8 bits
                out = daf.alloc_outputs(daf.make_params(daf.F32, n, 64, w.widths, 8.0), "cuda")
            sz = daf.daf_sizes(p)
            daf.daf_compress(p, x, out.packed, out.sizes.packed_capacity, out.bits, out.min, out.scale,
                             out.window_offsets, out.workspace, out.sizes.workspace)
            assert daf.daf_poll_status(out.workspace) == daf.OK
            torch.cuda.synchronize()
            with ThreadPoolExecutor(_host_threads()) as ex:          # window-aligned shards of groups
                gs = shard // G
                ref_bits = np.concatenate(list(ex.map(
                    lambda g0: oracle.choose_bits(ref_R[g0:g0 + gs], WE // G, w.widths, beta), range(0, n // G, gs))))
            ref_scale = oracle.group_params(ref_R, ref_bits)[0]
            label = f"cfg5/G{G}/b{beta}"
            assert np.array_equal(out.bits[:sz.n_groups].cpu().numpy(), ref_bits), label
            assert np.array_equal(out.min[:sz.n_groups].cpu().numpy().view(np.uint32), ref_mn.view(np.uint32)), label
            assert np.array_equal(out.scale[:sz.n_groups].cpu().numpy().view(np.uint32), ref_scale.view(np.uint32)), label
            goff = oracle.offsets(ref_bits, G)                        # byte offset of every group, and the total
            ref_woff = np.concatenate([goff[:-1:WE // G], goff[-1:]])
            assert np.array_equal(out.window_offsets[:sz.n_windows + 1].cpu().numpy().view(np.uint64), ref_woff), label
