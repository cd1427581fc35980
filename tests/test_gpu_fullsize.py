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
