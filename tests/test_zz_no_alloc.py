"""The workspace-free compress entry point, for callers that cannot allocate scratch memory
(a job whose device memory is fully committed to its own arena, code running inside an allocator
callback): it must produce exactly what daf_compress produces, call after call, although every
call reuses the same fixed scratch array inside the library.  Collected last on purpose."""
import numpy as np
import pytest

import oracle
import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import workloads as wl

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _outputs(params):
    sz = daf.daf_sizes(params)
    dev = "cuda"
    return dict(packed=torch.zeros(max(sz.packed_capacity, 16), dtype=torch.uint8, device=dev),
                bits=torch.zeros(sz.n_groups, dtype=torch.uint8, device=dev),
                mn=torch.zeros(sz.n_groups, dtype=torch.float32, device=dev),
                scale=torch.zeros(sz.n_groups, dtype=torch.float32, device=dev),
                woff=torch.zeros(sz.n_windows + 1, dtype=torch.int64, device=dev)), sz


def test_static_scratch_entry_point_matches_daf_compress_on_two_calls_in_a_row():
    # two different tensors, the second smaller and of another dtype: the second call finds the first one's leftovers
    cases = [(wl.TensorSpec("a", (16384 * 37 + 256 * 11,), "f32", "logscale", 5), 256, (1, 2, 4, 8), 3.0),
             (wl.TensorSpec("b", (16384 * 5 + 128 * 3,), "bf16", "t3_outliers", 9), 128, (2, 4, 8), 4.0)]
    for k, (spec, G, widths, beta) in enumerate(cases):
        a = wl.generate(90, k, spec)
        x = torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16) if spec.dtype == "bf16" else torch.from_numpy(a).cuda()
        params = daf.make_params(daf.dtype_code(x), x.numel(), G, widths, beta, seed=spec.philox_seed)
        ref, sz = _outputs(params)
        ws = torch.empty(sz.workspace, dtype=torch.uint8, device="cuda")
        daf.daf_compress(params, x, ref["packed"], sz.packed_capacity, ref["bits"], ref["mn"], ref["scale"], ref["woff"],
                         ws, sz.workspace)
        assert daf.daf_poll_status(ws) == daf.OK
        got, _ = _outputs(params)
        status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        # the call must not allocate: neither through torch's allocator nor behind its back
        held, (free, _) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
        daf.daf_compress_static(params, x, got["packed"], sz.packed_capacity, got["bits"], got["mn"], got["scale"],
                                got["woff"], status if k == 0 else None)     # the status word is optional
        torch.cuda.synchronize()
        if k > 0:                                                     # (the first call on a device may load the kernels)
            assert torch.cuda.memory_allocated() == held and torch.cuda.mem_get_info()[0] == free
        else:
            assert int(status.item()) == daf.OK
        total = int(ref["woff"][-1].item())
        assert total > 0 and torch.equal(got["woff"], ref["woff"])
        assert torch.equal(got["bits"], ref["bits"])
        assert torch.equal(got["mn"].view(torch.int32), ref["mn"].view(torch.int32))          # bit-exact, as everywhere
        assert torch.equal(got["scale"].view(torch.int32), ref["scale"].view(torch.int32))
        assert torch.equal(got["packed"][:total], ref["packed"][:total])
        # and against the CPU oracle, like every other entry point
        want = oracle.compress(a, G, widths, beta, dtype="bf16" if spec.dtype == "bf16" else None, seed=spec.philox_seed)
        assert np.array_equal(got["bits"].cpu().numpy(), want.bits)
        assert np.array_equal(got["mn"].cpu().numpy().view(np.uint32), want.mn.view(np.uint32))
        assert np.array_equal(got["scale"].cpu().numpy().view(np.uint32), want.scale.view(np.uint32))
        assert np.array_equal(got["woff"].cpu().numpy().view(np.uint64), want.window_offsets)
        assert total == want.packed.size and np.array_equal(got["packed"][:total].cpu().numpy(), want.packed)


def test_static_scratch_entry_point_rejects_tensors_beyond_its_fixed_size():
    n = (daf.STATIC_MAX_WINDOWS + 1) * 16384
    params = daf.make_params(daf.F32, n, 256, (4,), 4.0)
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(daf.DafError) as e:
        daf.daf_compress_static(params, dummy, dummy, 16, dummy, dummy, dummy, dummy)
    assert e.value.status == daf.ERR_CAPACITY
