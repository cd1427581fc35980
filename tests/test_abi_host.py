"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares,
validates arguments on the host, and the page pool keeps its books.  Nothing is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2507_07149_b200 as daf
from paper_2507_07149_b200 import build as daf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    daf_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "daf.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(daf_[a-z_0-9]+)\s*\(", header))
    assert declared == set(daf.SIGNATURES), declared ^ set(daf.SIGNATURES)
    handle = ctypes.CDLL(daf.LIB_PATH)
    for name in declared:
        assert hasattr(handle, name), name
    assert daf.daf_version() >= 0x000100
    assert daf.daf_status_string(daf.ERR_CAPACITY)


def test_params_struct_layout():
    assert ctypes.sizeof(daf.daf_params) == 56


def test_sizes_and_host_validation():
    import oracle
    p = daf.make_params(daf.F32, 16384 * 5 + 256 * 3, 256, (1, 2, 4, 8), 3.0)
    s = daf.daf_sizes(p)
    assert (s.n_groups, s.n_windows) == (64 * 5 + 3, 6)
    assert s.packed_capacity == oracle.packed_capacity(p.numel, 256, 16384, 3.0)
    assert s.workspace >= 256 + 8 * 6
    for G, We, beta in ((64, 4096, 2.5), (32, 16384, 8.0), (16384, 16384, 1.0), (128, 8192, 4.99)):
        n = We * 3 + G
        q = daf.make_params(daf.BF16, n, G, (1, 2, 4, 8), beta, window_elems=We)
        assert daf.daf_sizes(q).packed_capacity == oracle.packed_capacity(n, G, We, beta)

    # a budget above the largest width buys nothing: sizes are those of the largest width
    n = 16384 * 2 + 512
    for widths, top in (((1, 2, 4, 8), 8), ((1, 2, 4), 4), ((2,), 2)):
        big = daf.daf_sizes(daf.make_params(daf.F32, n, 256, widths, 12.0))
        at_top = daf.daf_sizes(daf.make_params(daf.F32, n, 256, widths, float(top)))
        assert big.packed_capacity == at_top.packed_capacity == n * top // 8

    def status(**kw):
        args = dict(dtype=daf.F32, numel=16384, group_size=256, widths=(2, 4, 8), bit_budget=4.0)
        args.update(kw)
        q = daf.make_params(args.pop("dtype"), args.pop("numel"), args.pop("group_size"), args.pop("widths"),
                            args.pop("bit_budget"), **args)
        try:
            daf.daf_sizes(q)
            return daf.OK
        except daf.DafError as e:
            return e.status

    assert status() == daf.OK
    assert status(group_size=48) == daf.ERR_INVALID_ARG            # not a power of two
    assert status(group_size=16) == daf.ERR_INVALID_ARG            # below 32
    assert status(group_size=32768) == daf.ERR_INVALID_ARG         # larger than the window
    assert status(numel=1000) == daf.ERR_SHAPE
    assert status(numel=0) == daf.ERR_SHAPE
    assert status(widths=()) == daf.ERR_INVALID_ARG
    assert status(widths=(3,)) == daf.ERR_INVALID_ARG
    assert status(bit_budget=1.5) == daf.ERR_BUDGET                 # below the smallest width
    assert status(window_elems=2048) == daf.ERR_UNSUPPORTED
    assert status(window_elems=5000) == daf.ERR_INVALID_ARG
    assert status(elem_index_base=4) == daf.ERR_INVALID_ARG
    # launch-policy flags: each alone and sensible pairs are fine, contradictory pairs and unknown bits are not
    for ok in (daf.FLAG_STREAM_ALWAYS, daf.FLAG_STREAM_NEVER, daf.FLAG_ONE_PASS, daf.FLAG_TWO_PASS, daf.FLAG_KEEP_WORKSPACE,
               daf.FLAG_STREAM_NEVER | daf.FLAG_TWO_PASS, daf.FLAG_STREAM_ALWAYS | daf.FLAG_ONE_PASS | daf.flag_poll_limit(100)):
        assert status(flags=ok) == daf.OK
    for bad_flags in (daf.FLAG_STREAM_ALWAYS | daf.FLAG_STREAM_NEVER, daf.FLAG_ONE_PASS | daf.FLAG_TWO_PASS, 0x20, 0x40, 0x80):
        assert status(flags=bad_flags) == daf.ERR_INVALID_ARG
    bad = daf.make_params(daf.F32, 16384, 256, (4,), 4.0)
    bad.struct_size = 8
    with pytest.raises(daf.DafError):
        daf.daf_sizes(bad)


def test_null_pointers_are_rejected_before_any_launch():
    p = daf.make_params(daf.F32, 16384, 256, (4,), 4.0)
    rc = daf.lib().daf_compress(ctypes.byref(p), None, None, 0, None, None, None, None, None, 0, None)
    assert rc == daf.ERR_INVALID_ARG
    rc = daf.lib().daf_decompress(ctypes.byref(p), None, None, None, None, None, None, None, 0, None)
    assert rc == daf.ERR_INVALID_ARG
    assert daf.lib().daf_group_offsets(None, 10, 256, None, None, 0, None) == daf.ERR_INVALID_ARG
    assert daf.lib().daf_poll_status(None, None) == daf.ERR_INVALID_ARG


def test_pool_first_fit_and_eviction():
    pool = daf.Pool(16 * 65536)
    a, off_a = pool.alloc(3 * 65536, importance=5.0)
    b, off_b = pool.alloc(65536 + 1, importance=1.0)                # two pages
    c, off_c = pool.alloc(4 * 65536, importance=9.0)
    assert (off_a, off_b, off_c) == (0, 3 * 65536, 5 * 65536)
    st = pool.stats()
    assert st["pages_used"] == 9 and st["live_allocations"] == 3 and st["largest_free_run_pages"] == 7
    pool.free(b)
    d, off_d = pool.alloc(65536, importance=2.0)                    # first fit reuses the lowest hole
    assert off_d == 3 * 65536
    e, off_e = pool.alloc(8 * 65536, importance=1.0)                # no run of 8 pages is free
    assert e == 0 and off_e is None
    # lowest importance per byte goes first: d (2 / 64Ki) < a (5 / 192Ki)?  no: a is lower per byte
    first = pool.evict_lowest()
    assert first == a
    assert pool.evict_lowest() == d
    assert pool.evict_lowest() == c
    assert pool.evict_lowest() == 0
    assert pool.stats()["evictions"] == 3 and pool.stats()["pages_used"] == 0
    with pytest.raises(daf.DafError):
        pool.free(12345)
    pool.close()


def test_training_integration_leaves_cpu_tensors_alone():
    """Host logic of the autograd integration: what does not qualify (here: CPU tensors) never reaches the
    library and is saved / computed as usual."""
    torch = pytest.importorskip("torch")
    from paper_2507_07149_b200.autograd import CompressedReLU, saved_activation_compression
    x = torch.randn(1 << 15, requires_grad=True)
    ctx = saved_activation_compression(min_numel=1024)
    with ctx:
        y = x.pow(2).sum()
    y.backward()
    assert ctx.stats["tensors"] == 0 and ctx.stats["passed_through"] >= 1
    assert torch.equal(x.grad, 2 * x.detach())
    layer = CompressedReLU(min_numel=1024)
    z = torch.randn(1 << 15, requires_grad=True)
    layer(z).sum().backward()
    assert torch.equal(z.grad, (z.detach() > 0).float())
    ctx.reseed(5)
    layer.reseed(5)
    assert ctx.seed == 5 and layer.seed == 5 and ctx._next_index == 0 and layer._next_index == 0
