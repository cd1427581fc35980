"""World-size-2 gloo test (CPU): sharding a tensor by whole windows, one shard per rank with its
element index base, reproduces the unsharded result byte for byte -- no exchange step on the path."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2507_07149_b200 import workloads as wl

G, WE, WIDTHS, BETA, SEED = 64, 4096, (1, 2, 4, 8), 3.0, 7
N = WE * 9 + G * 5                                             # ragged last window


def _data():
    rng = np.random.default_rng(3)
    return (rng.standard_normal(N) * np.repeat(10.0 ** rng.uniform(-1, 1, N // G), G)).astype(np.float32)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = _data()
    lo, hi = wl.shard_range(N, WE, rank, world)
    c = oracle.compress(x[lo:hi], G, WIDTHS, BETA, window_elems=WE, seed=SEED, base=lo)
    parts = [None] * world
    dist.all_gather_object(parts, (lo, hi, c.packed.tobytes(), c.bits.tobytes(), int(c.window_offsets[-1])))
    if rank == 0:
        full = oracle.compress(x, G, WIDTHS, BETA, window_elems=WE, seed=SEED)
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == N
        assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
        assert b"".join(p[2] for p in parts) == full.packed.tobytes()
        assert b"".join(p[3] for p in parts) == full.bits.tobytes()
        assert sum(p[4] for p in parts) == int(full.window_offsets[-1])
        out.put("ok")
    dist.barrier()
    dist.destroy_process_group()


def test_window_aligned_shards_reproduce_the_unsharded_bytes():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out.get(timeout=5) == "ok"


def test_shard_ranges_cover_the_tensor_in_whole_windows():
    for numel, world in ((WE * 9 + 5 * G, 2), (WE * 3, 4), (WE, 8), (WE * 16, 8)):
        cuts = [wl.shard_range(numel, WE, r, world) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == numel
        for (a, b), (c, d) in zip(cuts, cuts[1:]):
            assert b == c and a % WE == 0


def test_daf_shard_cuts_where_the_generator_of_the_bench_does():
    """The library's own sharding call against the window arithmetic written out here: whole windows, as even as
    possible, in order; bases move with the slices; ranks beyond the windows get nothing."""
    import paper_2507_07149_b200 as daf
    for numel, we, G in ((16384 * 10 + 256 * 3, 0, 256), (4096 * 7, 4096, 64), (16384, 0, 1024), (8192 * 5 + 128, 8192, 128)):
        WE_ = we or 16384
        p = daf.make_params(daf.F32, numel, G, (1, 2, 4, 8), 4.0, window_elems=we, seed=9, elem_index_base=8 * 5)
        for world in (1, 2, 3, 8, 64):
            at = 0
            for rank in range(world):
                shard, first = daf.daf_shard(p, rank, world)
                lo, hi = wl.shard_range(numel, WE_, rank, world)
                assert (first, int(shard.numel)) == (lo, hi - lo) and first == at
                assert int(shard.elem_index_base) == 40 + lo and int(shard.seed) == 9 and int(shard.group_size) == G
                assert lo % WE_ == 0 or lo == numel
                at += int(shard.numel)
            assert at == numel
    with pytest.raises(daf.DafError):
        daf.daf_shard(p, 3, 3)
    with pytest.raises(daf.DafError):
        daf.daf_shard(p, 0, 0)
