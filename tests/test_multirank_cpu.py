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
