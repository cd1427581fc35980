#!/usr/bin/env python
"""Benchmark of the activation compress / decompress hot path on B200.

One step = daf_compress followed by daf_decompress of one synthetic tensor (the whole hot
path).  Default workload: the 4 GiB fp32 Laplace tensor of the bandwidth sweep at group size
256 and a budget of 4 bits (widths {1,2,4,8}).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--group G] [--budget B] [--numel N]
  python bench.py --impl reference ...      # times the CPU oracle on a bounded sample
Under torchrun every rank compresses its own tensor (weak scaling, no collective on the path).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress+decompress throughput (uncompressed bytes)"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per element seen by ncu (dram__bytes_read.sum + dram__bytes_write.sum) for one launch
# on a 2^27-element fp32 slice of this workload (G = 256, budget 4): profiles/stream_compress_kernel_cfg5_G256_b4.md
# (546.50 MB read + 66.13 MB written) and profiles/decompress_kernel_cfg5_G256_b4.md (71.91 + 477.73 MB).
# Traffic grows in proportion to the element count, so it is scaled to the launch being timed.
NCU_TRAFFIC_BYTES_PER_ELEM = {"compress": 603.02e6 / (1 << 27), "decompress": 549.75e6 / (1 << 27)}
# (The decompress capture is a 512 MiB output: part of its stores still sits in L2 when the kernel ends, so the scaled
# figure understates the traffic of a full-size launch by the same amount.)
KERNEL_NAME = {"compress": "stream_compress_kernel", "decompress": "decompress_few_groups_kernel"}
# Kernels of this library launched per step on this workload: the streaming compress kernel, its verify kernel, the
# general compress kernel (which finds nothing to redo and returns), the decompress kernel.
LAUNCHES_PER_STEP = 4


def config_of(w, numel, dtype, G, beta, widths):
    """The `config` object of the JSON line: the same keys for the CUDA arm and the reference arm."""
    return {"workload": f"{w.name} ({numel} {dtype} Laplace(0,1) elements per GPU)",
            "numel_per_gpu": numel, "group_size": G, "bit_budget": beta, "widths": list(widths),
            "window_elems": 16384,
            "l2": "inputs (4 GiB) far exceed the 126 MB L2; no flush needed"}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--group", type=int, default=256)
    ap.add_argument("--budget", type=float, default=4.0)
    ap.add_argument("--numel", type=int, default=1 << 30)
    ap.add_argument("--dtype", default="f32", choices=["f32", "f16", "bf16"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--e2e-chunk", type=int, default=1 << 25, help="elements per chunk of the streamed end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(numel: int, itemsize: int, packed_bytes: int, G: int, n_windows: int) -> int:
    """Bytes a perfect implementation moves: the tensor once, the packed codes once, 9 bytes of
    metadata per group (width, min, scale) and 8 per window (offset).  Same for both directions."""
    return numel * itemsize + packed_bytes + 9 * (numel // G) + 8 * (n_windows + 1)


class ClockSampler:
    """Polls SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005, uuid: str = ""):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode() if uuid and not uuid.startswith("GPU-") else uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nvml = None

    def _run(self):
        n = self.nvml
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(int(n.nvmlDeviceGetClockInfo(self.h, n.NVML_CLOCK_SM)))
                try:
                    r = int(n.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nvml is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------------- CPU oracle timing
def oracle_sample(spec, cfg, sample_elems: int):
    from paper_2507_07149_b200 import workloads as wl
    sample_elems = min(sample_elems, spec.numel)
    return wl.generate(cfg, 0, spec, start=0, count=sample_elems)


def time_oracle(a, spec, G, widths, beta, threads: int):
    """Compress + decompress a window-aligned sample with the oracle as it stands, split into
    independent window-aligned shards over `threads` host threads (ctypes releases the GIL)."""
    from concurrent.futures import ThreadPoolExecutor
    import oracle
    oracle.build()
    n = a.size
    shard = max(16384, (n // threads) // 16384 * 16384)
    starts = list(range(0, n, shard))
    kw = {"dtype": "bf16"} if spec.dtype == "bf16" else {}

    def work(lo):
        hi = min(n, lo + shard)
        c = oracle.compress(a[lo:hi], G, widths, beta, seed=0, base=lo, want_codes=False, **kw)
        oracle.decompress(c)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(work, starts))
    dt = time.perf_counter() - t0
    return 2 * n * spec.itemsize / dt / 1e9, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2507_07149_b200 import workloads as wl
    w = wl.workload(5, numel=args.numel, group_size=args.group, bit_budget=args.budget)
    spec = wl.TensorSpec(w.tensors[0].name, w.tensors[0].shape, args.dtype, "laplace", 0)
    threads = os.cpu_count() or 1
    a = oracle_sample(spec, 5, 1 << 24)
    vals = []
    for i in range(args.warmup + args.steps):
        gbs, dt = time_oracle(a, spec, args.group, w.widths, args.budget, threads)
        if i >= args.warmup:
            vals.append((gbs, dt))
    v = float(np.mean([g for g, _ in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": float(np.mean([d for _, d in vals]) * 1e3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
            "config": config_of(w, args.numel, args.dtype, args.group, args.budget, w.widths),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"first {a.size} elements of the tensor per step (a bounded sample of the workload "
                                       "named in config), compress+decompress"},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------- CUDA arm
def run_cuda(args):
    import torch
    import paper_2507_07149_b200 as daf
    from paper_2507_07149_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if not os.path.exists(daf.LIB_PATH):
        if local == 0:
            from paper_2507_07149_b200 import build as daf_build
            daf_build.build()
        if dist is not None:
            dist.barrier()
    daf.lib()

    w = wl.workload(5, numel=args.numel, group_size=args.group, bit_budget=args.budget)
    spec = wl.TensorSpec(w.tensors[0].name, w.tensors[0].shape, args.dtype, "laplace", 0)
    G, widths, beta = w.group_size, w.widths, w.bit_budget
    tdt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[args.dtype]

    # synthetic input drawn into pinned host memory (rank r draws tensor index r), then resident in HBM
    h_in = torch.empty(spec.numel, dtype=tdt if args.dtype != "bf16" else torch.int16, pin_memory=True)
    wl.generate(5, rank, spec, out=h_in.numpy().view(wl.np_dtype(args.dtype)))
    if args.dtype == "bf16":
        h_in = h_in.view(torch.bfloat16)
    x = h_in.cuda(non_blocking=True)
    params = daf.make_params(daf.dtype_code(x), spec.numel, G, widths, beta, seed=0)
    c = daf.alloc_outputs(params, x.device)
    y = torch.empty_like(x)
    torch.cuda.synchronize()

    def step():
        daf.daf_compress(params, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                         c.workspace, c.sizes.workspace)
        daf.daf_decompress(params, c.packed, c.bits, c.min, c.scale, c.window_offsets, y)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert daf.daf_poll_status(c.workspace) == daf.OK
    packed_bytes = c.packed_bytes()

    # ---- timed region: device-resident inputs, CUDA events on the launching stream
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    sampler = ClockSampler(local, uuid=str(getattr(torch.cuda.get_device_properties(local), "uuid", "")))
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    for k in range(K):
        ev[k][0].record()
        daf.daf_compress(params, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                         c.workspace, c.sizes.workspace)
        ev[k][1].record()
        daf.daf_decompress(params, c.packed, c.bits, c.min, c.scale, c.window_offsets, y)
        ev[k][2].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if dist is not None:
        dist.barrier()
    total_ms = ev[0][0].elapsed_time(ev[K - 1][2])
    t_c = np.array([ev[k][0].elapsed_time(ev[k][1]) for k in range(K)])
    t_d = np.array([ev[k][1].elapsed_time(ev[k][2]) for k in range(K)])
    if dist is not None:
        t = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    assert daf.daf_poll_status(c.workspace) == daf.OK

    nbytes = spec.numel * spec.itemsize
    value = world * 2 * nbytes * K / (total_ms * 1e-3) / 1e9
    alg = algorithmic_bytes(spec.numel, spec.itemsize, packed_bytes, G, c.sizes.n_windows)
    peak, peak_src = measured_peak()
    dom = "compress" if t_c.mean() >= t_d.mean() else "decompress"
    dom_ms = float(max(t_c.mean(), t_d.mean()))
    # the ncu traffic figure was captured at fp32, G = 256, budget 4: use it for that configuration only
    profiled = args.dtype == "f32" and G == 256 and beta == 4.0

    def roof(kernel, ms):
        a = alg / (ms * 1e-3) / 1e9
        tr = NCU_TRAFFIC_BYTES_PER_ELEM[kernel] if profiled else None
        name = KERNEL_NAME[kernel]
        if kernel == "decompress" and G < 256:
            name = "decompress_kernel"                            # (groups below 256 elements take the variant with group records)
        return {"bound": "hbm", "kernel": name, "achieved": a, "peak": peak, "unit": "GB/s",
                "frac": a / peak, "peak_source": peak_src, "frac_of_nominal_8TBs": a / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": alg, "avg_launch_ms": ms,
                "traffic": None if tr is None else tr * spec.numel}

    other = "decompress" if dom == "compress" else "compress"
    roofline = roof(dom, dom_ms)
    roofline_other = roof(other, float(min(t_c.mean(), t_d.mean())))

    # ---- sampled parity against the oracle (outside the timed region): windows are independent
    parity = "skipped"
    if rank == 0:
        import oracle
        oracle.build()
        We = 16384
        n_w = c.sizes.n_windows
        pick = sorted(set([0, n_w - 1] + [int(v) for v in np.random.default_rng(0).integers(0, n_w, 256)]))   # first, last, 256 random
        woff = c.window_offsets.cpu().numpy()
        for wi in pick:
            lo, hi = wi * We, min(spec.numel, (wi + 1) * We)
            a = h_in[lo:hi].view(torch.int16).numpy().view(np.uint16) if args.dtype == "bf16" else h_in[lo:hi].numpy()
            ref = oracle.compress(a, G, widths, beta, dtype="bf16" if args.dtype == "bf16" else None, seed=0, base=lo)
            g0, g1 = lo // G, hi // G
            ok = np.array_equal(c.bits[g0:g1].cpu().numpy(), ref.bits)
            ok &= np.array_equal(c.packed[int(woff[wi]):int(woff[wi + 1])].cpu().numpy(), ref.packed)
            ok &= np.array_equal(c.min[g0:g1].cpu().numpy().view(np.uint32), ref.mn.view(np.uint32))
            got = y[lo:hi]
            got = got.view(torch.int16).cpu().numpy().view(np.uint16) if args.dtype != "f32" else got.cpu().numpy().view(np.uint32)
            want = oracle.decompress(ref)
            ok &= np.array_equal(got, want.view(got.dtype))
            if not ok:
                raise SystemExit(f"parity failure against the oracle in window {wi}")
        parity = f"bit-exact on {len(pick)} sampled windows (bits, min, packed bytes, decoded values)"

    # ---- end to end: pinned host input -> device, compress, decompress, output -> pinned host, through the package's own
    # streamed round trip (window-aligned chunks, 2^25 elements unless told otherwise; the copy in, the kernels and the copy out of
    # neighbouring chunks overlap on three streams; every byte still crosses the bus inside the timed region)
    e2e = None
    if not args.no_e2e:
        h_out = torch.empty_like(h_in, pin_memory=True)
        Ke = max(1, min(args.e2e_steps, K))
        round_trip = daf.HostRoundTrip(x.dtype, G, widths, beta, seed=0, chunk_elems=args.e2e_chunk)

        def e2e_step():
            round_trip(h_in, h_out)

        e2e_step()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(Ke):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        # the streamed result is the unsharded one (the chunks are shards with the counter base moved)
        same = bool(torch.equal(h_out.to(x.device).view(torch.int32 if args.dtype == "f32" else torch.int16),
                                y.view(torch.int32 if args.dtype == "f32" else torch.int16)))
        if not same:
            raise SystemExit("the streamed end-to-end result differs from the device-resident one")
        e2e = {"value": world * 2 * nbytes * Ke / (ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": nbytes,
               "d2h_bytes_per_step": nbytes, "steps": Ke, "how": f"HostRoundTrip: chunks of {args.e2e_chunk} elements, copies and kernels overlapped",
               "equals_device_resident_result": same}
        del h_out, round_trip

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        threads = os.cpu_count() or 1
        a = h_in[: min(spec.numel, 1 << 27)]
        a = a.view(torch.int16).numpy().view(np.uint16) if args.dtype == "bf16" else a.numpy()
        gbs, dt = time_oracle(a, spec, G, widths, beta, threads)
        cpu = {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"first {a.size} elements of the same tensor, compress+decompress, {dt:.1f} s wall"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
                "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": args.dtype, "data": "synthetic",
                "config": config_of(w, spec.numel, args.dtype, G, beta, widths), "packed_bytes": packed_bytes,
                "compress_gbs": nbytes / (t_c.mean() * 1e-3) / 1e9, "decompress_gbs": nbytes / (t_d.mean() * 1e-3) / 1e9,
                "compress_ms": float(t_c.mean()), "decompress_ms": float(t_d.mean()),
                "clocks": clocks, "e2e": e2e, "gpu_launches": LAUNCHES_PER_STEP * K, "roofline": roofline, "roofline_other": roofline_other,
                "cpu_baseline": cpu,
                "parity": parity}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
