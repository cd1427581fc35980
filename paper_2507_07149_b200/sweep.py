"""Times compress / decompress on the five benchmark workloads and the group-size x budget sweep.

    python -m paper_2507_07149_b200.sweep [--configs 1,2,3,4,5] [--sweep] [--relu] [--tensorwise] [--steps K] [--scale S]

Workloads 1-4 are sets of tensors: each set goes through ONE batched call (daf_compress_batch /
daf_decompress_batch) when it has at most DAF_BATCH_MAX tensors.  Inputs are the seeded synthetic
tensors of ``workloads.py``, resident in device memory before the timed region; the time of a call
is the median over K repetitions (after 3 warm-up calls), each bracketed by CUDA events; sets of
less than 512 MiB have the L2 flushed between repetitions.  ``--scale S`` divides the batch
dimension (or the element count of workload 5) by S for a quick look.  One markdown table row
per workload is printed: element count, input bytes, packed bytes, compress and decompress
time, and for each the algorithmic throughput: (tensor bytes + packed bytes + 9 bytes of
metadata per group + 8 per window) / time, the figure the roofline fractions are quoted on;
for the sets also the times of the same work issued as one call per tensor.
"""
from __future__ import annotations

import argparse

import numpy as np



def _device_tensor(torch, wl, cfg, ti, spec):
    tdt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.int16}[spec.dtype]
    h = torch.empty(spec.numel, dtype=tdt, pin_memory=True)
    wl.generate(cfg, ti, spec, out=h.numpy().view(wl.np_dtype(spec.dtype)))
    if spec.dtype == "bf16":
        h = h.view(torch.bfloat16)
    return h.cuda()


_FLUSH = None
_NVML = None


def _sm_mhz(torch):
    """SM clock right now (read while the GPU is still busy with the point just timed), or None without NVML."""
    global _NVML
    try:
        if _NVML is None:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
            _NVML = (pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid if not uuid.startswith("GPU-") else uuid).encode()))
        n, h = _NVML
        return int(n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM))
    except Exception:
        return None


COOLDOWN_S = 0.0


def _time(torch, fn, steps, flush):
    """Median over `steps` repetitions, each bracketed by its own pair of CUDA events.  With `flush`
    (working sets that would otherwise sit in the 126 MB L2) a 256 MiB buffer is overwritten
    between repetitions, outside the timed interval."""
    global _FLUSH
    if flush and _FLUSH is None:
        _FLUSH = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    if COOLDOWN_S > 0:
        import time
        torch.cuda.synchronize()
        time.sleep(COOLDOWN_S)
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    global LAST_MHZ
    for e0, e1 in ev:
        if flush:
            _FLUSH.fill_(1)
        e0.record()
        fn()
        e1.record()
    LAST_MHZ = _sm_mhz(torch)                                      # the queue is still draining: a clock under load
    torch.cuda.synchronize()
    return float(np.median([e0.elapsed_time(e1) for e0, e1 in ev]))


def run_set(torch, daf, wl, w, xs, steps):
    """(compress ms, decompress ms, packed bytes) for the tensors xs of workload w."""
    params = [daf.make_params(daf.dtype_code(x), x.numel(), w.group_size, w.widths, w.bit_budget, seed=t.philox_seed,
                              flags=FLAGS)
              for x, t in zip(xs, w.tensors)]
    outs = [daf.alloc_outputs(p, xs[0].device) for p in params]
    ys = [torch.empty_like(x) for x in xs]
    if len(xs) == 1:
        p, x, c, y = params[0], xs[0], outs[0], ys[0]

        def comp():
            daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                             c.workspace, c.sizes.workspace)

        def dec():
            daf.daf_decompress(p, c.packed, c.bits, c.min, c.scale, c.window_offsets, y)

        status = lambda: daf.daf_poll_status(c.workspace)
    else:
        assert len(xs) <= daf.BATCH_MAX
        ws_bytes = daf.daf_batch_workspace(params)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=xs[0].device)

        def comp():
            daf.daf_compress_batch(params, xs, [o.packed for o in outs], [o.sizes.packed_capacity for o in outs],
                                   [o.bits for o in outs], [o.min for o in outs], [o.scale for o in outs],
                                   [o.window_offsets for o in outs], ws, ws_bytes)

        def dec():
            daf.daf_decompress_batch(params, [o.packed for o in outs], [o.bits for o in outs], [o.min for o in outs],
                                     [o.scale for o in outs], [o.window_offsets for o in outs], ys)

        status = lambda: daf.daf_poll_status(ws)
    flush = sum(x.numel() * x.element_size() for x in xs) < (512 << 20)
    t_c = _time(torch, comp, steps, flush)
    assert status() == daf.OK, status()
    t_d = _time(torch, dec, steps, flush)
    packed = sum(o.packed_bytes() for o in outs)
    meta = sum(9 * (x.numel() // w.group_size) + 8 * (o.sizes.n_windows + 1) for x, o in zip(xs, outs))
    per_tensor = None
    if len(xs) > 1:                                              # the same set as one call per tensor
        def comp_each():
            for p, x, c in zip(params, xs, outs):
                daf.daf_compress(p, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                                 c.workspace, c.sizes.workspace)

        def dec_each():
            for p, c, y in zip(params, outs, ys):
                daf.daf_decompress(p, c.packed, c.bits, c.min, c.scale, c.window_offsets, y)

        per_tensor = (_time(torch, comp_each, steps, flush), _time(torch, dec_each, steps, flush))
    return t_c, t_d, packed, meta, per_tensor


LAST_MHZ = None
FLAGS = 0


def row(name, numel, nbytes, packed, meta, t_c, t_d, per_tensor=None):
    alg = nbytes + packed + meta
    each = "— | —" if per_tensor is None else f"{per_tensor[0]:.4f} | {per_tensor[1]:.4f}"
    return (f"| {name} | {numel} | {nbytes / 2**30:.3f} | {packed / 2**30:.3f} | {t_c:.4f} | {alg / t_c / 1e6:.0f} | "
            f"{t_d:.4f} | {alg / t_d / 1e6:.0f} | {each} | {LAST_MHZ if LAST_MHZ is not None else '—'} |")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--sweep", action="store_true", help="also the 16 (group size, budget) points of workload 5")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--scale", type=int, default=1)
    ap.add_argument("--relu", action="store_true",
                    help="also the fused producers and consumers (ReLU, ReLU6, GELU) on workload 5, each against torch's own "
                         "kernel followed / preceded by daf_compress / daf_decompress")
    ap.add_argument("--cooldown", type=float, default=1.0,
                    help="seconds of idle before every point, so that each is timed from the same state: back to back the points "
                         "run into the board's power cap and the SM clock falls from 1965 to about 1600 MHz (see the last column)")
    ap.add_argument("--tensorwise", action="store_true",
                    help="also the per-tensor path on workload 5: min / max reduction, Eq. 1 with one min / max / width, its inverse")
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0,
                    help="daf_params.flags of every call of the five workloads (launch policy, e.g. 8 = DAF_FLAG_ONE_PASS, "
                         "16 = DAF_FLAG_TWO_PASS, 2 = DAF_FLAG_STREAM_NEVER)")
    args = ap.parse_args()
    global FLAGS
    FLAGS = args.flags

    import torch
    import paper_2507_07149_b200 as daf
    from paper_2507_07149_b200 import workloads as wl

    daf.lib()
    global COOLDOWN_S
    COOLDOWN_S = args.cooldown
    print("| workload | elements | tensor GiB | packed GiB | compress ms | compress GB/s | decompress ms | decompress GB/s "
          "| compress ms, one call per tensor | decompress ms, one call per tensor | SM MHz under load |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    S = args.scale
    for cfg in [int(c) for c in args.configs.split(",")]:
        kw = {}
        if cfg in (2, 3, 4) and S > 1:
            kw["batch"] = max(1, {2: 64, 3: 128, 4: 64}[cfg] // S)
        if cfg == 5:
            kw["numel"] = (1 << 30) // S
        w = wl.workload(cfg, **kw)
        xs = [_device_tensor(torch, wl, cfg, i, t) for i, t in enumerate(w.tensors)]
        t_c, t_d, packed, meta, each = run_set(torch, daf, wl, w, xs, args.steps)
        print(row(w.name, w.numel, w.nbytes, packed, meta, t_c, t_d, each), flush=True)
        if cfg == 5 and args.sweep:
            for G in wl.SWEEP_GROUPS:
                for beta in wl.SWEEP_BUDGETS:
                    ws = wl.workload(5, numel=kw["numel"], group_size=G, bit_budget=beta)
                    t_c, t_d, packed, meta, each = run_set(torch, daf, wl, ws, xs, args.steps)
                    print(row(ws.name, ws.numel, ws.nbytes, packed, meta, t_c, t_d, each), flush=True)
        if cfg == 5 and args.relu:
            x = xs[0]
            p = daf.make_params(daf.dtype_code(x), x.numel(), w.group_size, w.widths, w.bit_budget, seed=0)
            c = daf.alloc_outputs(p, x.device)
            act = torch.empty_like(x)
            g = torch.randn_like(x)
            gi = torch.empty_like(x)
            F = torch.nn.functional
            # name, library code, the activation and its backward as torch runs them (separate kernels)
            variants = (
                ("ReLU", daf.ACT_RELU, lambda: torch.clamp_min(x, 0, out=act),
                 lambda: torch.ops.aten.threshold_backward.grad_input(g, act, 0.0, grad_input=gi)),
                ("ReLU6", daf.ACT_RELU6, lambda: torch.clamp(x, 0, 6, out=act),
                 lambda: torch.ops.aten.hardtanh_backward.grad_input(g, act, 0.0, 6.0, grad_input=gi)),
                ("GELU", daf.ACT_GELU, lambda: torch.ops.aten.gelu.out(x, out=act),
                 lambda: torch.ops.aten.gelu_backward.grad_input(g, act, grad_input=gi)))
            for name, code, torch_fwd, torch_bwd in variants:
                gelu = code == daf.ACT_GELU

                def fused():
                    daf.daf_act_compress(p, code, x, act, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale,
                                         c.window_offsets, c.workspace, c.sizes.workspace)

                def separate():
                    torch_fwd()
                    daf.daf_compress(p, x if gelu else act, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale,
                                     c.window_offsets, c.workspace, c.sizes.workspace)

                t_f = _time(torch, fused, args.steps, False)
                assert daf.daf_poll_status(c.workspace) == daf.OK
                packed = c.packed_bytes()
                t_s = _time(torch, separate, args.steps, False)
                alg = 2 * w.nbytes + packed + 9 * (x.numel() // w.group_size) + 8 * (c.sizes.n_windows + 1)
                print(f"| {w.name} {name} + compress, fused | {w.numel} | {w.nbytes / 2**30:.3f} | {packed / 2**30:.3f} | "
                      f"{t_f:.4f} | {alg / t_f / 1e6:.0f} | — | — | torch {name} + daf_compress: {t_s:.4f} | — |", flush=True)

                def fused_back():
                    daf.daf_decompress_act_grad(p, code, c.packed, c.bits, c.min, c.scale, c.window_offsets, g, gi)

                def separate_back():
                    daf.daf_decompress(p, c.packed, c.bits, c.min, c.scale, c.window_offsets, act)
                    torch_bwd()                                       # torch's backward kernel on the restored tensor

                t_fb = _time(torch, fused_back, args.steps, False)
                t_sb = _time(torch, separate_back, args.steps, False)
                print(f"| {w.name} {name} gradient from the packed form, fused | {w.numel} | {w.nbytes / 2**30:.3f} | "
                      f"{packed / 2**30:.3f} | — | — | {t_fb:.4f} | {alg / t_fb / 1e6:.0f} | — | daf_decompress + torch's "
                      f"{name} backward: {t_sb:.4f} |", flush=True)
            del act, c, g, gi
        if cfg == 5 and args.tensorwise:
            x = xs[0]
            width = int(w.bit_budget)
            stats = torch.empty(8, dtype=torch.int32, device=x.device)
            packed = torch.empty(x.numel() * width // 8, dtype=torch.uint8, device=x.device)
            ms = torch.empty(2, dtype=torch.float32, device=x.device)
            y = torch.empty_like(x)
            t_m = _time(torch, lambda: daf.daf_tensor_minmax(x, stats), args.steps, False)
            t_q = _time(torch, lambda: daf.daf_tensor_compress(x, width, stats, packed, ms), args.steps, False)
            t_d = _time(torch, lambda: daf.daf_tensor_decompress(packed, width, ms, y), args.steps, False)
            nb, pb = w.nbytes, packed.numel()
            print(f"| {w.name} per-tensor min / max | {w.numel} | {nb / 2**30:.3f} | — | {t_m:.4f} | {nb / t_m / 1e6:.0f} | — | — | — | — |")
            print(f"| {w.name} per-tensor quantize (width {width}) / dequantize | {w.numel} | {nb / 2**30:.3f} | {pb / 2**30:.3f} | "
                  f"{t_q:.4f} | {(nb + pb) / t_q / 1e6:.0f} | {t_d:.4f} | {(nb + pb) / t_d / 1e6:.0f} | — | — |", flush=True)
            del stats, packed, ms, y
        del xs
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
