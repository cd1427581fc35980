"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI on numpy inputs
and compare every artefact with the CPU oracle, reporting the first mismatch by stage."""
from __future__ import annotations

import numpy as np

import oracle
import paper_2507_07149_b200 as daf

TORCH_DT = {"f32": "float32", "f16": "float16", "bf16": "bfloat16"}
CODE = {"f32": daf.F32, "f16": daf.F16, "bf16": daf.BF16}


def to_device(a: np.ndarray, dtype: str):
    import torch
    if dtype == "bf16":
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def to_host(t, dtype: str) -> np.ndarray:
    import torch
    if dtype == "bf16":
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def bits_view(a: np.ndarray) -> np.ndarray:
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def gpu_compress(a: np.ndarray, dtype: str, G: int, widths, beta: float, **kw):
    x = to_device(np.ascontiguousarray(a).reshape(-1), dtype)
    c = daf.compress(x, G, widths, beta, check=True, **kw)
    return x, c


def first_mismatch(got: np.ndarray, want: np.ndarray):
    bad = np.flatnonzero(got != want)
    return None if bad.size == 0 else int(bad[0])


def assert_compress_parity(a: np.ndarray, dtype: str, G: int, widths, beta: float, *, window_elems: int = 16384,
                           rounding: int = 0, seed: int = 0, base: int = 0, label: str = ""):
    """GPU compress vs oracle: min, scale, bits, window offsets, codes, packed bytes -- all bit-exact."""
    import torch
    a = np.ascontiguousarray(a).reshape(-1)
    ref = oracle.compress(a, G, widths, beta, dtype="bf16" if dtype == "bf16" else None, window_elems=window_elems,
                          rounding=rounding, seed=seed, base=base)
    x, c = gpu_compress(a, dtype, G, widths, beta, window_elems=window_elems, rounding=rounding, seed=seed,
                        elem_index_base=base)
    torch.cuda.synchronize()
    W = window_elems // G

    def where(g):
        return f"{label} group {g} (window {g // W})"

    mn = c.min.cpu().numpy()
    i = first_mismatch(mn.view(np.uint32), ref.mn.view(np.uint32))
    assert i is None, f"min mismatch at {where(i)}: {mn[i]!r} vs {ref.mn[i]!r}"
    bits = c.bits.cpu().numpy()
    i = first_mismatch(bits, ref.bits)
    assert i is None, f"bits mismatch at {where(i)}: {bits[i]} vs {ref.bits[i]}"
    sc = c.scale.cpu().numpy()
    i = first_mismatch(sc.view(np.uint32), ref.scale.view(np.uint32))
    assert i is None, f"scale mismatch at {where(i)}: {sc[i]!r} vs {ref.scale[i]!r}"
    woff = c.window_offsets.cpu().numpy().view(np.uint64)
    i = first_mismatch(woff, ref.window_offsets)
    assert i is None, f"{label} window offset mismatch at window {i}: {woff[i]} vs {ref.window_offsets[i]}"
    total = int(woff[-1])
    packed = c.packed[:total].cpu().numpy()
    codes = oracle.unpack(packed, a.size, G, bits)
    i = first_mismatch(codes, ref.codes)
    assert i is None, (f"{label} code mismatch at element {i} (group {i // G}, window {i // window_elems}): "
                       f"{codes[i]} vs {ref.codes[i]}")
    i = first_mismatch(packed, ref.packed)
    assert i is None, f"{label} packed byte mismatch at byte {i}"
    return x, c, ref


def assert_decompress_parity(c, ref: "oracle.Compressed", dtype: str, label: str = ""):
    """GPU decompress of the GPU's own buffers vs oracle decode: 0 ulp for 16-bit outputs, <= 1 ulp for fp32."""
    import torch
    y = daf.decompress(c)
    torch.cuda.synchronize()
    got = to_host(y.reshape(-1), dtype)
    want = oracle.decompress(ref)
    if dtype == "f32":
        d = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        # the comparison is on bit patterns; +0 / -0 never differ here because both sides use the same fma
        i = first_mismatch(d <= 1, np.ones_like(d, bool))
        assert i is None, f"{label} decode mismatch at element {i}: {got[i]!r} vs {want[i]!r}"
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), f"{label}: decode within 1 ulp but not bit-equal"
    else:
        i = first_mismatch(bits_view(got), bits_view(want))
        assert i is None, f"{label} decode mismatch at element {i}: {got[i]!r} vs {want[i]!r}"
    return y
