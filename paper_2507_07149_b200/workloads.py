"""Seeded synthetic inputs for the five benchmark workloads.

This module only draws random tensors of the shapes, dtypes and value distributions the
workloads name; it holds none of the compression arithmetic and is the one module that both
the CUDA path's callers and the CPU oracle's callers may use.

Every tensor is drawn chunk by chunk (2^22 elements per chunk), chunk i of tensor t of
workload c from ``numpy.random.Generator(PCG64(SeedSequence([c, t, i])))``, always in
float32, then narrowed with round-to-nearest-even where the workload asks for a 16-bit
type.  Chunks are independent, so a tensor (or any chunk-aligned slice of it) can be drawn
on several threads and comes out the same.  bfloat16 tensors travel as uint16 bit patterns
(numpy has no bfloat16).
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
import os

import numpy as np

CHUNK = 1 << 22


@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: tuple
    dtype: str          # 'f32' | 'f16' | 'bf16'
    dist: str           # 'relu' | 'normal' | 'relu6' | 't3_outliers' | 'laplace' | 'logscale'
    philox_seed: int = 0

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape))

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == "f32" else 2


@dataclass(frozen=True)
class Workload:
    name: str
    cfg: int                     # workload number (also the first word of the seed sequence)
    tensors: tuple
    group_size: int
    widths: tuple
    bit_budget: float
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def nbytes(self) -> int:
        return sum(t.numel * t.itemsize for t in self.tensors)


# --------------------------------------------------------------------------- drawing
def _draw_chunk(dist: str, n: int, rng: np.random.Generator) -> np.ndarray:
    if dist == "normal":
        return rng.standard_normal(n, dtype=np.float32)
    if dist == "relu":                       # max(0, N(0,1))
        return np.maximum(rng.standard_normal(n, dtype=np.float32), np.float32(0))
    if dist == "relu6":                      # clip(N(0, sigma=2), 0, 6)
        return np.clip(rng.standard_normal(n, dtype=np.float32) * np.float32(2), np.float32(0), np.float32(6))
    if dist == "laplace":                    # Laplace(0,1) = Exp(1) with a random sign
        e = rng.standard_exponential(n, dtype=np.float32)
        neg = rng.random(n, dtype=np.float32) < np.float32(0.5)
        return np.where(neg, -e, e).astype(np.float32)
    if dist == "t3_outliers":                # Student-t(3); 0.1 % of entries set to +-20 sigma (sigma = sqrt(3))
        x = rng.standard_t(3.0, n).astype(np.float32)
        hit = rng.random(n, dtype=np.float32) < np.float32(1e-3)
        sign = np.where(rng.random(n, dtype=np.float32) < np.float32(0.5), np.float32(-1), np.float32(1))
        return np.where(hit, sign * np.float32(20.0 * np.sqrt(3.0)), x).astype(np.float32)
    if dist == "logscale":                   # N(0,1) times a per-256-run scale, log-uniform over 4 decades
        x = rng.standard_normal(n, dtype=np.float32)
        runs = -(-n // 256)
        s = np.float32(10.0) ** rng.uniform(-2.0, 2.0, runs).astype(np.float32)
        return (x * np.repeat(s, 256)[:n]).astype(np.float32)
    raise ValueError(dist)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even narrowing of finite float32 values to bfloat16 bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


def _narrow(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return x
    if dtype == "f16":
        return x.astype(np.float16)
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)


def np_dtype(dtype: str):
    return {"f32": np.float32, "f16": np.float16, "bf16": np.uint16}[dtype]


def generate(cfg: int, tensor_index: int, spec: TensorSpec, *, start: int = 0, count: int | None = None,
             threads: int | None = None, out: np.ndarray | None = None) -> np.ndarray:
    """Flat array of ``spec``'s elements [start, start+count); ``start`` must be chunk aligned."""
    n = spec.numel
    count = n - start if count is None else count
    assert start % CHUNK == 0 and 0 <= start and start + count <= n
    if out is None:
        out = np.empty(count, np_dtype(spec.dtype))
    first = start // CHUNK
    n_chunks = -(-count // CHUNK)

    def work(i: int):
        lo = i * CHUNK
        m = min(CHUNK, n - (start + lo))          # chunk length in the full tensor
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([cfg, tensor_index, first + i])))
        x = _narrow(_draw_chunk(spec.dist, m, rng), spec.dtype)
        take = min(m, count - lo)
        out[lo:lo + take] = x[:take]

    threads = threads or min(32, os.cpu_count() or 1)
    if n_chunks <= 1 or threads <= 1:
        for i in range(n_chunks):
            work(i)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, range(n_chunks)))
    return out


# --------------------------------------------------------------------------- the five workloads
def _resnet18_specs(batch: int):
    """Every conv / BN / ReLU output of ResNet-18 at 224x224 input (57 tensors)."""
    specs = []

    def add(kind, c, hw):
        dist = "relu" if kind == "relu" else "normal"
        specs.append((f"{kind}{len(specs)}_{c}x{hw}", (batch, c, hw, hw), dist))

    for kind in ("conv", "bn", "relu"):
        add(kind, 64, 112)
    for _ in range(2):                                   # layer1: two basic blocks, no downsample
        for kind in ("conv", "bn", "relu", "conv", "bn", "relu"):
            add(kind, 64, 56)
    for c, hw in ((128, 28), (256, 14), (512, 7)):       # layers 2-4: downsample block + plain block
        for kind in ("conv", "bn", "relu", "conv", "bn", "conv", "bn", "relu"):
            add(kind, c, hw)
        for kind in ("conv", "bn", "relu", "conv", "bn", "relu"):
            add(kind, c, hw)
    return specs


def _mobilenetv2_specs(batch: int):
    """(expanded, depthwise-output) ReLU6 activations of the 16 expansion-6 blocks (32 tensors)."""
    pairs = [((96, 112), (96, 56)), ((144, 56), (144, 56)), ((144, 56), (144, 28))]
    pairs += [((192, 28), (192, 28))] * 2 + [((192, 28), (192, 14))]
    pairs += [((384, 14), (384, 14))] * 3 + [((384, 14), (384, 14))]
    pairs += [((576, 14), (576, 14))] * 2 + [((576, 14), (576, 7))]
    pairs += [((960, 7), (960, 7))] * 2 + [((960, 7), (960, 7))]
    specs = []
    for exp, dw in pairs:
        for tag, (c, hw) in (("exp", exp), ("dw", dw)):
            specs.append((f"{tag}{len(specs)}_{c}x{hw}", (batch, c, hw, hw), "relu6"))
    return specs


def workload(cfg: int, **kw) -> Workload:
    """The benchmark workloads 1-5 (5 takes ``group_size`` and ``bit_budget``; ``numel`` to shrink it)."""
    if cfg == 1:
        t = (TensorSpec("relu_8x64x56x56", (8, 64, 56, 56), "f32", "relu", 0),)
        return Workload("cfg1_resnet18_stage1", 1, t, 256, (2, 4, 8), 4.0)
    if cfg == 2:
        batch = kw.get("batch", 64)
        t = tuple(TensorSpec(n, s, "f32", d, i) for i, (n, s, d) in enumerate(_resnet18_specs(batch)))
        return Workload(f"cfg2_resnet18_b{batch}", 2, t, 256, (1, 2, 4, 8), 3.0)
    if cfg == 3:
        batch = kw.get("batch", 128)
        t = tuple(TensorSpec(n, s, "f16", d, i) for i, (n, s, d) in enumerate(_mobilenetv2_specs(batch)))
        return Workload(f"cfg3_mobilenetv2_b{batch}", 3, t, 128, (1, 2, 4, 8), 2.0)
    if cfg == 4:
        batch, layers = kw.get("batch", 64), kw.get("layers", 12)
        t = []
        for l in range(layers):
            t.append(TensorSpec(f"ln{l}", (batch, 197, 768), "bf16", "t3_outliers", 2 * l))
            t.append(TensorSpec(f"gelu_in{l}", (batch, 197, 3072), "bf16", "t3_outliers", 2 * l + 1))
        return Workload(f"cfg4_vitb16_b{batch}", 4, tuple(t), 128, (2, 4, 8), 4.0)
    if cfg == 5:
        numel = kw.get("numel", 1 << 30)
        G, beta = kw.get("group_size", 256), kw.get("bit_budget", 4.0)
        t = (TensorSpec(f"laplace_{numel}", (numel,), "f32", "laplace", 0),)
        return Workload(f"cfg5_sweep_G{G}_b{beta:g}", 5, t, G, (1, 2, 4, 8), float(beta))
    raise ValueError(cfg)


SWEEP_GROUPS = (64, 256, 1024, 4096)
SWEEP_BUDGETS = (1.0, 2.0, 4.0, 8.0)


def shard_range(numel: int, window_elems: int, rank: int, world: int):
    """Window-aligned slice [lo, hi) of a flat tensor for one rank: whole windows, as even as possible.
    Compressing the slice with elem_index_base=lo reproduces the bytes of the unsharded run."""
    n_windows = -(-numel // window_elems)
    per, extra = divmod(n_windows, world)
    w_lo = rank * per + min(rank, extra)
    w_hi = w_lo + per + (1 if rank < extra else 0)
    return min(w_lo * window_elems, numel), min(w_hi * window_elems, numel)
