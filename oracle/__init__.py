"""CPU oracle for the DAF activation compress / decompress hot path (test infrastructure).

This package wraps ``daf_oracle.c`` -- a plain, slow restatement of the method in
IEEE binary32 -- through ctypes and numpy.  It is NOT part of the product: only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it, and it
imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "daf_oracle.c")
_LIB = os.path.join(_HERE, "libdaf_oracle.so")

F32, F16, BF16 = 0, 1, 2
ROUND_STOCHASTIC, ROUND_NEAREST = 0, 1
OK, ERR_ARG, ERR_NONFINITE, ERR_BUDGET, ERR_CAPACITY = 0, 1, 2, 3, 4

# No contraction, no fast-math: every operation is a single IEEE binary32 operation.
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
          "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source (gcc only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", *CFLAGS, "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int), ("numel", ctypes.c_uint64), ("group_size", ctypes.c_uint32),
                ("window_elems", ctypes.c_uint32), ("width_mask", ctypes.c_uint32),
                ("bit_budget", ctypes.c_float), ("rounding", ctypes.c_int), ("seed", ctypes.c_uint64),
                ("elem_index_base", ctypes.c_uint64)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.daf_oracle_raise_factor.restype = ctypes.c_float
        _lib.daf_oracle_raise_factor.argtypes = [ctypes.c_int, ctypes.c_int]
        _lib.daf_oracle_r15.restype = ctypes.c_uint32
        _lib.daf_oracle_r15.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        _lib.daf_oracle_beta_q8.restype = ctypes.c_uint32
        _lib.daf_oracle_beta_q8.argtypes = [ctypes.c_float]
        _lib.daf_oracle_half_to_float.restype = ctypes.c_float
        _lib.daf_oracle_half_to_float.argtypes = [ctypes.c_uint16]
        _lib.daf_oracle_float_to_half.restype = ctypes.c_uint16
        _lib.daf_oracle_float_to_half.argtypes = [ctypes.c_float]
        _lib.daf_oracle_float_to_bf16.restype = ctypes.c_uint16
        _lib.daf_oracle_float_to_bf16.argtypes = [ctypes.c_float]
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}")
        self.code = code


def _check(rc: int):
    if rc != OK:
        raise OracleError(rc)


# ---------------------------------------------------------------- dtype helpers
def dtype_code(a: np.ndarray, dtype: str | None = None) -> int:
    """dtype code of an input array; bf16 travels as uint16 bit patterns with dtype='bf16'."""
    if dtype in ("bf16", "bfloat16"):
        return BF16
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float16:
        return F16
    raise ValueError(f"unsupported dtype {a.dtype} / {dtype}")


def widen(a: np.ndarray, dtype: str | None = None) -> np.ndarray:
    code = dtype_code(a, dtype)
    a = np.ascontiguousarray(a).reshape(-1)
    x = np.empty(a.size, np.float32)
    _check(lib().daf_oracle_widen(code, _p(a), ctypes.c_uint64(a.size), _p(x)))
    return x


# ---------------------------------------------------------------- stage functions
def relu(a: np.ndarray, dtype: str | None = None) -> np.ndarray:
    """The producer that can be fused in front of the compression (Sec. 3.2.3): x where x > 0, else +0,
    in the array's own type (bf16 arrays are uint16 bit patterns: negative = sign bit set)."""
    if dtype == "bf16" or a.dtype == np.uint16:
        return np.where((a & 0x8000) != 0, np.uint16(0), a).astype(np.uint16)
    return np.where(a > 0, a, a.dtype.type(0)).astype(a.dtype)


def relu6(a: np.ndarray, dtype: str | None = None) -> np.ndarray:
    """ReLU6 as a fused producer (Sec. 3.2.3): min(max(x, +0), 6) in the array's own type."""
    if dtype == "bf16" or a.dtype == np.uint16:
        six = np.uint16(0x40C0)                                    # 6.0; positive bf16 patterns order like integers
        r = np.where((a & 0x8000) != 0, np.uint16(0), a)
        return np.where(r > six, six, r).astype(np.uint16)
    r = np.where(a > 0, a, a.dtype.type(0))
    return np.where(r > 6, a.dtype.type(6), r).astype(a.dtype)


def gelu(x) -> np.ndarray:
    """GELU(x) = x Phi(x) = x/2 erfc(-x / sqrt 2) in binary64 (the reference the fused producer is held to)."""
    import math
    x = np.asarray(x, np.float64)
    erfc = np.vectorize(math.erfc, otypes=[np.float64])
    return 0.5 * x * erfc(-x / math.sqrt(2.0))


def gelu_grad(x) -> np.ndarray:
    """d/dx GELU(x) = Phi(x) + x phi(x) in binary64."""
    import math
    x = np.asarray(x, np.float64)
    erfc = np.vectorize(math.erfc, otypes=[np.float64])
    return 0.5 * erfc(-x / math.sqrt(2.0)) + x * np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)


def to_bf16_bits(x) -> np.ndarray:
    """binary32 -> bf16 bit patterns, round to nearest even (the oracle's own conversion, element by element)."""
    f = lib().daf_oracle_float_to_bf16
    return np.array([f(float(v)) for v in np.asarray(x, np.float32).reshape(-1)], np.uint16)


def stats(x, G: int):
    x = _c(x, np.float32).reshape(-1)
    ng = x.size // G
    mn, mx, R = (np.empty(ng, np.float32) for _ in range(3))
    _check(lib().daf_oracle_stats(_p(x), ctypes.c_uint64(x.size), ctypes.c_uint32(G), _p(mn), _p(mx), _p(R)))
    return mn, mx, R


def width_mask(widths) -> int:
    m = 0
    for b in widths:
        m |= 1 << int(b)
    return m


def beta_q8(bit_budget: float) -> int:
    return int(lib().daf_oracle_beta_q8(ctypes.c_float(bit_budget)))


def choose_bits(R, groups_per_window: int, widths, bit_budget: float) -> np.ndarray:
    R = _c(R, np.float32)
    bits = np.empty(R.size, np.uint8)
    _check(lib().daf_oracle_choose_bits(_p(R), ctypes.c_uint64(R.size), ctypes.c_uint32(groups_per_window),
                                        ctypes.c_uint32(width_mask(widths)), ctypes.c_uint32(beta_q8(bit_budget)),
                                        _p(bits)))
    return bits


def raise_factor(b_lo: int, b_hi: int) -> np.float32:
    return np.float32(lib().daf_oracle_raise_factor(b_lo, b_hi))


def group_params(R, bits):
    R = _c(R, np.float32)
    bits = _c(bits, np.uint8)
    scale, inv = np.empty(R.size, np.float32), np.empty(R.size, np.float32)
    lib().daf_oracle_group_params(_p(R), _p(bits), ctypes.c_uint64(R.size), _p(scale), _p(inv))
    return scale, inv


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().daf_oracle_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def philox_round(ctr, key):
    ctr = _c(ctr, np.uint32).copy()
    key = _c(key, np.uint32).copy()
    lib().daf_oracle_philox_round(_p(ctr), _p(key))
    return ctr, key


def r15(seed: int, j: int) -> int:
    return int(lib().daf_oracle_r15(ctypes.c_uint64(seed), ctypes.c_uint64(j)))


def codes(x, G: int, mn, inv, bits, rounding: int = ROUND_STOCHASTIC, seed: int = 0, base: int = 0) -> np.ndarray:
    x = _c(x, np.float32).reshape(-1)
    mn, inv, bits = _c(mn, np.float32), _c(inv, np.float32), _c(bits, np.uint8)
    out = np.empty(x.size, np.uint8)
    _check(lib().daf_oracle_codes(_p(x), ctypes.c_uint64(x.size), ctypes.c_uint32(G), _p(mn), _p(inv), _p(bits),
                                  ctypes.c_int(rounding), ctypes.c_uint64(seed), ctypes.c_uint64(base), _p(out)))
    return out


def codes_r15(x, G: int, mn, inv, bits, r15_) -> np.ndarray:
    """Step 5 with the 15-bit rounding offsets supplied by the caller."""
    x = _c(x, np.float32).reshape(-1)
    mn, inv, bits, r15_ = _c(mn, np.float32), _c(inv, np.float32), _c(bits, np.uint8), _c(r15_, np.uint16)
    out = np.empty(x.size, np.uint8)
    _check(lib().daf_oracle_codes_r15(_p(x), ctypes.c_uint64(x.size), ctypes.c_uint32(G), _p(mn), _p(inv), _p(bits),
                                      _p(r15_), _p(out)))
    return out


def offsets(bits, G: int) -> np.ndarray:
    bits = _c(bits, np.uint8)
    off = np.empty(bits.size + 1, np.uint64)
    lib().daf_oracle_offsets(_p(bits), ctypes.c_uint64(bits.size), ctypes.c_uint32(G), _p(off))
    return off


def pack(codes_, G: int, bits, off=None) -> np.ndarray:
    codes_, bits = _c(codes_, np.uint8), _c(bits, np.uint8)
    off = offsets(bits, G) if off is None else _c(off, np.uint64)
    packed = np.empty(int(off[-1]), np.uint8)
    _check(lib().daf_oracle_pack(_p(codes_), ctypes.c_uint64(codes_.size), ctypes.c_uint32(G), _p(bits), _p(off),
                                 _p(packed), ctypes.c_uint64(packed.size)))
    return packed


def unpack(packed, n: int, G: int, bits, off=None) -> np.ndarray:
    packed, bits = _c(packed, np.uint8), _c(bits, np.uint8)
    off = offsets(bits, G) if off is None else _c(off, np.uint64)
    out = np.empty(n, np.uint8)
    _check(lib().daf_oracle_unpack(_p(packed), ctypes.c_uint64(n), ctypes.c_uint32(G), _p(bits), _p(off), _p(out)))
    return out


def _out_array(n: int, code: int) -> np.ndarray:
    return np.empty(n, np.float32 if code == F32 else (np.float16 if code == F16 else np.uint16))


def decode(codes_, G: int, mn, scale, dtype_code_: int = F32) -> np.ndarray:
    codes_, mn, scale = _c(codes_, np.uint8), _c(mn, np.float32), _c(scale, np.float32)
    out = _out_array(codes_.size, dtype_code_)
    _check(lib().daf_oracle_decode(_p(codes_), ctypes.c_uint64(codes_.size), ctypes.c_uint32(G), _p(mn), _p(scale),
                                   ctypes.c_int(dtype_code_), _p(out)))
    return out


# ---------------------------------------------------------------- whole path
@dataclass
class Compressed:
    """Everything the compress step stores, plus the oracle-only extras (mx, codes)."""
    dtype: int
    numel: int
    group_size: int
    window_elems: int
    widths: tuple
    bit_budget: float
    rounding: int
    seed: int
    base: int
    packed: np.ndarray          # uint8, total bytes = window_offsets[-1]
    bits: np.ndarray            # uint8 per group
    mn: np.ndarray              # float32 per group
    scale: np.ndarray           # float32 per group
    window_offsets: np.ndarray  # uint64, n_windows + 1
    mx: np.ndarray | None = None
    codes: np.ndarray | None = None


def _params(code, numel, G, We, widths, budget, rounding, seed, base) -> _Params:
    return _Params(code, numel, G, We, width_mask(widths), budget, rounding, seed, base)


def packed_capacity(numel: int, G: int, We: int, bit_budget: float) -> int:
    """Upper bound on the packed bytes: per window floor(beta_q8 * n / 256) * G / 8."""
    ng = numel // G
    W = We // G
    q8 = beta_q8(bit_budget)
    full, last = divmod(ng, W)
    return full * ((q8 * W) >> 8) * G // 8 + ((q8 * last) >> 8) * G // 8


def compress(a: np.ndarray, G: int, widths, bit_budget: float, *, dtype: str | None = None,
             window_elems: int = 16384, rounding: int = ROUND_STOCHASTIC, seed: int = 0, base: int = 0,
             want_codes: bool = True) -> Compressed:
    code = dtype_code(a, dtype)
    a = np.ascontiguousarray(a).reshape(-1)
    n = a.size
    ng = n // G
    nw = -(-ng // (window_elems // G))
    cap = packed_capacity(n, G, window_elems, bit_budget)
    packed = np.empty(max(cap, 1), np.uint8)
    bits = np.empty(ng, np.uint8)
    mn, scale, mx = (np.empty(ng, np.float32) for _ in range(3))
    woff = np.empty(nw + 1, np.uint64)
    codes_ = np.empty(n, np.uint8) if want_codes else None
    p = _params(code, n, G, window_elems, widths, bit_budget, rounding, seed, base)
    _check(lib().daf_oracle_compress(ctypes.byref(p), _p(a), _p(packed), ctypes.c_uint64(cap), _p(bits), _p(mn),
                                     _p(scale), _p(woff), _p(mx), _p(codes_) if want_codes else None))
    return Compressed(code, n, G, window_elems, tuple(widths), bit_budget, rounding, seed, base,
                      packed[: int(woff[-1])].copy(), bits, mn, scale, woff, mx, codes_)


def decompress(c: Compressed) -> np.ndarray:
    out = _out_array(c.numel, c.dtype)
    p = _params(c.dtype, c.numel, c.group_size, c.window_elems, c.widths, c.bit_budget, c.rounding, c.seed, c.base)
    packed = _c(c.packed, np.uint8)
    _check(lib().daf_oracle_decompress(ctypes.byref(p), _p(packed), _p(_c(c.bits, np.uint8)), _p(_c(c.mn, np.float32)),
                                       _p(_c(c.scale, np.float32)), _p(_c(c.window_offsets, np.uint64)), _p(out)))
    return out
