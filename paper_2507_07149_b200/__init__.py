"""B200-native activation compress / decompress (the DAF hot path): thin Python binding.

Every function here only marshals arguments for the C ABI declared in ``include/daf.h``
(``libdaf.so``, hand-written sm_100a kernels).  PyTorch supplies device memory and streams;
all arithmetic of the path runs in the CUDA library.  There is no CPU fallback: if the
library is missing or fails to load, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdaf.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_BUDGET, ERR_CAPACITY, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = range(8)
F32, F16, BF16 = 0, 1, 2
ROUND_STOCHASTIC, ROUND_NEAREST = 0, 1
FLAG_STREAM_ALWAYS, FLAG_STREAM_NEVER, FLAG_KEEP_WORKSPACE, FLAG_ONE_PASS, FLAG_TWO_PASS = 1, 2, 4, 8, 16


# daf_params.flags used by make_params when the caller gives none (the GPU tests set FLAG_STREAM_ALWAYS here so
# that their small tensors still go through both compress kernels).
DEFAULT_FLAGS = 0


def flag_poll_limit(n: int) -> int:
    """daf_params.flags value that makes bounded device-side waits give up after n polls (diagnostic)."""
    return int(n) << 8

BATCH_MAX = 64
DEFAULT_WINDOW = 16384


class daf_params(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("dtype", ctypes.c_uint32), ("numel", ctypes.c_uint64),
                ("group_size", ctypes.c_uint32), ("window_elems", ctypes.c_uint32), ("width_mask", ctypes.c_uint32),
                ("bit_budget", ctypes.c_float), ("rounding", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("seed", ctypes.c_uint64), ("elem_index_base", ctypes.c_uint64)]


class daf_pool_stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in ("arena_bytes", "page_bytes", "pages_total", "pages_used",
                                               "live_allocations", "bytes_requested", "largest_free_run_pages",
                                               "evictions")]


class daf_store_config(ctypes.Structure):
    _fields_ = [("mem_budget_bytes", ctypes.c_uint64), ("time_budget", ctypes.c_double), ("page_bytes", ctypes.c_uint64),
                ("step_bytes", ctypes.c_uint64), ("width_mask", ctypes.c_uint32), ("reserved", ctypes.c_uint32)]


class daf_store_move(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in ("id", "from_offset", "to_offset", "bytes")]


class daf_store_stats(ctypes.Structure):
    _fields_ = ([(n, ctypes.c_uint64) for n in ("arena_bytes", "mem_budget_bytes", "used_bytes", "planned_bytes")]
                + [("time_budget", ctypes.c_double), ("used_time", ctypes.c_double)]
                + [(n, ctypes.c_uint64) for n in ("entries", "kept", "evictions", "resizes", "grows", "shrinks", "moves")])


class DafError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().daf_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{where}: {msg} (status {status})")


_lib = None
_u64p = ctypes.POINTER(ctypes.c_uint64)
_vp = ctypes.c_void_p

# name -> (restype, argtypes): every symbol include/daf.h declares
SIGNATURES = {
    "daf_sizes": (ctypes.c_int, [ctypes.POINTER(daf_params), _u64p, _u64p, _u64p, _u64p]),
    "daf_shard": (ctypes.c_int, [ctypes.POINTER(daf_params), ctypes.c_uint32, ctypes.c_uint32, ctypes.POINTER(daf_params), _u64p]),
    "daf_compress": (ctypes.c_int, [ctypes.POINTER(daf_params), _vp, _vp, ctypes.c_uint64, _vp, _vp, _vp, _vp, _vp,
                                    ctypes.c_uint64, _vp]),
    "daf_relu_compress": (ctypes.c_int, [ctypes.POINTER(daf_params), _vp, _vp, _vp, ctypes.c_uint64, _vp, _vp, _vp, _vp, _vp,
                                         ctypes.c_uint64, _vp]),
    "daf_act_compress": (ctypes.c_int, [ctypes.POINTER(daf_params), ctypes.c_uint32, _vp, _vp, _vp, ctypes.c_uint64, _vp, _vp,
                                        _vp, _vp, _vp, ctypes.c_uint64, _vp]),
    "daf_decompress_act_grad": (ctypes.c_int, [ctypes.POINTER(daf_params), ctypes.c_uint32, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                               _vp]),
    "daf_compress_static": (ctypes.c_int, [ctypes.POINTER(daf_params), _vp, _vp, ctypes.c_uint64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "daf_decompress": (ctypes.c_int, [ctypes.POINTER(daf_params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_uint64, _vp]),
    "daf_decompress_relu_grad": (ctypes.c_int, [ctypes.POINTER(daf_params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "daf_group_offsets": (ctypes.c_int, [_vp, ctypes.c_uint64, ctypes.c_uint32, _vp, _vp, ctypes.c_uint64, _vp]),
    "daf_group_offsets_diag": (ctypes.c_int, [_vp, ctypes.c_uint64, ctypes.c_uint32, _vp, _vp, ctypes.c_uint64, ctypes.c_uint32,
                                              _vp]),
    "daf_group_offsets_workspace": (ctypes.c_uint64, [ctypes.c_uint64]),
    "daf_poll_status": (ctypes.c_int, [_vp, _vp]),
    "daf_batch_workspace": (ctypes.c_uint64, [ctypes.c_uint32, ctypes.POINTER(daf_params)]),
    "daf_compress_batch": (ctypes.c_int, [ctypes.c_uint32, ctypes.POINTER(daf_params), _vp, _vp, _u64p, _vp, _vp, _vp, _vp,
                                          _vp, ctypes.c_uint64, _vp]),
    "daf_decompress_batch": (ctypes.c_int, [ctypes.c_uint32, ctypes.POINTER(daf_params), _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "daf_tensor_minmax": (ctypes.c_int, [ctypes.c_uint32, _vp, ctypes.c_uint64, _vp, _vp]),
    "daf_tensor_compress": (ctypes.c_int, [ctypes.c_uint32, _vp, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32,
                                           ctypes.c_uint64, ctypes.c_uint64, _vp, _vp, _vp, _vp]),
    "daf_tensor_decompress": (ctypes.c_int, [ctypes.c_uint32, _vp, ctypes.c_uint64, ctypes.c_uint32, _vp, _vp, _vp]),
    "daf_pool_create": (_vp, [ctypes.c_uint64, ctypes.c_uint64]),
    "daf_pool_destroy": (None, [_vp]),
    "daf_pool_alloc": (ctypes.c_uint64, [_vp, ctypes.c_uint64, ctypes.c_double, _u64p]),
    "daf_pool_free": (ctypes.c_int, [_vp, ctypes.c_uint64]),
    "daf_pool_evict_lowest": (ctypes.c_uint64, [_vp]),
    "daf_pool_get_stats": (ctypes.c_int, [_vp, ctypes.POINTER(daf_pool_stats)]),
    "daf_store_bytes": (ctypes.c_uint64, [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32]),
    "daf_store_create": (_vp, [ctypes.POINTER(daf_store_config)]),
    "daf_store_destroy": (None, [_vp]),
    "daf_store_estimate": (ctypes.c_int, [_vp, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_double,
                                          ctypes.c_double, ctypes.POINTER(ctypes.c_uint32), _u64p,
                                          ctypes.POINTER(ctypes.c_uint32)]),
    "daf_store_admit": (ctypes.c_int, [_vp, ctypes.c_uint64, ctypes.c_double, ctypes.POINTER(ctypes.c_uint32), _u64p, _u64p,
                                       ctypes.POINTER(ctypes.c_uint32)]),
    "daf_store_width": (ctypes.c_int, [_vp, ctypes.c_uint64, ctypes.POINTER(ctypes.c_uint32), _u64p]),
    "daf_store_release": (ctypes.c_int, [_vp, ctypes.c_uint64]),
    "daf_store_set_budget": (ctypes.c_int, [_vp, ctypes.c_uint64, ctypes.c_double, ctypes.POINTER(daf_store_move),
                                            ctypes.POINTER(ctypes.c_uint32), _u64p, ctypes.POINTER(ctypes.c_uint32)]),
    "daf_store_get_stats": (ctypes.c_int, [_vp, ctypes.POINTER(daf_store_stats)]),
    "daf_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "daf_version": (ctypes.c_uint32, []),
}


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2507_07149_b200.build` "
                               "(nvcc, sm_100a); there is no CPU fallback")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise DafError(status, where)


# ------------------------------------------------------------------------------------ params / sizes
def width_mask(widths) -> int:
    m = 0
    for b in widths:
        m |= 1 << int(b)
    return m


def make_params(dtype: int, numel: int, group_size: int, widths, bit_budget: float, *, window_elems: int = 0,
                rounding: int = ROUND_STOCHASTIC, seed: int = 0, elem_index_base: int = 0,
                flags: int | None = None) -> daf_params:
    if flags is None:
        flags = DEFAULT_FLAGS
    return daf_params(ctypes.sizeof(daf_params), dtype, numel, group_size, window_elems, width_mask(widths),
                      bit_budget, rounding, flags, seed, elem_index_base)


@dataclass
class Sizes:
    n_groups: int
    n_windows: int
    packed_capacity: int
    workspace: int


def daf_sizes(params: daf_params) -> Sizes:
    v = [ctypes.c_uint64() for _ in range(4)]
    _check(lib().daf_sizes(ctypes.byref(params), *[ctypes.byref(x) for x in v]), "daf_sizes")
    return Sizes(*[int(x.value) for x in v])


def daf_shard(params: daf_params, rank: int, world: int):
    """(parameters of rank's window-aligned slice, its first element); the slice's numel is 0 when there is none."""
    shard, first = daf_params(), ctypes.c_uint64()
    _check(lib().daf_shard(ctypes.byref(params), rank, world, ctypes.byref(shard), ctypes.byref(first)), "daf_shard")
    return shard, int(first.value)


def _torch():
    import torch
    return torch


def dtype_code(t) -> int:
    torch = _torch()
    return {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}[t.dtype]


def _call(fn, ref, stream, *args) -> int:
    """Calls fn(*args, stream) with the device of tensor `ref` current in this thread (the library launches on the
    current device) and, unless a stream is given, on torch's current stream OF THAT DEVICE.  Returns the status."""
    torch = _torch()
    dev = ref.device
    if stream is None:
        stream = torch.cuda.current_stream(dev)
    if dev.index == torch.cuda.current_device():
        return int(fn(*args, int(stream.cuda_stream)))
    with torch.cuda.device(dev):
        return int(fn(*args, int(stream.cuda_stream)))


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


# ------------------------------------------------------------------------------------ raw entry points
def daf_compress(params, d_in, d_packed, packed_capacity, d_bits, d_min, d_scale, d_window_offsets, d_workspace,
                 workspace_bytes, stream=None):
    """Tensors (or None) in, status checked; everything else is the C call."""
    status = _call(lib().daf_compress, d_in, stream, ctypes.byref(params), _ptr(d_in), _ptr(d_packed),
                   packed_capacity, _ptr(d_bits), _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets),
                   _ptr(d_workspace), workspace_bytes)
    _check(status, "daf_compress")


def daf_relu_compress(params, d_in, d_act, d_packed, packed_capacity, d_bits, d_min, d_scale, d_window_offsets, d_workspace,
                      workspace_bytes, stream=None):
    """Fused producer: d_act = max(d_in, +0) is written and compressed in one pass (d_act may be d_in)."""
    status = _call(lib().daf_relu_compress, d_in, stream, ctypes.byref(params), _ptr(d_in), _ptr(d_act),
                   _ptr(d_packed), packed_capacity, _ptr(d_bits), _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets),
                   _ptr(d_workspace), workspace_bytes)
    _check(status, "daf_relu_compress")


ACT_RELU, ACT_RELU6, ACT_GELU = 1, 2, 3


def daf_act_compress(params, act, d_in, d_act, d_packed, packed_capacity, d_bits, d_min, d_scale, d_window_offsets, d_workspace,
                     workspace_bytes, stream=None):
    """Fused producer for ReLU / ReLU6 / GELU: d_act = act(d_in) written in the same pass that compresses (the
    activation for ReLU and ReLU6, the input for GELU)."""
    status = _call(lib().daf_act_compress, d_in, stream, ctypes.byref(params), act, _ptr(d_in), _ptr(d_act),
                   _ptr(d_packed), packed_capacity, _ptr(d_bits), _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets),
                   _ptr(d_workspace), workspace_bytes)
    _check(status, "daf_act_compress")


def daf_decompress_act_grad(params, act, d_packed, d_bits, d_min, d_scale, d_window_offsets, d_grad_out, d_grad_in, stream=None):
    """Fused consumer: the gradient of the activation from its compressed form (may be in place)."""
    status = _call(lib().daf_decompress_act_grad, d_grad_out, stream, ctypes.byref(params), act, _ptr(d_packed),
                   _ptr(d_bits), _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets), _ptr(d_grad_out),
                   _ptr(d_grad_in))
    _check(status, "daf_decompress_act_grad")


STATIC_MAX_WINDOWS = 65536


def daf_compress_static(params, d_in, d_packed, packed_capacity, d_bits, d_min, d_scale, d_window_offsets, d_status=None,
                        stream=None):
    """daf_compress for callers that cannot allocate a workspace: the kernel's scratch is a fixed
    array inside the library (at most STATIC_MAX_WINDOWS windows; calls must not overlap on the GPU).
    d_status: optional int32 tensor of one element that receives the device status word."""
    status = _call(lib().daf_compress_static, d_in, stream, ctypes.byref(params), _ptr(d_in), _ptr(d_packed),
                   packed_capacity, _ptr(d_bits), _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets), _ptr(d_status))
    _check(status, "daf_compress_static")


def daf_decompress_relu_grad(params, d_packed, d_bits, d_min, d_scale, d_window_offsets, d_grad_out, d_grad_in, stream=None):
    """Fused consumer: d_grad_in = d_grad_out where the restored activation is > 0, else 0 (may be in place)."""
    status = _call(lib().daf_decompress_relu_grad, d_grad_out, stream, ctypes.byref(params), _ptr(d_packed),
                   _ptr(d_bits), _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets), _ptr(d_grad_out),
                   _ptr(d_grad_in))
    _check(status, "daf_decompress_relu_grad")


def daf_decompress(params, d_packed, d_bits, d_min, d_scale, d_window_offsets, d_out, d_workspace=None,
                   workspace_bytes=0, stream=None):
    status = _call(lib().daf_decompress, d_out, stream, ctypes.byref(params), _ptr(d_packed), _ptr(d_bits),
                   _ptr(d_min), _ptr(d_scale), _ptr(d_window_offsets), _ptr(d_out), _ptr(d_workspace),
                   workspace_bytes)
    _check(status, "daf_decompress")


def daf_group_offsets_workspace(n_groups: int) -> int:
    return int(lib().daf_group_offsets_workspace(n_groups))


def daf_group_offsets(d_bits, n_groups, group_size, d_offsets, d_ws, ws_bytes, stream=None):
    status = _call(lib().daf_group_offsets, d_bits, stream, _ptr(d_bits), n_groups, group_size, _ptr(d_offsets),
                   _ptr(d_ws), ws_bytes)
    _check(status, "daf_group_offsets")


def daf_group_offsets_diag(d_bits, n_groups, group_size, d_offsets, d_ws, ws_bytes, flags, stream=None):
    """daf_group_offsets with diagnostic flags (FLAG_KEEP_WORKSPACE, flag_poll_limit(n)): for tests of the bounded wait."""
    status = _call(lib().daf_group_offsets_diag, d_bits, stream, _ptr(d_bits), n_groups, group_size, _ptr(d_offsets),
                   _ptr(d_ws), ws_bytes, flags)
    _check(status, "daf_group_offsets_diag")


def daf_poll_status(d_workspace, stream=None) -> int:
    return _call(lib().daf_poll_status, d_workspace, stream, _ptr(d_workspace))


def _ptr_array(tensors):
    return (ctypes.c_void_p * len(tensors))(*[_ptr(t) for t in tensors])


def daf_batch_workspace(params_list) -> int:
    arr = (daf_params * len(params_list))(*params_list)
    return int(lib().daf_batch_workspace(len(params_list), arr))


def daf_compress_batch(params_list, d_in, d_packed, capacities, d_bits, d_min, d_scale, d_window_offsets, d_workspace,
                       workspace_bytes, stream=None):
    n = len(params_list)
    arr = (daf_params * n)(*params_list)
    caps = (ctypes.c_uint64 * n)(*capacities)
    status = _call(lib().daf_compress_batch, d_in[0], stream, n, arr, _ptr_array(d_in), _ptr_array(d_packed), caps,
                   _ptr_array(d_bits), _ptr_array(d_min), _ptr_array(d_scale), _ptr_array(d_window_offsets),
                   _ptr(d_workspace), workspace_bytes)
    _check(status, "daf_compress_batch")


def daf_decompress_batch(params_list, d_packed, d_bits, d_min, d_scale, d_window_offsets, d_out, stream=None):
    n = len(params_list)
    arr = (daf_params * n)(*params_list)
    status = _call(lib().daf_decompress_batch, d_out[0], stream, n, arr, _ptr_array(d_packed), _ptr_array(d_bits),
                   _ptr_array(d_min), _ptr_array(d_scale), _ptr_array(d_window_offsets), _ptr_array(d_out))
    _check(status, "daf_decompress_batch")


def daf_version() -> int:
    return int(lib().daf_version())


def daf_status_string(status: int) -> str:
    return lib().daf_status_string(status).decode()


# ------------------------------------------------------------------------------------ conveniences (allocation only)
@dataclass
class CompressedTensor:
    """Device buffers written by daf_compress for one tensor (owned by torch)."""
    params: daf_params
    shape: tuple
    packed: object
    bits: object
    min: object
    scale: object
    window_offsets: object
    workspace: object
    sizes: Sizes

    def packed_bytes(self) -> int:
        return int(self.window_offsets[-1].item())


def alloc_outputs(params: daf_params, device, shape=None) -> CompressedTensor:
    torch = _torch()
    sz = daf_sizes(params)
    return CompressedTensor(
        params, tuple(shape) if shape is not None else (int(params.numel),),
        torch.empty(max(sz.packed_capacity, 16), dtype=torch.uint8, device=device),
        torch.empty(sz.n_groups, dtype=torch.uint8, device=device),
        torch.empty(sz.n_groups, dtype=torch.float32, device=device),
        torch.empty(sz.n_groups, dtype=torch.float32, device=device),
        torch.empty(sz.n_windows + 1, dtype=torch.int64, device=device),
        torch.empty(sz.workspace, dtype=torch.uint8, device=device), sz)


def compress(x, group_size: int, widths, bit_budget: float, *, window_elems: int = 0, rounding: int = ROUND_STOCHASTIC,
             seed: int = 0, elem_index_base: int = 0, flags: int | None = None, out: CompressedTensor | None = None,
             check: bool = False, stream=None) -> CompressedTensor:
    """Allocate outputs with torch (unless given) and call daf_compress on the current stream."""
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("compress expects a contiguous CUDA tensor")
    params = make_params(dtype_code(x), x.numel(), group_size, widths, bit_budget, window_elems=window_elems,
                         rounding=rounding, seed=seed, elem_index_base=elem_index_base, flags=flags)
    c = out if out is not None else alloc_outputs(params, x.device, x.shape)
    c.params = params
    daf_compress(params, x, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets, c.workspace,
                 c.sizes.workspace, stream)
    if check:
        _check(daf_poll_status(c.workspace, stream), "daf_compress (device status)")
    return c


def relu_compress(x, group_size: int, widths, bit_budget: float, *, rounding: int = ROUND_STOCHASTIC, seed: int = 0,
                  elem_index_base: int = 0, flags: int | None = None, inplace: bool = False, out: CompressedTensor | None = None,
                  check: bool = False, stream=None, act: int = ACT_RELU):
    """(act(x), compressed form) in one pass over x (daf_act_compress); ``inplace`` overwrites x.  The compressed
    form holds act(x) for ReLU and ReLU6, and x itself for GELU."""
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("relu_compress expects a contiguous CUDA tensor")
    params = make_params(dtype_code(x), x.numel(), group_size, widths, bit_budget, rounding=rounding, seed=seed,
                         elem_index_base=elem_index_base, flags=flags)
    c = out if out is not None else alloc_outputs(params, x.device, x.shape)
    c.params = params
    y = x if inplace else _torch().empty_like(x)
    daf_act_compress(params, act, x, y, c.packed, c.sizes.packed_capacity, c.bits, c.min, c.scale, c.window_offsets,
                     c.workspace, c.sizes.workspace, stream)
    if check:
        _check(daf_poll_status(c.workspace, stream), "daf_act_compress (device status)")
    return y, c


def decompress(c: CompressedTensor, out=None, stream=None):
    torch = _torch()
    dt = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16}[int(c.params.dtype)]
    if out is None:
        out = torch.empty(c.shape, dtype=dt, device=c.packed.device)
    daf_decompress(c.params, c.packed, c.bits, c.min, c.scale, c.window_offsets, out, None, 0, stream)
    return out


def relu_grad(c: CompressedTensor, grad_out, out=None, stream=None, act: int = ACT_RELU):
    """Gradient of the activation from its compressed form (daf_decompress_act_grad)."""
    torch = _torch()
    if not grad_out.is_contiguous():
        grad_out = grad_out.contiguous()
    if out is None:
        out = torch.empty_like(grad_out)
    daf_decompress_act_grad(c.params, act, c.packed, c.bits, c.min, c.scale, c.window_offsets, grad_out, out, stream)
    return out


# ------------------------------------------------------------------------------------ per-tensor path
def daf_tensor_minmax(d_in, d_stats, stream=None):
    """min, max and range of the whole tensor into d_stats (8 x 32-bit words on the device: floats 0-2, scratch 4-7)."""
    status = _call(lib().daf_tensor_minmax, d_in, stream, dtype_code(d_in), _ptr(d_in), d_in.numel(), _ptr(d_stats))
    _check(status, "daf_tensor_minmax")


def daf_tensor_compress(d_in, width, d_stats, d_packed, d_min_scale, *, rounding=ROUND_STOCHASTIC, seed=0, elem_index_base=0,
                        stream=None):
    status = _call(lib().daf_tensor_compress, d_in, stream, dtype_code(d_in), _ptr(d_in), d_in.numel(), width, rounding, seed,
                   elem_index_base, _ptr(d_stats), _ptr(d_packed), _ptr(d_min_scale))
    _check(status, "daf_tensor_compress")


def daf_tensor_decompress(d_packed, width, d_min_scale, d_out, stream=None):
    status = _call(lib().daf_tensor_decompress, d_out, stream, dtype_code(d_out), _ptr(d_packed), d_out.numel(), width,
                   _ptr(d_min_scale), _ptr(d_out))
    _check(status, "daf_tensor_decompress")


def tensor_compress(x, width: int, *, rounding: int = ROUND_STOCHASTIC, seed: int = 0, elem_index_base: int = 0, stream=None):
    """Eq. 1 with one min / max / width for the whole tensor: (packed uint8 tensor, min_scale float tensor, stats)."""
    torch = _torch()
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("tensor_compress expects a contiguous CUDA tensor")
    stats = torch.empty(8, dtype=torch.int32, device=x.device)
    packed = torch.empty(max(x.numel() * width // 8, 16), dtype=torch.uint8, device=x.device)
    min_scale = torch.empty(2, dtype=torch.float32, device=x.device)
    daf_tensor_minmax(x, stats, stream)
    daf_tensor_compress(x, width, stats, packed, min_scale, rounding=rounding, seed=seed, elem_index_base=elem_index_base,
                        stream=stream)
    return packed, min_scale, stats


def tensor_decompress(packed, width: int, min_scale, shape, dtype, stream=None):
    out = _torch().empty(shape, dtype=dtype, device=packed.device)
    daf_tensor_decompress(packed, width, min_scale, out, stream)
    return out


class Pool:
    """Host-side page pool (bookkeeping only) over a caller-owned arena."""

    def __init__(self, arena_bytes: int, page_bytes: int = 0):
        self._h = lib().daf_pool_create(arena_bytes, page_bytes)
        if not self._h:
            raise DafError(ERR_INVALID_ARG, "daf_pool_create")

    def alloc(self, nbytes: int, importance: float):
        off = ctypes.c_uint64()
        h = int(lib().daf_pool_alloc(self._h, nbytes, importance, ctypes.byref(off)))
        return (h, int(off.value)) if h else (0, None)

    def free(self, handle: int):
        _check(lib().daf_pool_free(self._h, handle), "daf_pool_free")

    def evict_lowest(self) -> int:
        return int(lib().daf_pool_evict_lowest(self._h))

    def stats(self) -> dict:
        s = daf_pool_stats()
        _check(lib().daf_pool_get_stats(self._h, ctypes.byref(s)), "daf_pool_get_stats")
        return {n: int(getattr(s, n)) for n, _ in daf_pool_stats._fields_}

    def close(self):
        if self._h:
            lib().daf_pool_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def store_bytes(numel: int, group_size: int, width: int) -> int:
    """Bytes one activation occupies in a store at the given width (see daf_store_bytes)."""
    return int(lib().daf_store_bytes(numel, group_size, width))


class Store:
    """Importance-aware store (Sec. 3.4 of the paper): per-activation width under a memory and a time budget, two
    ordered indices, first-fit pages in an arena that follows the budget in steps.  Bookkeeping only."""

    NOT_STORED = (1 << 64) - 1
    _MAX_OUT = 4096

    def __init__(self, mem_budget_bytes: int, time_budget: float, widths=(1, 2, 4, 8), page_bytes: int = 0,
                 step_bytes: int = 0):
        cfg = daf_store_config(mem_budget_bytes, time_budget, page_bytes, step_bytes, width_mask(widths), 0)
        self._h = lib().daf_store_create(ctypes.byref(cfg))
        if not self._h:
            raise DafError(ERR_INVALID_ARG, "daf_store_create")

    def estimate(self, ident: int, numel: int, group_size: int, importance: float, time_cost: float, evicted=None) -> int:
        """Width planned for the activation; ids that lost their place in the call are appended to `evicted`."""
        w, n = ctypes.c_uint32(), ctypes.c_uint32(self._MAX_OUT)
        ev = (ctypes.c_uint64 * self._MAX_OUT)()
        _check(lib().daf_store_estimate(self._h, ident, numel, group_size, importance, time_cost, ctypes.byref(w), ev,
                                        ctypes.byref(n)), "daf_store_estimate")
        if evicted is not None:
            evicted.extend(int(ev[i]) for i in range(min(n.value, self._MAX_OUT)))
        return int(w.value)

    def admit(self, ident: int, importance: float):
        """(width, offset or None, ids evicted to make room)"""
        w, off, n = ctypes.c_uint32(), ctypes.c_uint64(), ctypes.c_uint32(self._MAX_OUT)
        ev = (ctypes.c_uint64 * self._MAX_OUT)()
        _check(lib().daf_store_admit(self._h, ident, importance, ctypes.byref(w), ctypes.byref(off), ev, ctypes.byref(n)),
               "daf_store_admit")
        return int(w.value), (None if off.value == self.NOT_STORED else int(off.value)), [int(ev[i]) for i in range(min(n.value, self._MAX_OUT))]

    def width(self, ident: int):
        w, off = ctypes.c_uint32(), ctypes.c_uint64()
        _check(lib().daf_store_width(self._h, ident, ctypes.byref(w), ctypes.byref(off)), "daf_store_width")
        return int(w.value), (None if off.value == self.NOT_STORED else int(off.value))

    def release(self, ident: int):
        _check(lib().daf_store_release(self._h, ident), "daf_store_release")

    def set_budget(self, mem_budget_bytes: int, time_budget: float):
        """(moves as (id, from, to, bytes), ids evicted)"""
        nm, ne = ctypes.c_uint32(self._MAX_OUT), ctypes.c_uint32(self._MAX_OUT)
        mv, ev = (daf_store_move * self._MAX_OUT)(), (ctypes.c_uint64 * self._MAX_OUT)()
        _check(lib().daf_store_set_budget(self._h, mem_budget_bytes, time_budget, mv, ctypes.byref(nm), ev, ctypes.byref(ne)),
               "daf_store_set_budget")
        return ([(int(m.id), int(m.from_offset), int(m.to_offset), int(m.bytes)) for m in mv[:min(nm.value, self._MAX_OUT)]],
                [int(ev[i]) for i in range(min(ne.value, self._MAX_OUT))])

    def stats(self) -> dict:
        s = daf_store_stats()
        _check(lib().daf_store_get_stats(self._h, ctypes.byref(s)), "daf_store_get_stats")
        return {n: getattr(s, n) for n, _ in daf_store_stats._fields_}

    def close(self):
        if self._h:
            lib().daf_store_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class HostRoundTrip:
    """Compress + decompress of a tensor that lives in pinned HOST memory, streamed through the device in window-aligned
    chunks: while chunk i is compressed and restored, chunk i+1 is on its way in and chunk i-1 on its way out (three
    streams, two sets of device buffers).  The chunks are shards in the sense of daf_shard -- same seed, counter base
    moved -- so the restored values are exactly those of one call on the whole tensor.  The packed form of a chunk only
    lives until the next chunk reuses its slot: this is the end-to-end path of the benchmark and of callers that want
    the effect of the round trip (what the backward pass will see), not a way to keep the packed bytes."""

    def __init__(self, dtype, group_size: int, widths, bit_budget: float, *, seed: int = 0, rounding: int = ROUND_STOCHASTIC,
                 chunk_elems: int = 1 << 25, device="cuda"):
        torch = _torch()
        if chunk_elems % DEFAULT_WINDOW:
            raise ValueError("chunk_elems must be a multiple of the window")
        self.kw = dict(group_size=group_size, widths=tuple(widths), bit_budget=float(bit_budget), seed=seed, rounding=rounding)
        self.chunk, self.device = int(chunk_elems), torch.device(device)
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream(self.device) for _ in range(3))
        self.x = [torch.empty(self.chunk, dtype=dtype, device=self.device) for _ in range(2)]
        self.y = [torch.empty(self.chunk, dtype=dtype, device=self.device) for _ in range(2)]
        code = dtype_code(self.x[0])
        full = make_params(code, self.chunk, group_size, widths, bit_budget, rounding=rounding, seed=seed)
        self.c = [alloc_outputs(full, self.device) for _ in range(2)]
        self.free = [torch.cuda.Event() for _ in range(2)]

    def __call__(self, h_in, h_out) -> None:
        """h_in, h_out: flat pinned host tensors of the same length (a multiple of the group size).  Returns when the
        work has been enqueued; the calling stream waits for it (so events recorded on it afterwards see it done)."""
        torch = _torch()
        n = h_in.numel()
        cur = torch.cuda.current_stream(self.device)
        for s in (self.s_in, self.s_run, self.s_out):
            s.wait_stream(cur)
        for i, lo in enumerate(range(0, n, self.chunk)):
            m, k = min(self.chunk, n - lo), i & 1
            ev_in, ev_run = torch.cuda.Event(), torch.cuda.Event()
            with torch.cuda.stream(self.s_in):
                if i >= 2:
                    self.s_in.wait_event(self.free[k])            # the slot's last chunk has left the device
                self.x[k][:m].copy_(h_in[lo:lo + m], non_blocking=True)
                ev_in.record()
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(ev_in)
                kw = self.kw
                c = compress(self.x[k][:m], kw["group_size"], kw["widths"], kw["bit_budget"], rounding=kw["rounding"],
                             seed=kw["seed"], elem_index_base=lo, out=self.c[k] if m == self.chunk else None)
                decompress(c, out=self.y[k][:m])
                ev_run.record()
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(ev_run)
                h_out[lo:lo + m].copy_(self.y[k][:m], non_blocking=True)
                self.free[k].record()
        cur.wait_stream(self.s_out)
