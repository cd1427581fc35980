"""Training integration: saved activations held in compressed form between forward and backward.

``saved_activation_compression`` is a ``torch.autograd.graph.saved_tensors_hooks`` context.  Inside
it every eligible tensor that autograd saves for the backward pass is compressed (``daf_compress_batch``)
and restored with ``daf_decompress`` when the backward pass asks for it (the end-to-end flow of
Sec. 3.1 / Fig. 3(a): compress after the layer's forward, keep the packed form, restore right before
the layer's backward).  Both steps run in the CUDA kernels behind the C ABI; this module only decides
which tensors take the path, where their packed form lives, and keeps the handles.

Which saved tensors are compressed.  The hook sees EVERY tensor an operation saves, not only layer
outputs: inputs of convolutions and matrix products, outputs of ReLU / softmax / GELU inputs,
normalisation inputs, and also tensors derived from weights (a transposed or cast copy of a weight
under autocast is no longer a ``Parameter``).  Eligible are CUDA tensors of dtype float32 / float16 /
bfloat16 that are not ``Parameter``s (nor views of one), hold at least ``min_numel`` elements, whose
element count is a multiple of the group size, and for which ``exclude(tensor)`` (if given) is false.
Everything else (weights, index tensors, small or ragged tensors) is saved as it is.  A tensor that
is not contiguous or does not start on a 32-byte boundary (an offset view) is copied first.

Launches.  Saved tensors are queued and compressed ``batch`` at a time (at most 64) by ONE call of
``daf_compress_batch`` per dtype and width; the queue is also flushed when its tensors hold more than
``batch_bytes``, when the context exits and before anything queued is read back.  Until a tensor's
batch is flushed it stays alive uncompressed, so ``batch`` and ``batch_bytes`` bound the extra memory.
Nothing in the forward path reads a value back from the device: the packed form gets the capacity
the bit budget guarantees (``numel * width / 8``) and keeps it; ``check_status`` reads the status
words of all batches since the last call, once.

Where the packed form lives.  Without a memory budget each batch gets one torch allocation, carved
into the tensors' parts.  With ``mem_budget`` the context owns one arena of that size and a
``Store`` (Sec. 3.4: Alg. 3) that decides, per activation, the width (the context's ``bit_budget`` at
most) and the pages, under the memory budget and an optional time budget, from an importance the
caller supplies (``importance(index, tensor) -> float``, 1 for all by default; the store sees its
moving average before the activation arrives and the value itself when it does).  An activation the
store drops (width 0), or evicts later to make room, is NOT kept: the backward pass gets zeros in its
place, so the weight gradient that needed it is zero for that step (the paper's "fewer weights
updated").

Stochastic rounding draws from one Philox stream per context: tensor i starts at the element index
where tensor i-1 ended (rounded up to a multiple of 8), so no two saved tensors of one step share
random numbers; ``reseed`` moves to a new key for the next step.
"""
from __future__ import annotations

import weakref

import torch

import ctypes

from . import (ACT_GELU, ACT_RELU, ACT_RELU6, BATCH_MAX, ROUND_STOCHASTIC, Store, _call, _check, daf_params, daf_poll_status,
               daf_sizes, dtype_code, lib, make_params)

_DTYPES = (torch.float32, torch.float16, torch.bfloat16)
_ALIGN = 32


def _aligned_contiguous(t):
    """t itself when the kernels can read it in place, else a contiguous copy (fresh allocations are aligned)."""
    x = t.detach()
    if not x.is_contiguous():
        x = x.contiguous()
    if x.data_ptr() % _ALIGN:
        x = x.clone()
    return x


def _up16(v: int) -> int:
    return (v + 15) & ~15


def _layout(params, packed_bytes=None):
    """Byte offsets of one compressed tensor's parts inside its allocation, in the order and with the padding of
    daf_store_bytes: window offsets, min, scale, packed codes (packed_bytes of them; by default the capacity the
    budget guarantees), widths.  Returns (sizes, (o_min, o_scale, o_packed, o_bits, total))."""
    sz = daf_sizes(params)
    ng, nw = sz.n_groups, sz.n_windows
    pb = sz.packed_capacity if packed_bytes is None else packed_bytes
    assert sz.packed_capacity <= pb
    o_min = _up16(8 * (nw + 1))
    o_scale = o_min + _up16(4 * ng)
    o_packed = o_scale + _up16(4 * ng)
    o_bits = o_packed + _up16(pb)
    return sz, (o_min, o_scale, o_packed, o_bits, o_bits + _up16(ng))


class _Saved:
    """What the context keeps for one saved activation: the tensor itself while it is queued, then its parts."""

    # block, at, lay, params: where the compressed form lives (a uint8 tensor, the byte it starts at, the offsets of its parts
    # as _layout gives them) and the parameters it was compressed with; set when the handle's batch has been launched
    __slots__ = ("owner", "ident", "x", "block", "at", "lay", "params", "shape", "dtype", "device", "width", "offset",
                 "dropped", "kept", "__weakref__")

    def __init__(self, owner, ident, x, shape, width, offset):
        self.owner, self.ident, self.x = owner, ident, x
        self.block, self.at, self.lay, self.params = None, 0, None, None
        self.shape, self.dtype, self.device = shape, x.dtype, x.device
        self.width, self.offset, self.dropped, self.kept = width, offset, width == 0, 0

    def __del__(self):
        owner = self.owner
        if owner is not None and owner._store is not None:
            try:
                owner._store.release(self.ident)
                owner._announced.discard(self.ident)
            except Exception:
                pass


class saved_activation_compression(torch.autograd.graph.saved_tensors_hooks):
    """Context manager: compress what autograd saves, decompress when the backward pass reads it.

    group_size, widths, bit_budget, rounding: as for ``compress``.  With a store, bit_budget must be an allowed
    width: the largest one an activation can get (each window then has that width throughout).
    min_numel: tensors smaller than this stay uncompressed.  exclude: predicate on the saved tensor.
    batch, batch_bytes: queue limits (see the module text).
    mem_budget (bytes), time_budget (seconds per step; None = unlimited), importance, step_bytes: the store.
    """

    def __init__(self, group_size: int = 256, widths=(1, 2, 4, 8), bit_budget: float = 4.0, *, seed: int = 0,
                 rounding: int = ROUND_STOCHASTIC, min_numel: int = 16384, exclude=None, batch: int = 16,
                 batch_bytes: int = 256 << 20, mem_budget: int | None = None, time_budget: float | None = None,
                 importance=None, step_bytes: int = 0, device=None):
        self.group_size, self.widths = int(group_size), tuple(sorted(int(w) for w in widths))
        if mem_budget is not None and (int(bit_budget) != bit_budget or int(bit_budget) not in self.widths):
            raise ValueError("with a store, bit_budget must be one of the allowed widths")
        self.bit_budget = int(bit_budget) if mem_budget is not None else float(bit_budget)
        self.seed, self.rounding, self.min_numel = int(seed), int(rounding), int(min_numel)
        self.exclude, self.importance = exclude, importance
        self.batch, self.batch_bytes = max(1, min(int(batch), BATCH_MAX)), int(batch_bytes)
        self._next_index = 0
        self._count = 0                                             # saved tensors seen this step (the store's ids)
        self._queue, self._queued_bytes, self._queued_by_key = [], 0, {}
        self._workspaces = []                                       # one per batch since the last check_status
        self._ma = {}                                               # position in the step -> moving average of the importance
        self._shapes = {}                                           # position in the step -> (numel, time cost) seen last
        self._base, self._announced = 0, set()                      # the step's id range; ids the store has an entry for
        self._handles = weakref.WeakValueDictionary()
        self._store, self._arena = None, None
        self._layouts = {}                                          # (dtype, numel, budget, packed bytes) -> (params, sizes, offsets)
        if mem_budget is not None:
            allowed = [w for w in self.widths if w <= self.bit_budget]
            self._store = Store(int(mem_budget), float("1e30") if time_budget is None else float(time_budget), allowed,
                                step_bytes=step_bytes)
            self._arena = torch.empty(int(mem_budget), dtype=torch.uint8, device=device if device is not None else "cuda")
        self.stats = {"tensors": 0, "bytes_in": 0, "bytes_kept": 0, "passed_through": 0, "dropped": 0, "launches": 0, "shared": 0}
        super().__init__(self._pack, self._unpack)

    # ---------------------------------------------------------------------------------------- step bookkeeping
    def reseed(self, seed: int) -> None:
        """New Philox key and a fresh element counter (call once per training step, before the forward pass).  With a
        store, this is also the pre-iteration estimate of Alg. 3: every activation seen last step is announced with its
        size and the moving average of its importance."""
        self.seed, self._next_index = int(seed), 0
        self._new_step()

    def _new_step(self) -> None:
        self.flush()
        if self._store is not None:
            for ident in self._announced:                           # announced last step but never saved
                if ident not in self._handles:
                    self._store.release(ident)
            self._base += 1 << 24                                   # ids are never reused while old handles may live
            self._announced = set()
            gone = []
            for pos, (numel, cost) in self._shapes.items():
                self._store.estimate(self._base + pos, numel, self.group_size, self._ma.get(pos, 1.0), cost, gone)
                self._announced.add(self._base + pos)
            for e in gone:                                          # something of an earlier step that is still alive
                h = self._handles.get(e)
                if h is not None:
                    self._drop(h)
        self._count = 0

    def __enter__(self):
        if self._count and not len(self._handles):                  # a new forward pass and nothing of the last one is alive
            self._new_step()
        return super().__enter__()

    def check_status(self) -> None:
        """Waits for the work queued so far and raises if a batch recorded a device-side error."""
        self.flush()
        ws, self._workspaces = self._workspaces, []
        for w in ws:
            _check(daf_poll_status(w), "daf_compress_batch (device status)")

    def __exit__(self, *exc):
        out = super().__exit__(*exc)
        self.flush()
        return out

    def set_budget(self, mem_budget: int, time_budget: float | None = None) -> None:
        """New budgets for the store (Sec. 3.4.4); activations that no longer fit are dropped, those beyond the new end
        of the arena are copied to where the store moved them.  The arena tensor itself keeps its size."""
        if self._store is None or mem_budget > self._arena.numel():
            raise ValueError("set_budget needs a store and a budget within the arena that was reserved")
        self.flush()
        moves, evicted = self._store.set_budget(int(mem_budget), float("1e30") if time_budget is None else float(time_budget))
        for e in evicted:
            h = self._handles.get(e)
            if h is not None:
                self._drop(h)
        for ident, src, dst, nbytes in moves:
            h = self._handles.get(ident)
            if h is None:
                continue
            self._arena[dst:dst + nbytes].copy_(self._arena[src:src + nbytes].clone())   # the ranges may overlap
            h.offset = dst
            if h.block is not None:
                h.at = dst

    # ---------------------------------------------------------------------------------------- hooks
    def _eligible(self, t) -> bool:
        if not (t.is_cuda and t.dtype in _DTYPES and t.numel() >= self.min_numel and t.numel() % self.group_size == 0):
            return False
        if isinstance(t, torch.nn.Parameter) or isinstance(getattr(t, "_base", None), torch.nn.Parameter):
            return False
        if self._arena is not None and t.device != self._arena.device:
            return False
        return not (self.exclude is not None and self.exclude(t))

    @staticmethod
    def _time_cost(x) -> float:
        return 2.0 * x.numel() * x.element_size() / 5.0e12          # read once to compress, written once to restore

    def _pack(self, t):
        if not self._eligible(t):
            self.stats["passed_through"] += 1
            return t
        # the same tensor is often saved twice in a row (a ReLU keeps its output, the next layer its input): while the
        # first handle is still queued, and so keeps the storage alive, the second save shares it
        key = (t.data_ptr(), t._version, tuple(t.shape), t.stride(), t.dtype)
        h = self._queued_by_key.get(key)
        if h is not None:
            self.stats["shared"] += 1
            return h
        x = _aligned_contiguous(t)
        pos, self._count = self._count, self._count + 1
        ident = self._base + pos
        width, offset = self.bit_budget, None
        if self._store is not None:
            measured = 1.0 if self.importance is None else float(self.importance(pos, t))
            shape = (x.numel(), self._time_cost(x))
            ma = self._ma.get(pos)
            gone = []
            if ident not in self._announced or self._shapes.get(pos) != shape:
                self._store.estimate(ident, shape[0], self.group_size, measured if ma is None else ma, shape[1], gone)
                self._announced.add(ident)
            self._shapes[pos] = shape
            self._ma[pos] = measured if ma is None else 0.9 * ma + 0.1 * measured
            width, offset, evicted = self._store.admit(ident, measured)
            evicted = gone + evicted
            for e in evicted:
                h = self._handles.get(e)
                if h is not None and e != ident:
                    self._drop(h)
        h = _Saved(self, ident, x, t.shape, width, offset)
        self._handles[ident] = h
        nbytes = x.numel() * x.element_size()
        self.stats["tensors"] += 1
        self.stats["bytes_in"] += nbytes
        if width == 0:
            h.x = None
            self.stats["dropped"] += 1
            return h
        h.kept = self._layout_of(dtype_code(x), x.numel(), width)[2][4]
        self.stats["bytes_kept"] += h.kept
        self._queue.append(h)
        self._queued_bytes += nbytes
        if x.data_ptr() == t.data_ptr():
            self._queued_by_key[key] = h
        if len(self._queue) >= self.batch or self._queued_bytes >= self.batch_bytes:
            self.flush()
        return h

    def _drop(self, h) -> None:
        """The store took this activation's pages away: forget its data."""
        if not h.dropped:
            self.stats["dropped"] += 1
            self.stats["bytes_kept"] -= h.kept
        h.dropped, h.x, h.block = True, None, None
        if h in self._queue:
            self._queue.remove(h)
            for k in [k for k, v in self._queued_by_key.items() if v is h]:
                del self._queued_by_key[k]

    def _unpack(self, s):
        if not isinstance(s, _Saved):
            return s
        if s.dropped:
            return torch.zeros(s.shape, dtype=s.dtype, device=s.device)
        if s.block is None:
            self.flush()
        out = torch.empty(s.shape, dtype=s.dtype, device=s.device)
        b = s.block.data_ptr() + s.at
        o_min, o_scale, o_packed, o_bits, _ = s.lay
        status = _call(lib().daf_decompress, out, None, ctypes.byref(s.params), b + o_packed, b + o_bits, b + o_min, b + o_scale, b,
                       out.data_ptr(), 0, 0)
        _check(status, "daf_decompress")
        return out

    def _layout_of(self, code: int, numel: int, width):
        """(parameters without seed and counter base, sizes, offsets of the parts) for a tensor of this type, size and
        budget; remembered, since a model saves the same shapes every step."""
        key = (code, numel, width)
        v = self._layouts.get(key)
        if v is None:
            p = make_params(code, numel, self.group_size, self.widths, float(width), rounding=self.rounding)
            sz, offs = _layout(p, numel * int(width) // 8 if self._arena is not None else None)
            v = self._layouts[key] = (p, sz, offs)
        return v

    # ---------------------------------------------------------------------------------------- the batched launch
    def flush(self) -> None:
        """Compresses everything queued: one daf_compress_batch call per (device, dtype, width)."""
        queue, self._queue, self._queued_bytes = self._queue, [], 0
        self._queued_by_key.clear()
        groups = {}
        for h in queue:
            if not h.dropped:
                groups.setdefault((h.device, h.dtype, h.width), []).append(h)
        for (device, _, width), hs in groups.items():
            for i in range(0, len(hs), BATCH_MAX):
                self._launch(device, width, hs[i:i + BATCH_MAX])

    def _launch(self, device, width, hs) -> None:
        n = len(hs)
        lays = [self._layout_of(dtype_code(h.x), h.x.numel(), width) for h in hs]
        if self._arena is not None:
            block, starts = self._arena, [h.offset for h in hs]
        else:
            starts, total = [], 0
            for lay in lays:
                starts.append(total)
                total += (lay[2][4] + 255) & ~255
            block = torch.empty(total, dtype=torch.uint8, device=device)
        base = block.data_ptr()
        arr = (daf_params * n)()
        ptrs = [(ctypes.c_void_p * n)() for _ in range(6)]          # in, packed, bits, min, scale, window offsets
        caps = (ctypes.c_uint64 * n)()
        for i, (h, (tmpl, sz, (o_min, o_scale, o_packed, o_bits, _)), at) in enumerate(zip(hs, lays, starts)):
            arr[i] = tmpl
            arr[i].seed, arr[i].elem_index_base = self.seed, self._next_index
            self._next_index += (h.x.numel() + 7) & ~7
            b = base + at
            ptrs[0][i], ptrs[1][i], ptrs[2][i] = h.x.data_ptr(), b + o_packed, b + o_bits
            ptrs[3][i], ptrs[4][i], ptrs[5][i] = b + o_min, b + o_scale, b
            caps[i] = sz.packed_capacity
        ws_bytes = int(lib().daf_batch_workspace(n, arr))
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        status = _call(lib().daf_compress_batch, hs[0].x, None, n, arr, ptrs[0], ptrs[1], caps, ptrs[2], ptrs[3], ptrs[4], ptrs[5],
                       ws.data_ptr(), ws_bytes)
        _check(status, "daf_compress_batch")
        self._workspaces.append(ws)
        self.stats["launches"] += 1
        for i, (h, lay, at) in enumerate(zip(hs, lays, starts)):
            h.block, h.at, h.lay, h.params = block, at, lay[2], daf_params.from_buffer_copy(arr[i])
            h.x = None                                              # the uncompressed tensor can go now


class _ReluSavedCompressed(torch.autograd.Function):
    """Activation whose output is written and whose saved tensor is compressed in one pass (daf_act_compress); the
    backward pass forms the gradient from the packed form (daf_decompress_act_grad: the restored tensor is never
    written).  ReLU and ReLU6 keep their output, GELU its input."""

    @staticmethod
    def forward(ctx, x, module):
        from . import relu_compress
        xin = _aligned_contiguous(x)
        act, c = relu_compress(xin, module.group_size, module.widths, module.bit_budget, rounding=module.rounding,
                               seed=module.seed, elem_index_base=module._next_index, check=module.trim, act=module.act)
        module._next_index += (x.numel() + 7) & ~7
        if module.trim:
            c.packed = c.packed[:max(c.packed_bytes(), 16)].clone()
        c.workspace = None
        ctx.saved = c
        ctx.shape = x.shape
        ctx.act = module.act
        return act.view(x.shape)

    @staticmethod
    def backward(ctx, grad_out):
        from . import relu_grad
        c = ctx.saved
        if dtype_code(grad_out) != int(c.params.dtype):
            # autograd hands a function gradients in the type of its forward output, so this is a caller's error
            raise TypeError("the gradient of a CompressedReLU must have the dtype of its output")
        g = grad_out.reshape(-1)
        if not g.is_contiguous() or g.data_ptr() % _ALIGN:
            g = g.contiguous() if not g.is_contiguous() else g.clone()
            if g.data_ptr() % _ALIGN:
                g = g.clone()
        return relu_grad(c, g, act=ctx.act).view(ctx.shape), None   # one pass: packed + gradient in, gradient out


class CompressedReLU(torch.nn.Module):
    """ReLU layer that keeps its output for the backward pass in compressed form only, produced by the
    fused kernel (the activation crosses device memory once: read x, write relu(x) and its packed form).
    Inputs that do not qualify (see ``saved_activation_compression``) go through ``torch.relu``; an input that is
    not contiguous or not 32-byte aligned is copied first.  ``trim`` copies the used part of the packed buffer into
    a right-sized allocation, at the price of one device-to-host read per call; without it the buffer keeps the
    capacity the budget guarantees and the forward pass never waits for the device."""

    act = ACT_RELU
    _plain = staticmethod(torch.relu)

    def __init__(self, group_size: int = 256, widths=(1, 2, 4, 8), bit_budget: float = 4.0, *, seed: int = 0,
                 rounding: int = ROUND_STOCHASTIC, min_numel: int = 16384, trim: bool = False):
        super().__init__()
        self.group_size, self.widths, self.bit_budget = int(group_size), tuple(widths), float(bit_budget)
        self.seed, self.rounding, self.min_numel, self.trim = int(seed), int(rounding), int(min_numel), bool(trim)
        self._next_index = 0

    def reseed(self, seed: int) -> None:
        self.seed, self._next_index = int(seed), 0

    def forward(self, x):
        ok = (x.is_cuda and x.dtype in _DTYPES and x.numel() >= self.min_numel and x.numel() % self.group_size == 0
              and torch.is_grad_enabled() and x.requires_grad)
        return _ReluSavedCompressed.apply(x, self) if ok else self._plain(x)


class CompressedReLU6(CompressedReLU):
    """ReLU6 with its output kept compressed; the gradient passes where the restored output is strictly inside (0, 6)."""
    act = ACT_RELU6
    _plain = staticmethod(torch.nn.functional.relu6)


class CompressedGELU(CompressedReLU):
    """GELU (erf form) that keeps its INPUT compressed; the backward pass multiplies the gradient by GELU' at the
    restored input."""
    act = ACT_GELU
    _plain = staticmethod(torch.nn.functional.gelu)
