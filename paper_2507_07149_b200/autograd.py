"""Training integration: saved activations held in compressed form between forward and backward.

``saved_activation_compression`` is a ``torch.autograd.graph.saved_tensors_hooks`` context.  Inside
it every eligible tensor that autograd saves for the backward pass goes through ``daf_compress``
when it is saved and through ``daf_decompress`` when the backward pass asks for it (the end-to-end
flow of Sec. 3.1 / Fig. 3(a): compress after the layer's forward, keep the packed form, restore
right before the layer's backward).  Both steps run in the CUDA kernels behind the C ABI; this
module only decides which tensors take the path and keeps the handles.

Eligible: CUDA tensors of dtype float32 / float16 / bfloat16 that are not parameters, hold at least
``min_numel`` elements and whose element count is a multiple of the group size.  Everything else
(weights, index tensors, small or ragged tensors) is saved as it is.

Stochastic rounding draws from one Philox stream per context: tensor i starts at the element index
where tensor i-1 ended (rounded up to a multiple of 8), so no two saved tensors of one step share
random numbers; ``reseed`` moves to a new key for the next step.
"""
from __future__ import annotations

import torch

from . import ROUND_STOCHASTIC, CompressedTensor, compress, decompress

_DTYPES = (torch.float32, torch.float16, torch.bfloat16)


class _Saved:
    """What the context keeps for one compressed activation."""

    __slots__ = ("c", "shape", "nbytes_in", "nbytes_kept")

    def __init__(self, c: CompressedTensor, shape, nbytes_in: int, nbytes_kept: int):
        self.c, self.shape, self.nbytes_in, self.nbytes_kept = c, shape, nbytes_in, nbytes_kept


class saved_activation_compression(torch.autograd.graph.saved_tensors_hooks):
    """Context manager: compress what autograd saves, decompress when the backward pass reads it.

    group_size, widths, bit_budget, rounding: as for ``compress``.
    min_numel: tensors smaller than this stay uncompressed.
    trim: copy the used prefix of the packed buffer into a right-sized allocation and drop the
        worst-case-sized one and the workspace (one device-to-host read of the total size per
        tensor); without it the packed buffer keeps its worst-case capacity.
    """

    def __init__(self, group_size: int = 256, widths=(1, 2, 4, 8), bit_budget: float = 4.0, *, seed: int = 0,
                 rounding: int = ROUND_STOCHASTIC, min_numel: int = 16384, trim: bool = True):
        self.group_size, self.widths, self.bit_budget = int(group_size), tuple(widths), float(bit_budget)
        self.seed, self.rounding, self.min_numel, self.trim = int(seed), int(rounding), int(min_numel), bool(trim)
        self._next_index = 0
        self.stats = {"tensors": 0, "bytes_in": 0, "bytes_kept": 0, "passed_through": 0}
        super().__init__(self._pack, self._unpack)

    def reseed(self, seed: int) -> None:
        """New Philox key and a fresh element counter (call once per training step)."""
        self.seed, self._next_index = int(seed), 0

    def _eligible(self, t) -> bool:
        return (t.is_cuda and t.dtype in _DTYPES and not isinstance(t, torch.nn.Parameter)
                and t.numel() >= self.min_numel and t.numel() % self.group_size == 0)

    def _pack(self, t):
        if not self._eligible(t):
            self.stats["passed_through"] += 1
            return t
        x = t.detach().contiguous()
        c = compress(x, self.group_size, self.widths, self.bit_budget, rounding=self.rounding, seed=self.seed,
                     elem_index_base=self._next_index, check=self.trim)
        self._next_index += (x.numel() + 7) & ~7
        if self.trim:
            c.packed = c.packed[:max(c.packed_bytes(), 16)].clone()
            c.workspace = None
        kept = sum(b.numel() * b.element_size() for b in (c.packed, c.bits, c.min, c.scale, c.window_offsets))
        nbytes = x.numel() * x.element_size()
        self.stats["tensors"] += 1
        self.stats["bytes_in"] += nbytes
        self.stats["bytes_kept"] += kept
        return _Saved(c, t.shape, nbytes, kept)

    def _unpack(self, s):
        if not isinstance(s, _Saved):
            return s
        return decompress(s.c).view(s.shape)


class _ReluSavedCompressed(torch.autograd.Function):
    """ReLU whose output is written and compressed in one pass (daf_relu_compress); the backward pass
    masks the gradient with the output restored from the packed form (daf_decompress_relu_grad: the
    restored output is never written)."""

    @staticmethod
    def forward(ctx, x, module):
        from . import relu_compress
        act, c = relu_compress(x.contiguous(), module.group_size, module.widths, module.bit_budget, rounding=module.rounding,
                               seed=module.seed, elem_index_base=module._next_index, check=module.trim)
        module._next_index += (x.numel() + 7) & ~7
        if module.trim:
            c.packed = c.packed[:max(c.packed_bytes(), 16)].clone()
            c.workspace = None
        ctx.saved = c
        ctx.shape = x.shape
        return act.view(x.shape)

    @staticmethod
    def backward(ctx, grad_out):
        from . import relu_grad
        c = ctx.saved
        if grad_out.dtype != {0: torch.float32, 1: torch.float16, 2: torch.bfloat16}[int(c.params.dtype)]:
            y = decompress(c).view(ctx.shape)                     # gradient in another type: mask in torch
            return grad_out * (y > 0).to(grad_out.dtype), None
        return relu_grad(c, grad_out.reshape(-1)).view(ctx.shape), None   # one pass: packed + gradient in, gradient out


class CompressedReLU(torch.nn.Module):
    """ReLU layer that keeps its output for the backward pass in compressed form only, produced by the
    fused kernel (the activation crosses device memory once: read x, write relu(x) and its packed form).
    Inputs that do not qualify (see ``saved_activation_compression``) go through ``torch.relu``."""

    def __init__(self, group_size: int = 256, widths=(1, 2, 4, 8), bit_budget: float = 4.0, *, seed: int = 0,
                 rounding: int = ROUND_STOCHASTIC, min_numel: int = 16384, trim: bool = True):
        super().__init__()
        self.group_size, self.widths, self.bit_budget = int(group_size), tuple(widths), float(bit_budget)
        self.seed, self.rounding, self.min_numel, self.trim = int(seed), int(rounding), int(min_numel), bool(trim)
        self._next_index = 0

    def reseed(self, seed: int) -> None:
        self.seed, self._next_index = int(seed), 0

    def forward(self, x):
        ok = (x.is_cuda and x.dtype in _DTYPES and x.numel() >= self.min_numel and x.numel() % self.group_size == 0
              and torch.is_grad_enabled() and x.requires_grad)
        return _ReluSavedCompressed.apply(x, self) if ok else torch.relu(x)
