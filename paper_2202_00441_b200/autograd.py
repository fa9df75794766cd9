"""Drop-in activation modules over the C ABI (Listing 1 as a PyTorch layer).

``FewBitActivation("gelu", bits=3)`` replaces ``nn.GELU()``: the forward pass
returns the exact activation, autograd keeps only ``bits`` bits per element
(the packed interval codes) instead of the input, and the backward pass
multiplies the incoming gradient by the level of each element's interval.
Only argument marshalling happens here; both passes run in the CUDA library.
"""
from __future__ import annotations

import torch
from torch import nn

from .binding import Table, fewbit_bwd, fewbit_fwd, fewbit_fwd_bias, fewbit_table_create, fewbit_table_create_folded


def _flat_aligned(t: torch.Tensor) -> torch.Tensor:
    t = t.contiguous().view(-1)
    if t.data_ptr() % 32:                 # a view into the middle of a buffer: the library wants 32-byte alignment
        t = t.clone()
    return t


class _FewBitFunction(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x: torch.Tensor, table: Table):
        if x.dtype not in (torch.float32, torch.bfloat16, torch.float16) or not x.is_cuda:
            raise TypeError("FewBitActivation needs a CUDA tensor of dtype float32, bfloat16 or float16")
        y, packed = fewbit_fwd(table, _flat_aligned(x))
        ctx.table = table
        ctx.save_for_backward(packed)     # bits/8 bytes per element; x itself is not kept
        return y.view(x.shape)

    @staticmethod
    def backward(ctx, grad_out: torch.Tensor):
        (packed,) = ctx.saved_tensors
        grad_in = fewbit_bwd(ctx.table, packed, _flat_aligned(grad_out))
        return grad_in.view(grad_out.shape), None


class _FewBitBiasFunction(torch.autograd.Function):
    """f(x + bias) with the bias add inside the forward kernel; the gradient with respect to the
    bias is the column sum of the gradient with respect to x (accumulated in binary32)."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, bias: torch.Tensor, table: Table):
        if x.dtype not in (torch.float32, torch.bfloat16, torch.float16) or not x.is_cuda:
            raise TypeError("FewBitActivation needs a CUDA tensor of dtype float32, bfloat16 or float16")
        cols = bias.numel()
        xf = x.contiguous()
        if xf.data_ptr() % 32:
            xf = xf.clone()
        y, packed = fewbit_fwd_bias(table, xf.view(-1, cols), _flat_aligned(bias.to(x.dtype)))
        ctx.table, ctx.bias_dtype = table, bias.dtype
        ctx.save_for_backward(packed)
        return y.view(x.shape)

    @staticmethod
    def backward(ctx, grad_out: torch.Tensor):
        (packed,) = ctx.saved_tensors
        grad_in = fewbit_bwd(ctx.table, packed, _flat_aligned(grad_out)).view(grad_out.shape)
        grad_bias = grad_in.reshape(-1, grad_out.shape[-1]).sum(0, dtype=torch.float32).to(ctx.bias_dtype)
        return grad_in, grad_bias, None


class FewBitActivation(nn.Module):
    """Activation whose backward pass uses a ``bits``-bit piecewise-constant derivative.

    act: gelu | silu | sigmoid | tanh | elu | softplus | leaky_relu | relu | selu.
    folded: for sigmoid / tanh, quantise |x| (one more effective bit)."""

    def __init__(self, act: str = "gelu", bits: int = 3, folded: bool = False):
        super().__init__()
        self.act, self.bits, self.folded = act, int(bits), bool(folded)
        self.table = fewbit_table_create_folded(act, bits) if folded else fewbit_table_create(act, bits)

    def forward(self, x: torch.Tensor, bias: torch.Tensor | None = None) -> torch.Tensor:
        """``bias`` (optional): one value per element of the last dimension of ``x`` (a multiple of
        8), added to ``x`` inside the kernel."""
        if bias is not None:
            return _FewBitBiasFunction.apply(x, bias, self.table)
        return _FewBitFunction.apply(x, self.table)

    def extra_repr(self) -> str:
        return f"act={self.act}, bits={self.bits}, folded={self.folded}"


def fewbit_activation(x: torch.Tensor, table: Table, bias: torch.Tensor | None = None) -> torch.Tensor:
    """Functional form: ``table`` from ``fewbit_table_create``; with ``bias``, f(x + bias)."""
    if bias is not None:
        return _FewBitBiasFunction.apply(x, bias, table)
    return _FewBitFunction.apply(x, table)
