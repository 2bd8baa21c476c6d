"""torch.autograd wrapper around the C-ABI calls, for use inside a model.

    from paper_2603_08343_b200.autograd import wht_affine
    out = wht_affine(heads_concat, a, b)                 # y = a (.) (x H)/sqrt(d) + b
    out = wht_affine(heads_concat, a, b, resid=hidden)   # y = resid + ...   (one kernel)

Argument marshalling only: the forward is wht_affine_fwd / wht_affine_fwd_residual, the backward
is wht_affine_bwd (which recomputes z from the saved x); the gradient of the residual input is
the incoming gradient itself.  x may have any leading shape; its last dimension is d.
"""
from __future__ import annotations

import torch

from . import binding as B


class _WhtAffine(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, a, b, resid):
        xc = x.contiguous()
        rc = None if resid is None else resid.contiguous()
        y = B.forward(xc.view(-1, xc.shape[-1]), a, b, resid=None if rc is None else rc.view(-1, rc.shape[-1]))
        ctx.save_for_backward(xc, a)
        ctx.has_resid = resid is not None
        ctx.param_dtype = a.dtype
        return y.view(xc.shape)

    @staticmethod
    def backward(ctx, dy):
        x, a = ctx.saved_tensors
        d = x.shape[-1]
        dyc = dy.contiguous().view(-1, d)
        dx, da, db = B.backward(dyc, x.view(-1, d), a)
        return (dx.view(x.shape), da.to(ctx.param_dtype), db.to(ctx.param_dtype),
                dy if ctx.has_resid else None)


def wht_affine(x: torch.Tensor, a: torch.Tensor, b: torch.Tensor, resid: torch.Tensor | None = None) -> torch.Tensor:
    """Differentiable y = [resid +] a (.) (x H_d)/sqrt(d) + b over the last dimension of x."""
    return _WhtAffine.apply(x, a, b, resid)


class _WhtAffineGrouped(torch.autograd.Function):
    """Block-diagonal form (d = groups * block): every block of channels has its own transform."""

    @staticmethod
    def forward(ctx, x, a, b, block):
        xc = x.contiguous()
        d = xc.shape[-1]
        T = xc.numel() // d
        y = torch.empty_like(xc)
        B.wht_affine_fwd_grouped(xc, a, b, y, T, d, block, B.dtype_code(xc, a))
        ctx.save_for_backward(xc, a)
        ctx.block = block
        return y

    @staticmethod
    def backward(ctx, dy):
        x, a = ctx.saved_tensors
        d, block = x.shape[-1], ctx.block
        T = x.numel() // d
        code = B.dtype_code(x, a)
        dyc = dy.contiguous()
        dx = torch.empty_like(x)
        da = torch.empty(d, dtype=torch.float32, device=x.device)
        db = torch.empty_like(da)
        need = B.wht_affine_bwd_grouped_workspace_bytes(T, d, block, code)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=x.device)
        B.wht_affine_bwd_grouped(dyc, x, a, dx, da, db, T, d, block, code, ws)
        return dx, da.to(a.dtype), db.to(a.dtype), None


class WhtAffine(torch.nn.Module):
    """The layer that stands in for the dense attention output projection (Eq. 1): a fixed Walsh-Hadamard
    transform over the d concatenated head channels followed by the learned per-channel scale a and shift b
    (2*d parameters instead of d*d).  Starts as the plain orthonormal transform: a = 1, b = 0.

    d must be a power of two, or, with `block` given, a multiple of a power-of-two block (each block of
    channels is then transformed on its own: the block-diagonal form; the paper does not say what it does
    at its widths 768 and 1536, so that choice is this library's).  `forward(x, resid=None)` takes
    x[..., d]; with `resid` the residual add that follows the attention block is fused into the kernel
    (power-of-two d only).
    Rows are stored in x's dtype (fp32 or bf16); parameters are fp32 unless `param_dtype` says bf16.
    """

    def __init__(self, d: int, block: int | None = None, param_dtype=torch.float32, device=None):
        super().__init__()
        if block is None and d & (d - 1):
            raise ValueError(f"d = {d} is not a power of two: pass block= for the block-diagonal form")
        if block is not None and (block & (block - 1) or d % block):
            raise ValueError(f"block = {block} must be a power of two that divides d = {d}")
        self.d, self.block = d, block
        self.a = torch.nn.Parameter(torch.ones(d, dtype=param_dtype, device=device))
        self.b = torch.nn.Parameter(torch.zeros(d, dtype=param_dtype, device=device))

    def forward(self, x: torch.Tensor, resid: torch.Tensor | None = None) -> torch.Tensor:
        if x.shape[-1] != self.d:
            raise ValueError(f"last dimension {x.shape[-1]} != d = {self.d}")
        if self.block is not None and self.block != self.d:
            if resid is not None:
                raise ValueError("the block-diagonal form has no fused residual: add it outside the layer")
            return _WhtAffineGrouped.apply(x, self.a, self.b, self.block)
        return wht_affine(x, self.a, self.b, resid)

    def extra_repr(self) -> str:
        return f"d={self.d}" + (f", block={self.block}" if self.block else "")
