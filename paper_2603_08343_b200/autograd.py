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
