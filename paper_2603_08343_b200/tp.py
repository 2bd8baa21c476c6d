"""Tensor parallelism for the path: the d = g*w channels split over g ranks.

Rank s holds channels [s*w, (s+1)*w) of every row as its own contiguous [T, w]
tensor.  H_d = H_g (x) H_w in Sylvester order, so the transform is the local one
of width w applied to a signed sum of the g blocks, with sign H_g[s][r] =
(-1)^popcount(s & r) for source s at rank r: the exchange is "every rank reads
every rank's block" (all-gather volume, bf16 as stored), and the library's
`wht_affine_fwd_tp` / `wht_affine_bwd_tp` kernels do the reads themselves through
peer pointers, fused with the transform.  Parameter gradients stay local: rank r
owns a_r, b_r and gets da_r, db_r complete (over its rows).

This module is the host logic: the sign rule, the column split, and a small
wrapper that keeps the pointer tables and the scratch buffer.  How peer pointers
are obtained (CUDA IPC, symmetric memory) is the caller's business; ranks must
synchronise before a call (inputs complete everywhere) and after it (nobody
overwrites inputs that a peer may still be reading).
"""
from __future__ import annotations

import torch


def tp_sign(s: int, r: int) -> int:
    """H_g[s][r] of the Sylvester matrix: the sign of source block s in the output block of rank r."""
    return -1 if bin(s & r).count("1") & 1 else 1


def tp_signs(g: int, r: int):
    if g < 1 or g & (g - 1) or not 0 <= r < g:
        raise ValueError(f"bad rank {r} of {g} (g must be a power of two)")
    return [tp_sign(s, r) for s in range(g)]


def split_columns(x: torch.Tensor, g: int):
    """The g contiguous [T, w] column blocks of x[T, d] (copies: each rank's block is its own tensor)."""
    d = x.shape[-1]
    if d % g:
        raise ValueError(f"d = {d} is not a multiple of g = {g}")
    w = d // g
    return [x[..., s * w:(s + 1) * w].contiguous() for s in range(g)]


class TpWht:
    """Rank r's side of the column-sharded op.

    `forward(x_parts, a, b)` and `backward(dy_parts, x_parts, a_parts)` take, for every
    rank, either a tensor on this device (single-GPU emulation, tests) or an integer
    device address valid on this GPU (a peer mapping); entry r is this rank's own block.
    """

    def __init__(self, g: int, r: int):
        tp_signs(g, r)  # validates
        self.g, self.r = g, r
        self._ws = None

    def forward(self, x_parts, a, b, T: int, w: int, out=None, stream=None):
        from . import binding
        y = out
        if y is None:
            y = torch.empty((T, w), dtype=_dtype_of(x_parts[self.r], a), device=a.device)
        binding.wht_affine_fwd_tp(x_parts, a, b, y, T, w, self.g, self.r, _code(y, a), stream)
        return y

    def backward(self, dy_parts, x_parts, a_parts, T: int, w: int, like=None, stream=None):
        from . import binding
        a = a_parts[self.r]
        if like is None:
            like = dy_parts[self.r]
        dx = torch.empty((T, w), dtype=like.dtype, device=a.device)
        da = torch.empty(w, dtype=torch.float32, device=a.device)
        db = torch.empty(w, dtype=torch.float32, device=a.device)
        code = _code(dx, a)
        need = binding.wht_affine_bwd_tp_workspace_bytes(T, w, self.g, code)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(max(need, 16), dtype=torch.uint8, device=a.device)
        binding.wht_affine_bwd_tp(dy_parts, x_parts, a_parts, dx, da, db, T, w, self.g, self.r, code, self._ws,
                                  stream)
        return dx, da, db


def _dtype_of(part, a):
    if isinstance(part, int):
        raise ValueError("pass out= when this rank's own block is given as an address")
    return part.dtype


def _code(rows, a):
    from . import binding
    return binding.dtype_code(rows, a)


class SymmetricBlocks:
    """This rank's [T, w] block in torch symmetric memory, with every rank's address of it.

    `tensor` is the local block (fill it, or have the producing kernel write into it);
    `addresses[s]` is rank s's block as mapped into THIS process (entry `rank` is the local
    one), ready to be passed as `x_parts` / `dy_parts` / `a_parts`.  `barrier()` is the
    cross-rank synchronisation the calls need: once after every rank has written its block
    and before any rank launches, once after the launches and before anybody overwrites.
    All ranks of `group` must construct it together (the rendezvous is collective).
    """

    def __init__(self, T: int, w: int, dtype, group=None, device=None):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem
        if group is None:
            group = dist.group.WORLD
        device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.tensor = symm_mem.empty((T, w), dtype=dtype, device=device)
        self.handle = symm_mem.rendezvous(self.tensor, group)
        self.rank = int(self.handle.rank)
        self.world_size = int(self.handle.world_size)
        self.addresses = [int(p) for p in self.handle.buffer_ptrs]
        if self.addresses[self.rank] != self.tensor.data_ptr():
            raise RuntimeError("symmetric memory handed back a block that is not at the tensor's address")

    def barrier(self):
        self.handle.barrier()
