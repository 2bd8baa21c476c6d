"""Data parallelism for the path: rows are independent, so T rows split over ranks.

Every rank runs the forward and backward calls on its own contiguous row range
with the full (replicated) a and b.  The forward needs no exchange.  In the
backward, dx is local; da and db are sums over ALL rows, so each rank's partial
da|db (2*d fp32 values, written by the library straight into one bucket) is
summed with a single all-reduce -- the only collective of the path.  This module
holds that host logic only; it runs unchanged over NCCL (GPU ranks) and gloo
(CPU ranks, as in the tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(T: int, world_size: int, rank: int):
    """Contiguous row range [r0, r1) of `rank` when T rows are split over ranks.

    The first T % world_size ranks take one extra row.
    """
    if world_size < 1 or not 0 <= rank < world_size:
        raise ValueError(f"bad rank {rank} of {world_size}")
    base, extra = divmod(T, world_size)
    r0 = rank * base + min(rank, extra)
    return r0, r0 + base + (1 if rank < extra else 0)


class GradBucket:
    """One contiguous fp32 buffer da|db, so that the all-reduce is a single message.

    `da` and `db` are views of the bucket (both 16-byte aligned for d >= 4), to
    be passed as the da/db outputs of the backward call.
    """

    def __init__(self, d: int, device="cpu"):
        self.d = d
        self.flat = torch.zeros(2 * d, dtype=torch.float32, device=device)
        self.da = self.flat[:d]
        self.db = self.flat[d:]

    def all_reduce(self, group=None):
        """Sums the bucket over the ranks of `group` in place (no-op without a process group)."""
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(self.flat, op=dist.ReduceOp.SUM, group=group)
        return self.da, self.db
