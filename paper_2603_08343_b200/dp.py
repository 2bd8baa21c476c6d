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


class GradBucketRing:
    """`n` GradBuckets used in turn, each step's all-reduce left in flight while the next step computes.

    The sum over ranks is needed by whoever consumes the gradients (an optimizer), not by the next
    forward pass, so a step need not wait for its own all-reduce: it is started asynchronously and
    waited for only when its bucket comes round again (or at `drain`).  On GPU ranks the wait is a
    stream dependency, not a host block.

        bucket = ring.acquire()                 # its previous all-reduce, if any, is waited for
        wht_affine_bwd(..., bucket.da, bucket.db, ...)
        ring.all_reduce_async(bucket)           # returns at once
        ...
        ring.drain()                            # before reading the last steps' sums
    """

    def __init__(self, d: int, device="cpu", n: int = 2):
        if n < 1:
            raise ValueError("at least one bucket")
        self.buckets = [GradBucket(d, device) for _ in range(n)]
        self._pending = [None] * n
        self._next = 0

    def acquire(self) -> GradBucket:
        i = self._next
        self._next = (i + 1) % len(self.buckets)
        self._wait(i)
        return self.buckets[i]

    def all_reduce_async(self, bucket: GradBucket, group=None) -> None:
        i = next(k for k, b in enumerate(self.buckets) if b is bucket)
        self._wait(i)
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            self._pending[i] = dist.all_reduce(bucket.flat, op=dist.ReduceOp.SUM, group=group, async_op=True)

    def drain(self) -> None:
        for i in range(len(self.buckets)):
            self._wait(i)

    def _wait(self, i: int) -> None:
        work, self._pending[i] = self._pending[i], None
        if work is not None:
            work.wait()
