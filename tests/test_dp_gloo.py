"""World-size-2 run of the data-parallel host logic on CPU ranks (gloo).

Each rank takes its row shard, stands in for the CUDA calls with the oracle on that
shard (the kernels need a GPU; the sharding, the da|db bucket and the all-reduce do
not), and the reduced gradients must equal the oracle's on all rows.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from helpers import to_f64
from paper_2603_08343_b200 import dp
from paper_2603_08343_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, T, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.CONFIGS["tiny"].with_rows(T)
        r0, r1 = dp.shard_rows(T, world, rank)
        x = to_f64(wl.gen_rows(w, "x", r0, r1))
        dy = to_f64(wl.gen_rows(w, "dy", r0, r1))
        a, b = (to_f64(t) for t in wl.gen_params(w))
        y = oracle.wht_affine_fwd(x, a, b)
        dx, da, db = oracle.wht_affine_bwd(dy, x, a)
        bucket = dp.GradBucket(w.d)
        bucket.da.copy_(torch.from_numpy(da).float())
        bucket.db.copy_(torch.from_numpy(db).float())
        assert bucket.flat.data_ptr() % 16 == 0 and bucket.db.data_ptr() % 16 == 0
        da_all, db_all = bucket.all_reduce()
        torch.save({"r0": r0, "r1": r1, "y": y, "dx": dx, "da": da_all.clone(), "db": db_all.clone()},
                   os.path.join(out, f"rank{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_rows_and_reduce_grads(tmp_path):
    world, T = 2, 37  # odd row count: the shards differ in size
    mp.spawn(_rank_main, args=(world, _free_port(), T, str(tmp_path)), nprocs=world, join=True)
    w = wl.CONFIGS["tiny"].with_rows(T)
    x, dy = to_f64(wl.gen_full(w, "x")), to_f64(wl.gen_full(w, "dy"))
    a, b = (to_f64(t) for t in wl.gen_params(w))
    y = oracle.wht_affine_fwd(x, a, b)
    dx, da, db = oracle.wht_affine_bwd(dy, x, a)
    parts = [torch.load(os.path.join(tmp_path, f"rank{r}.pt"), weights_only=False) for r in range(world)]
    assert parts[0]["r0"] == 0 and parts[0]["r1"] == parts[1]["r0"] and parts[1]["r1"] == T
    np.testing.assert_array_equal(np.concatenate([p["y"] for p in parts]), y)
    np.testing.assert_array_equal(np.concatenate([p["dx"] for p in parts]), dx)
    for p in parts:  # every rank holds the full-row sums after the all-reduce
        np.testing.assert_allclose(p["da"].numpy(), da, rtol=0, atol=1e-4 * np.max(np.abs(da)))
        np.testing.assert_allclose(p["db"].numpy(), db, rtol=0, atol=1e-4 * np.max(np.abs(db)))
    assert torch.equal(parts[0]["da"], parts[1]["da"]) and torch.equal(parts[0]["db"], parts[1]["db"])


def test_bucket_without_process_group_is_local():
    bucket = dp.GradBucket(8)
    bucket.da.fill_(2.0)
    da, db = bucket.all_reduce()
    assert torch.all(da == 2.0) and torch.all(db == 0.0)


def _ring_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        d, steps = 16, 5
        ring = dp.GradBucketRing(d, n=2)
        seen = []
        for step in range(steps):
            bucket = ring.acquire()          # the sum of step - 2 sits here until it is overwritten now
            if step >= 2:
                seen.append((step - 2, bucket.flat.clone()))
            bucket.da.fill_(float(10 * step + rank + 1))
            bucket.db.fill_(float(-(10 * step + rank + 1)))
            ring.all_reduce_async(bucket)
        ring.drain()
        for k in (steps - 2, steps - 1):
            seen.append((k, ring.buckets[k % 2].flat.clone()))
        torch.save(seen, os.path.join(out, f"ring{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_overlapped_bucket_ring_on_two_ranks(tmp_path):
    # every step's all-reduce stays in flight until its bucket comes round again: each step's sum over the
    # two ranks must be what that step wrote (1 + 2 + 20 * step), on both ranks, for all five steps
    world = 2
    mp.spawn(_ring_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        seen = torch.load(os.path.join(tmp_path, f"ring{rank}.pt"), weights_only=False)
        assert sorted(k for k, _ in seen) == [0, 1, 2, 3, 4]
        for step, flat in seen:
            want = float(20 * step + 3)
            assert torch.all(flat[:16] == want) and torch.all(flat[16:] == -want), (rank, step)


def test_bucket_ring_without_process_group_is_local():
    ring = dp.GradBucketRing(8, n=3)
    b0 = ring.acquire()
    b0.da.fill_(5.0)
    ring.all_reduce_async(b0)
    assert ring.acquire() is ring.buckets[1] and ring.acquire() is ring.buckets[2] and ring.acquire() is b0
    ring.drain()
    assert torch.all(b0.da == 5.0)
