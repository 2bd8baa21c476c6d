"""Column-sharded (tensor-parallel) form on CPU: the Kronecker identity it rests on, the sign rule the
host hands to the kernels, the argument checks of its C ABI, and a world-size-2 gloo run in which
each rank owns one column block and the blocks are exchanged with a collective."""
import ctypes
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from helpers import to_f64
from paper_2603_08343_b200 import tp
from paper_2603_08343_b200 import workloads as wl


def test_sylvester_matrix_is_a_kronecker_product():
    # H_d = H_g (x) H_w: entry ((s, i'), (r, j')) = H_g[s][r] * H_w[i'][j'], block index = top bits
    for g, w in [(2, 8), (4, 16), (8, 32), (2, 256)]:
        H = oracle.sylvester_hadamard(g * w)
        np.testing.assert_array_equal(H, np.kron(oracle.sylvester_hadamard(g), oracle.sylvester_hadamard(w)))


def test_sign_rule_is_the_small_sylvester_matrix():
    for g in (1, 2, 4, 8):
        Hg = oracle.sylvester_hadamard(g)
        for r in range(g):
            assert tp.tp_signs(g, r) == [int(Hg[s][r]) for s in range(g)]
    with pytest.raises(ValueError):
        tp.tp_signs(3, 0)
    with pytest.raises(ValueError):
        tp.tp_signs(4, 4)


def _rank_forward(x_blocks, a_r, b_r, g, r):
    """What rank r computes, written with the host's sign rule and the oracle's width-w matrix."""
    w = x_blocks[0].shape[1]
    mixed = sum(sgn * xb for sgn, xb in zip(tp.tp_signs(g, r), x_blocks))
    return a_r * (mixed @ oracle.sylvester_hadamard(w).astype(np.float64)) / np.sqrt(g * w) + b_r


def _rank_backward(dy_blocks, x_blocks, a_blocks, g, r):
    w = x_blocks[0].shape[1]
    Hw = oracle.sylvester_hadamard(w).astype(np.float64)
    signs = tp.tp_signs(g, r)
    z = (sum(sgn * xb for sgn, xb in zip(signs, x_blocks)) @ Hw) / np.sqrt(g * w)
    gsum = sum(sgn * ab * dyb for sgn, ab, dyb in zip(signs, a_blocks, dy_blocks))
    return (gsum @ Hw) / np.sqrt(g * w), np.sum(dy_blocks[r] * z, axis=0), np.sum(dy_blocks[r], axis=0)


@pytest.mark.parametrize("g,w,T", [(2, 64, 9), (4, 32, 5), (8, 16, 7)])
def test_column_blocks_reproduce_the_full_width_oracle(g, w, T):
    rng = np.random.default_rng(40 + g)
    d = g * w
    x, dy = rng.standard_normal((T, d)), rng.standard_normal((T, d))
    a, b = rng.uniform(0.5, 1.5, d), rng.normal(0, 0.1, d)
    y = oracle.wht_affine_fwd(x, a, b)
    dx, da, db = oracle.wht_affine_bwd(dy, x, a)
    xs = [p.numpy() for p in tp.split_columns(torch.from_numpy(x), g)]
    dys = [p.numpy() for p in tp.split_columns(torch.from_numpy(dy), g)]
    as_ = [a[s * w:(s + 1) * w] for s in range(g)]
    for r in range(g):
        cols = slice(r * w, (r + 1) * w)
        np.testing.assert_allclose(_rank_forward(xs, as_[r], b[cols], g, r), y[:, cols], rtol=0, atol=1e-12)
        dx_r, da_r, db_r = _rank_backward(dys, xs, as_, g, r)
        np.testing.assert_allclose(dx_r, dx[:, cols], rtol=0, atol=1e-12)
        np.testing.assert_allclose(da_r, da[cols], rtol=0, atol=1e-11)
        np.testing.assert_allclose(db_r, db[cols], rtol=0, atol=1e-12)


def test_argument_errors_need_no_gpu():
    from paper_2603_08343_b200 import build
    build.build()
    from paper_2603_08343_b200 import binding
    lib = binding.lib()
    buf = (ctypes.c_char * 4096)()
    p = ctypes.c_void_p((ctypes.addressof(buf) + 15) & ~15)
    off = p.value + 4
    parts = (ctypes.c_void_p * 8)(*([p.value] * 8))
    bad = (ctypes.c_void_p * 8)(*([p.value, off] + [p.value] * 6))
    hole = (ctypes.c_void_p * 8)(*([p.value, None] + [p.value] * 6))
    s = None
    assert lib.wht_affine_fwd_tp(parts, p, p, p, 4, 256, 3, 0, 0, s) == -2      # g not a power of two
    assert lib.wht_affine_fwd_tp(parts, p, p, p, 4, 256, 16, 0, 0, s) == -2     # more than 8 ranks
    assert lib.wht_affine_fwd_tp(parts, p, p, p, 4, 256, 4, 4, 0, s) == -2      # r outside [0, g)
    assert lib.wht_affine_fwd_tp(parts, p, p, p, 4, 100, 4, 0, 0, s) == -2      # w not a power of two
    assert lib.wht_affine_fwd_tp(parts, p, p, p, 4, 256, 4, 0, 9, s) == -4
    assert lib.wht_affine_fwd_tp(None, p, p, p, 4, 256, 4, 0, 0, s) == -1
    assert lib.wht_affine_fwd_tp(hole, p, p, p, 4, 256, 4, 0, 0, s) == -1
    assert lib.wht_affine_fwd_tp(bad, p, p, p, 4, 256, 4, 0, 0, s) == -5
    assert lib.wht_affine_fwd_tp(parts, p, p, p, 0, 256, 4, 0, 0, s) == 0       # no rows: nothing to do
    assert lib.wht_affine_bwd_tp(parts, parts, parts, p, None, p, 4, 256, 2, 1, 0, p, 64, s) == -1
    assert lib.wht_affine_bwd_tp(parts, hole, parts, p, p, p, 4, 256, 2, 1, 0, p, 64, s) == -1
    assert lib.wht_affine_bwd_tp(parts, parts, bad, p, p, p, 4, 256, 2, 1, 0, p, 64, s) == -5
    assert lib.wht_affine_bwd_tp(parts, parts, parts, p, p, p, 4, 256, 2, 2, 0, p, 64, s) == -2
    assert lib.wht_affine_bwd_tp_workspace_bytes(4, 256, 3, 0) == 0


# ---- two CPU ranks (gloo): each owns one column block, blocks travel by all_gather -----------------

def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, T, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.CONFIGS["tiny"].with_rows(T)           # d = 256 -> two blocks of 128 channels
        wd = w.d // world
        cols = slice(rank * wd, (rank + 1) * wd)
        x = wl.gen_full(w, "x")[:, cols].contiguous()  # this rank's own blocks only
        dy = wl.gen_full(w, "dy")[:, cols].contiguous()
        a, b = (t[cols].contiguous() for t in wl.gen_params(w))

        def exchange(t):  # stands in for the peer reads of the CUDA kernel
            parts = [torch.empty_like(t) for _ in range(world)]
            dist.all_gather(parts, t)
            return [to_f64(p) for p in parts]

        xs, dys, as_ = exchange(x), exchange(dy), exchange(a)
        y = _rank_forward(xs, to_f64(a), to_f64(b), world, rank)
        dx, da, db = _rank_backward(dys, xs, as_, world, rank)
        torch.save({"y": y, "dx": dx, "da": da, "db": db}, os.path.join(out, f"rank{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_ranks_own_column_blocks(tmp_path):
    world, T = 2, 11
    mp.spawn(_rank_main, args=(world, _free_port(), T, str(tmp_path)), nprocs=world, join=True)
    w = wl.CONFIGS["tiny"].with_rows(T)
    x, dy = to_f64(wl.gen_full(w, "x")), to_f64(wl.gen_full(w, "dy"))
    a, b = (to_f64(t) for t in wl.gen_params(w))
    y = oracle.wht_affine_fwd(x, a, b)
    dx, da, db = oracle.wht_affine_bwd(dy, x, a)
    parts = [torch.load(os.path.join(tmp_path, f"rank{r}.pt"), weights_only=False) for r in range(world)]
    np.testing.assert_allclose(np.concatenate([p["y"] for p in parts], axis=1), y, rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.concatenate([p["dx"] for p in parts], axis=1), dx, rtol=0, atol=1e-12)
    # parameter gradients are complete on the owning rank: no reduction over the column ranks
    np.testing.assert_allclose(np.concatenate([p["da"] for p in parts]), da, rtol=0, atol=1e-11)
    np.testing.assert_allclose(np.concatenate([p["db"] for p in parts]), db, rtol=0, atol=1e-12)
