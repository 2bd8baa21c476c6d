"""Column-sharded (tensor-parallel) calls on one GPU: the g ranks' blocks live in separate tensors of
the same device and every rank's call runs in turn (the calls only read their inputs, no kernel waits
for another), then the concatenated blocks are compared with the fp64 oracle at the full width."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_grad_vec, assert_rows_bf16, assert_rows_fp32, to_f64
from paper_2603_08343_b200 import tp
from paper_2603_08343_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2603_08343_b200 import build
    build.build()
    from paper_2603_08343_b200 import binding
    yield binding
    binding.wht_affine_set_variant(0)
    binding.wht_affine_device_status()


CASES = [
    (2, 128, wl.WHT_F32, 70), (4, 64, wl.WHT_F32, 33), (8, 8, wl.WHT_F32, 100),
    (2, 1024, wl.WHT_BF16, 300), (4, 512, wl.WHT_BF16_PF32, 129), (8, 256, wl.WHT_BF16, 517),
    (8, 1024, wl.WHT_BF16_PF32, 65), (2, 4096, wl.WHT_BF16, 19), (4, 2048, wl.WHT_BF16_PF32, 1111),
    (1, 2048, wl.WHT_BF16, 40),
]


# the tcgen05 form of the forward (one product per source block, signs by the negate-A bit): forced by
# variant 4 on small cases, and chosen by itself once T*w reaches 4 Mi elements
UMMA_CASES = [
    (2, 1024, wl.WHT_BF16, 300, 4), (8, 1024, wl.WHT_BF16_PF32, 65, 4), (4, 2048, wl.WHT_BF16_PF32, 1111, 4),
    (2, 4096, wl.WHT_BF16, 19, 4), (8, 2048, wl.WHT_BF16, 7, 4), (4, 4096, wl.WHT_BF16_PF32, 130, 4),
    (2, 1024, wl.WHT_BF16_PF32, 4100, 0), (1, 1024, wl.WHT_BF16, 129, 4),
]


@pytest.mark.parametrize("g,w,dtype,T,variant", [c + (0,) for c in CASES] + UMMA_CASES)
def test_column_sharded_calls_match_the_full_width_oracle(B, g, w, dtype, T, variant):
    B.wht_affine_set_variant(variant)
    d = g * w
    wk = wl.Workload("tp", T, d, dtype, "normal", 900 + d + g, True, "")
    x, dy = wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")
    a, b = wl.gen_params(wk)
    xs = [p.cuda() for p in tp.split_columns(x, g)]
    dys = [p.cuda() for p in tp.split_columns(dy, g)]
    as_ = [a[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
    bs = [b[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
    ys, dxs, das, dbs = [], [], [], []
    for r in range(g):
        rank = tp.TpWht(g, r)
        ys.append(rank.forward(xs, as_[r], bs[r], T, w))
        dx, da, db = rank.backward(dys, xs, as_, T, w)
        dxs.append(dx); das.append(da); dbs.append(db)
    torch.cuda.synchronize()
    y = torch.cat(ys, dim=1).cpu()
    dx = torch.cat(dxs, dim=1).cpu()
    da, db = torch.cat(das).cpu(), torch.cat(dbs).cpu()
    ref_y = oracle.wht_affine_fwd(to_f64(x), to_f64(a), to_f64(b))
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    if dtype == wl.WHT_F32:
        assert_rows_fp32(to_f64(y), ref_y, to_f64(x), "tp y")
        assert_rows_fp32(to_f64(dx), ref_dx, to_f64(a)[None, :] * to_f64(dy), "tp dx")
    else:
        assert_rows_bf16(to_f64(y), ref_y, "tp y")
        assert_rows_bf16(to_f64(dx), ref_dx, "tp dx")
    assert_grad_vec(to_f64(da), ref_da, "tp da")
    assert_grad_vec(to_f64(db), ref_db, "tp db")
    if g == 1:  # one rank is the plain call of the same kernel family
        B.wht_affine_set_variant(variant or 1)
        assert torch.equal(ys[0], B.forward(xs[0], as_[0], bs[0]))
    B.wht_affine_set_variant(0)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("g,w,T,dtype", [(2, 1024, 148 * 16 * 2 + 5, wl.WHT_BF16_PF32), (4, 1024, 148 * 16 + 3, wl.WHT_BF16),
                                         (8, 1024, 148 * 16 + 1, wl.WHT_BF16_PF32), (2, 2048, 148 * 8 * 2 + 7, wl.WHT_BF16),
                                         (4, 2048, 148 * 8 + 4, wl.WHT_BF16_PF32), (2, 4096, 148 * 4 + 3, wl.WHT_BF16_PF32)])
def test_column_sharded_backward_on_the_tensor_core_many_rows(B, g, w, T, dtype, mode):
    """The tcgen05 backward of the column-sharded form over several tiles per CTA (the ring and both
    accumulators wrap, the last tile is ragged), in both operand modes, every rank in turn, against the
    full-width chain rule of Eq. 1.  Repeating a call must give the same bits (fixed summation order)."""
    B.wht_affine_set_variant(0)
    B.wht_affine_set_bwd_operand_mode(mode)
    try:
        d = g * w
        wk = wl.Workload("tp-bwd", T, d, dtype, "normal", 1200 + d + g, True, "")
        x, dy = wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")
        a, _ = wl.gen_params(wk)
        xs = [p.cuda() for p in tp.split_columns(x, g)]
        dys = [p.cuda() for p in tp.split_columns(dy, g)]
        as_ = [a[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
        outs = [tp.TpWht(g, r).backward(dys, xs, as_, T, w) for r in range(g)]
        again = tp.TpWht(g, g - 1).backward(dys, xs, as_, T, w)
        torch.cuda.synchronize()
        assert all(torch.equal(u, v) for u, v in zip(outs[g - 1], again))
        dx = torch.cat([o[0] for o in outs], dim=1).cpu()
        da, db = torch.cat([o[1] for o in outs]).cpu(), torch.cat([o[2] for o in outs]).cpu()
        ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
        assert_rows_bf16(to_f64(dx), ref_dx, f"tp dx g={g} w={w} mode={mode}")
        assert_grad_vec(to_f64(da), ref_da, f"tp da g={g} w={w}")
        assert_grad_vec(to_f64(db), ref_db, f"tp db g={g} w={w}")
        # the same bits as the butterfly kernels' reductions is not required; the same values within the bound is:
        B.wht_affine_set_variant(1)
        dx_b, da_b, db_b = tp.TpWht(g, 0).backward(dys, xs, as_, T, w)
        torch.cuda.synchronize()
        assert_rows_bf16(to_f64(outs[0][0].cpu()), to_f64(dx_b.cpu()), "tcgen05 vs butterfly dx")
        assert_grad_vec(to_f64(outs[0][1].cpu()), to_f64(da_b.cpu()), "tcgen05 vs butterfly da")
    finally:
        B.wht_affine_set_variant(0)
        B.wht_affine_set_bwd_operand_mode(0)
    B.wht_affine_device_status()


def test_blocks_given_as_addresses_and_repeat_calls_are_bit_identical(B):
    g, w, T, dtype = 4, 512, 257, wl.WHT_BF16_PF32
    wk = wl.Workload("tp", T, g * w, dtype, "normal", 77, True, "")
    x, dy = wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")
    a, b = wl.gen_params(wk)
    xs = [p.cuda() for p in tp.split_columns(x, g)]
    dys = [p.cuda() for p in tp.split_columns(dy, g)]
    as_ = [a[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
    r = 3
    rank = tp.TpWht(g, r)
    b_r = b[r * w:(r + 1) * w].contiguous().cuda()
    y1 = rank.forward(xs, as_[r], b_r, T, w)
    y2 = torch.empty_like(y1)
    rank.forward([t.data_ptr() for t in xs], as_[r], b_r, T, w, out=y2)   # peer mappings arrive as addresses
    out1 = rank.backward(dys, xs, as_, T, w)
    out2 = rank.backward([t.data_ptr() for t in dys], [t.data_ptr() for t in xs], as_, T, w, like=dys[r])
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)
    for u, v in zip(out1, out2):
        assert torch.equal(u, v)


@pytest.mark.parametrize("variant", [0, 1])
def test_blocks_past_two_to_the_31_elements(B, variant):
    # g = 2 ranks, blocks of 2^21 + 5 rows x 1024 columns: 2^31 + 5120 elements per block.  All rows are zero
    # but the first and the last 100; those are checked against the full-width oracle, a zero row must come out
    # as b and as zero, and da, db follow from the non-zero rows alone.
    B.wht_affine_set_variant(variant)
    g, w, dtype = 2, 1024, wl.WHT_BF16_PF32
    d, T, n = g * w, (1 << 21) + 5, 100
    wk = wl.Workload("tpbig", 2 * n, d, dtype, "normal", 990, True, "")
    x, dy = wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")
    a, b = wl.gen_params(wk)
    xs = [torch.zeros(T, w, dtype=torch.bfloat16, device="cuda") for _ in range(g)]
    dys = [torch.zeros(T, w, dtype=torch.bfloat16, device="cuda") for _ in range(g)]
    for s in range(g):
        for blocks, src in ((xs, x), (dys, dy)):
            blocks[s][:n].copy_(src[:n, s * w:(s + 1) * w])
            blocks[s][T - n:].copy_(src[n:, s * w:(s + 1) * w])
    as_ = [a[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
    bs = [b[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
    ref_y = oracle.wht_affine_fwd(to_f64(x), to_f64(a), to_f64(b))
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    pick = lambda t: torch.cat([t[:n], t[T - n:]]).cpu()
    ys, dxs, das, dbs = [], [], [], []
    for r in range(g):
        rank = tp.TpWht(g, r)
        y = rank.forward(xs, as_[r], bs[r], T, w)
        dx, da, db = rank.backward(dys, xs, as_, T, w)
        torch.cuda.synchronize()
        for row in (n, T // 2, T - n - 1):
            assert torch.equal(y[row], bs[r].bfloat16()) and torch.count_nonzero(dx[row]).item() == 0
        ys.append(pick(y)); dxs.append(pick(dx)); das.append(da.cpu()); dbs.append(db.cpu())
        del y, dx
    assert_rows_bf16(to_f64(torch.cat(ys, dim=1)), ref_y, "tp y past 2^31")
    assert_rows_bf16(to_f64(torch.cat(dxs, dim=1)), ref_dx, "tp dx past 2^31")
    assert_grad_vec(to_f64(torch.cat(das)), ref_da, "tp da past 2^31")
    assert_grad_vec(to_f64(torch.cat(dbs)), ref_db, "tp db past 2^31")
    B.wht_affine_set_variant(0)
    B.wht_affine_device_status()


def test_no_rows(B):
    g, w = 2, 256
    rank = tp.TpWht(g, 1)
    a = torch.ones(w, device="cuda")
    empty = [torch.empty((0, w), device="cuda") for _ in range(g)]
    y = rank.forward(empty, a, a, 0, w)
    dx, da, db = rank.backward(empty, empty, [a, a], 0, w)
    torch.cuda.synchronize()
    assert y.shape == (0, w) and dx.shape == (0, w)
    assert torch.all(da == 0) and torch.all(db == 0)


def test_blocks_in_symmetric_memory_single_rank(B):
    """The helper that hands out peer addresses, with a process group of one rank (all that one GPU allows):
    the address table has this rank's own block, and a call through it equals the plain call."""
    import os
    import socket
    import torch.distributed as dist
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    started = not dist.is_initialized()
    if started:
        try:
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
        except Exception as exc:
            pytest.skip(f"no NCCL process group on this box: {exc}")
    try:
        T, w = 257, 1024
        try:
            blk = tp.SymmetricBlocks(T, w, torch.bfloat16)
        except Exception as exc:  # driver or build without symmetric memory support
            pytest.skip(f"torch symmetric memory is not available here: {exc}")
        assert blk.world_size == 1 and blk.rank == 0 and blk.addresses == [blk.tensor.data_ptr()]
        wk = wl.Workload("tp", T, w, wl.WHT_BF16_PF32, "normal", 31, True, "")
        x = wl.gen_full(wk, "x").cuda()
        a, b = (t.cuda() for t in wl.gen_params(wk))
        blk.tensor.copy_(x)
        blk.barrier()
        y = torch.empty_like(x)
        tp.TpWht(1, 0).forward(blk.addresses, a, b, T, w, out=y)
        blk.barrier()
        torch.cuda.synchronize()
        B.wht_affine_set_variant(1)
        assert torch.equal(y, B.forward(x, a, b))
        B.wht_affine_set_variant(0)
    finally:
        if started:
            dist.destroy_process_group()
