"""The -DWHT_DEBUG build: the same kernels, with every output and the scratch of a call placed between
guard regions that are checked after the kernels have run (the stand-in for a memory checker).  The small
parity cases run through it, in every kernel family: results must be the regular build's bit for bit and
no call may report a damaged guard; the checker itself must notice a byte written on either side."""
import ctypes

import pytest
import torch

import oracle
from helpers import assert_grad_vec, assert_rows_bf16, assert_rows_fp32, to_f64
from paper_2603_08343_b200 import workloads as wl

pytestmark = pytest.mark.gpu

WHT_ERR_GUARD = -10


@pytest.fixture(scope="module")
def libs():
    from paper_2603_08343_b200 import build
    build.build()
    dbg_path = build.build(debug=True)
    from paper_2603_08343_b200 import binding
    dbg = binding.load_library(dbg_path)
    assert dbg.wht_affine_debug_build() == 1 and binding.lib().wht_affine_debug_build() == 0
    yield binding, dbg
    binding.wht_affine_set_variant(0)
    dbg.wht_affine_set_variant(0)
    assert dbg.wht_affine_device_status() == 0


def _p(t):
    return ctypes.c_void_p(t.data_ptr())


def test_the_guard_check_notices_a_byte_on_either_side(libs):
    B, dbg = libs
    assert dbg.wht_affine_debug_selftest_guard(0) == 0
    assert dbg.wht_affine_debug_selftest_guard(1) == WHT_ERR_GUARD
    assert dbg.wht_affine_debug_selftest_guard(2) == WHT_ERR_GUARD
    assert b"outside" in dbg.wht_affine_status_string(WHT_ERR_GUARD)
    assert B.lib().wht_affine_debug_selftest_guard(1) == -8  # not a debug build


CASES = [(256, wl.WHT_F32, 64), (8, wl.WHT_F32, 1031), (64, wl.WHT_BF16, 257), (256, wl.WHT_BF16, 130),
         (512, wl.WHT_BF16_PF32, 257), (1024, wl.WHT_BF16, 257), (2048, wl.WHT_BF16_PF32, 148 * 8 + 3),
         (4096, wl.WHT_BF16, 37), (8192, wl.WHT_BF16_PF32, 21), (16384, wl.WHT_F32, 5), (32768, wl.WHT_BF16, 3)]


@pytest.mark.parametrize("variant", [0, 1, 2, 3, 4, 5])
def test_small_parity_cases_through_the_guarded_build(libs, variant):
    B, dbg = libs
    B.wht_affine_set_variant(variant)
    assert dbg.wht_affine_set_variant(variant) == 0
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    for d, dtype, T in CASES:
        w = wl.Workload("guard", T, d, dtype, "normal", 3100 + d, True, "")
        x, dy = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
        a, b = wl.gen_params(w)
        xd, dyd, ad, bd = x.cuda(), dy.cuda(), a.cuda(), b.cuda()
        what = f"d={d} dtype={dtype} T={T} variant={variant}"
        # forward, fused residual, decode shape
        y_ref = B.forward(xd, ad, bd)
        y = torch.full_like(xd, float("nan"))
        assert dbg.wht_affine_fwd(_p(xd), _p(ad), _p(bd), _p(y), T, d, dtype, s) == 0, what
        yr_ref = B.forward(xd, ad, bd, resid=dyd)
        yr = torch.full_like(xd, float("nan"))
        assert dbg.wht_affine_fwd_residual(_p(xd), _p(ad), _p(bd), _p(dyd), _p(yr), T, d, dtype, s) == 0, what
        yd = torch.full_like(xd, float("nan"))
        assert dbg.wht_affine_fwd_decode(_p(xd), _p(ad), _p(bd), _p(yd), T, d, dtype, s) == 0, what
        yd_ref = B.forward(xd, ad, bd, decode=True)
        # backward through the three entry points
        dx_ref, da_ref, db_ref = B.backward(dyd, xd, ad)
        outs = []
        need = B.wht_affine_bwd_workspace_bytes(T, d, dtype)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
        for which in ("bwd", "ws", "noalloc"):
            dx = torch.full_like(xd, float("nan"))
            da = torch.full((d,), float("nan"), device="cuda")
            db = torch.full((d,), float("nan"), device="cuda")
            if which == "bwd":
                rc = dbg.wht_affine_bwd(_p(dyd), _p(xd), _p(ad), _p(dx), _p(da), _p(db), T, d, dtype, s)
            elif which == "ws":
                rc = dbg.wht_affine_bwd_ws(_p(dyd), _p(xd), _p(ad), _p(dx), _p(da), _p(db), T, d, dtype, _p(ws),
                                           ws.numel(), s)
            else:
                if need > 16 * 1024 * 1024:
                    continue
                rc = dbg.wht_affine_bwd_noalloc(_p(dyd), _p(xd), _p(ad), _p(dx), _p(da), _p(db), T, d, dtype, s)
            assert rc == 0, f"{what} {which}: status {rc}"
            outs.append((dx, da, db))
        torch.cuda.synchronize()
        assert torch.equal(y, y_ref) and torch.equal(yr, yr_ref) and torch.equal(yd, yd_ref), what
        for dx, da, db in outs:
            assert torch.equal(dx, dx_ref) and torch.equal(da, da_ref) and torch.equal(db, db_ref), what
        # in place over the input, as the regular build allows
        x2 = xd.clone()
        assert dbg.wht_affine_fwd(_p(x2), _p(ad), _p(bd), _p(x2), T, d, dtype, s) == 0
        torch.cuda.synchronize()
        assert torch.equal(x2, y_ref), what
    # and against the definition itself (Eq. 1 and its chain rule) for the last case
    ref_y = oracle.wht_affine_fwd(to_f64(x), to_f64(a), to_f64(b))
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    assert_rows_bf16(to_f64(y.cpu()), ref_y, "guarded y")
    assert_rows_bf16(to_f64(outs[0][0].cpu()), ref_dx, "guarded dx")
    assert_grad_vec(to_f64(outs[0][1].cpu()), ref_da, "guarded da")
    assert_grad_vec(to_f64(outs[0][2].cpu()), ref_db, "guarded db")


def test_grouped_and_column_sharded_calls_through_the_guarded_build(libs):
    B, dbg = libs
    from paper_2603_08343_b200 import tp
    B.wht_affine_set_variant(0)
    dbg.wht_affine_set_variant(0)
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    for d, block, dtype, T in ((768, 256, wl.WHT_BF16_PF32, 300), (1536, 512, wl.WHT_BF16, 129), (96, 32, wl.WHT_F32, 77)):
        g = torch.Generator().manual_seed(d)
        io = torch.float32 if dtype == wl.WHT_F32 else torch.bfloat16
        pt = torch.bfloat16 if dtype == wl.WHT_BF16 else torch.float32
        x = torch.randn(T, d, generator=g).to(io).cuda()
        dy = torch.randn(T, d, generator=g).to(io).cuda()
        a = (torch.rand(d, generator=g) + 0.5).to(pt).cuda()
        b = (torch.randn(d, generator=g) * 0.1).to(pt).cuda()
        y_ref = torch.empty_like(x)
        B.wht_affine_fwd_grouped(x, a, b, y_ref, T, d, block, dtype)
        y = torch.full_like(x, float("nan"))
        assert dbg.wht_affine_fwd_grouped(_p(x), _p(a), _p(b), _p(y), T, d, block, dtype, s) == 0
        need = B.wht_affine_bwd_grouped_workspace_bytes(T, d, block, dtype)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
        ref = [torch.empty_like(x), torch.empty(d, device="cuda"), torch.empty(d, device="cuda")]
        B.wht_affine_bwd_grouped(dy, x, a, ref[0], ref[1], ref[2], T, d, block, dtype, ws)
        got = [torch.full_like(x, float("nan")), torch.empty(d, device="cuda"), torch.empty(d, device="cuda")]
        assert dbg.wht_affine_bwd_grouped(_p(dy), _p(x), _p(a), _p(got[0]), _p(got[1]), _p(got[2]), T, d, block, dtype,
                                          _p(ws), ws.numel(), s) == 0
        torch.cuda.synchronize()
        assert torch.equal(y, y_ref) and all(torch.equal(u, v) for u, v in zip(got, ref)), f"grouped d={d}"
    for g_, w_, dtype, T in ((2, 1024, wl.WHT_BF16_PF32, 300), (4, 256, wl.WHT_BF16, 129), (8, 1024, wl.WHT_BF16, 148 * 16 + 1)):
        wk = wl.Workload("guard-tp", T, g_ * w_, dtype, "normal", 3300 + g_, True, "")
        x, dy = wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")
        a, b = wl.gen_params(wk)
        xs = [p.cuda() for p in tp.split_columns(x, g_)]
        dys = [p.cuda() for p in tp.split_columns(dy, g_)]
        as_ = [a[k * w_:(k + 1) * w_].contiguous().cuda() for k in range(g_)]
        r = g_ - 1
        b_r = b[r * w_:(r + 1) * w_].contiguous().cuda()
        rank = tp.TpWht(g_, r)
        y_ref = rank.forward(xs, as_[r], b_r, T, w_)
        ref = rank.backward(dys, xs, as_, T, w_)
        arr = lambda parts: (ctypes.c_void_p * g_)(*[p.data_ptr() for p in parts])  # noqa: E731
        y = torch.full_like(y_ref, float("nan"))
        assert dbg.wht_affine_fwd_tp(arr(xs), _p(as_[r]), _p(b_r), _p(y), T, w_, g_, r, dtype, s) == 0
        need = B.wht_affine_bwd_tp_workspace_bytes(T, w_, g_, dtype)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
        got = [torch.full_like(ref[0], float("nan")), torch.empty(w_, device="cuda"), torch.empty(w_, device="cuda")]
        assert dbg.wht_affine_bwd_tp(arr(dys), arr(xs), arr(as_), _p(got[0]), _p(got[1]), _p(got[2]), T, w_, g_, r,
                                     dtype, _p(ws), ws.numel(), s) == 0
        torch.cuda.synchronize()
        assert torch.equal(y, y_ref) and all(torch.equal(u, v) for u, v in zip(got, ref)), f"tp g={g_} w={w_}"


def test_a_failed_guard_buffer_allocation_is_an_error(libs):
    # the guarded build allocates on every call: an injected out-of-memory answer must surface as
    # WHT_ERR_WORKSPACE, the output must stay as it was, and the next call must work
    B, dbg = libs
    w = wl.Workload("guard", 130, 1024, wl.WHT_BF16, "normal", 3300, True, "")
    x = wl.gen_full(w, "x")
    a, b = wl.gen_params(w)
    xd, ad, bd = x.cuda(), a.cuda(), b.cuda()
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    y = torch.full_like(xd, 7.0)
    assert dbg.wht_affine_test_fail_allocations(1) == 0
    try:
        assert dbg.wht_affine_fwd(_p(xd), _p(ad), _p(bd), _p(y), w.T, w.d, w.dtype, s) == -6
        torch.cuda.synchronize()
        assert torch.all(y == 7.0)
    finally:
        assert dbg.wht_affine_test_fail_allocations(0) == 0
    assert dbg.wht_affine_fwd(_p(xd), _p(ad), _p(bd), _p(y), w.T, w.d, w.dtype, s) == 0
    torch.cuda.synchronize()
    assert_rows_bf16(to_f64(y.cpu()), oracle.wht_affine_fwd(to_f64(x), to_f64(a), to_f64(b)), "after the failed allocation")
