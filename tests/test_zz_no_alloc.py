"""wht_affine_bwd_noalloc against wht_affine_bwd, through the C ABI.

The no-allocation entry point serves callers that may not call cudaMalloc (all device
memory owned by a pool, or allocation forbidden once a serving loop is running), so
its scratch is a fixed array inside the library that every call shares and that keeps
the previous call's contents.  Two calls in a row, on different shapes, must each give
what the allocating entry point gives: the second call must not be disturbed by what
the first one left behind.  This file sorts last so that a failure here cannot hide
another test's result in a run that stops at the first failure.
"""
import pytest
import torch

import oracle
from helpers import assert_grad_vec, assert_rows_bf16, assert_rows_fp32, to_f64
from paper_2603_08343_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2603_08343_b200 import build
    build.build()
    from paper_2603_08343_b200 import binding
    binding.wht_affine_set_variant(0)
    return binding


def _both(B, w):
    x = wl.gen_full(w, "x").cuda()
    dy = wl.gen_full(w, "dy").cuda()
    a = wl.gen_params(w)[0].cuda()
    outs = []
    for fn in (B.wht_affine_bwd, B.wht_affine_bwd_noalloc):
        dx = torch.empty_like(x)
        da = torch.full((w.d,), float("nan"), device="cuda")
        db = torch.full((w.d,), float("nan"), device="cuda")
        fn(dy, x, a, dx, da, db, w.T, w.d, w.dtype)
        torch.cuda.synchronize()
        outs.append((dx.cpu(), da.cpu(), db.cpu()))
    return outs, a.cpu(), dy.cpu()


def test_two_calls_in_a_row_match_the_allocating_entry_point(B):
    cases = [
        wl.Workload("noalloc", 5000, 2048, wl.WHT_BF16_PF32, "normal", 41, True, ""),  # 148 CTAs x 16 KiB of partial sums
        wl.Workload("noalloc", 301, 1024, wl.WHT_BF16, "normal", 42, True, ""),        # fewer, smaller partials over stale data
        wl.Workload("noalloc", 600, 8192, wl.WHT_F32, "normal", 45, True, ""),         # butterfly family, 64 KiB per CTA: most of the array
        wl.Workload("noalloc", 300, 4096, wl.WHT_BF16_PF32, "normal", 46, True, ""),
        wl.Workload("noalloc", 64, 256, wl.WHT_F32, "normal", 43, True, ""),
    ]
    for w in cases:
        (ref, got), a, dy = _both(B, w)
        # against the definition itself (chain rule on Eq. 1), not only against the other entry point
        x = wl.gen_full(w, "x")
        o_dx, o_da, o_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
        if w.dtype == wl.WHT_F32:
            assert_rows_fp32(to_f64(got[0]), o_dx, to_f64(a)[None, :] * to_f64(dy), "noalloc dx vs oracle")
        else:
            assert_rows_bf16(to_f64(got[0]), o_dx, "noalloc dx vs oracle")
        assert_grad_vec(to_f64(got[1]), o_da, "noalloc da vs oracle")
        assert_grad_vec(to_f64(got[2]), o_db, "noalloc db vs oracle")
        if w.dtype == wl.WHT_F32:
            assert_rows_fp32(to_f64(got[0]), to_f64(ref[0]), to_f64(a)[None, :] * to_f64(dy), "noalloc dx")
        else:
            assert_rows_bf16(to_f64(got[0]), to_f64(ref[0]), "noalloc dx")
        assert_grad_vec(to_f64(got[1]), to_f64(ref[1]), "noalloc da")
        assert_grad_vec(to_f64(got[2]), to_f64(ref[2]), "noalloc db")
        # same kernels, same launch shape, fixed summation order: the results are in fact identical
        assert all(torch.equal(g, r) for g, r in zip(got, ref))


def test_every_width_up_to_8192_fits_the_builtin_array(B):
    # the header promises that d <= 8192 fits for any T: the scratch need grows with the CTA count, which
    # stops growing once every SM is full, so a large T gives the maximum
    for logd in range(3, 14):
        for dtype in (wl.WHT_F32, wl.WHT_BF16, wl.WHT_BF16_PF32):
            need = B.wht_affine_bwd_workspace_bytes(1 << 22, 1 << logd, dtype)
            assert 0 < need <= 16 * 1024 * 1024, f"d={1 << logd} dtype={dtype}: {need} bytes"


def test_oversized_problem_is_rejected_without_launching(B):
    # d = 32768 with 128 rows needs 128 CTAs x 256 KiB of partial sums, twice the built-in 16 MiB
    w = wl.Workload("noalloc", 128, 32768, wl.WHT_F32, "normal", 44, True, "")
    assert B.wht_affine_bwd_workspace_bytes(w.T, w.d, w.dtype) > 16 * 1024 * 1024
    x = torch.zeros(w.T, w.d, device="cuda")
    a = torch.ones(w.d, device="cuda")
    da = torch.full((w.d,), 7.0, device="cuda")
    db = torch.full((w.d,), 7.0, device="cuda")
    dx = torch.full_like(x, 7.0)
    with pytest.raises(B.WhtError) as err:
        B.wht_affine_bwd_noalloc(x, x, a, dx, da, db, w.T, w.d, w.dtype)
    assert err.value.status == -6
    torch.cuda.synchronize()
    assert torch.all(da == 7.0) and torch.all(db == 7.0) and torch.all(dx == 7.0)
