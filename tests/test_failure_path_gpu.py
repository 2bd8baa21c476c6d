"""The bounded waits of the streamed kernels, made to run out on purpose -- without faulting or hanging
anything: the library's self-test kernel waits on a barrier that nothing completes, with a limit of a few
hundred microseconds, through the very routine the tcgen05 kernels wait with.  The host must then read
WHT_ERR_DEVICE_WAIT exactly once, and the library must go on working."""
import time

import numpy as np
import pytest
import torch

import oracle
from helpers import assert_rows_bf16, to_f64
from paper_2603_08343_b200 import workloads as wl

pytestmark = pytest.mark.gpu

WHT_ERR_DEVICE_WAIT = -9


@pytest.fixture(scope="module")
def B():
    from paper_2603_08343_b200 import build
    build.build()
    from paper_2603_08343_b200 import binding
    binding.wht_affine_set_variant(0)
    return binding


def test_an_expired_wait_is_reported_once_and_the_library_goes_on(B):
    torch.cuda.synchronize()
    B.wht_affine_device_status()            # clean before the test (raises if an earlier kernel gave up)
    out = torch.zeros(3, dtype=torch.int32, device="cuda")
    t0 = time.time()
    B.wht_affine_selftest_wait_expiry(300, out)
    torch.cuda.synchronize()                # the kernel returns by itself
    assert time.time() - t0 < 5.0
    got = out.cpu().tolist()
    assert got[0] == 1, "the short wait should have run out"
    assert got[1] == 1, "the second warp should have left through the abort flag"
    with pytest.raises(B.WhtError) as err:
        B.wht_affine_device_status()
    assert err.value.status == WHT_ERR_DEVICE_WAIT
    B.wht_affine_device_status()            # cleared by the query: reported once
    # the context is intact: a tcgen05 forward right after it matches the oracle (Eq. 1)
    w = wl.CONFIGS["training"].with_rows(148 * 8 + 3)
    x = wl.gen_full(w, "x")
    a, b = wl.gen_params(w)
    B.wht_affine_set_variant(4)
    try:
        y = B.forward(x.cuda(), a.cuda(), b.cuda())
        torch.cuda.synchronize()
    finally:
        B.wht_affine_set_variant(0)
    assert_rows_bf16(to_f64(y.cpu()), oracle.wht_affine_fwd(to_f64(x), to_f64(a), to_f64(b)), "forward after the self-test")
    B.wht_affine_device_status()


def test_selftest_arguments_are_checked(B):
    out = torch.zeros(3, dtype=torch.int32, device="cuda")
    for bad in (0, 2_000_000):
        with pytest.raises(B.WhtError):
            B.wht_affine_selftest_wait_expiry(bad, out)
    torch.cuda.synchronize()
    assert out.cpu().tolist() == [0, 0, 0]
    B.wht_affine_device_status()


def test_a_failed_scratch_allocation_is_an_error_and_nothing_runs(B):
    # host-side injection: the library's next allocation answers "out of memory" without the allocator being
    # called.  The backward that needs the scratch must return WHT_ERR_WORKSPACE before any launch, leave its
    # outputs alone, and the next call must allocate and give the oracle's result.
    from helpers import assert_grad_vec
    w = wl.Workload("allocfail", 301, 2048, wl.WHT_BF16_PF32, "normal", 71, True, "")
    x, dy = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
    a, _ = wl.gen_params(w)
    xd, dyd, ad = x.cuda(), dy.cuda(), a.cuda()
    dx = torch.full_like(xd, 7.0)
    da = torch.full((w.d,), 7.0, device="cuda")
    db = torch.full((w.d,), 7.0, device="cuda")
    torch.cuda.synchronize()
    B.wht_affine_shutdown()                      # the library owns no scratch now: the next backward allocates
    assert B.wht_affine_test_fail_allocations(1) == 0
    try:
        with pytest.raises(B.WhtError) as err:
            B.wht_affine_bwd(dyd, xd, ad, dx, da, db, w.T, w.d, w.dtype)
        assert err.value.status == -6            # WHT_ERR_WORKSPACE
        torch.cuda.synchronize()
        assert torch.all(dx == 7.0) and torch.all(da == 7.0) and torch.all(db == 7.0)
        assert B.wht_affine_test_fail_allocations(0) == 0   # the one injected failure was used up
        # the calls that bring their own scratch, or need none, never allocate
        B.wht_affine_test_fail_allocations(5)
        if not B.lib().wht_affine_debug_build():
            y = B.forward(xd, ad, ad)
            B.wht_affine_bwd_noalloc(dyd, xd, ad, dx, da, db, w.T, w.d, w.dtype)
            torch.cuda.synchronize()
            assert B.wht_affine_test_fail_allocations(0) == 5
    finally:
        B.wht_affine_test_fail_allocations(0)
    B.wht_affine_bwd(dyd, xd, ad, dx, da, db, w.T, w.d, w.dtype)
    torch.cuda.synchronize()
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    assert_rows_bf16(to_f64(dx.cpu()), ref_dx, "dx after the failed allocation")
    assert_grad_vec(to_f64(da.cpu()), ref_da, "da after the failed allocation")
    assert_grad_vec(to_f64(db.cpu()), ref_db, "db after the failed allocation")
    with pytest.raises(B.WhtError):
        B.wht_affine_test_fail_allocations(-1)
    B.wht_affine_device_status()
