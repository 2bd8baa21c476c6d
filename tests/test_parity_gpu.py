"""CUDA path vs the fp64 oracle, element by element, through the C ABI (ctypes binding).

Tolerances (written out in tests/helpers.py):
  fp32 storage : max_j |err| <= 1e-5 * ||transform input row||_2      per row
  bf16 storage : max_j |err| <= 1e-2 * max_j |reference row|           per row
  da, db       : max_j |err| <= 1e-4 * max_j |reference|               per vector
"""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import assert_grad_vec, assert_rows_bf16, assert_rows_fp32, to_f64
from paper_2603_08343_b200 import workloads as wl

pytestmark = pytest.mark.gpu

# butterfly; mma.sync with direct loads; with streamed rows; tcgen05; tcgen05 with half-size products in the
# backward (each falls back where unsupported)
VARIANTS = [1, 2, 3, 4, 5]


@pytest.fixture(scope="module")
def B():
    from paper_2603_08343_b200 import build
    build.build()
    from paper_2603_08343_b200 import binding
    yield binding
    binding.wht_affine_set_variant(0)
    binding.wht_affine_device_status()  # raises if any kernel's bounded wait expired during the module


def _check_fwd(w, y_gpu, x_cpu, a_cpu, b_cpu, what):
    ref = oracle.wht_affine_fwd(to_f64(x_cpu), to_f64(a_cpu), to_f64(b_cpu))
    got = to_f64(y_gpu)
    if w.dtype == wl.WHT_F32:
        return assert_rows_fp32(got, ref, to_f64(x_cpu), what)
    return assert_rows_bf16(got, ref, what)


def _check_bwd(w, dx_gpu, da_gpu, db_gpu, dy_cpu, x_cpu, a_cpu, what):
    dy64, x64, a64 = to_f64(dy_cpu), to_f64(x_cpu), to_f64(a_cpu)
    dx, da, db = oracle.wht_affine_bwd(dy64, x64, a64)
    got = to_f64(dx_gpu)
    if w.dtype == wl.WHT_F32:
        assert_rows_fp32(got, dx, a64[None, :] * dy64, what + " dx")
    else:
        assert_rows_bf16(got, dx, what + " dx")
    assert_grad_vec(to_f64(da_gpu), da, what + " da")
    assert_grad_vec(to_f64(db_gpu), db, what + " db")


def _run_case(B, w, variant, decode=False, bwd=True):
    B.wht_affine_set_variant(variant)
    x = wl.gen_full(w, "x")
    a, b = wl.gen_params(w)
    xd, ad, bd = x.cuda(), a.cuda(), b.cuda()
    y = B.forward(xd, ad, bd, decode=decode)
    torch.cuda.synchronize()
    _check_fwd(w, y.cpu(), x, a, b, f"{w.name} T={w.T} d={w.d} v{variant} fwd")
    if bwd:
        dy = wl.gen_full(w, "dy")
        dx, da, db = B.backward(dy.cuda(), xd, ad)
        torch.cuda.synchronize()
        _check_bwd(w, dx.cpu(), da.cpu(), db.cpu(), dy, x, a, f"{w.name} T={w.T} d={w.d} v{variant} bwd")


# ------------------------------------------------------------------ configs[0]: Tiny

@pytest.mark.parametrize("variant", VARIANTS)
def test_tiny_fwd_bwd(B, variant):
    _run_case(B, wl.CONFIGS["tiny"], variant)


# ------------------------------------------------------------------ every supported d, every dtype, ragged T

@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("dtype", [wl.WHT_F32, wl.WHT_BF16, wl.WHT_BF16_PF32])
@pytest.mark.parametrize("logd", list(range(3, 14)))
def test_all_sizes_ragged_rows(B, logd, dtype, variant):
    d = 1 << logd
    # row counts that leave a ragged last tile for every rows-per-CTA setting, over several tiles
    T = 1031 if d <= 64 else (257 if d <= 1024 else 37)
    w = wl.Workload("sweep", T, d, dtype, "normal", 100 + logd, True, "")
    _run_case(B, w, variant)


@pytest.mark.parametrize("dtype", [wl.WHT_F32, wl.WHT_BF16_PF32])
def test_d16384(B, dtype):
    w = wl.Workload("sweep", 5, 16384, dtype, "normal", 77, True, "")
    _run_case(B, w, 0)


@pytest.mark.parametrize("T", [1, 2, 3, 7, 8, 9, 255, 256, 300])
def test_row_count_tails(B, T):
    for d, dtype in [(256, wl.WHT_F32), (1024, wl.WHT_BF16), (2048, wl.WHT_BF16_PF32)]:
        w = wl.Workload("tails", T, d, dtype, "normal", 200 + T, True, "")
        for variant in VARIANTS:
            _run_case(B, w, variant)


# ------------------------------------------------------------------ configs[1]: Prefill, every row

@pytest.mark.parametrize("variant", VARIANTS)
def test_prefill_full(B, variant):
    _run_case(B, wl.CONFIGS["prefill"], variant, bwd=False)


# ------------------------------------------------------------------ configs[2]: Decode

@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("T", wl.DECODE_T)
def test_decode(B, T, variant):
    w = wl.CONFIGS["decode"].with_rows(T)
    _run_case(B, w, variant, decode=True, bwd=False)


def test_prepared_call_equals_the_plain_wrapper(B):
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["decode"].with_rows(8)
    x = wl.gen_full(w, "x").cuda()
    a, b = (t.cuda() for t in wl.gen_params(w))
    y1 = B.forward(x, a, b, decode=True)
    y2 = torch.zeros_like(x)
    call = B.prepare("wht_affine_fwd_decode", x, a, b, y2, w.T, w.d, w.dtype)
    call()
    call()
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)
    bad = B.prepare("wht_affine_fwd_decode", x, a, b, y2, w.T, 100, w.dtype)  # errors surface at the call
    with pytest.raises(B.WhtError):
        bad()
    with pytest.raises(ValueError):
        B.prepare("no_such_call", x)


def test_decode_equals_fwd_bitwise(B):
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["decode"].with_rows(64)
    x = wl.gen_full(w, "x").cuda()
    a, b = (t.cuda() for t in wl.gen_params(w))
    y1 = B.forward(x, a, b, decode=True)
    y2 = B.forward(x, a, b, decode=False)
    torch.cuda.synchronize()
    # both run fp32 accumulation over the same 4096 terms; orders may differ, the rounding target not
    assert_rows_bf16(to_f64(y1.cpu()), to_f64(y2.cpu()), "decode vs fwd")


# ------------------------------------------------------------------ configs[3], [4]: full size, sampled

def _sample_rows(T, n, seed):
    rng = np.random.default_rng(seed)
    rows = set(range(64)) | set(range(T - 64, T)) | set(rng.integers(0, T, n).tolist())
    return np.array(sorted(rows))


def _spread_columns(d, per_cell, seed):
    """Column sample that reaches every part of the kernels' channel layouts: for every 1024-channel
    piece of a row and every group of 32 consecutive 8-channel chunks (the tensor-memory lane quarter
    that owns them in the tcgen05 kernels; both halves of the channels at d >= 4096), `per_cell` random
    columns, plus the corners."""
    rng = np.random.default_rng(seed)
    cols = {0, 1, d // 2 - 1, d // 2, d - 2, d - 1}
    for piece in range(max(1, d // 1024)):
        for quarter in range(4):
            m = rng.integers(quarter * 32, quarter * 32 + 32, per_cell)
            n = rng.integers(0, 8, per_cell)
            cols |= set((piece * 1024 + m * 8 + n).tolist())
    return np.array(sorted(c for c in cols if 0 <= c < d))


def _full_size_case(B, w, n_rows, cols, variant):
    """Full-size run of a config in the launch configuration the benchmark times.  y and dx: sampled rows
    against the oracle (Eq. 1 and its chain rule).  da, db need every row: the oracle's column form over
    all T rows, on the columns given (None = every column)."""
    B.wht_affine_set_variant(variant)
    a, b = wl.gen_params(w)
    ad, bd = a.cuda(), b.cuda()
    x = wl.gen_full(w, "x", out=torch.empty(w.T, w.d, dtype=w.io_torch_dtype).pin_memory(), threads=32)
    dy = wl.gen_full(w, "dy", out=torch.empty(w.T, w.d, dtype=w.io_torch_dtype).pin_memory(), threads=32)
    xd, dyd = x.cuda(), dy.cuda()
    y = B.forward(xd, ad, bd)
    dx, da, db = B.backward(dyd, xd, ad)
    torch.cuda.synchronize()
    rows = _sample_rows(w.T, n_rows, w.seed)
    ridx = torch.from_numpy(rows)
    xs, dys = x[ridx], dy[ridx]
    ys, dxs = y[ridx.cuda()].cpu(), dx[ridx.cuda()].cpu()
    a64 = to_f64(a)
    ref_y = oracle.wht_affine_fwd(to_f64(xs), a64, to_f64(b))
    assert_rows_bf16(to_f64(ys), ref_y, f"{w.name} fwd sampled rows")
    ref_dx, _, _ = oracle.wht_affine_bwd(to_f64(dys), to_f64(xs), a64)
    assert_rows_bf16(to_f64(dxs), ref_dx, f"{w.name} dx sampled rows")
    every = cols is None
    cols = np.arange(w.d) if every else np.asarray(cols)
    da_ref = np.zeros(cols.size)
    db_ref = np.zeros(cols.size)
    blk = 8192
    for r0 in range(0, w.T, blk):
        pa, pb = oracle.da_db_columns(to_f64(dy[r0:r0 + blk]), to_f64(x[r0:r0 + blk]), cols)
        da_ref += pa
        db_ref += pb
    da_got = to_f64(da.cpu())[cols]
    db_got = to_f64(db.cpu())[cols]
    # the bound is 1e-4 * max|g_ref| over the vector; a column sample gives a lower estimate of that
    # maximum, which only makes the check stricter
    which = "all columns" if every else f"{cols.size} columns"
    assert_grad_vec(da_got, da_ref, f"{w.name} da {which}")
    assert_grad_vec(db_got, db_ref, f"{w.name} db {which}")
    if not every:
        # db over ALL columns against plain column sums in fp64 (cheap at any size)
        db_all = np.zeros(w.d)
        for r0 in range(0, w.T, blk):
            db_all += to_f64(dy[r0:r0 + blk]).sum(axis=0)
        assert_grad_vec(to_f64(db.cpu()), db_all, f"{w.name} db all columns")


@pytest.mark.parametrize("variant", VARIANTS)
def test_training_full_size(B, variant):
    # the automatic selection (what the benchmark times) is checked on every column of da and db; the
    # forced families on a spread sample
    w = wl.CONFIGS["training"]
    _full_size_case(B, w, n_rows=1024, cols=_spread_columns(w.d, 12, w.seed + 1), variant=variant)


def test_training_full_size_every_column(B):
    _full_size_case(B, wl.CONFIGS["training"], n_rows=1024, cols=None, variant=0)


def test_large_full_size(B):
    w = wl.CONFIGS["large"]
    cols = _spread_columns(w.d, 16, w.seed + 1)  # 8 pieces x 4 lane quarters x 16 = about 500 columns
    assert cols.size >= 256
    _full_size_case(B, w, n_rows=256, cols=cols, variant=0)


# ------------------------------------------------------------------ the paper's own inference shapes

@pytest.mark.parametrize("d", [1024, 2048])
def test_paper_prefill_shape(B, d):
    """The paper's prefill benchmark: batch 1024 x 64 input tokens = 65536 rows, at its two power-of-two
    model widths (Small d = 1024, Large d = 2048), bf16 rows and parameters; sampled rows against Eq. 1."""
    B.wht_affine_set_variant(0)
    w = wl.Workload("paper_prefill", 1024 * 64, d, wl.WHT_BF16, "normal", 10 + d, False, "")
    a, b = wl.gen_params(w)
    x = wl.gen_full(w, "x", threads=32)
    y = B.forward(x.cuda(), a.cuda(), b.cuda())
    torch.cuda.synchronize()
    ridx = torch.from_numpy(_sample_rows(w.T, 2048, w.seed))
    ref = oracle.wht_affine_fwd(to_f64(x[ridx]), to_f64(a), to_f64(b))
    assert_rows_bf16(to_f64(y[ridx.cuda()].cpu()), ref, f"paper prefill d={d}")
    B.wht_affine_device_status()


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d", [1024, 2048])
def test_paper_decode_shape(B, d, variant):
    """The paper's decode benchmark: batch 2048, one new token per sequence = 2048 rows per call, through
    wht_affine_fwd_decode; every row against Eq. 1."""
    w = wl.Workload("paper_decode", 2048, d, wl.WHT_BF16, "normal", 20 + d, False, "")
    _run_case(B, w, variant, decode=True, bwd=False)


# ------------------------------------------------------------------ structure that needs no oracle

@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d", [256, 4096, 32768])
def test_impulse_rows_closed_form(B, d, variant):
    # x = e_k  =>  y = a (.) (row k of H)/sqrt(d) + b with sign (-1)^popcount(k & j)
    B.wht_affine_set_variant(variant)
    ks = [0, 1, 5, d // 2, d - 1]
    x = torch.zeros(len(ks), d, dtype=torch.float32)
    for r, k in enumerate(ks):
        x[r, k] = 1.0
    w = wl.Workload("imp", len(ks), d, wl.WHT_F32, "normal", 9, False, "")
    a, b = wl.gen_params(w)
    y = B.forward(x.cuda(), a.cuda(), b.cuda()).cpu().numpy().astype(np.float64)
    j = np.arange(d)
    for r, k in enumerate(ks):
        par = np.zeros(d, dtype=np.int64)
        v = j & k
        while np.any(v):
            par ^= v & 1
            v >>= 1
        want = a.numpy().astype(np.float64) * (1 - 2 * par) / math.sqrt(d) + b.numpy().astype(np.float64)
        assert np.max(np.abs(y[r] - want)) <= 1e-5


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,dtype", [(32768, torch.float32), (8192, torch.float32), (1024, torch.float32)])
def test_involution_and_norm(B, d, dtype, variant):
    B.wht_affine_set_variant(variant)
    g = torch.Generator().manual_seed(d)
    x = torch.randn(9, d, generator=g, dtype=dtype).cuda()
    one = torch.ones(d, dtype=dtype).cuda()
    zero = torch.zeros(d, dtype=dtype).cuda()
    z = B.forward(x, one, zero)
    back = B.forward(z, one, zero)
    torch.cuda.synchronize()
    xn = x.double().norm(dim=1)
    assert torch.all((z.double().norm(dim=1) - xn).abs() <= 1e-5 * xn)
    assert torch.all((back.double() - x.double()).abs().amax(dim=1) <= 2e-5 * xn)


@pytest.mark.parametrize("variant", VARIANTS)
def test_in_place_and_empty(B, variant):
    B.wht_affine_set_variant(variant)
    for name in ("tiny", "prefill"):
        w = wl.CONFIGS[name].with_rows(300)
        x = wl.gen_full(w, "x").cuda()
        a, b = (t.cuda() for t in wl.gen_params(w))
        y = B.forward(x, a, b)
        x2 = x.clone()
        B.forward(x2, a, b, out=x2)
        assert torch.equal(y, x2)
        dy = wl.gen_full(w, "dy").cuda()
        dx, da, db = B.backward(dy, x, a)
        dy2 = dy.clone()
        da2, db2 = torch.empty_like(da), torch.empty_like(db)
        B.wht_affine_bwd(dy2, x, a, dy2, da2, db2, w.T, w.d, w.dtype)
        assert torch.equal(dx, dy2) and torch.equal(da, da2) and torch.equal(db, db2)
        # T == 0: forward is a no-op, backward writes zeros
        e = torch.empty(0, w.d, dtype=x.dtype, device="cuda")
        B.forward(e, a, b)
        da0 = torch.full((w.d,), 3.0, device="cuda")
        db0 = torch.full((w.d,), 3.0, device="cuda")
        B.wht_affine_bwd(e, e, a, e, da0, db0, 0, w.d, w.dtype)
        torch.cuda.synchronize()
        assert torch.count_nonzero(da0) == 0 and torch.count_nonzero(db0) == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_bwd_reproducible_and_workspace_forms_agree(B, variant):
    B.wht_affine_set_variant(variant)
    w = wl.CONFIGS["training"].with_rows(5000)
    x = wl.gen_full(w, "x").cuda()
    dy = wl.gen_full(w, "dy").cuda()
    a, _ = wl.gen_params(w)
    a = a.cuda()
    dx1, da1, db1 = B.backward(dy, x, a)
    dx2, da2, db2 = B.backward(dy, x, a)
    assert torch.equal(dx1, dx2) and torch.equal(da1, da2) and torch.equal(db1, db2)
    need = B.wht_affine_bwd_workspace_bytes(w.T, w.d, w.dtype)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    dx3 = torch.empty_like(dx1)
    da3, db3 = torch.empty_like(da1), torch.empty_like(db1)
    B.wht_affine_bwd_ws(dy, x, a, dx3, da3, db3, w.T, w.d, w.dtype, ws)
    assert torch.equal(dx1, dx3) and torch.equal(da1, da3) and torch.equal(db1, db3)
    small = torch.empty(max(need // 2, 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.WhtError) as err:
        B.wht_affine_bwd_ws(dy, x, a, dx3, da3, db3, w.T, w.d, w.dtype, small)
    assert err.value.status == -6


def test_heavy_tailed_rows(B):
    # Student-t(3) rows in bf16: single spikes dominate a row; fp32 accumulation must hold the bound
    for variant in VARIANTS:
        w = wl.CONFIGS["large"].with_rows(48)
        _run_case(B, w, variant)


def test_streamed_kernels_on_many_rows(B):
    # enough rows that every row group loops through its ring several times, ragged tail
    B.wht_affine_set_variant(3)
    for d, dtype, T in [(512, wl.WHT_BF16, 9001), (1024, wl.WHT_BF16, 20011), (2048, wl.WHT_BF16_PF32, 9973),
                        (4096, wl.WHT_BF16, 3001), (8192, wl.WHT_BF16_PF32, 1501)]:
        w = wl.Workload("stream", T, d, dtype, "normal", 300 + d, True, "")
        _run_case(B, w, 3)
    B.wht_affine_device_status()


def test_fp32_rows_on_the_tensor_core_passes(B):
    # fp32 rows enter every H_16 pass as three bf16 terms; the fp32 bound (1e-5 of the row norm) must hold as
    # for the register butterflies.  Direct loads (2), streamed (3: every ring wraps several times, ragged
    # tail), and the automatic choice from the row count on at which it streams.
    for d, T in [(256, 20011), (512, 9001), (1024, 9973), (2048, 5003), (4096, 3001), (8192, 1501)]:
        w = wl.Workload("f32mma", T, d, wl.WHT_F32, "normal", 900 + d, True, "")
        _run_case(B, w, 3)
    for d, T in [(256, 1031), (1024, 2053), (2048, 1201), (8192, 301)]:
        w = wl.Workload("f32mma", T, d, wl.WHT_F32, "normal", 950 + d, True, "")
        _run_case(B, w, 2)
    for d, T in [(512, 148 * 32 + 5), (1024, 148 * 32 + 1), (2048, 148 * 32 + 3)]:
        w = wl.Workload("f32mma", T, d, wl.WHT_F32, "student_t3", 970 + d, True, "")
        _run_case(B, w, 0)
    B.wht_affine_device_status()


@pytest.mark.parametrize("d,dtype,variants", [(1024, wl.WHT_BF16_PF32, [0, 1, 2, 3]), (1024, wl.WHT_F32, [0, 1, 2]),
                                              (8192, wl.WHT_BF16_PF32, [0, 3]), (256, wl.WHT_BF16, [0, 1])])
def test_tensors_past_two_to_the_31_elements(B, d, dtype, variants):
    # e.g. 2^21 + 5 rows of 1024: 2^31 + 5120 elements per tensor, byte offsets past 4 GiB (bf16) and 8 GiB (fp32), so
    # any 32-bit element or byte index in a kernel or on the way to it shows.  Only three blocks of rows are
    # non-zero (the first rows, rows around the middle, the last 133): they are checked against the oracle row by
    # row; a zero row must come out as b (forward) and as zero (backward), exactly; and da, db are sums over rows
    # to which the zero rows add nothing, so the oracle on the three blocks alone gives them.
    T = (1 << 31) // d + 5
    blocks = [(0, 128), (T // 2 - 3, 128), (T - 133, 133)]
    zero_rows = [128, 5000, T // 3, T // 2 + 200, T - 134]
    proto = wl.Workload("big", 1, d, dtype, "normal", 1234, True, "")
    a, b = wl.gen_params(proto)
    tdt = proto.io_torch_dtype
    x_d = torch.zeros(T, d, dtype=tdt, device="cuda")
    dy_d = torch.zeros(T, d, dtype=tdt, device="cuda")
    xs, dys = [], []
    for i, (r0, n) in enumerate(blocks):
        wb = wl.Workload("big", n, d, dtype, "normal", 1300 + i, True, "")
        xs.append(wl.gen_full(wb, "x"))
        dys.append(wl.gen_full(wb, "dy"))
        x_d[r0:r0 + n].copy_(xs[-1])
        dy_d[r0:r0 + n].copy_(dys[-1])
    x_all, dy_all = torch.cat(xs), torch.cat(dys)
    a64, b64 = to_f64(a), to_f64(b)
    y_ref = oracle.wht_affine_fwd(to_f64(x_all), a64, b64)
    dx_ref, da_ref, db_ref = oracle.wht_affine_bwd(to_f64(dy_all), to_f64(x_all), a64)
    ad, bd = a.cuda(), b.cuda()
    b_stored = bd.to(tdt)
    y_d = torch.empty_like(x_d)
    for variant in variants:
        B.wht_affine_set_variant(variant)
        y_d.fill_(7.0)
        B.forward(x_d, ad, bd, out=y_d)
        got = torch.cat([y_d[r0:r0 + n] for r0, n in blocks]).cpu()
        what = f"2^31 elements, dtype {dtype}, v{variant}"
        if dtype == wl.WHT_F32:
            assert_rows_fp32(to_f64(got), y_ref, to_f64(x_all), what + " y")
        else:
            assert_rows_bf16(to_f64(got), y_ref, what + " y")
        for r in zero_rows:
            assert torch.equal(y_d[r], b_stored), f"{what}: y of zero row {r}"
        # fused residual add, in place over the residual stream (here: dy)
        y_d.copy_(dy_d)
        B.forward(x_d, ad, bd, out=y_d, resid=y_d)
        got = torch.cat([y_d[r0:r0 + n] for r0, n in blocks]).cpu()
        res_ref = oracle.wht_affine_fwd_residual(to_f64(x_all), a64, b64, to_f64(dy_all))
        if dtype == wl.WHT_F32:
            err = np.max(np.abs(to_f64(got) - res_ref), axis=1)
            assert np.all(err <= 1e-5 * (np.linalg.norm(to_f64(x_all), axis=1) + np.max(np.abs(to_f64(dy_all)), axis=1)))
        else:
            assert_rows_bf16(to_f64(got), res_ref, what + " y + resid")
        for r in zero_rows:
            assert torch.equal(y_d[r], b_stored), f"{what}: residual form, zero row {r}"
        y_d.fill_(7.0)
        da = torch.empty(d, dtype=torch.float32, device="cuda")
        db = torch.empty(d, dtype=torch.float32, device="cuda")
        B.wht_affine_bwd(dy_d, x_d, ad, y_d, da, db, T, d, dtype)
        got = torch.cat([y_d[r0:r0 + n] for r0, n in blocks]).cpu()
        if dtype == wl.WHT_F32:
            assert_rows_fp32(to_f64(got), dx_ref, a64[None, :] * to_f64(dy_all), what + " dx")
        else:
            assert_rows_bf16(to_f64(got), dx_ref, what + " dx")
        for r in zero_rows:
            assert torch.count_nonzero(y_d[r]).item() == 0, f"{what}: dx of zero row {r}"
        assert_grad_vec(to_f64(da.cpu()), da_ref, what + " da")
        assert_grad_vec(to_f64(db.cpu()), db_ref, what + " db")
    B.wht_affine_set_variant(0)
    B.wht_affine_device_status()


def test_tcgen05_kernels_on_many_rows(B):
    # several tiles per CTA on every SM (the ring and both accumulator sets wrap), ragged last tile
    for d, dtype, T in [(1024, wl.WHT_BF16, 148 * 16 * 5 + 7), (2048, wl.WHT_BF16_PF32, 148 * 8 * 4 + 3),
                        (4096, wl.WHT_BF16, 148 * 4 * 3 + 1), (8192, wl.WHT_BF16_PF32, 148 * 2 * 3 + 1)]:
        w = wl.Workload("tc5", T, d, dtype, "normal", 400 + d, True, "")
        _run_case(B, w, 4)
        _run_case(B, w, 5)
    B.wht_affine_device_status()


def test_back_to_back_calls_see_each_others_results(B):
    # The kernels are launched so that a call may be scheduled while its predecessor in the stream
    # still drains; each must nevertheless read what the predecessor wrote.  A chain of calls that
    # feed one another must give the same bits with and without a synchronisation after every call.
    B.wht_affine_set_variant(0)
    for d, dtype, T in [(2048, wl.WHT_BF16_PF32, 148 * 8 * 3 + 5), (1024, wl.WHT_BF16, 148 * 16 * 2 + 3),
                        (4096, wl.WHT_BF16, 64)]:
        w = wl.Workload("chain", T, d, dtype, "normal", 500 + d, True, "")
        x0 = wl.gen_full(w, "x").cuda()
        dy = wl.gen_full(w, "dy").cuda()
        a, b = (t.cuda() for t in wl.gen_params(w))

        def chain(sync):
            bufs = [x0.clone(), torch.empty_like(x0)]
            da = torch.empty(d, dtype=torch.float32, device="cuda")
            db = torch.empty_like(da)
            dx = torch.empty_like(x0)
            for k in range(6):
                B.wht_affine_fwd(bufs[k % 2], a, b, bufs[(k + 1) % 2], T, d, dtype)
                if sync:
                    torch.cuda.synchronize()
            # the backward reads the row tensor the last forward has just written, twice in a row
            for _ in range(2):
                B.wht_affine_bwd(dy, bufs[0], a, dx, da, db, T, d, dtype)
                if sync:
                    torch.cuda.synchronize()
            torch.cuda.synchronize()
            return bufs[0].clone(), dx, da, db

        got, ref = chain(False), chain(True)
        assert all(torch.equal(g, r) for g, r in zip(got, ref)), f"d={d}: chained calls differ"
        assert torch.isfinite(got[0].float()).all()
    B.wht_affine_device_status()


# ------------------------------------------------------------------ fused residual forward

@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,dtype,T", [(256, wl.WHT_F32, 64), (64, wl.WHT_BF16, 1031), (1024, wl.WHT_BF16, 257),
                                       (2048, wl.WHT_BF16_PF32, 300), (4096, wl.WHT_BF16, 37),
                                       (8192, wl.WHT_BF16_PF32, 21), (16384, wl.WHT_F32, 5),
                                       (2048, wl.WHT_F32, 300), (1024, wl.WHT_F32, 148 * 32 + 9)])
def test_fwd_residual(B, d, dtype, T, variant):
    B.wht_affine_set_variant(variant)
    w = wl.Workload("res", T, d, dtype, "normal", 600 + d, True, "")
    x, r = wl.gen_full(w, "x"), wl.gen_full(w, "dy")  # the second seeded tensor serves as the residual stream
    a, b = wl.gen_params(w)
    xd, rd, ad, bd = x.cuda(), r.cuda(), a.cuda(), b.cuda()
    y = B.forward(xd, ad, bd, resid=rd)
    torch.cuda.synchronize()
    ref = oracle.wht_affine_fwd_residual(to_f64(x), to_f64(a), to_f64(b), to_f64(r))
    if dtype == wl.WHT_F32:
        # the transform's error scales with ||x||, the final add with |resid|: one rounding of the sum
        err = np.max(np.abs(to_f64(y.cpu()) - ref), axis=1)
        assert np.all(err <= 1e-5 * (np.linalg.norm(to_f64(x), axis=1) + np.max(np.abs(to_f64(r)), axis=1)))
    else:
        assert_rows_bf16(to_f64(y.cpu()), ref, f"residual d={d} v{variant}")
    # in place over the residual stream (out == resid), as a model would call it
    r2 = rd.clone()
    B.forward(xd, ad, bd, out=r2, resid=r2)
    assert torch.equal(r2, y)


def test_fwd_residual_many_rows(B):
    # the tcgen05 kernels' residual path over several tiles per CTA with a ragged tail
    B.wht_affine_set_variant(0)
    for d, dtype, T in [(1024, wl.WHT_BF16, 148 * 16 * 3 + 5), (2048, wl.WHT_BF16_PF32, 148 * 8 * 2 + 3),
                        (8192, wl.WHT_BF16_PF32, 148 * 2 * 2 + 1)]:
        w = wl.Workload("res", T, d, dtype, "normal", 700 + d, True, "")
        x, r = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
        a, b = wl.gen_params(w)
        y = B.forward(x.cuda(), a.cuda(), b.cuda(), resid=r.cuda())
        torch.cuda.synchronize()
        ref = oracle.wht_affine_fwd_residual(to_f64(x), to_f64(a), to_f64(b), to_f64(r))
        assert_rows_bf16(to_f64(y.cpu()), ref, f"residual many rows d={d}")
    B.wht_affine_device_status()


def test_fwd_residual_training_full_size(B):
    # the fused residual forward in the launch configuration the benchmark times (65536 x 2048), sampled rows
    # against y = resid + Eq. 1
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["training"]
    a, b = wl.gen_params(w)
    x = wl.gen_full(w, "x", threads=32)
    r = wl.gen_full(w, "dy", threads=32)  # the second seeded tensor serves as the residual stream
    y = B.forward(x.cuda(), a.cuda(), b.cuda(), resid=r.cuda())
    torch.cuda.synchronize()
    ridx = torch.from_numpy(_sample_rows(w.T, 1024, w.seed + 9))
    ref = oracle.wht_affine_fwd_residual(to_f64(x[ridx]), to_f64(a), to_f64(b), to_f64(r[ridx]))
    assert_rows_bf16(to_f64(y[ridx.cuda()].cpu()), ref, "residual forward, training size")
    B.wht_affine_device_status()


def test_host_pipeline_matches_direct_calls(B):
    # end-to-end helpers: pinned host -> device -> C ABI -> pinned host, rows moving in chunks on two
    # copy streams; same results as the plain device-resident calls
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["training"].with_rows(5000)
    x, dy = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
    a, b = wl.gen_params(w)
    xd, dyd, ad, bd = x.cuda(), dy.cuda(), a.cuda(), b.cuda()
    y_ref = B.forward(xd, ad, bd)
    dx_ref, da_ref, db_ref = B.backward(dyd, xd, ad)
    torch.cuda.synchronize()
    st = {"x": torch.empty_like(xd), "a": torch.empty_like(ad), "b": torch.empty_like(bd), "y": torch.empty_like(xd),
          "dy": torch.empty_like(xd), "dx": torch.empty_like(xd), "da": torch.empty_like(da_ref),
          "db": torch.empty_like(db_ref)}
    xp, dyp, ap, bp = x.pin_memory(), dy.pin_memory(), a.pin_memory(), b.pin_memory()
    for pipe in (None, B.HostPipe(chunk_rows=1024)):
        yp, dxp = torch.empty_like(xp).pin_memory(), torch.empty_like(xp).pin_memory()
        dap, dbp = torch.empty(w.d).pin_memory(), torch.empty(w.d).pin_memory()
        B.forward_host(xp, ap, bp, yp, st, pipe=pipe)
        B.backward_host(dyp, xp, ap, dxp, dap, dbp, st, pipe=pipe, x_resident=True)
        if pipe is not None:
            pipe.join()
        torch.cuda.synchronize()
        if pipe is None:
            assert torch.equal(yp, y_ref.cpu())
        else:
            # a 1024-row chunk is below the tcgen05 cross-over: another kernel family, another
            # summation order, the same rounding target
            assert_rows_bf16(to_f64(yp), to_f64(y_ref.cpu()), "chunked forward")
        if pipe is None:
            assert torch.equal(dxp, dx_ref.cpu())
            assert torch.equal(dap, da_ref.cpu()) and torch.equal(dbp, db_ref.cpu())
        else:
            assert_rows_bf16(to_f64(dxp), to_f64(dx_ref.cpu()), "chunked backward dx")
            assert_grad_vec(to_f64(dap), to_f64(da_ref.cpu()), "chunked backward da")
            assert_grad_vec(to_f64(dbp), to_f64(db_ref.cpu()), "chunked backward db")


def test_host_backward_twice_in_a_row_without_a_sync(B):
    # Two end-to-end backward calls on different inputs through the SAME staging buffers, no host or
    # stream synchronisation in between: the second call's copies in must wait for the first call's
    # kernels, and its kernels for the first call's copies out.  Both results against the oracle.
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["training"].with_rows(6000)
    a, _ = wl.gen_params(w)
    sets = []
    for k in range(2):
        wk = wl.Workload(w.name, w.T, w.d, w.dtype, w.dist, w.seed + 50 + k, True, "")
        sets.append((wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")))
    dev = lambda t: torch.empty_like(t, device="cuda")  # noqa: E731
    for pipe in (None, B.HostPipe(chunk_rows=1024)):
        st = {"x": dev(sets[0][0]), "a": dev(a), "dy": dev(sets[0][0]), "dx": dev(sets[0][0]),
              "da": torch.empty(w.d, device="cuda"), "db": torch.empty(w.d, device="cuda")}
        ap = a.pin_memory()
        outs = []
        for x, dy in sets:
            xp, dyp = x.pin_memory(), dy.pin_memory()
            dxp = torch.empty_like(xp).pin_memory()
            dap, dbp = torch.empty(w.d).pin_memory(), torch.empty(w.d).pin_memory()
            B.backward_host(dyp, xp, ap, dxp, dap, dbp, st, pipe=pipe, x_resident=False)
            outs.append((xp, dyp, dxp, dap, dbp))
        if pipe is not None:
            pipe.join()
        torch.cuda.synchronize()
        for k, (xp, dyp, dxp, dap, dbp) in enumerate(outs):
            ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dyp), to_f64(xp), to_f64(a))
            tag = f"host backward call {k} ({'plain' if pipe is None else 'piped'})"
            assert_rows_bf16(to_f64(dxp), ref_dx, tag + " dx")
            assert_grad_vec(to_f64(dap), ref_da, tag + " da")
            assert_grad_vec(to_f64(dbp), ref_db, tag + " db")


def test_reduce_grads(B):
    # gradients of disjoint row sets add: chunked backward + wht_affine_reduce_grads == one backward
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["training"].with_rows(3001)
    x, dy = wl.gen_full(w, "x").cuda(), wl.gen_full(w, "dy").cuda()
    a = wl.gen_params(w)[0].cuda()
    bounds = [0, 7, 1500, 1501, 3001]
    parts = torch.full((len(bounds) - 1, 2, w.d), float("nan"), device="cuda")
    dx = torch.empty_like(x)
    for i in range(len(bounds) - 1):
        r0, r1 = bounds[i], bounds[i + 1]
        B.wht_affine_bwd(dy[r0:r1], x[r0:r1], a, dx[r0:r1], parts[i, 0], parts[i, 1], r1 - r0, w.d, w.dtype)
    da, db = torch.empty(w.d, device="cuda"), torch.empty(w.d, device="cuda")
    B.wht_affine_reduce_grads(parts, parts.shape[0], w.d, da, db)
    da2, db2 = torch.empty_like(da), torch.empty_like(db)
    B.wht_affine_reduce_grads(parts, parts.shape[0], w.d, da2, db2)
    torch.cuda.synchronize()
    assert torch.equal(da, da2) and torch.equal(db, db2)
    _, da_ref, db_ref = oracle.wht_affine_bwd(to_f64(dy.cpu()), to_f64(x.cpu()), to_f64(a.cpu()))
    assert_grad_vec(to_f64(da.cpu()), da_ref, "reduced da")
    assert_grad_vec(to_f64(db.cpu()), db_ref, "reduced db")
    np.testing.assert_allclose(to_f64(da.cpu()), parts[:, 0].double().sum(0).cpu().numpy(), rtol=1e-6, atol=1e-4)
    B.wht_affine_reduce_grads(parts, 0, w.d, da, db)
    torch.cuda.synchronize()
    assert torch.count_nonzero(da) == 0 and torch.count_nonzero(db) == 0


def _round_to_bf16_bits(v64: np.ndarray) -> np.ndarray:
    """fp64 -> nearest-even bfloat16 bit patterns, done on the integer representation of fp32."""
    f32 = v64.astype(np.float32)
    # where the fp32 rounding of the fp64 value is itself a tie-breaker it could double-round; such
    # values have measure ~2^-29 and do not move the statistics below
    u = f32.view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


@pytest.mark.parametrize("variant", [0, 3, 4, 5])
def test_outputs_are_the_correctly_rounded_values_almost_everywhere(B, variant):
    # fp32 accumulation then ONE rounding: the stored bf16 must be the nearest bf16 of the exact
    # result except where the fp32 error (~1e-7 relative to the row scale) straddles a rounding
    # boundary (bf16 spacing ~4e-3 relative): a fraction of order 1e-3.  An intermediate kept in
    # bf16 anywhere on the path would push the fraction to tens of per cent.
    B.wht_affine_set_variant(variant)
    w = wl.CONFIGS["training"].with_rows(2400)
    x, dy = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
    a, b = wl.gen_params(w)
    xd, dyd, ad, bd = x.cuda(), dy.cuda(), a.cuda(), b.cuda()
    y = B.forward(xd, ad, bd)
    B.wht_affine_set_bwd_operand_mode(1)  # the mode in which dx is rounded once (g carried as a bf16 pair)
    try:
        dx, _, _ = B.backward(dyd, xd, ad)
        torch.cuda.synchronize()
    finally:
        B.wht_affine_set_bwd_operand_mode(0)
    ref_y = oracle.wht_affine_fwd(to_f64(x), to_f64(a), to_f64(b))
    ref_dx, _, _ = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    # (tensor, reference, name, allowed fraction not nearest, absolute slack relative to the row maximum:
    #  fp32 accumulation for y; for dx the bf16 hi + lo operand split adds 2^-17 of the operand scale)
    # the mma.sync family splits an fp32 operand into bf16 hi + lo in the forward too
    y_slack = 4e-5 if variant == 3 else 2e-6
    for got, ref, what, bound, slack in ((y, ref_y, "y", 5e-3, y_slack), (dx, ref_dx, "dx", 2e-2, 4e-5)):
        bits = got.cpu().view(torch.int16).numpy().view(np.uint16)
        want = _round_to_bf16_bits(ref)
        frac = float(np.mean(bits != want))
        assert frac <= bound, f"{what} v{variant}: {frac:.2e} of the outputs are not the nearest bf16"
        # every output within half a bf16 step of the exact value plus the arithmetic's own error
        half_step = np.exp2(np.floor(np.log2(np.maximum(np.abs(ref), 1e-300))) - 8)
        err = np.abs(to_f64(got.cpu()) - ref)
        allowed = half_step * (1 + 1e-6) + slack * np.max(np.abs(ref), axis=1, keepdims=True)
        worst = float(np.max(err / allowed))
        assert worst <= 1.0, f"{what} v{variant}: an output is {worst:.2f}x beyond half a bf16 step + {slack:g}*max|row|"


# ------------------------------------------------------------------ bf16-operand mode of the tcgen05 backward

@pytest.mark.parametrize("name,rows", [("training", 148 * 8 * 2 + 3), ("large", 148 * 2 * 2 + 1), ("prefill", 148 * 16 + 5)])
@pytest.mark.parametrize("variant", [4, 5])
def test_bwd_bf16_operand_mode(B, name, rows, variant):
    """The two settings of wht_affine_set_bwd_operand_mode.  In the default one g = (a/sqrt d) (.) dy is
    rounded to bf16 once before the second +-1 product; with mode 1 it is carried as a bf16 pair.  In both,
    dx must meet the bound for bf16 storage, 1e-2 * max|dx_row|, on every row of the chain rule of Eq. 1
    -- also on the heavy-tailed rows of the Large config, where one spike dominates a row -- with half
    of the bound to spare, and da, db (which never pass through g) must have the same bits in both."""
    B.wht_affine_set_variant(variant)
    base = wl.CONFIGS[name]
    w = wl.Workload(base.name, rows, base.d, base.dtype, base.dist, base.seed + 7, True, "")
    x, dy = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
    a, _ = wl.gen_params(w)
    xd, dyd, ad = x.cuda(), dy.cuda(), a.cuda()
    assert B.wht_affine_get_bwd_operand_mode() == 0
    dx0, da0, db0 = B.backward(dyd, xd, ad)
    B.wht_affine_set_bwd_operand_mode(1)
    try:
        dx1, da1, db1 = B.backward(dyd, xd, ad)
        torch.cuda.synchronize()
    finally:
        B.wht_affine_set_bwd_operand_mode(0)
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    worst0 = assert_rows_bf16(to_f64(dx0.cpu()), ref_dx, f"{name} dx, bf16 operand (default)")
    worst1 = assert_rows_bf16(to_f64(dx1.cpu()), ref_dx, f"{name} dx, bf16 pair")
    assert worst0 <= 0.5, f"{name}: the default mode uses {worst0:.2f} of the bound (pair mode {worst1:.2f})"
    assert worst1 <= worst0 + 1e-9
    assert torch.equal(da0, da1) and torch.equal(db0, db1)
    assert_grad_vec(to_f64(da0.cpu()), ref_da, f"{name} da")
    assert_grad_vec(to_f64(db0.cpu()), ref_db, f"{name} db")
    with pytest.raises(B.WhtError):
        B.wht_affine_set_bwd_operand_mode(2)
    B.wht_affine_set_variant(0)
    B.wht_affine_device_status()


# ------------------------------------------------------------------ grouped (block-diagonal) form

@pytest.mark.parametrize("variant", [0, 1, 2, 3])
@pytest.mark.parametrize("d,block,dtype,T", [(768, 256, wl.WHT_F32, 70), (768, 256, wl.WHT_BF16, 300),
                                             (1280, 256, wl.WHT_BF16_PF32, 1237), (3072, 512, wl.WHT_F32, 611),
                                             (1536, 512, wl.WHT_BF16_PF32, 129), (3072, 1024, wl.WHT_BF16, 33),
                                             (96, 32, wl.WHT_F32, 1000), (1024, 1024, wl.WHT_BF16, 40),
                                             (768, 256, wl.WHT_BF16_PF32, 148 * 32 + 77), (1536, 512, wl.WHT_BF16, 148 * 32 + 5),
                                             (512, 256, wl.WHT_BF16, 3), (6144, 2048, wl.WHT_BF16_PF32, 21),
                                             (768, 256, wl.WHT_F32, 148 * 32 + 9)])
def test_grouped_form(B, d, block, dtype, T, variant):
    B.wht_affine_set_variant(variant)
    w = wl.Workload("grp", T, block, dtype, "normal", 800 + d, True, "")  # generators take a power of two:
    G = d // block                                                          # draw G blocks side by side
    x = torch.cat([wl.gen_full(wl.Workload("grp", T, block, dtype, "normal", 800 + d + g, True, ""), "x")
                   for g in range(G)], dim=1).contiguous()
    dy = torch.cat([wl.gen_full(wl.Workload("grp", T, block, dtype, "normal", 800 + d + g, True, ""), "dy")
                    for g in range(G)], dim=1).contiguous()
    ab = [wl.gen_params(wl.Workload("grp", T, block, dtype, "normal", 800 + d + g, True, "")) for g in range(G)]
    a = torch.cat([p[0] for p in ab]).contiguous()
    b = torch.cat([p[1] for p in ab]).contiguous()
    xd, dyd, ad, bd = x.cuda(), dy.cuda(), a.cuda(), b.cuda()
    y = torch.empty_like(xd)
    B.wht_affine_fwd_grouped(xd, ad, bd, y, T, d, block, dtype)
    need = B.wht_affine_bwd_grouped_workspace_bytes(T, d, block, dtype)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    dx = torch.empty_like(xd)
    da = torch.empty(d, dtype=torch.float32, device="cuda")
    db = torch.empty_like(da)
    B.wht_affine_bwd_grouped(dyd, xd, ad, dx, da, db, T, d, block, dtype, ws)
    torch.cuda.synchronize()
    ref_y = oracle.wht_affine_fwd_grouped(to_f64(x), to_f64(a), to_f64(b), block)
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd_grouped(to_f64(dy), to_f64(x), to_f64(a), block)
    if dtype == wl.WHT_F32:
        assert_rows_fp32(to_f64(y.cpu()), ref_y, to_f64(x), "grouped y")
        assert_rows_fp32(to_f64(dx.cpu()), ref_dx, to_f64(a)[None, :] * to_f64(dy), "grouped dx")
    else:
        assert_rows_bf16(to_f64(y.cpu()), ref_y, "grouped y")
        assert_rows_bf16(to_f64(dx.cpu()), ref_dx, "grouped dx")
    assert_grad_vec(to_f64(da.cpu()), ref_da, "grouped da")
    assert_grad_vec(to_f64(db.cpu()), ref_db, "grouped db")
    if G == 1:  # one group is the plain call
        assert torch.equal(y, B.forward(xd, ad, bd))
    with pytest.raises(B.WhtError) as err:
        B.wht_affine_fwd_grouped(xd, ad, bd, y, T, d, 48, dtype)
    assert err.value.status == -2
    B.wht_affine_set_variant(0)


def test_grouped_form_past_two_to_the_31_elements(B):
    # d = 768 = 3 blocks of 256, 2^31 / 768 + 7 rows: as in the plain test of that name, three blocks of rows are
    # non-zero, the rest must come out as b and as zero, and da, db follow from the non-zero rows alone
    d, block, dtype = 768, 256, wl.WHT_BF16_PF32
    G = d // block
    T = (1 << 31) // d + 7
    rows = [(0, 96), (T // 2 + 1, 96), (T - 77, 77)]
    zero_rows = [96, T // 3, T - 78]
    gen = lambda n, seed, which: torch.cat(
        [wl.gen_full(wl.Workload("grpbig", n, block, dtype, "normal", seed + g, True, ""), which) for g in range(G)],
        dim=1).contiguous()
    ab = [wl.gen_params(wl.Workload("grpbig", 1, block, dtype, "normal", 1500 + g, True, "")) for g in range(G)]
    a = torch.cat([p[0] for p in ab]).contiguous()
    b = torch.cat([p[1] for p in ab]).contiguous()
    x_d = torch.zeros(T, d, dtype=torch.bfloat16, device="cuda")
    dy_d = torch.zeros_like(x_d)
    xs, dys = [], []
    for i, (r0, n) in enumerate(rows):
        xs.append(gen(n, 1600 + 10 * i, "x"))
        dys.append(gen(n, 1600 + 10 * i, "dy"))
        x_d[r0:r0 + n].copy_(xs[-1])
        dy_d[r0:r0 + n].copy_(dys[-1])
    x_all, dy_all = torch.cat(xs), torch.cat(dys)
    ref_y = oracle.wht_affine_fwd_grouped(to_f64(x_all), to_f64(a), to_f64(b), block)
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd_grouped(to_f64(dy_all), to_f64(x_all), to_f64(a), block)
    ad, bd = a.cuda(), b.cuda()
    out = torch.empty_like(x_d)
    da = torch.empty(d, dtype=torch.float32, device="cuda")
    db = torch.empty_like(da)
    for variant in (0, 1):
        B.wht_affine_set_variant(variant)
        out.fill_(7.0)
        B.wht_affine_fwd_grouped(x_d, ad, bd, out, T, d, block, dtype)
        got = torch.cat([out[r0:r0 + n] for r0, n in rows]).cpu()
        assert_rows_bf16(to_f64(got), ref_y, f"grouped y past 2^31, v{variant}")
        for r in zero_rows:
            assert torch.equal(out[r], bd.bfloat16())
        ws = torch.empty(max(B.wht_affine_bwd_grouped_workspace_bytes(T, d, block, dtype), 16), dtype=torch.uint8,
                         device="cuda")
        out.fill_(7.0)
        B.wht_affine_bwd_grouped(dy_d, x_d, ad, out, da, db, T, d, block, dtype, ws)
        got = torch.cat([out[r0:r0 + n] for r0, n in rows]).cpu()
        assert_rows_bf16(to_f64(got), ref_dx, f"grouped dx past 2^31, v{variant}")
        for r in zero_rows:
            assert torch.count_nonzero(out[r]).item() == 0
        assert_grad_vec(to_f64(da.cpu()), ref_da, "grouped da past 2^31")
        assert_grad_vec(to_f64(db.cpu()), ref_db, "grouped db past 2^31")
    B.wht_affine_set_variant(0)


def test_autograd_wrapper(B):
    from paper_2603_08343_b200.autograd import wht_affine
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["training"].with_rows(6 * 50)
    x, dy, r = wl.gen_full(w, "x"), wl.gen_full(w, "dy"), wl.gen_full(w.with_rows(300), "x").flip(0)
    a, b = wl.gen_params(w)
    xd = x.cuda().view(6, 50, w.d).requires_grad_(True)        # [batch, seq, d]
    ad, bd = a.cuda().requires_grad_(True), b.cuda().requires_grad_(True)
    rd = r.cuda().view(6, 50, w.d).requires_grad_(True)
    out = wht_affine(xd, ad, bd, resid=rd)
    out.backward(dy.cuda().view(6, 50, w.d))
    torch.cuda.synchronize()
    ref_y = oracle.wht_affine_fwd_residual(to_f64(x), to_f64(a), to_f64(b), to_f64(r))
    ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), to_f64(a))
    assert_rows_bf16(to_f64(out.detach().cpu().view(-1, w.d)), ref_y, "autograd y")
    assert_rows_bf16(to_f64(xd.grad.cpu().view(-1, w.d)), ref_dx, "autograd dx")
    assert_grad_vec(to_f64(ad.grad.cpu()), ref_da, "autograd da")
    assert_grad_vec(to_f64(bd.grad.cpu()), ref_db, "autograd db")
    assert torch.equal(rd.grad.view(-1, w.d).cpu(), dy)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,T,dtype", [(2048, 301, wl.WHT_BF16_PF32), (8192, 37, wl.WHT_BF16_PF32),
                                       (256, 100, wl.WHT_BF16_PF32), (1024, 257, wl.WHT_F32),
                                       (2048, 148 * 32 + 3, wl.WHT_F32)])
def test_a_non_finite_row_stays_in_its_row(B, d, T, dtype, variant):
    """Rows are independent: Inf or NaN in one row of x (or dy) must leave every other row of y (dx)
    bit-identical -- tiles hold several rows side by side in shared and tensor memory -- while da, db,
    which sum over rows, follow the arithmetic (non-finite)."""
    B.wht_affine_set_variant(variant)
    w = wl.Workload("poison", T, d, dtype, "normal", 4242 + d, True, "")
    x, dy = wl.gen_full(w, "x").cuda(), wl.gen_full(w, "dy").cuda()
    a, b = (t.cuda() for t in wl.gen_params(w))
    y0 = B.forward(x, a, b)
    dx0, da0, db0 = B.backward(dy, x, a)
    bad_row, other = T // 2, [r for r in range(T) if r != T // 2]
    xp = x.clone()
    xp[bad_row, 7] = float("inf")
    xp[bad_row, d - 3] = float("nan")
    y1 = B.forward(xp, a, b)
    dx1, da1, db1 = B.backward(dy, xp, a)          # x enters da only
    dyp = dy.clone()
    dyp[bad_row, 1] = float("-inf")
    dx2, da2, db2 = B.backward(dyp, x, a)
    torch.cuda.synchronize()
    assert torch.equal(y1[other], y0[other]) and not torch.isfinite(y1[bad_row]).any()
    assert torch.equal(dx1, dx0) and torch.equal(db1, db0) and not torch.isfinite(da1).any()
    assert torch.equal(dx2[other], dx0[other]) and not torch.isfinite(dx2[bad_row]).any()
    assert not torch.isfinite(db2[1]) and torch.isfinite(db2[2:]).all()
    B.wht_affine_set_variant(0)


@pytest.mark.parametrize("d,dtype,T,decode", [(256, wl.WHT_F32, 64, False), (4096, wl.WHT_BF16, 8, True),
                                              (1024, wl.WHT_BF16, 257, False), (2048, wl.WHT_BF16_PF32, 148 * 8 + 3, False),
                                              (1024, wl.WHT_F32, 148 * 32 + 1, False)])
def test_calls_captured_in_a_cuda_graph(B, d, dtype, T, decode):
    # every compute call is asynchronous on its stream and, once its first call has sized the library's caches,
    # free of allocation and synchronisation: a graph of forward, fused residual forward and the three backward
    # entry points is captured once and replayed on NEW data in the same tensors; the replay must give the
    # oracle's values for the new data (Eq. 1 and its chain rule)
    B.wht_affine_set_variant(0)
    w0 = wl.Workload("graph", T, d, dtype, "normal", 4100 + d, True, "")
    w1 = wl.Workload("graph", T, d, dtype, "normal", 4200 + d, True, "")
    a, b = wl.gen_params(w0)
    ad, bd = a.cuda(), b.cuda()
    x, dy = wl.gen_full(w0, "x").cuda(), wl.gen_full(w0, "dy").cuda()
    y, yr = torch.empty_like(x), torch.empty_like(x)
    dxs = [torch.empty_like(x) for _ in range(3)]
    das = [torch.empty(d, dtype=torch.float32, device="cuda") for _ in range(3)]
    dbs = [torch.empty(d, dtype=torch.float32, device="cuda") for _ in range(3)]
    ws = torch.empty(max(B.wht_affine_bwd_workspace_bytes(T, d, dtype), 16), dtype=torch.uint8, device="cuda")

    def calls():
        (B.wht_affine_fwd_decode if decode else B.wht_affine_fwd)(x, ad, bd, y, T, d, dtype)
        B.wht_affine_fwd_residual(x, ad, bd, dy, yr, T, d, dtype)
        B.wht_affine_bwd(dy, x, ad, dxs[0], das[0], dbs[0], T, d, dtype)
        B.wht_affine_bwd_ws(dy, x, ad, dxs[1], das[1], dbs[1], T, d, dtype, ws)
        B.wht_affine_bwd_noalloc(dy, x, ad, dxs[2], das[2], dbs[2], T, d, dtype)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        calls()                                 # sizes the scratch, looks up the built-in array, fills the caches
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        calls()
    x1, dy1 = wl.gen_full(w1, "x"), wl.gen_full(w1, "dy")
    x.copy_(x1)
    dy.copy_(dy1)
    for t in [y, yr] + dxs + das + dbs:
        t.fill_(7.0)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    what = f"graph replay d={d} dtype={dtype} T={T}"
    _check_fwd(w1, y.cpu(), x1, a, b, what + " fwd")
    ref_r = oracle.wht_affine_fwd_residual(to_f64(x1), to_f64(a), to_f64(b), to_f64(dy1))
    if dtype == wl.WHT_F32:
        err = np.max(np.abs(to_f64(yr.cpu()) - ref_r), axis=1)
        assert np.all(err <= 1e-5 * (np.linalg.norm(to_f64(x1), axis=1) + np.max(np.abs(to_f64(dy1)), axis=1)))
    else:
        assert_rows_bf16(to_f64(yr.cpu()), ref_r, what + " residual")
    for k in range(3):
        _check_bwd(w1, dxs[k].cpu(), das[k].cpu(), dbs[k].cpu(), dy1, x1, a, what + f" bwd entry {k}")
    assert all(torch.equal(dxs[0], t) for t in dxs[1:]) and all(torch.equal(das[0], t) for t in das[1:])
    B.wht_affine_device_status()


def test_calls_on_two_streams_at_once(B):
    """A forward and a backward (caller-owned scratch) issued on two streams with no ordering between them
    give the bits of the serial calls: the kernels share SMs, tensor memory and the device-wide status word
    but no data."""
    B.wht_affine_set_variant(0)
    w = wl.CONFIGS["training"].with_rows(8192)
    x1, x2, dy2 = wl.gen_full(w, "x").cuda(), wl.gen_full(w, "dy").cuda(), wl.gen_full(w, "x").cuda().flip(0).contiguous()
    a, b = (t.cuda() for t in wl.gen_params(w))
    y_ref = B.forward(x1, a, b)
    dx_ref, da_ref, db_ref = B.backward(dy2, x2, a)
    ws = torch.empty(max(B.wht_affine_bwd_workspace_bytes(w.T, w.d, w.dtype), 16), dtype=torch.uint8, device="cuda")
    y, dx = torch.empty_like(x1), torch.empty_like(x2)
    da, db = torch.empty_like(da_ref), torch.empty_like(db_ref)
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(10):
        B.wht_affine_fwd(x1, a, b, y, w.T, w.d, w.dtype, stream=s1)
        B.wht_affine_bwd_ws(dy2, x2, a, dx, da, db, w.T, w.d, w.dtype, ws, stream=s2)
    torch.cuda.synchronize()
    assert torch.equal(y, y_ref) and torch.equal(dx, dx_ref)
    assert torch.equal(da, da_ref) and torch.equal(db, db_ref)


def test_layer_module(B):
    from paper_2603_08343_b200.autograd import WhtAffine
    B.wht_affine_set_variant(0)
    for d, block, T in ((1024, None, 130), (768, 256, 77)):
        layer = WhtAffine(d, block=block, device="cuda")
        assert sorted(n for n, _ in layer.named_parameters()) == ["a", "b"] and layer.a.numel() == d
        gen = torch.Generator().manual_seed(d)
        x = torch.randn(T, d, generator=gen).bfloat16()
        dy = torch.randn(T, d, generator=gen).bfloat16()
        with torch.no_grad():  # move the parameters off their initial 1 / 0 so that they matter
            layer.a.copy_(torch.rand(d, generator=gen) + 0.5)
            layer.b.copy_(torch.randn(d, generator=gen) * 0.1)
        xd = x.cuda().view(1, T, d).requires_grad_(True)
        out = layer(xd)
        out.backward(dy.cuda().view(1, T, d))
        torch.cuda.synchronize()
        a64, b64 = to_f64(layer.a.detach().cpu()), to_f64(layer.b.detach().cpu())
        if block is None:
            ref_y = oracle.wht_affine_fwd(to_f64(x), a64, b64)
            ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(to_f64(dy), to_f64(x), a64)
        else:
            ref_y = oracle.wht_affine_fwd_grouped(to_f64(x), a64, b64, block)
            ref_dx, ref_da, ref_db = oracle.wht_affine_bwd_grouped(to_f64(dy), to_f64(x), a64, block)
        assert_rows_bf16(to_f64(out.detach().cpu().view(T, d)), ref_y, "layer y")
        assert_rows_bf16(to_f64(xd.grad.cpu().view(T, d)), ref_dx, "layer dx")
        assert_grad_vec(to_f64(layer.a.grad.cpu()), ref_da, "layer da")
        assert_grad_vec(to_f64(layer.b.grad.cpu()), ref_db, "layer db")
    with pytest.raises(ValueError):
        WhtAffine(768)


def test_copy_rows(B):
    src = torch.arange(3 * 1024, dtype=torch.float32, device="cuda").view(3, 1024)
    dst = torch.zeros_like(src)
    B.wht_copy_rows(src, dst, 3, 1024, wl.WHT_F32)
    assert torch.equal(src, dst)
