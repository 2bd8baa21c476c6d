"""Mixed launches back to back, with no synchronisation in between, at seeded random shapes around and above the
sizes at which the automatic selection changes kernel family: forward, fused residual forward, backward and a small
forward right behind them, three times over.  Sampled rows are compared with the oracle (rows are independent, so a
sample of rows is checked at the oracle's full fidelity); every row is compared with the butterfly family's result
(itself checked against the oracle in test_parity_gpu.py) at the storage type's bound; the three repetitions must be
bit-identical; and no kernel's bounded wait may have expired."""
import random

import numpy as np
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
    yield binding
    binding.wht_affine_set_variant(0)
    binding.wht_affine_set_bwd_operand_mode(0)
    binding.wht_affine_device_status()


def _shapes(seed, count, fp32):
    rng = random.Random(seed)
    out = []
    for _ in range(count):
        logd = rng.choice([8, 9, 10, 10, 11, 11, 12, 13])
        d = 1 << logd
        tile = max(1, 16384 // d)
        T = rng.choice([rng.randint(1, 6000), rng.randint(148 * 32 - 40, 148 * 32 + 40),
                        rng.randint(148 * tile * 4, 148 * tile * 12) + rng.choice([0, 1, tile - 1, tile // 2 + 1])])
        T = min(T, (1 << 27) // d)
        dtype = wl.WHT_F32 if fp32 else rng.choice([wl.WHT_BF16, wl.WHT_BF16_PF32])
        out.append((d, T, dtype, rng.choice([0, 0, 0, 2, 3] if fp32 else [0, 0, 0, 3, 4, 5]), rng.choice([0, 1])))
    return out


@pytest.mark.parametrize("fp32", [False, True])
def test_mixed_back_to_back_launches(B, fp32):
    rng = np.random.default_rng(17)
    for case, (d, T, dtype, variant, mode) in enumerate(_shapes(5 + fp32, 60, fp32)):
        tdt = torch.float32 if dtype == wl.WHT_F32 else torch.bfloat16
        gen = torch.Generator(device="cuda").manual_seed(9000 + case)
        x = torch.randn(T, d, device="cuda", generator=gen).to(tdt)
        dy = torch.randn(T, d, device="cuda", generator=gen).to(tdt)
        a, b = (t.cuda() for t in wl.gen_params(wl.Workload("stress", 1, d, dtype, "normal", 9100 + case, True, "")))
        what = f"case {case}: d={d} T={T} dtype={dtype} variant={variant} mode={mode}"
        B.wht_affine_set_variant(1)
        y_ref = B.forward(x, a, b)
        dx_ref, da_ref, db_ref = B.backward(dy, x, a)
        B.wht_affine_set_variant(variant)
        B.wht_affine_set_bwd_operand_mode(mode)
        small = max(1, T // 7)
        outs = []
        for _ in range(3):  # no synchronisation anywhere in this loop
            y = B.forward(x, a, b)
            yr = B.forward(x, a, b, resid=dy)
            dx, da, db = B.backward(dy, x, a)
            outs.append((y, yr, dx, da, db, B.forward(x[:small], a, b)))
        torch.cuda.synchronize()
        B.wht_affine_set_bwd_operand_mode(0)
        assert all(torch.equal(outs[0][k], outs[r][k]) for k in range(6) for r in (1, 2)), what + ": not reproducible"
        y, yr, dx, da, db, ys = outs[0]
        # (the small call may run in another kernel family than the large one: same bound, not the same bits)
        tol = 2e-5 * x[:small].double().norm(dim=1) if dtype == wl.WHT_F32 else 2e-2 * y[:small].float().abs().amax(dim=1)
        assert bool(((ys.double() - y[:small].double()).abs().amax(dim=1) <= tol).all()), what + ": the small call"
        # every row against the butterfly family, at the storage type's bound
        if dtype == wl.WHT_F32:
            xn = x.double().norm(dim=1)
            gn = (a[None, :] * dy).double().norm(dim=1)
            assert bool(((y.double() - y_ref.double()).abs().amax(dim=1) <= 2e-5 * xn).all()), what + ": y"
            assert bool(((dx.double() - dx_ref.double()).abs().amax(dim=1) <= 2e-5 * gn).all()), what + ": dx"
        else:
            for got, ref, name in ((y, y_ref, "y"), (dx, dx_ref, "dx")):
                bound = 2e-2 * ref.float().abs().amax(dim=1)
                assert bool(((got.float() - ref.float()).abs().amax(dim=1) <= bound).all()), what + ": " + name
        assert float((da - da_ref).abs().max()) <= 2e-4 * float(da_ref.abs().max()) + 1e-6, what + ": da"
        assert float((db - db_ref).abs().max()) <= 2e-4 * float(db_ref.abs().max()) + 1e-6, what + ": db"
        # a sample of rows against the oracle (Eq. 1 and its chain rule, fp64)
        rows = np.unique(np.concatenate([[0, T - 1], rng.integers(0, T, 6)]))
        ridx = torch.from_numpy(rows).cuda()
        xs, dys = x[ridx].cpu(), dy[ridx].cpu()
        a64, b64 = to_f64(a.cpu()), to_f64(b.cpu())
        o_y = oracle.wht_affine_fwd(to_f64(xs), a64, b64)
        o_dx = oracle.wht_affine_bwd(to_f64(dys), to_f64(xs), a64)[0]
        o_yr = oracle.wht_affine_fwd_residual(to_f64(xs), a64, b64, to_f64(dys))
        if dtype == wl.WHT_F32:
            assert_rows_fp32(to_f64(y[ridx].cpu()), o_y, to_f64(xs), what + ": y vs oracle")
            assert_rows_fp32(to_f64(dx[ridx].cpu()), o_dx, a64[None, :] * to_f64(dys), what + ": dx vs oracle")
        else:
            assert_rows_bf16(to_f64(y[ridx].cpu()), o_y, what + ": y vs oracle")
            assert_rows_bf16(to_f64(dx[ridx].cpu()), o_dx, what + ": dx vs oracle")
            assert_rows_bf16(to_f64(yr[ridx].cpu()), o_yr, what + ": y + resid vs oracle")
        B.wht_affine_device_status()
        del x, dy, outs
