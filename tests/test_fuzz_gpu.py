"""Seeded random sweep of shapes, storage types and kernel families against the oracle.

Row counts are drawn both at random and right around multiples of the tcgen05 kernels' tile
height (one row short, exact, one over, half a tile), where ragged-tile handling lives.
"""
import random

import numpy as np
import pytest
import torch

import oracle
from helpers import to_f64
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


def _ratio_rows(got, ref, dtype, fp32_scale):
    err = np.max(np.abs(got - ref), axis=1)
    bound = 1e-5 * fp32_scale if dtype == wl.WHT_F32 else 1e-2 * np.max(np.abs(ref), axis=1)
    return float(np.max(err / np.maximum(bound, 1e-300)))


def _cases(seed, count):
    rng = random.Random(seed)
    out = []
    for case in range(count):
        logd = rng.choice([3, 5, 8, 9, 10, 10, 11, 11, 12, 12, 13, 13, 14])
        d = 1 << logd
        dtype = rng.choice([wl.WHT_F32, wl.WHT_BF16, wl.WHT_BF16_PF32, wl.WHT_BF16_PF32, wl.WHT_BF16])
        variant = rng.choice([0, 0, 1, 2, 3, 4, 5])
        max_rows = max(1, min(6000, (1 << 25) // (d * d // 64 + 1)))  # keeps the dense oracle to a fraction of a second
        if 10 <= logd <= 13 and rng.random() < 0.5:
            tile = 128 // (8 * (d // 1024))
            k = rng.randint(1, max(1, min(max_rows // tile, 148 * 3)))
            T = max(1, k * tile + rng.choice([-1, 0, 1, tile // 2]))
        else:
            T = rng.randint(1, max_rows)
        out.append((case, d, min(T, max_rows), dtype, variant, rng.choice(["normal", "student_t3"])))
    return out


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_match_the_oracle(B, seed):
    for case, d, T, dtype, variant, dist in _cases(seed, 24):
        w = wl.Workload("fuzz", T, d, dtype, dist, 5000 + 100 * seed + case, True, "")
        x, dy = wl.gen_full(w, "x"), wl.gen_full(w, "dy")
        a, b = wl.gen_params(w)
        B.wht_affine_set_variant(variant)
        xd, dyd, ad, bd = x.cuda(), dy.cuda(), a.cuda(), b.cuda()
        y = B.forward(xd, ad, bd)
        yr = B.forward(xd, ad, bd, resid=dyd)
        dx, da, db = B.backward(dyd, xd, ad)
        torch.cuda.synchronize()
        x64, dy64, a64, b64 = to_f64(x), to_f64(dy), to_f64(a), to_f64(b)
        ref_y = oracle.wht_affine_fwd(x64, a64, b64)
        ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(dy64, x64, a64)
        xn = np.linalg.norm(x64, axis=1)
        what = f"d={d} T={T} dtype={dtype} variant={variant} {dist}"
        assert _ratio_rows(to_f64(y.cpu()), ref_y, dtype, xn) <= 1.0, what + ": y"
        assert _ratio_rows(to_f64(yr.cpu()), ref_y + dy64, dtype, xn + np.max(np.abs(dy64), axis=1)) <= 1.0, \
            what + ": y with residual"
        assert _ratio_rows(to_f64(dx.cpu()), ref_dx, dtype, np.linalg.norm(a64[None, :] * dy64, axis=1)) <= 1.0, \
            what + ": dx"
        assert np.max(np.abs(to_f64(da.cpu()) - ref_da)) <= 1e-4 * np.max(np.abs(ref_da)), what + ": da"
        assert np.max(np.abs(to_f64(db.cpu()) - ref_db)) <= 1e-4 * np.max(np.abs(ref_db)), what + ": db"


def _tp_cases(seed, count):
    rng = random.Random(seed)
    out = []
    for case in range(count):
        g = rng.choice([2, 2, 4, 4, 8])
        logw = rng.choice([3, 6, 8, 9, 10, 10, 11, 11, 12])
        while g << logw > 16384:      # keeps the dense oracle at the full width small
            logw -= 1
        w = 1 << logw
        dtype = rng.choice([wl.WHT_F32, wl.WHT_BF16, wl.WHT_BF16_PF32, wl.WHT_BF16_PF32])
        variant = rng.choice([0, 1, 4, 4])
        d = g * w
        max_rows = max(1, min(3000, (1 << 25) // (d * d // 64 + 1)))
        if logw >= 10 and rng.random() < 0.5:
            tile = 128 // (8 * (w // 1024))
            T = max(1, rng.randint(1, max(1, max_rows // tile)) * tile + rng.choice([-1, 0, 1, tile // 2]))
        else:
            T = rng.randint(1, max_rows)
        out.append((case, g, w, min(T, max_rows), dtype, variant))
    return out


@pytest.mark.parametrize("seed", [21, 22])
def test_random_column_sharded_shapes_match_the_oracle(B, seed):
    from paper_2603_08343_b200 import tp
    for case, g, w, T, dtype, variant in _tp_cases(seed, 20):
        B.wht_affine_set_bwd_operand_mode(case & 1)  # both operand modes of the tcgen05 backward
        d = g * w
        wk = wl.Workload("fuzz-tp", T, d, dtype, "normal", 7000 + 100 * seed + case, True, "")
        x, dy = wl.gen_full(wk, "x"), wl.gen_full(wk, "dy")
        a, b = wl.gen_params(wk)
        B.wht_affine_set_variant(variant)
        xs = [p.cuda() for p in tp.split_columns(x, g)]
        dys = [p.cuda() for p in tp.split_columns(dy, g)]
        as_ = [a[s * w:(s + 1) * w].contiguous().cuda() for s in range(g)]
        outs = []
        for r in range(g):
            rank = tp.TpWht(g, r)
            y = rank.forward(xs, as_[r], b[r * w:(r + 1) * w].contiguous().cuda(), T, w)
            outs.append((y,) + rank.backward(dys, xs, as_, T, w))
        torch.cuda.synchronize()
        y = torch.cat([o[0] for o in outs], dim=1).cpu()
        dx = torch.cat([o[1] for o in outs], dim=1).cpu()
        da, db = torch.cat([o[2] for o in outs]).cpu(), torch.cat([o[3] for o in outs]).cpu()
        x64, dy64, a64, b64 = to_f64(x), to_f64(dy), to_f64(a), to_f64(b)
        ref_y = oracle.wht_affine_fwd(x64, a64, b64)
        ref_dx, ref_da, ref_db = oracle.wht_affine_bwd(dy64, x64, a64)
        what = f"g={g} w={w} T={T} dtype={dtype} variant={variant}"
        assert _ratio_rows(to_f64(y), ref_y, dtype, np.linalg.norm(x64, axis=1)) <= 1.0, what + ": y"
        assert _ratio_rows(to_f64(dx), ref_dx, dtype, np.linalg.norm(a64[None, :] * dy64, axis=1)) <= 1.0, what + ": dx"
        assert np.max(np.abs(to_f64(da) - ref_da)) <= 1e-4 * np.max(np.abs(ref_da)), what + ": da"
        assert np.max(np.abs(to_f64(db) - ref_db)) <= 1e-4 * np.max(np.abs(ref_db)), what + ": db"
    B.wht_affine_set_bwd_operand_mode(0)


def _grouped_cases(seed, count):
    rng = random.Random(seed)
    out = []
    for case in range(count):
        groups = rng.choice([2, 3, 3, 5, 6, 7])
        logb = rng.choice([3, 5, 7, 8, 8, 9, 9, 10, 11])
        block = 1 << logb
        dtype = rng.choice([wl.WHT_F32, wl.WHT_BF16, wl.WHT_BF16_PF32, wl.WHT_BF16_PF32])
        variant = rng.choice([0, 0, 1, 2, 3])
        d = groups * block
        max_rows = max(1, min(5000, (1 << 24) // (d * d // 64 + 1)))
        out.append((case, groups, block, rng.randint(1, max_rows), dtype, variant))
    return out


@pytest.mark.parametrize("seed", [31])
def test_random_block_diagonal_shapes_match_the_oracle(B, seed):
    """The grouped form (d = groups * block, every block transformed on its own) over random group counts,
    block widths, storage types and kernel families, against its plain block-diagonal definition."""
    for case, groups, block, T, dtype, variant in _grouped_cases(seed, 24):
        d = groups * block
        gen = torch.Generator().manual_seed(9000 + 100 * seed + case)
        io = torch.float32 if dtype == wl.WHT_F32 else torch.bfloat16
        pt = torch.bfloat16 if dtype == wl.WHT_BF16 else torch.float32
        x = torch.randn(T, d, generator=gen).to(io)
        dy = torch.randn(T, d, generator=gen).to(io)
        a = (torch.rand(d, generator=gen) + 0.5).to(pt)
        b = (torch.randn(d, generator=gen) * 0.1).to(pt)
        B.wht_affine_set_variant(variant)
        xd, dyd, ad, bd = x.cuda(), dy.cuda(), a.cuda(), b.cuda()
        y = torch.empty_like(xd)
        B.wht_affine_fwd_grouped(xd, ad, bd, y, T, d, block, dtype)
        ws = torch.empty(max(B.wht_affine_bwd_grouped_workspace_bytes(T, d, block, dtype), 16), dtype=torch.uint8, device="cuda")
        dx = torch.empty_like(xd)
        da, db = torch.empty(d, device="cuda"), torch.empty(d, device="cuda")
        B.wht_affine_bwd_grouped(dyd, xd, ad, dx, da, db, T, d, block, dtype, ws)
        torch.cuda.synchronize()
        x64, dy64, a64, b64 = to_f64(x), to_f64(dy), to_f64(a), to_f64(b)
        ref_y = oracle.wht_affine_fwd_grouped(x64, a64, b64, block)
        ref_dx, ref_da, ref_db = oracle.wht_affine_bwd_grouped(dy64, x64, a64, block)
        what = f"groups={groups} block={block} T={T} dtype={dtype} variant={variant}"
        # the fp32 bound is per transform input: here the norm of the row's block, the smallest over the blocks
        blocks_x = np.linalg.norm(x64.reshape(T, groups, block), axis=2).min(axis=1)
        blocks_g = np.linalg.norm((a64[None, :] * dy64).reshape(T, groups, block), axis=2).min(axis=1)
        if dtype == wl.WHT_F32:
            # per block the error is bounded by 1e-5 of ITS norm; the largest block norm bounds the row's maximum
            nx = np.linalg.norm(x64.reshape(T, groups, block), axis=2).max(axis=1)
            ng = np.linalg.norm((a64[None, :] * dy64).reshape(T, groups, block), axis=2).max(axis=1)
            assert _ratio_rows(to_f64(y.cpu()), ref_y, dtype, nx) <= 1.0, what + ": y"
            assert _ratio_rows(to_f64(dx.cpu()), ref_dx, dtype, ng) <= 1.0, what + ": dx"
        else:
            assert _ratio_rows(to_f64(y.cpu()), ref_y, dtype, blocks_x) <= 1.0, what + ": y"
            assert _ratio_rows(to_f64(dx.cpu()), ref_dx, dtype, blocks_g) <= 1.0, what + ": dx"
        assert np.max(np.abs(to_f64(da.cpu()) - ref_da)) <= 1e-4 * np.max(np.abs(ref_da)), what + ": da"
        assert np.max(np.abs(to_f64(db.cpu()) - ref_db)) <= 1e-4 * np.max(np.abs(ref_db)), what + ": db"
    B.wht_affine_set_variant(0)
