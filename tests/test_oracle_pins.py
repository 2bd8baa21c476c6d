"""Pins for the CPU oracle: what the paper prints and what the mathematics fixes.

Each test is chosen so that one plausible mistake in oracle/wht_oracle.py (another
ordering of the transform, a missing or doubled 1/sqrt(d), a dropped bias, x used
where z belongs in da, a wrong sign in a butterfly) makes it fail.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.linalg

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- ordering

def test_h4_matches_printed_sign_pattern():
    # Fig. 1 prints H_4; sequency (Walsh) or dyadic (Paley) order would permute rows 1..3.
    rows = _golden_lines("h4_sign_pattern.txt")
    printed = np.array([[1.0 if c == "+" else -1.0 for c in r] for r in rows])
    assert printed.shape == (4, 4)
    np.testing.assert_array_equal(oracle.sylvester_hadamard(4), printed)


@pytest.mark.parametrize("d", [1, 2, 4, 8, 16, 64, 256, 1024])
def test_matches_kronecker_recursion_and_scipy(d):
    # Sylvester's construction H_2n = [[H, H], [H, -H]] is a second, independent
    # definition; scipy.linalg.hadamard implements it as a library routine.
    H = oracle.sylvester_hadamard(d)
    K = np.array([[1.0]])
    while K.shape[0] < d:
        K = np.block([[K, K], [K, -K]])
    np.testing.assert_array_equal(H, K)
    np.testing.assert_array_equal(H, scipy.linalg.hadamard(d).astype(np.float64))


@pytest.mark.parametrize("d", [2, 8, 64, 512, 1024])
def test_h_ht_is_d_identity_in_integers(d):
    # Eq. 1's condition H^T H = I for the normalised matrix <=> H H^T = d I unnormalised.
    H = oracle.sylvester_hadamard(d).astype(np.int64)
    np.testing.assert_array_equal(H @ H.T, d * np.eye(d, dtype=np.int64))
    np.testing.assert_array_equal(H, H.T)


def test_d_must_be_power_of_two():
    for bad in (0, 3, 12, 768):
        with pytest.raises(ValueError):
            oracle.sylvester_hadamard(bad)


# ---------------------------------------------------------------- normalisation

@pytest.mark.parametrize("d", [2, 16, 256, 2048])
def test_norm_preserved_and_involution(d):
    rng = np.random.default_rng(d)
    x = rng.standard_normal((5, d))
    z = oracle.wht_normalised(x)
    np.testing.assert_allclose(np.linalg.norm(z, axis=1), np.linalg.norm(x, axis=1), rtol=1e-13)
    # the normalised transform is its own inverse: H(Hx) = d x
    np.testing.assert_allclose(oracle.wht_normalised(z), x, rtol=0, atol=1e-12)
    ones = np.ones(d)
    zero = np.zeros(d)
    np.testing.assert_allclose(oracle.wht_affine_fwd(z, ones, zero), x, rtol=0, atol=1e-12)


@pytest.mark.parametrize("d", [4, 32, 1024])
def test_constant_and_impulse_rows(d):
    rng = np.random.default_rng(7 + d)
    a = rng.uniform(0.5, 1.5, d)
    b = rng.normal(0, 0.1, d)
    # H . 1 = d e_0  =>  y = a_0 sqrt(d) e_0 + b
    y = oracle.wht_affine_fwd(np.ones((1, d)), a, b)[0]
    expect = b.copy()
    expect[0] += a[0] * math.sqrt(d)
    np.testing.assert_allclose(y, expect, rtol=0, atol=1e-12)
    # x = e_k  =>  y = a (.) (row k of H)/sqrt(d) + b, signs from popcount parity
    for k in (0, 1, d // 2, d - 1):
        e = np.zeros((1, d))
        e[0, k] = 1.0
        signs = np.array([(-1.0) ** bin(k & j).count("1") for j in range(d)])
        np.testing.assert_allclose(oracle.wht_affine_fwd(e, a, b)[0],
                                   a * signs / math.sqrt(d) + b, rtol=0, atol=1e-14)
    # x = 0  =>  y = b
    np.testing.assert_array_equal(oracle.wht_affine_fwd(np.zeros((2, d)), a, b),
                                  np.broadcast_to(b, (2, d)))


# ---------------------------------------------------------------- brute force

@pytest.mark.parametrize("d", [2, 4, 8, 16])
def test_brute_force_small(d):
    # pure-Python triple loop from the recursive sign rule, exact rationals for the sum
    def sign(i, j, n):
        # entry (i, j) of H_n via the quadrant rule of Sylvester's construction
        s = 1
        while n > 1:
            n //= 2
            if i >= n and j >= n:
                s = -s
            i %= n
            j %= n
        return s

    rng = np.random.default_rng(100 + d)
    x = rng.integers(-4, 5, size=(3, d)).astype(np.float64)
    a = rng.integers(1, 4, size=d).astype(np.float64)
    b = rng.integers(-2, 3, size=d).astype(np.float64)
    y = oracle.wht_affine_fwd(x, a, b)
    for t, j in itertools.product(range(3), range(d)):
        acc = 0
        for i in range(d):
            acc += int(x[t, i]) * sign(i, j, d)
        assert y[t, j] == pytest.approx(a[j] * acc / math.sqrt(d) + b[j], abs=1e-13)


@pytest.mark.parametrize("d", [2, 8, 16])
def test_residual_form_brute_force_and_special_cases(d):
    # out = resid + a (.) z + b: pure-Python sum from the popcount sign rule, then the cases that
    # reduce to something known (x = 0 -> resid + b exactly; resid = 0 -> the plain forward).
    rng = np.random.default_rng(300 + d)
    x = rng.integers(-3, 4, size=(2, d)).astype(np.float64)
    r = rng.integers(-5, 6, size=(2, d)).astype(np.float64)
    a = rng.integers(1, 4, size=d).astype(np.float64)
    b = rng.integers(-2, 3, size=d).astype(np.float64)
    out = oracle.wht_affine_fwd_residual(x, a, b, r)
    for t, j in itertools.product(range(2), range(d)):
        acc = sum(int(x[t, i]) * (-1) ** bin(i & j).count("1") for i in range(d))
        assert out[t, j] == pytest.approx(r[t, j] + a[j] * acc / math.sqrt(d) + b[j], abs=1e-13)
    np.testing.assert_array_equal(oracle.wht_affine_fwd_residual(np.zeros((2, d)), a, b, r), r + b)
    np.testing.assert_array_equal(oracle.wht_affine_fwd_residual(x, a, b, np.zeros((2, d))),
                                  oracle.wht_affine_fwd(x, a, b))
    # a dropped or doubled residual term is caught by the first loop; a sign error too
    assert not np.allclose(oracle.wht_affine_fwd(x, a, b) - r, out)


# ---------------------------------------------------------------- grouped (block-diagonal) form

@pytest.mark.parametrize("d,block", [(24, 8), (768, 256), (48, 16), (64, 64)])
def test_grouped_form(d, block):
    rng = np.random.default_rng(d + block)
    T, G = 4, d // block
    x = rng.standard_normal((T, d))
    dy = rng.standard_normal((T, d))
    a = rng.uniform(0.5, 1.5, d)
    b = rng.normal(0, 0.1, d)
    y = oracle.wht_affine_fwd_grouped(x, a, b, block)
    # each group is the plain transform of its own slice (and of nothing else)
    for g in range(G):
        sl = slice(g * block, (g + 1) * block)
        np.testing.assert_allclose(y[:, sl], oracle.wht_affine_fwd(x[:, sl], a[sl], b[sl]), rtol=0, atol=1e-12)
    # orthonormal: norms preserved, and the matrix squares to block * I in integers
    M = oracle.grouped_hadamard(d, block).astype(np.int64)
    np.testing.assert_array_equal(M @ M.T, block * np.eye(d, dtype=np.int64))
    z = oracle.wht_affine_fwd_grouped(x, np.ones(d), np.zeros(d), block)
    np.testing.assert_allclose(np.linalg.norm(z, axis=1), np.linalg.norm(x, axis=1), rtol=1e-13)
    # gradients: adjoint identity and finite differences on a few entries
    dx, da, db = oracle.wht_affine_bwd_grouped(dy, x, a, block)
    assert np.sum(dy * (y - b)) == pytest.approx(np.sum(dx * x), rel=1e-12)
    h = 1e-3
    for j in (0, block - 1, d - 1):
        ap, am = a.copy(), a.copy()
        ap[j] += h
        am[j] -= h
        fd = (np.sum(dy * oracle.wht_affine_fwd_grouped(x, ap, b, block)) -
              np.sum(dy * oracle.wht_affine_fwd_grouped(x, am, b, block))) / (2 * h)
        assert fd == pytest.approx(da[j], rel=1e-8, abs=1e-8)
    np.testing.assert_allclose(db, dy.sum(axis=0), rtol=0, atol=1e-13)
    if G == 1:
        np.testing.assert_array_equal(y, oracle.wht_affine_fwd(x, a, b))
    with pytest.raises(ValueError):
        oracle.grouped_hadamard(d + 1, block)


# ---------------------------------------------------------------- Fig. 2 butterfly

def test_butterfly_pairs_of_figure():
    # the stage wiring printed in Fig. 2 for d = 8 is what fwht_butterfly walks
    for line in _golden_lines("butterfly_pairs_d8.txt"):
        parts = line.split()
        stride = int(parts[0])
        pairs = {tuple(int(p) - 1 for p in s.split("-")) for s in parts[1:]}
        walked = {(i, i + stride) for i in range(8) if not i & stride}
        assert pairs == walked


@pytest.mark.parametrize("d", [2, 8, 64, 256, 1024, 4096])
def test_butterfly_equals_matrix_and_op_count(d):
    rng = np.random.default_rng(d + 1)
    v = rng.standard_normal(d)
    got, ops = oracle.fwht_butterfly(v)
    want = v @ oracle.sylvester_hadamard(d)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-9 * math.sqrt(d))
    assert ops == d * int(math.log2(d))


def test_butterfly_op_counts_match_figure():
    for line in _golden_lines("fwht_op_counts.txt"):
        d, count = (int(s) for s in line.split())
        _, ops = oracle.fwht_butterfly(np.zeros(d))
        assert ops == count


# ---------------------------------------------------------------- gradients

def _loss(x, a, b, dy):
    return float(np.sum(dy * oracle.wht_affine_fwd(x, a, b)))


@pytest.mark.parametrize("T,d", [(3, 8), (5, 64), (4, 256)])
def test_gradients_by_central_differences(T, d):
    rng = np.random.default_rng(T * 1000 + d)
    x = rng.standard_normal((T, d))
    dy = rng.standard_normal((T, d))
    a = rng.uniform(0.5, 1.5, d)
    b = rng.normal(0, 0.1, d)
    dx, da, db = oracle.wht_affine_bwd(dy, x, a)
    h = 1e-3  # the loss is linear in each of x, a, b alone, so the difference is exact up to rounding
    cols = sorted(set([0, 1, d // 2, d - 1]) | set(rng.integers(0, d, 4).tolist()))
    for j in cols:
        ap, am = a.copy(), a.copy()
        ap[j] += h
        am[j] -= h
        assert (_loss(x, ap, b, dy) - _loss(x, am, b, dy)) / (2 * h) == pytest.approx(da[j], rel=1e-8, abs=1e-8)
        bp, bm = b.copy(), b.copy()
        bp[j] += h
        bm[j] -= h
        assert (_loss(x, a, bp, dy) - _loss(x, a, bm, dy)) / (2 * h) == pytest.approx(db[j], rel=1e-8, abs=1e-8)
    for t, i in [(0, 0), (T - 1, d - 1), (1, d // 2), (T // 2, 1)]:
        xp, xm = x.copy(), x.copy()
        xp[t, i] += h
        xm[t, i] -= h
        assert (_loss(xp, a, b, dy) - _loss(xm, a, b, dy)) / (2 * h) == pytest.approx(dx[t, i], rel=1e-8, abs=1e-8)


@pytest.mark.parametrize("d", [16, 512])
def test_adjoint_identity_and_db_column_sums(d):
    rng = np.random.default_rng(d * 3)
    T = 6
    x = rng.standard_normal((T, d))
    dy = rng.standard_normal((T, d))
    a = rng.uniform(0.5, 1.5, d)
    b = rng.normal(0, 0.1, d)
    dx, da, db = oracle.wht_affine_bwd(dy, x, a)
    y = oracle.wht_affine_fwd(x, a, b)
    # <dy, y - b> = <dx, x>  (the map x -> y - b is linear with adjoint dy -> dx)
    assert np.sum(dy * (y - b)) == pytest.approx(np.sum(dx * x), rel=1e-12)
    # <dy, y - b> = <da, a> as well, since y - b = a (.) z
    assert np.sum(dy * (y - b)) == pytest.approx(np.sum(da * a), rel=1e-12)
    col = np.zeros(d)
    for t in range(T):
        col += dy[t]
    np.testing.assert_allclose(db, col, rtol=0, atol=1e-13)


def test_da_db_columns_agrees_with_full():
    rng = np.random.default_rng(11)
    T, d = 37, 128
    x = rng.standard_normal((T, d)).astype(np.float32)
    dy = rng.standard_normal((T, d)).astype(np.float32)
    a = rng.uniform(0.5, 1.5, d)
    _, da, db = oracle.wht_affine_bwd(dy, x, a)
    cols = np.array([0, 5, 64, 127])
    da_c, db_c = oracle.da_db_columns(dy, x, cols)
    np.testing.assert_allclose(da_c, da[cols], rtol=1e-12)
    np.testing.assert_allclose(db_c, db[cols], rtol=1e-12, atol=1e-13)


def test_da_db_columns_over_several_row_blocks():
    """The column form walks the rows in blocks of 4096: with T = 9001 it takes three trips, the last
    one ragged.  Pinned against the full definition (chain rule on Eq. 1; itself pinned by finite
    differences above) on ALL columns and on a sample, and against a plain per-row loop written from
    the definition da[j] = sum_t dy[t, j] * (sum_i x[t, i] H[i][j]) / sqrt(d).  A block read without its
    row offset, a dropped last block or a block counted twice fails it."""
    rng = np.random.default_rng(2603)
    T, d = 9001, 64
    x = rng.standard_normal((T, d)).astype(np.float32)
    dy = rng.standard_normal((T, d)).astype(np.float32)
    # rows differ in scale from block to block, so that a block taken for another cannot cancel out
    x *= (1.0 + np.arange(T) // 4096)[:, None].astype(np.float32)
    _, da, db = oracle.wht_affine_bwd(dy, x, np.ones(d))
    every = np.arange(d)
    da_c, db_c = oracle.da_db_columns(dy, x, every)
    np.testing.assert_allclose(da_c, da, rtol=1e-11, atol=1e-9)
    np.testing.assert_allclose(db_c, db, rtol=1e-11, atol=1e-9)
    some = np.array([0, 1, 31, 32, 63])
    da_s, db_s = oracle.da_db_columns(dy, x, some)
    np.testing.assert_allclose(da_s, da[some], rtol=1e-11, atol=1e-9)
    np.testing.assert_allclose(db_s, db[some], rtol=1e-11, atol=1e-9)
    # the definition as a loop over rows, for two columns
    H = oracle.sylvester_hadamard(d)
    for j in (1, 63):
        acc_a = acc_b = 0.0
        for t in range(T):
            acc_a += float(dy[t, j]) * float(np.dot(x[t].astype(np.float64), H[:, j])) / math.sqrt(d)
            acc_b += float(dy[t, j])
        assert da_c[j] == pytest.approx(acc_a, rel=1e-10, abs=1e-9)
        assert db_c[j] == pytest.approx(acc_b, rel=1e-10, abs=1e-9)
    # what the pin would catch: the sums over the first two blocks only, or with the first block twice
    da_short, _ = oracle.da_db_columns(dy[:8192], x[:8192], every)
    da_twice = da_short + oracle.da_db_columns(dy[:4096], x[:4096], every)[0] \
        - oracle.da_db_columns(dy[4096:8192], x[4096:8192], every)[0]
    assert np.max(np.abs(da_short - da)) > 1e-3 * np.max(np.abs(da))
    assert np.max(np.abs(da_twice - da)) > 1e-3 * np.max(np.abs(da))


def test_da_db_columns_adds_over_row_blocks_like_the_parity_tests_use_it():
    """The full-size parity tests call the column form on 8192-row slices and add the results; the sum
    over slices must be the value over all rows (da and db are sums over rows)."""
    rng = np.random.default_rng(8343)
    T, d = 20000, 32
    x = rng.standard_normal((T, d))
    dy = rng.standard_normal((T, d))
    cols = np.array([0, 7, 16, 31])
    whole_a, whole_b = oracle.da_db_columns(dy, x, cols)
    parts_a, parts_b = np.zeros(cols.size), np.zeros(cols.size)
    for r0 in range(0, T, 8192):
        pa, pb = oracle.da_db_columns(dy[r0:r0 + 8192], x[r0:r0 + 8192], cols)
        parts_a += pa
        parts_b += pb
    np.testing.assert_allclose(parts_a, whole_a, rtol=1e-11, atol=1e-9)
    np.testing.assert_allclose(parts_b, whole_b, rtol=1e-11, atol=1e-9)
    _, da, db = oracle.wht_affine_bwd(dy, x, np.ones(d))
    np.testing.assert_allclose(whole_a, da[cols], rtol=1e-11, atol=1e-9)
    np.testing.assert_allclose(whole_b, db[cols], rtol=1e-11, atol=1e-9)


def test_widen_bf16_bits_exact():
    # 0x3F80 = 1.0, 0xC000 = -2.0, 0x3DCD ~ 0.100098 (bf16 nearest to 0.1), 0x0000 = 0
    bits = np.array([0x3F80, 0xC000, 0x3DCD, 0x0000, 0x7F7F], dtype=np.uint16)
    got = oracle.widen_bf16_bits(bits)
    want = np.array([1.0, -2.0, 0.10009765625, 0.0, 3.3895313892515355e38])
    np.testing.assert_array_equal(got, want)


# ---------------------------------------------------------------- planted mistakes are caught

def test_pins_catch_planted_mistakes(monkeypatch):
    # A wrong ordering (sequency order) still satisfies H H^T = d I, so the printed
    # pattern is what must catch it; check that it would.
    H = oracle.sylvester_hadamard(4)
    sequency = H[[0, 2, 3, 1]]
    rows = _golden_lines("h4_sign_pattern.txt")
    printed = np.array([[1.0 if c == "+" else -1.0 for c in r] for r in rows])
    assert not np.array_equal(sequency, printed)
    # da computed from x instead of z fails the finite-difference pin
    rng = np.random.default_rng(5)
    x = rng.standard_normal((3, 8))
    dy = rng.standard_normal((3, 8))
    a = rng.uniform(0.5, 1.5, 8)
    b = np.zeros(8)
    wrong_da = np.sum(dy * x, axis=0)
    h = 1e-3
    ap, am = a.copy(), a.copy()
    ap[3] += h
    am[3] -= h
    fd = (_loss(x, ap, b, dy) - _loss(x, am, b, dy)) / (2 * h)
    assert abs(fd - wrong_da[3]) > 1e-3
