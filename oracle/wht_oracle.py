"""Plain fp64 definition of the Hadamard head-mixing operation and its gradients.

TEST INFRASTRUCTURE.  This file is the parity authority for the CUDA library; it
shares no code with it and must never be imported by the product package.  It is
deliberately slow and literal: the method reaches exactly (up to rounding order)
the result of a dense product with the explicitly constructed matrix, so the
oracle is that dense product written out.  numpy's matmul is the only library
primitive used as a step.

What the paper fixes, and where:
  * Eq. 1:   MHA_Had(X) = alpha (.) (Y H) + beta, with H the normalised
             Walsh-Hadamard matrix, H^T H = I  (hence the 1/sqrt(d) scale).
  * Fig. 1:  the printed 4x4 sign pattern  ++++ / +-+- / ++-- / +--+  fixes the
             ordering as Sylvester ("natural"): H[i][j] = (-1)^popcount(i & j).
  * Fig. 2:  the in-place butterfly, stages with stride 1, 2, 4, ..., each pair
             (i, i+stride) replaced by (sum, difference); no reordering.
  * Table "dense vs Hadamard": the backward pass costs O(d log d); its formulas
             are not printed, they follow from Eq. 1 by the chain rule:
               dx = ((a (.) dy) H^T) / sqrt(d),   da = sum_t dy (.) z,   db = sum_t dy,
             where z = (x H)/sqrt(d).

Pins (tests/test_oracle_pins.py): the printed H_4, scipy's Sylvester matrix,
the Kronecker recursion, H H^T = d I in integers, norm preservation, involution,
impulse and constant rows, brute force at d <= 16 (also with a residual row added),
the Fig. 2 butterfly with its
d*log2(d) operation count, central finite differences and the adjoint identity
for the gradients; the column form of da, db over several of its row blocks (ragged
last block) against the full definition and a per-row loop.  No function here is
"parity unpinned".
"""
from __future__ import annotations

import functools
import math

import numpy as np


def _log2_exact(d: int) -> int:
    if d < 1 or (d & (d - 1)) != 0:
        raise ValueError(f"d must be a power of two, got {d}")
    return d.bit_length() - 1


@functools.lru_cache(maxsize=3)
def sylvester_hadamard(d: int) -> np.ndarray:
    """Unnormalised d x d matrix of +-1 in Sylvester order (Fig. 1 sign pattern).

    H[i][j] = +1 when popcount(i & j) is even, -1 when it is odd.  The matrix is
    a constant of d, so the last few sizes are kept (read-only) between calls.
    """
    _log2_exact(d)
    idx = np.arange(d, dtype=np.int32)
    both = idx[:, None] & idx[None, :]
    parity = np.zeros((d, d), dtype=np.int8)
    bit = 1
    while bit < d:
        parity ^= ((both & bit) != 0).astype(np.int8)
        bit <<= 1
    H = (1 - 2 * parity).astype(np.float64)
    H.setflags(write=False)
    return H


def widen_bf16_bits(bits: np.ndarray) -> np.ndarray:
    """Exact bfloat16 -> float64 widening of raw 16-bit patterns (stored inputs).

    A bfloat16 is the upper half of an IEEE binary32, so the value is obtained
    by placing the pattern in the high 16 bits of a 32-bit word.
    """
    u = np.ascontiguousarray(bits).astype(np.uint16, copy=False)
    as_f32 = (u.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return as_f32.astype(np.float64)


def wht_normalised(x: np.ndarray) -> np.ndarray:
    """z = (x H) / sqrt(d) for every row of x[T, d]  (Eq. 1, the factor Y H)."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    H = sylvester_hadamard(d)
    return (x @ H) / math.sqrt(float(d))


def wht_affine_fwd(x: np.ndarray, a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """y[t, j] = a[j] * z[t, j] + b[j],  z = (x H)/sqrt(d)   (Eq. 1)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    z = wht_normalised(x)
    return a[None, :] * z + b[None, :]


def wht_affine_fwd_residual(x: np.ndarray, a: np.ndarray, b: np.ndarray, resid: np.ndarray) -> np.ndarray:
    """out[t, j] = resid[t, j] + a[j] * z[t, j] + b[j]: Eq. 1 followed by the residual
    connection of the attention block that the projection's output feeds (Sec. 3)."""
    return np.asarray(resid, dtype=np.float64) + wht_affine_fwd(x, a, b)


def wht_affine_bwd(dy: np.ndarray, x: np.ndarray, a: np.ndarray):
    """Gradients of L = sum(dy (.) y) with y from Eq. 1.

    dx[t, i] = (sum_j a[j] dy[t, j] H[j][i]) / sqrt(d)
    da[j]    = sum_t dy[t, j] z[t, j]
    db[j]    = sum_t dy[t, j]
    Returns (dx, da, db), all float64.
    """
    dy = np.asarray(dy, dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    a = np.asarray(a, dtype=np.float64)
    d = x.shape[-1]
    H = sylvester_hadamard(d)
    root = math.sqrt(float(d))
    z = (x @ H) / root
    g = a[None, :] * dy
    dx = (g @ H.T) / root
    da = np.sum(dy * z, axis=0)
    db = np.sum(dy, axis=0)
    return dx, da, db


def grouped_hadamard(d: int, block: int) -> np.ndarray:
    """Unnormalised block-diagonal matrix diag(H_block, ..., H_block) of order d = groups * block."""
    _log2_exact(block)
    if d < block or d % block:
        raise ValueError(f"d={d} is not a multiple of block={block}")
    return np.kron(np.eye(d // block), sylvester_hadamard(block))


def wht_affine_fwd_grouped(x: np.ndarray, a: np.ndarray, b: np.ndarray, block: int) -> np.ndarray:
    """Eq. 1 with H replaced by diag(H_block, ...)/sqrt(block): a reading offered for widths that are
    not a power of two (the paper's d = 768, 1536), about which the paper itself is silent."""
    x = np.asarray(x, dtype=np.float64)
    G = grouped_hadamard(x.shape[-1], block)
    z = (x @ G) / math.sqrt(float(block))
    return np.asarray(a, dtype=np.float64)[None, :] * z + np.asarray(b, dtype=np.float64)[None, :]


def wht_affine_bwd_grouped(dy: np.ndarray, x: np.ndarray, a: np.ndarray, block: int):
    """Gradients of the grouped form (chain rule, G symmetric): (dx, da, db)."""
    dy = np.asarray(dy, dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    a = np.asarray(a, dtype=np.float64)
    G = grouped_hadamard(x.shape[-1], block)
    root = math.sqrt(float(block))
    z = (x @ G) / root
    dx = ((a[None, :] * dy) @ G.T) / root
    return dx, np.sum(dy * z, axis=0), np.sum(dy, axis=0)


def da_db_columns(dy: np.ndarray, x: np.ndarray, cols: np.ndarray):
    """da[j], db[j] for the listed columns j only, over ALL rows.

    z[t, j] = (sum_i x[t, i] H[i][j]) / sqrt(d) needs only column j of H, so a
    sample of columns can be checked at sizes where the full product is too
    slow.  Returns (da[cols], db[cols]).
    """
    dy = np.asarray(dy)
    x = np.asarray(x)
    cols = np.asarray(cols, dtype=np.int64)
    d = x.shape[-1]
    Hc = sylvester_hadamard(d)[:, cols]
    root = math.sqrt(float(d))
    da = np.zeros(cols.shape[0], dtype=np.float64)
    db = np.zeros(cols.shape[0], dtype=np.float64)
    step = 4096
    for r0 in range(0, x.shape[0], step):
        xb = x[r0:r0 + step].astype(np.float64)
        dyb = dy[r0:r0 + step][:, cols].astype(np.float64)
        zc = (xb @ Hc) / root
        da += np.sum(dyb * zc, axis=0)
        db += np.sum(dyb, axis=0)
    return da, db


def fwht_butterfly(v: np.ndarray):
    """Unnormalised transform of one vector by the butterfly network of Fig. 2.

    Stage s = 1, 2, ... uses stride 2^(s-1); every pair (i, i + stride) with
    bit `stride` of i clear becomes (v[i] + v[i+stride], v[i] - v[i+stride]).
    Returns (H v, number of additions and subtractions performed).  Kept only
    as a cross-check of the figure against the matrix definition; the oracle
    proper never calls it.
    """
    out = np.array(v, dtype=np.float64, copy=True)
    d = out.shape[0]
    _log2_exact(d)
    ops = 0
    stride = 1
    while stride < d:
        for i in range(d):
            if i & stride:
                continue
            lo = out[i]
            hi = out[i + stride]
            out[i] = lo + hi
            out[i + stride] = lo - hi
            ops += 2
        stride *= 2
    return out, ops
