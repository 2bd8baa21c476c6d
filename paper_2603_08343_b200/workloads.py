"""Seeded synthetic inputs shaped like the paper's prefill, decode and training runs.

This module holds NO arithmetic of the method: it only draws random tensors.
It is the one module that both the CPU oracle's tests and the CUDA path's tests
use, so that both sides see identical bits.

Every tensor is drawn on the CPU in blocks of ROWS_PER_BLOCK rows; block k of
tensor `which` of a workload uses its own torch.Generator seeded from
(seed, which, k).  Any row range can therefore be regenerated without drawing
the rest, which is how the full-size parity tests sample rows.

Draw recipe (values are drawn in fp32, then rounded once, round-to-nearest-even,
to the storage type):
  x, dy : N(0, 1), or 0.5 * Student-t(nu=3) built as n0 / sqrt((n1^2+n2^2+n3^2)/3)
  a     : U(0.5, 1.5)
  b     : N(0, sigma = 0.1)
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import torch

# dtype codes of the C ABI (include/wht_affine.h)
WHT_F32 = 0
WHT_BF16 = 1
WHT_BF16_PF32 = 2

ROWS_PER_BLOCK = 1024
_TENSOR_ID = {"x": 1, "dy": 2, "a": 3, "b": 4}


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    d: int
    dtype: int          # WHT_F32 / WHT_BF16 / WHT_BF16_PF32
    dist: str           # "normal" or "student_t3"
    seed: int
    has_bwd: bool
    note: str

    @property
    def io_torch_dtype(self):
        return torch.float32 if self.dtype == WHT_F32 else torch.bfloat16

    @property
    def param_torch_dtype(self):
        return torch.bfloat16 if self.dtype == WHT_BF16 else torch.float32

    @property
    def io_bytes(self) -> int:
        return 4 if self.dtype == WHT_F32 else 2

    def with_rows(self, T: int) -> "Workload":
        return Workload(self.name, T, self.d, self.dtype, self.dist, self.seed,
                        self.has_bwd, self.note)


CONFIGS = {
    "tiny": Workload("tiny", 64, 256, WHT_F32, "normal", 0, True,
                     "64 rows, d=256, fp32 everywhere"),
    "prefill": Workload("prefill", 8 * 2048, 1024, WHT_BF16, "normal", 1, False,
                        "batch 8 x seq 2048, d=1024 (16 heads x 64), bf16 x/a/b"),
    "decode": Workload("decode", 256, 4096, WHT_BF16, "normal", 2, False,
                       "one token per sequence, T in {1,8,64,256}, d=4096 (32 x 128), bf16"),
    "training": Workload("training", 16 * 4096, 2048, WHT_BF16_PF32, "normal", 3, True,
                         "batch 16 x seq 4096, d=2048, bf16 x/dy, fp32 a/b/da/db"),
    "large": Workload("large", 4 * 32768, 8192, WHT_BF16_PF32, "student_t3", 4, True,
                      "batch 4 x seq 32768, d=8192 (64 x 128), bf16 heavy-tailed x/dy, fp32 a/b"),
}
DECODE_T = (1, 8, 64, 256)


def _generator(w: Workload, which: str, block: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((w.seed * 1_000_003 + _TENSOR_ID[which]) * 1_000_033 + block)
    return g


def _draw_block(w: Workload, which: str, block: int, rows: int) -> torch.Tensor:
    """fp32 values of one block (always drawn at full block height)."""
    g = _generator(w, which, block)
    n0 = torch.randn(ROWS_PER_BLOCK, w.d, generator=g, dtype=torch.float32)
    if w.dist == "student_t3":
        chi = torch.zeros_like(n0)
        for _ in range(3):
            n = torch.randn(ROWS_PER_BLOCK, w.d, generator=g, dtype=torch.float32)
            chi.addcmul_(n, n)
        n0 = 0.5 * n0 / torch.sqrt(chi / 3.0)
    elif w.dist != "normal":
        raise ValueError(w.dist)
    return n0[:rows]


def gen_rows(w: Workload, which: str, r0: int, r1: int) -> torch.Tensor:
    """Rows [r0, r1) of tensor `which` ("x" or "dy") in storage dtype, on the CPU."""
    assert which in ("x", "dy") and 0 <= r0 <= r1
    out = torch.empty(r1 - r0, w.d, dtype=w.io_torch_dtype)
    r = r0
    while r < r1:
        block = r // ROWS_PER_BLOCK
        b0 = block * ROWS_PER_BLOCK
        hi = min(r1, b0 + ROWS_PER_BLOCK)
        vals = _draw_block(w, which, block, ROWS_PER_BLOCK)
        out[r - r0:hi - r0] = vals[r - b0:hi - b0].to(w.io_torch_dtype)
        r = hi
    return out


def gen_full(w: Workload, which: str, out: torch.Tensor | None = None,
             threads: int = 8) -> torch.Tensor:
    """All T rows of `which`; blocks are drawn in parallel (same bits as gen_rows)."""
    if out is None:
        out = torch.empty(w.T, w.d, dtype=w.io_torch_dtype)
    nblocks = (w.T + ROWS_PER_BLOCK - 1) // ROWS_PER_BLOCK

    def fill(block: int) -> None:
        b0 = block * ROWS_PER_BLOCK
        hi = min(w.T, b0 + ROWS_PER_BLOCK)
        out[b0:hi] = _draw_block(w, which, block, ROWS_PER_BLOCK)[:hi - b0].to(out.dtype)

    if nblocks <= 1 or threads <= 1:
        for k in range(nblocks):
            fill(k)
    else:
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(fill, range(nblocks)))
    return out


def gen_params(w: Workload):
    """(a, b) in the workload's parameter storage dtype, on the CPU."""
    ga = _generator(w, "a", 0)
    gb = _generator(w, "b", 0)
    a = torch.rand(w.d, generator=ga, dtype=torch.float32) + 0.5
    b = torch.randn(w.d, generator=gb, dtype=torch.float32) * 0.1
    return a.to(w.param_torch_dtype), b.to(w.param_torch_dtype)
