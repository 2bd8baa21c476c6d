"""Shared test helpers: moving stored tensors between torch and the numpy oracle."""
import numpy as np
import torch

import oracle


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a stored CPU tensor (fp32 or bf16) to float64 for the oracle."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        bits = t.view(torch.int16).numpy().view(np.uint16)
        return oracle.widen_bf16_bits(bits)
    return t.numpy().astype(np.float64)


# ---- tolerances of the parity tests (norm-wise, per row or per vector) ----------

def rowwise_max_err(got: np.ndarray, ref: np.ndarray) -> np.ndarray:
    return np.max(np.abs(got.astype(np.float64) - ref), axis=1)


def assert_rows_fp32(got, ref, transform_input, what=""):
    """fp32 storage: max_j |err| <= 1e-5 * ||input row||_2, input = what the transform saw."""
    err = rowwise_max_err(got, ref)
    bound = 1e-5 * np.linalg.norm(transform_input, axis=1)
    bad = np.nonzero(err > bound)[0]
    assert bad.size == 0, f"{what}: {bad.size} rows over 1e-5*||row||, worst ratio {np.max(err / np.maximum(bound, 1e-300)):.3g}"
    return float(np.max(err / np.maximum(bound, 1e-300)))


def assert_rows_bf16(got, ref, what=""):
    """bf16 storage, fp32 accumulation: max_j |err| <= 1e-2 * max_j |ref row|."""
    err = rowwise_max_err(got, ref)
    bound = 1e-2 * np.max(np.abs(ref), axis=1)
    bad = np.nonzero(err > bound)[0]
    assert bad.size == 0, f"{what}: {bad.size} rows over 1e-2*max|row|, worst ratio {np.max(err / np.maximum(bound, 1e-300)):.3g}"
    return float(np.max(err / np.maximum(bound, 1e-300)))


def assert_grad_vec(got, ref, what=""):
    """da, db in fp32: max_j |err| <= 1e-4 * max_j |ref|."""
    err = np.max(np.abs(got.astype(np.float64) - ref))
    bound = 1e-4 * np.max(np.abs(ref))
    assert err <= bound, f"{what}: max err {err:.3g} > {bound:.3g}"
    return float(err / max(bound, 1e-300))
