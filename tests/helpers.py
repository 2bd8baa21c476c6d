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
