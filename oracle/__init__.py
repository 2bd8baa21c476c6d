"""CPU fp64 oracle for the Walsh-Hadamard head-mixing path (test infrastructure only).

Nothing in the product package imports this directory.  Only the test suite,
the smoke check and the benchmark's CPU-baseline leg may use it.
"""
from .wht_oracle import (  # noqa: F401
    sylvester_hadamard,
    widen_bf16_bits,
    wht_affine_fwd,
    wht_affine_fwd_residual,
    wht_affine_bwd,
    grouped_hadamard,
    wht_affine_fwd_grouped,
    wht_affine_bwd_grouped,
    wht_normalised,
    da_db_columns,
    fwht_butterfly,
)
