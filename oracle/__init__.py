"""CPU oracle for PCG verification -- test infrastructure, not product code.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA library and never imports it.
"""
from .pcg_oracle import (  # noqa: F401
    F32,
    BF16,
    F16,
    FLAG_ZERO_RESIDUAL,
    FLAG_THINNING_EXHAUSTED,
    build,
    max_threads,
    softmax,
    group_probs,
    verify,
    OracleResult,
)
