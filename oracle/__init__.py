"""CPU oracle for the BitLinear forward (BitNet b1.58).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA library.
"""
from .oracle import (  # noqa: F401
    Oracle,
    build_oracle,
    load_oracle,
)
