"""CPU oracle for the stencil sweep.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package imports nothing from them.
"""
from .stencil_oracle import (  # noqa: F401
    ZERO,
    PERIODIC,
    apply,
    apply_points,
    build,
    num_threads,
)
