"""CPU oracle for the LLMem peak-memory estimator.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.
"""
from .binding import *  # noqa: F401,F403
