"""Test-infrastructure oracle for the MoHGE expert layer (fp64, numpy, CPU).

This package is NOT part of the product path. Only the test-suite, the smoke
check and the benchmark's CPU-baseline leg may import it. It shares no code
with the CUDA library and never imports it.
"""
from .mohge_oracle import *  # noqa: F401,F403
