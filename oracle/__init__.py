"""CPU oracle for the 8-bit quantized convolution path.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the CPU-baseline
leg of the benchmark.  The CUDA package never imports this module.
"""
from .q8_oracle import *  # noqa: F401,F403
