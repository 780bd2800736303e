"""Seeded synthetic inputs shaped like the paper's workloads.

This package only draws random tensors and runs the pre-existing FP32 model
(with library convolutions) to obtain calibration samples.  It contains none
of the quantization method's arithmetic and is shared by the oracle-side
tests and the CUDA-side code as the single source of input bytes.
"""
from .synth import *  # noqa: F401,F403
