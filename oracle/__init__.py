"""CPU float64 oracle for the CAMERA micro-expert analysis.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain reference the CUDA
path is checked against.  It shares no code with the CUDA library or its
Python binding and must never be imported by them; only the test-suite, the
smoke check and the benchmark's CPU-baseline leg call it.
"""
from .camera_oracle import *  # noqa: F401,F403
from .adapters import f64, to_oracle_layer  # noqa: F401
