"""Plain, slow, FP64 CPU oracle of the FP-Sketch verifier.

TEST INFRASTRUCTURE ONLY.  This package is the correctness reference that the
CUDA path is compared with.  It shares no code, table or constant generator
with the CUDA path and must never be imported by the product package; only the
test-suite, the smoke check and the benchmark's CPU-baseline leg use it.
"""
from .fpsk_oracle import *  # noqa: F401,F403
