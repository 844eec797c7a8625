"""Float64 CPU oracle for the SignMuon optimizer step.

TEST INFRASTRUCTURE ONLY. Nothing in the product path imports this package; it is
used by the tests, by the smoke check and by the CPU-baseline leg of the benchmark.
It shares no code with the CUDA path.
"""
from .signmuon_oracle import *  # noqa: F401,F403
