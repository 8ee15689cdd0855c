"""CPU oracle for the DropIT layer path (arXiv 2202.13808).

TEST INFRASTRUCTURE ONLY.  A plain C restatement of the paper's definitions
(`dropit_oracle.c`) behind a numpy/ctypes binding (`oracle.py`).  It is imported
by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by
nothing on the product path; it shares no code with the CUDA library.
"""
from .oracle import *  # noqa: F401,F403
