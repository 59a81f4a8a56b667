"""CPU oracle for two-sided adaptive rounding (GPTQ-2D).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, obviously-correct
restatement of what the paper defines.  It exists so that the CUDA path can be
checked against something written independently of it.  It shares no code,
headers, tables or helpers with the CUDA path and must never be imported by
the product package; only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may call it.

Everything here is fp64 numpy (LAPACK/BLAS routines serve as single steps);
`cref` wraps a plain-C restatement of the sequential sweeps for sizes where
Python loops are too slow.
"""
from .gptq2d_oracle import *  # noqa: F401,F403
