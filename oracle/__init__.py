"""CPU oracle for Sparse Binary Compression -- TEST INFRASTRUCTURE ONLY.

A plain single-threaded C implementation of the paper's Algorithms 1-4
(``sbc_oracle.c``) with a ctypes/numpy wrapper.  Nothing in the CUDA package
imports this; only the tests, the smoke check and the benchmark's CPU-baseline
leg do.
"""
from .sbc_oracle import *  # noqa: F401,F403
