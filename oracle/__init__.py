"""CPU oracle for CD-Adam.  TEST INFRASTRUCTURE ONLY.

A ctypes front end over ``cdadam_oracle.c`` (plain single-threaded C written from the
paper's Algorithm 1 and Appendix A).  Nothing in the CUDA library or its Python binding
imports this package; it is used by the tests, the smoke check and the CPU-baseline leg of
the benchmark only.
"""
from .oracle import (Oracle, build, compress_sign, compress_topk, compress_randk, l1_exact,
                     SIGN, TOPK, IDENTITY, RANDK, MARKOV, EF, NAIVE, STATE_NAMES)

__all__ = ["Oracle", "build", "compress_sign", "compress_topk", "compress_randk", "l1_exact",
           "SIGN", "TOPK", "IDENTITY", "RANDK", "MARKOV", "EF", "NAIVE", "STATE_NAMES"]
