"""CPU oracle for the Goldilocks sumcheck matmul proof -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It wraps ``imm_oracle.c`` (plain C, ``% p`` on 128-bit integers) through ctypes and shares no
code with the CUDA library.  See the header of ``imm_oracle.c`` for the conventions and the
list of pins.
"""
from .imm_oracle import *  # noqa: F401,F403
