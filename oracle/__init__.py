"""CPU oracles -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; it
shares no code with the CUDA library.

* the Goldilocks sumcheck matmul proof: ``imm_oracle.c`` (plain C, ``% p`` on 128-bit integers)
  wrapped through ctypes and re-exported here; its header lists the conventions and the pins;
* the logit distance distribution (TV / KL distances, Top-K distance, the per-request tail
  statistic): ``oracle.ldd`` (plain numpy in float64); its header lists the readings and the pins;
* the hash commitment (SHA-256 Merkle tree, ``hashlib`` as the library step): ``oracle.commitment``;
* the non-interactive (Fiat-Shamir) form of the matmul proof: ``oracle.fs``;
* the element-wise links between proved products (requantisation): ``oracle.glue``.
"""
from . import commit_oracle as commitment  # noqa: F401
from . import fs_oracle as fs  # noqa: F401
from . import glue_oracle as glue  # noqa: F401
from . import ldd_oracle as ldd  # noqa: F401
from .imm_oracle import *  # noqa: F401,F403
