"""B200-native prover for sumcheck proofs of int8 matrix products over the Goldilocks field.

``imm`` is the thin binding of the C-ABI CUDA library (argument marshalling only);
``synth`` holds the seeded synthetic input generators.  Importing the package does not load the
CUDA library; the first call into ``imm`` does, and raises if it is missing.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "imm"]


def __getattr__(name):
    if name == "imm":
        import importlib
        return importlib.import_module(".imm", __name__)
    raise AttributeError(name)
