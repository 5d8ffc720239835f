"""Regenerates the stored transcripts under tests/golden/ by calling ONLY the CPU oracle.

    python tests/golden/make_golden.py [--check]

``--check`` compares instead of writing.  The two small worked examples were first derived with
big-integer arithmetic straight from the definitions before the oracle existed; the oracle
reproduces them, and the test-suite additionally re-derives the 2x4x2 example by exhaustive
hypercube summation.  The larger cases are regression values of the oracle alone.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
HERE = os.path.dirname(os.path.abspath(__file__))

import oracle  # noqa: E402
from paper_2602_22700_b200 import synth  # noqa: E402  (input generators only)


def cases():
    A = np.array([[1, -2, 3, -4], [5, 6, -7, 8]], dtype=np.int8)
    B = np.array([[1, 2], [-3, 4], [5, -6], [7, 8]], dtype=np.int8)
    C = np.array([[-6, -56], [8, 140]], dtype=np.int32)
    yield ("example_2x4x2", "A=[[1,-2,3,-4],[5,6,-7,8]] B=[[1,2],[-3,4],[5,-6],[7,8]] "
           "C=A*B seed=1 proof_id=0", oracle.sumcheck_matmul_prove(A, B, C, 1, 0))
    p = synth.single_small(1, 64, 64, 64)[0]
    yield ("uniform_64x64x64", "uniform int8 A (tid 0), B (tid 1), data seed 1; proof seed 1, id 0",
           oracle.sumcheck_matmul_prove(p.A.numpy(), p.B.numpy(), p.C.numpy(), 1, 0))
    p = synth.qkv_projection(1, 24, 100, 72)[0]
    yield ("gauss_24x100x72", "qkv_projection(seed 1, tokens 24, d_model 100, d_out 72); proof seed 5, id 3",
           oracle.sumcheck_matmul_prove(p.A.numpy(), p.B.numpy(), p.C.numpy(), 5, 3))


def render(name, what, words):
    lines = [f"# {name}: {what}",
             "# transcript words, hex: c0, then g_j(0) g_j(1) g_j(2) per round, then a_fin, b_fin",
             "# written by tests/golden/make_golden.py from the CPU oracle"]
    lines += [f"{int(w):016x}" for w in words]
    return "\n".join(lines) + "\n"


def main():
    check = "--check" in sys.argv
    bad = 0
    for name, what, words in cases():
        path = os.path.join(HERE, name + ".txt")
        text = render(name, what, words)
        if check:
            if open(path).read() != text:
                print("MISMATCH", name)
                bad += 1
        else:
            open(path, "w").write(text)
            print("wrote", path)
    sys.exit(1 if bad else 0)


if __name__ == "__main__":
    main()
