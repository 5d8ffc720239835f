"""CPU oracle for the element-wise links between proved matrix products -- TEST INFRASTRUCTURE ONLY.

Plain numpy on 64-bit integers, one definition per function, no blocking.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import it; it shares no code with the CUDA library.

What it follows.  The reference execution F_theta* is a chain of attention, MLP and normalisation
steps (Section 4.1), and the proof must establish that these continuous transformations were
computed with the committed model (Section 5.2, item 2).  The sumcheck proofs cover the matrix
products one by one; what ties one product's output to the next product's input is an element-wise
map.  In an int8-quantised execution that map is the requantisation of the int32 accumulators

    H[i, j] = clamp( floor( (C[i, j] + rnd) / 2^shift ), lo, hi )

(round-half-up division by a power of two when rnd = 2^(shift-1), then saturation), and a verifier
that holds the opened tensors checks it by recomputing it: the link holds iff no entry of H differs.

Readings (the paper names the parts of F_theta* and nothing about their arithmetic): the division
rounds toward minus infinity (floor), which is what an arithmetic right shift of a two's-complement
integer computes; 0 <= rnd < 2^shift; the check reports how many entries differ and the row-major
position i*cols + j of the first one (-1 if none), so that a failing audit can name the entry.

The gated feed-forward block of the decoder models the paper audits (Section 6.1: LLaMA3, Qwen3)
has one more element-wise step between its products: an activation of the gate projection and its
product with the up projection.  In an int8 execution both are integer maps,

    g[i, j] = act[ clamp(floor((G[i, j] + rnd) / 2^shift), -128, 127) + 128 ]        (a 256-entry table)
    u[i, j] =      clamp(floor((U[i, j] + rnd) / 2^shift), -128, 127)
    H[i, j] = clamp( floor( (g[i, j] * u[i, j] + rnd2) / 2^shift2 ), lo, hi )

with G, U the int32 outputs of the gate and up products and H the int8 input of the down product;
without U the link is the activation alone, H = g.  Readings: the activation is whatever int8 -> int8
table the committed model ships (the paper fixes no integer arithmetic; the table is an input here);
both products are requantised with the same shift and rounding and saturate to the full int8 range
before the table is indexed; floor division as above.

Pins (tests/test_oracle_glue.py): Python big-integer floor division and exact fractions
(round-half-up of C / 2^shift) on hand-written values at the rounding boundaries, both signs, the
clamp edges and the int32 extremes; shift = 0; idempotence under the clamp; monotonicity; the input
generator's own hidden activations; counts and first positions of planted differences; the gated link
entry by entry in Python integers, with the identity table and no gate reducing to the plain
requantisation, a ReLU table to a clamp at zero, and products at the rounding boundaries of both signs.
No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


def requantize(C, shift: int, rnd: int, lo: int, hi: int) -> np.ndarray:
    """H = clamp(floor((C + rnd) / 2^shift), lo, hi) as int8; C holds int32 values."""
    assert 0 <= shift <= 30 and 0 <= rnd < (1 << shift) or (shift == 0 and rnd == 0)
    assert -128 <= lo <= hi <= 127
    t = np.asarray(C, dtype=np.int64) + int(rnd)
    q = np.floor_divide(t, np.int64(1) << np.int64(shift))
    return np.clip(q, lo, hi).astype(np.int8)


def requant_check(C, H, shift: int, rnd: int, lo: int, hi: int):
    """(number of entries where H differs from requantize(C), row-major index of the first or -1)."""
    C = np.asarray(C)
    H = np.asarray(H)
    assert C.shape == H.shape
    bad = np.flatnonzero((requantize(C, shift, rnd, lo, hi) != H.astype(np.int8)).reshape(-1))
    return int(bad.size), (int(bad[0]) if bad.size else -1)


def activation(G, act, shift: int, rnd: int) -> np.ndarray:
    """g = act[clamp(floor((G + rnd) / 2^shift), -128, 127) + 128] as int8; act holds 256 int8 values."""
    act = np.asarray(act, dtype=np.int8)
    assert act.shape == (256,)
    q = requantize(G, shift, rnd, -128, 127).astype(np.int64)
    return act[q + 128]


def gated_link(G, U, act, shift: int, rnd: int, shift2: int, rnd2: int, lo: int, hi: int) -> np.ndarray:
    """H = clamp(floor((g * u + rnd2) / 2^shift2), lo, hi) with g = activation(G), u = requantize(U) to the
    full int8 range; U None: H = g."""
    g = activation(G, act, shift, rnd)
    if U is None:
        return g
    assert 0 <= shift2 <= 14 and (0 <= rnd2 < (1 << shift2) or (shift2 == 0 and rnd2 == 0))
    assert -128 <= lo <= hi <= 127
    u = requantize(U, shift, rnd, -128, 127)
    t = g.astype(np.int64) * u.astype(np.int64) + int(rnd2)
    q = np.floor_divide(t, np.int64(1) << np.int64(shift2))
    return np.clip(q, lo, hi).astype(np.int8)


def gated_link_check(G, U, H, act, shift: int, rnd: int, shift2: int, rnd2: int, lo: int, hi: int):
    """(number of entries where H differs from gated_link(...), row-major index of the first or -1)."""
    want = gated_link(G, U, act, shift, rnd, shift2, rnd2, lo, hi)
    H = np.asarray(H)
    assert want.shape == H.shape
    bad = np.flatnonzero((want != H.astype(np.int8)).reshape(-1))
    return int(bad.size), (int(bad[0]) if bad.size else -1)
