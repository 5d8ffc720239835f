"""Pins of the glue oracle (oracle/glue_oracle.py): the requantisation link between two proved
products against big-integer and exact-fraction arithmetic on hand-written cases.  CPU only."""
from fractions import Fraction
import math

import numpy as np
import pytest

from oracle import glue


def by_hand(c: int, shift: int, rnd: int, lo: int, hi: int) -> int:
    """The definition in Python integers: floor division, then saturation."""
    return max(lo, min(hi, (c + rnd) // (1 << shift)))


def half_up(c: int, shift: int) -> int:
    """Round-half-up of the exact quotient c / 2^shift."""
    return math.floor(Fraction(c, 1 << shift) + Fraction(1, 2))


EDGES_9 = [0, 1, -1, 255, 256, 257, -255, -256, -257, 511, 512, 513, 767, 768, 769, -767, -768, -769,
           # the clamp edges of [-127, 127]: quotients 126.5 / 127.5 / -126.5 / -127.5 / -128.5
           127 * 512 - 257, 127 * 512 - 256, 127 * 512 + 255, 127 * 512 + 256, 128 * 512,
           -127 * 512 + 255, -127 * 512 - 256, -127 * 512 - 257, -128 * 512 - 256, -128 * 512 - 257,
           2**31 - 1, 2**31 - 256, 2**31 - 257, -2**31, -2**31 + 255, -2**31 + 256]


def test_requantize_is_round_half_up_then_clamp_on_hand_written_values():
    got = glue.requantize(np.array(EDGES_9, dtype=np.int32), 9, 256, -127, 127)
    for c, g in zip(EDGES_9, got):
        assert int(g) == by_hand(c, 9, 256, -127, 127) == max(-127, min(127, half_up(c, 9))), c
    # spelled out: the boundary between q and q+1 sits at C = 512 q + 256 (ties go up), for both signs
    assert glue.requantize(np.array([255, 256, -257, -256, 767, 768, -769, -768]), 9, 256, -127, 127).tolist() == \
        [0, 1, -1, 0, 1, 2, -2, -1]
    # saturation: 127.5 and above -> 127; -127.5 rounds up to -127; below -127.5 still -127
    assert glue.requantize(np.array([127 * 512 + 255, 127 * 512 + 256, 2**31 - 1]), 9, 256, -127, 127).tolist() == [127] * 3
    assert glue.requantize(np.array([-127 * 512 - 256, -127 * 512 - 257, -2**31]), 9, 256, -127, 127).tolist() == [-127] * 3
    assert glue.requantize(np.array([-128 * 512 - 256, -128 * 512 - 257, -2**31]), 9, 256, -128, 127).tolist() == [-128] * 3


@pytest.mark.parametrize("shift,rnd", [(0, 0), (1, 0), (1, 1), (4, 8), (9, 0), (9, 256), (9, 511), (16, 1 << 15), (30, 1 << 29)])
def test_requantize_matches_big_integer_floor_division(shift, rnd):
    rng = np.random.default_rng(shift * 7 + rnd % 5)
    vals = np.concatenate([rng.integers(-2**31, 2**31, 4000, dtype=np.int64),
                           rng.integers(-70000, 70000, 4000, dtype=np.int64),
                           np.array([-2**31, 2**31 - 1, 0, -1, 1], dtype=np.int64)]).astype(np.int32)
    for lo, hi in ((-127, 127), (-128, 127), (0, 15), (-3, -3)):
        got = glue.requantize(vals, shift, rnd, lo, hi)
        want = [by_hand(int(c), shift, rnd, lo, hi) for c in vals]
        assert got.tolist() == want
    # negative values really take the floor, not truncation toward zero
    if shift > 0 and rnd == 0:
        assert int(glue.requantize(np.array([-1]), shift, 0, -128, 127)[0]) == -1


def test_requantize_properties():
    rng = np.random.default_rng(3)
    c = np.sort(rng.integers(-100000, 100000, 5000)).astype(np.int32)
    h = glue.requantize(c, 9, 256, -127, 127).astype(np.int64)
    assert (np.diff(h) >= 0).all()                                   # monotone
    assert h.min() == -127 and h.max() == 127
    inside = np.abs(c.astype(np.int64)) < 127 * 512 - 256
    assert (np.abs(h[inside] * 512 - c[inside]) <= 256).all()        # within half a step where nothing saturates
    # shift 0 is the plain clamp
    assert glue.requantize(np.array([-300, -5, 7, 300]), 0, 0, -127, 127).tolist() == [-127, -5, 7, 127]


def test_requant_check_counts_and_locates_differences():
    rng = np.random.default_rng(4)
    C = rng.integers(-80000, 80000, (37, 53)).astype(np.int32)
    H = glue.requantize(C, 9, 256, -127, 127)
    assert glue.requant_check(C, H, 9, 256, -127, 127) == (0, -1)
    H2 = H.copy()
    H2[5, 7] += 1
    assert glue.requant_check(C, H2, 9, 256, -127, 127) == (1, 5 * 53 + 7)
    H2[2, 50] -= 1
    H2[36, 52] ^= 0x40
    assert glue.requant_check(C, H2, 9, 256, -127, 127) == (3, 2 * 53 + 50)
    # one altered accumulator: seen iff it crosses a rounding boundary
    C2 = C.copy()
    C2[0, 0] += 512
    assert glue.requant_check(C2, H, 9, 256, -127, 127) == (1, 0)
    r = int(C[1, 1]) & 511                                            # stay on the same side of the boundary at 256
    C3 = C.copy()
    C3[1, 1] += 1 if r != 255 else -1
    assert glue.requant_check(C3, H, 9, 256, -127, 127) == (0, -1)
    # other parameters give other answers (the check is of THIS map)
    assert glue.requant_check(C, H, 9, 255, -127, 127)[0] > 0
    assert glue.requant_check(C, H, 8, 128, -127, 127)[0] > 0


def test_the_input_generators_hidden_activations_satisfy_the_link():
    """synth.requantize_i8 (torch, used to manufacture the down projection's input) is this map."""
    import torch
    from paper_2602_22700_b200 import synth
    up, down = synth.ffn_pair(1, 16, 64, 96, device="cpu")
    assert glue.requant_check(up.C.numpy(), down.A.numpy(), 9, 256, -127, 127) == (0, -1)
    x = torch.tensor(EDGES_9, dtype=torch.int32)
    assert synth.requantize_i8(x).tolist() == glue.requantize(np.array(EDGES_9, dtype=np.int32), 9, 256, -127, 127).tolist()


# ---------------------------------------------------------------- activation and gating link

def relu_table():
    return np.array([max(0, v) for v in range(-128, 128)], dtype=np.int8)


def silu_like_table():
    """An arbitrary odd-looking int8 table (round(x * sigmoid(x / 16))): any table is valid input."""
    return np.array([int(round(v / (1.0 + math.exp(-v / 16.0)))) for v in range(-128, 128)], dtype=np.int8)


def gated_by_hand(g: int, u, act, shift, rnd, shift2, rnd2, lo, hi) -> int:
    """The definition entry by entry in Python integers."""
    q = max(-128, min(127, (g + rnd) // (1 << shift)))
    a = int(act[q + 128])
    if u is None:
        return a
    w = max(-128, min(127, (u + rnd) // (1 << shift)))
    return max(lo, min(hi, (a * w + rnd2) // (1 << shift2)))


def test_activation_alone_reduces_to_known_maps():
    rng = np.random.default_rng(11)
    G = np.concatenate([rng.integers(-90000, 90000, 3000), np.array(EDGES_9)]).astype(np.int32)
    ident = np.arange(-128, 128, dtype=np.int8)
    # identity table: the plain requantisation to the full int8 range
    assert (glue.gated_link(G, None, ident, 9, 256, 0, 0, -128, 127) == glue.requantize(G, 9, 256, -128, 127)).all()
    # ReLU table: the requantisation clamped at zero
    assert (glue.gated_link(G, None, relu_table(), 9, 256, 0, 0, -128, 127) == glue.requantize(G, 9, 256, 0, 127)).all()
    # a constant table ignores its input; a reversed table negates (except at -128, which has no negative)
    assert (glue.activation(G, np.full(256, 7, dtype=np.int8), 9, 256) == 7).all()
    rev = np.array([max(-128, min(127, -v)) for v in range(-128, 128)], dtype=np.int8)
    q = glue.requantize(G, 9, 256, -128, 127).astype(np.int64)
    assert (glue.activation(G, rev, 9, 256).astype(np.int64) == np.clip(-q, -128, 127)).all()
    # the table is indexed by value + 128: entry 0 answers -128, entry 255 answers 127
    probe = np.zeros(256, dtype=np.int8); probe[0] = 11; probe[255] = 22; probe[128] = 33
    assert glue.activation(np.array([-2**31, 2**31 - 1, 0, 255, 256]), probe, 9, 256).tolist() == [11, 22, 33, 33, 0]


@pytest.mark.parametrize("shift2,rnd2", [(0, 0), (6, 32), (7, 64), (7, 0), (7, 127), (14, 1 << 13)])
def test_gated_link_matches_python_integers(shift2, rnd2):
    rng = np.random.default_rng(100 + shift2 + rnd2)
    n = 3000
    G = np.concatenate([rng.integers(-70000, 70000, n), np.array(EDGES_9)]).astype(np.int32)
    U = np.concatenate([rng.integers(-70000, 70000, n), np.array(EDGES_9[::-1])]).astype(np.int32)
    for act in (silu_like_table(), relu_table(), np.arange(-128, 128, dtype=np.int8)):
        for lo, hi in ((-127, 127), (-128, 127), (0, 100)):
            got = glue.gated_link(G, U, act, 9, 256, shift2, rnd2, lo, hi)
            want = [gated_by_hand(int(g), int(u), act, 9, 256, shift2, rnd2, lo, hi) for g, u in zip(G, U)]
            assert got.tolist() == want


def test_gated_link_rounding_boundaries_of_the_product():
    """g * u = 64 (2 t + 1) sits exactly between t and t + 1 at shift2 = 7: ties go up, for both signs;
    the extreme products (-128 * -128 = 16384, -128 * 127) saturate."""
    ident = np.arange(-128, 128, dtype=np.int8)
    pairs = [(8, 8), (8, -8), (-8, -8), (24, 8), (-24, 8), (1, 63), (1, 64), (1, 65), (-1, 64), (-1, 65), (-128, -128), (-128, 127), (127, 127)]
    G = np.array([g for g, _ in pairs], dtype=np.int32)          # shift 0: the accumulators are the int8 values
    U = np.array([u for _, u in pairs], dtype=np.int32)
    got = glue.gated_link(G, U, ident, 0, 0, 7, 64, -127, 127).tolist()
    exact = [max(-127, min(127, math.floor(Fraction(g * u, 128) + Fraction(1, 2)))) for g, u in pairs]
    assert got == exact == [1, 0, 1, 2, -1, 0, 1, 1, 0, -1, 127, -127, 126]


def test_gated_link_check_counts_and_locates():
    rng = np.random.default_rng(12)
    G = rng.integers(-60000, 60000, (19, 23)).astype(np.int32)
    U = rng.integers(-60000, 60000, (19, 23)).astype(np.int32)
    act = silu_like_table()
    H = glue.gated_link(G, U, act, 9, 256, 7, 64, -127, 127)
    args = (act, 9, 256, 7, 64, -127, 127)
    assert glue.gated_link_check(G, U, H, *args) == (0, -1)
    H2 = H.copy(); H2[3, 4] += 1; H2[18, 22] -= 1
    assert glue.gated_link_check(G, U, H2, *args) == (2, 3 * 23 + 4)
    # another table, or the gate and up operands swapped, is another map
    assert glue.gated_link_check(G, U, H, relu_table(), 9, 256, 7, 64, -127, 127)[0] > 0
    assert glue.gated_link_check(U, G, H, *args)[0] > 0
    # without U the check is of the activation alone
    A = glue.gated_link(G, None, act, 9, 256, 0, 0, -128, 127)
    assert glue.gated_link_check(G, None, A, act, 9, 256, 0, 0, -128, 127) == (0, -1)
