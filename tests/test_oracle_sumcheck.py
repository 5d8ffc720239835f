"""Pins for the oracle's sumcheck prover and verifier (CPU only)."""
import os
import random
import subprocess
import sys

import numpy as np
import pytest

from bigint_defs import P, clog2, interp_deg2, mle, round_poly_by_definition

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def rand_problem(rng, m, k, n, lo=-128, hi=127):
    A = np.array([[rng.randint(lo, hi) for _ in range(k)] for _ in range(m)], dtype=np.int8)
    B = np.array([[rng.randint(lo, hi) for _ in range(n)] for _ in range(k)], dtype=np.int8)
    C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
    return A, B, C


def chal(oracle, seed, pid, dom, cnt):
    return [oracle.challenge(seed, pid, dom, i) for i in range(cnt)]


def read_golden(name):
    with open(os.path.join(GOLD, name + ".txt")) as f:
        return [int(line, 16) for line in f if line.strip() and not line.startswith("#")]


def test_worked_example_2x4x2(oracle):
    """Small case worked by hand: avec[0] = 1 + 4 r_row, bvec[0] = 1 + r_col, and the whole
    transcript re-derived by exhaustive hypercube sums in big integers."""
    A = [[1, -2, 3, -4], [5, 6, -7, 8]]
    B = [[1, 2], [-3, 4], [5, -6], [7, 8]]
    C = [[-6, -56], [8, 140]]
    t = oracle.sumcheck_matmul_prove(np.array(A, np.int8), np.array(B, np.int8), np.array(C, np.int32), 1, 0)
    r_row, r_col, r_k = chal(oracle, 1, 0, 1, 1), chal(oracle, 1, 0, 2, 1), chal(oracle, 1, 0, 3, 2)
    assert r_row == [1105691118476636830] and r_col == [9648468725782202765]
    Er = oracle.eq_table(r_row)
    avec = oracle.mle_partial_eval(np.array(A, np.int8), oracle.BIND_ROWS, Er)
    bvec = oracle.mle_partial_eval(np.array(B, np.int8), oracle.BIND_COLS, oracle.eq_table(r_col))
    assert int(avec[0]) == (1 + 4 * r_row[0]) % P == 4422764473906547321
    assert int(bvec[0]) == (1 + r_col[0]) % P == 9648468725782202766
    want = [mle(C, r_row, r_col)]
    for j in range(2):
        want += [round_poly_by_definition(A, B, r_row, r_col, r_k[:j], X) for X in (0, 1, 2)]
    want += [mle(A, r_row, r_k), mle(B, r_k, r_col)]
    assert [int(w) for w in t] == want == read_golden("example_2x4x2")


def test_golden_files_match_oracle():
    rc = subprocess.call([sys.executable, os.path.join(GOLD, "make_golden.py"), "--check"])
    assert rc == 0


def test_config1_pins(oracle):
    """64x64x64 uniform case: entries and transcript words derived independently of the oracle
    with big-integer arithmetic from the definitions."""
    from paper_2602_22700_b200 import synth
    p = synth.single_small(1, 64, 64, 64)[0]
    A, B, C = p.A.numpy(), p.B.numpy(), p.C.numpy()
    assert int(C[0, 0]) == 32385 and int(C[63, 63]) == 726
    assert (oracle.matmul_i8_i32(A, B) == C).all()
    t = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 1, 0)]
    assert len(t) == 21 == oracle.transcript_len(64)
    assert t[0] == 0x6CAD3A2AE63675D3
    assert t[1:4] == [0x6AF518A51574908C, 0x01B82185D0C1E547, 0xA4BB34060DD55395]
    assert t[-2] == 0x7C45DE3AD3039288 and t[-1] == 0xED65A9B19C31CE3B
    h = 0
    for w in t:
        h = oracle.mix64(h ^ w)
    assert h == 0xA256C9D8D03EB32B
    assert t == read_golden("uniform_64x64x64")
    assert oracle.sumcheck_verify(t, 6, 1, 0) == (oracle.OK, -1)


@pytest.mark.parametrize("m,k,n", [(2, 4, 2), (3, 5, 2), (1, 8, 1), (4, 3, 7), (5, 6, 3), (2, 2, 8)])
def test_round_polynomials_match_exhaustive_definition(oracle, m, k, n):
    rng = random.Random(100 * m + 10 * k + n)
    A, B, C = rand_problem(rng, m, k, n)
    seed, pid = 17, 5
    t = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, seed, pid)]
    a, b, c = clog2(m), clog2(k), clog2(n)
    assert len(t) == 3 * b + 3
    r_row, r_col, r_k = chal(oracle, seed, pid, 1, a), chal(oracle, seed, pid, 2, c), chal(oracle, seed, pid, 3, b)
    Al, Bl, Cl = A.tolist(), B.tolist(), C.tolist()
    assert t[0] == mle(Cl, r_row, r_col)
    claim = t[0]
    for j in range(b):
        g = [round_poly_by_definition(Al, Bl, r_row, r_col, r_k[:j], X) for X in (0, 1, 2)]
        assert t[1 + 3 * j:4 + 3 * j] == g
        assert (g[0] + g[1]) % P == claim                     # running-claim invariant
        claim = interp_deg2(g[0], g[1], g[2], r_k[j])
        assert oracle.interp_deg2(g[0], g[1], g[2], r_k[j]) == claim
        # the interpolated value is the true g_j(r_j)
        assert claim == round_poly_by_definition(Al, Bl, r_row, r_col, r_k[:j], r_k[j])
    assert t[-2] == mle(Al, r_row, r_k) and t[-1] == mle(Bl, r_k, r_col)
    assert claim == t[-2] * t[-1] % P
    assert oracle.sumcheck_verify(t, b, seed, pid, t[0], t[-2], t[-1]) == (oracle.OK, -1)


def test_k_equal_one_has_no_rounds(oracle):
    rng = random.Random(9)
    A, B, C = rand_problem(rng, 3, 1, 4)
    t = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 2, 0)]
    r_row, r_col = chal(oracle, 2, 0, 1, 2), chal(oracle, 2, 0, 2, 2)
    assert t == [mle(C.tolist(), r_row, r_col), mle(A.tolist(), r_row, []), mle(B.tolist(), [], r_col)]
    assert t[0] == t[1] * t[2] % P
    assert oracle.sumcheck_verify(t, 0, 2, 0) == (oracle.OK, -1)


def test_inner_product_special_case(oracle):
    """m = n = 1: a plain inner-product sumcheck; avec and bvec are the lifted vectors."""
    rng = random.Random(10)
    A, B, C = rand_problem(rng, 1, 8, 1)
    t = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 4, 1)]
    assert t[0] == int(C[0, 0]) % P
    assert t[1] == sum(int(A[0, y]) * int(B[y, 0]) for y in range(4)) % P
    assert t[2] == sum(int(A[0, y]) * int(B[y, 0]) for y in range(4, 8)) % P


def test_sum_of_products_equals_claim_iff_product_is_right(oracle):
    rng = random.Random(11)
    A, B, C = rand_problem(rng, 6, 12, 5)
    seed, pid = 3, 2
    Er = oracle.eq_table(chal(oracle, seed, pid, 1, 3))
    Ec = oracle.eq_table(chal(oracle, seed, pid, 2, 3))
    av = oracle.mle_partial_eval(A, oracle.BIND_ROWS, Er)
    bv = oracle.mle_partial_eval(B, oracle.BIND_COLS, Ec)
    c0 = oracle.mle_eval_point(C, Er, Ec)
    assert sum(int(x) * int(y) for x, y in zip(av, bv)) % P == c0
    C2 = C.copy()
    C2[2, 3] += 1
    assert oracle.mle_eval_point(C2, Er, Ec) == (c0 + int(Er[2]) * int(Ec[3])) % P != c0


def test_rejections(oracle):
    rng = random.Random(12)
    A, B, C = rand_problem(rng, 6, 16, 5)
    seed, pid, b = 8, 1, 4
    good = oracle.sumcheck_matmul_prove(A, B, C, seed, pid)
    assert oracle.sumcheck_verify(good, b, seed, pid) == (oracle.OK, -1)
    # a single altered C entry: the round-0 sum no longer matches the claim
    C2 = C.copy()
    C2[1, 4] += 1
    bad = oracle.sumcheck_matmul_prove(A, B, C2, seed, pid)
    assert oracle.sumcheck_verify(bad, b, seed, pid) == (oracle.REJECT, 0)
    # a single int8 weight changed by +-1 with C unchanged
    for delta in (1, -1):
        B2 = B.copy()
        B2[7, 2] = np.int8(int(B2[7, 2]) + delta if abs(int(B2[7, 2]) + delta) <= 127 else int(B2[7, 2]) - delta)
        bad = oracle.sumcheck_matmul_prove(A, B2, C, seed, pid)
        assert oracle.sumcheck_verify(bad, b, seed, pid) == (oracle.REJECT, 0)
        # prover consistent with the tampered weight (C recomputed): passes the rounds, but the
        # verifier's own evaluation of the true B exposes it
        C3 = (A.astype(np.int64) @ B2.astype(np.int64)).astype(np.int32)
        sneaky = oracle.sumcheck_matmul_prove(A, B2, C3, seed, pid)
        assert oracle.sumcheck_verify(sneaky, b, seed, pid) == (oracle.OK, -1)
        r_k = chal(oracle, seed, pid, 3, b)
        true_b = oracle.mle_eval_bruteforce(B, r_k, chal(oracle, seed, pid, 2, 3))
        assert oracle.sumcheck_verify(sneaky, b, seed, pid, None, None, true_b) == (oracle.REJECT, b + 3)
    # any single transcript word altered
    for pos in range(len(good)):
        t = good.copy()
        t[pos] = np.uint64((int(t[pos]) + 1) % P)
        rc, where = oracle.sumcheck_verify(t, b, seed, pid)
        assert rc == oracle.REJECT
        # c0, g_j(0), g_j(1) break round j's sum; g_j(2) only shifts the next claim
        j, e = divmod(pos - 1, 3)
        assert where == (0 if pos == 0 else b if pos > 3 * b else j + (1 if e == 2 else 0))
    # wrong seed / proof id, non-canonical word
    assert oracle.sumcheck_verify(good, b, seed + 1, pid)[0] == oracle.REJECT
    assert oracle.sumcheck_verify(good, b, seed, pid + 1)[0] == oracle.REJECT
    t = good.copy()
    t[3] = np.uint64(P)
    assert oracle.sumcheck_verify(t, b, seed, pid)[0] < 0


def test_implicit_padding_equals_explicit_padding(oracle):
    rng = random.Random(13)
    for (m, k, n) in ((3, 3, 3), (5, 14, 6), (2, 9, 7)):
        A, B, C = rand_problem(rng, m, k, n)
        mp, kp, np_ = 1 << clog2(m), 1 << clog2(k), 1 << clog2(n)
        Ap = np.zeros((mp, kp), np.int8); Ap[:m, :k] = A
        Bp = np.zeros((kp, np_), np.int8); Bp[:k, :n] = B
        Cp = np.zeros((mp, np_), np.int32); Cp[:m, :n] = C
        t1 = oracle.sumcheck_matmul_prove(A, B, C, 6, 4)
        t2 = oracle.sumcheck_matmul_prove(Ap, Bp, Cp, 6, 4)
        assert (t1 == t2).all()
        # leading dimensions larger than the extents change nothing
        t3 = oracle.sumcheck_matmul_prove(Ap[:m, :k], Bp[:k, :n], Cp[:m, :n], 6, 4)
        assert (t1 == t3).all()


def test_transposed_operands_change_the_transcript(oracle):
    """Guards the row/column roles: proving with A and B swapped-and-transposed is a different
    statement and must not give the same words."""
    rng = random.Random(14)
    A, B, C = rand_problem(rng, 4, 4, 4)
    t1 = oracle.sumcheck_matmul_prove(A, B, C, 1, 0)
    t2 = oracle.sumcheck_matmul_prove(np.ascontiguousarray(B.T), np.ascontiguousarray(A.T),
                                      np.ascontiguousarray(C.T), 1, 0)
    assert not (t1 == t2).all()
    assert oracle.sumcheck_verify(t2, 2, 1, 0) == (oracle.OK, -1)
