"""Pins for the oracle's eq tables and multilinear-extension evaluation (CPU only)."""
import random

import numpy as np

from bigint_defs import P, bits_msb_first, clog2, eq_point, mle


def rand_fe(rng, n):
    return [rng.randrange(P) for _ in range(n)]


def test_eq_table_closed_form_sum_and_onehot(oracle):
    rng = random.Random(1)
    for n in range(0, 7):
        r = rand_fe(rng, n)
        E = oracle.eq_table(r)
        assert len(E) == 1 << n
        for i in range(1 << n):
            want = eq_point(r, bits_msb_first(i, n))
            assert int(E[i]) == want == oracle.eq_closed(r, i)
        assert sum(int(e) for e in E) % P == 1
    r = rand_fe(rng, 1)
    assert [int(e) for e in oracle.eq_table(r)] == [(1 - r[0]) % P, r[0]]
    # Boolean r selects one entry; the index reads r most-significant-bit first
    for idx in (0, 5, 6, 15):
        E = oracle.eq_table(bits_msb_first(idx, 4))
        assert [int(e) for e in E] == [1 if i == idx else 0 for i in range(16)]
    # variable 0 is the top bit: r = (t, 0, 0) puts weight t on index 4 and 1-t on index 0
    t = rng.randrange(P)
    E = oracle.eq_table([t, 0, 0])
    assert int(E[4]) == t and int(E[0]) == (1 - t) % P and sum(int(e) for e in E) % P == 1


def test_mle_at_boolean_points_is_the_entry(oracle):
    rng = random.Random(2)
    for rows, cols, dt, lo, hi in ((3, 5, np.int8, -128, 127), (4, 4, np.int32, -2**31, 2**31 - 1),
                                   (1, 6, np.int8, -128, 127), (7, 1, np.int32, -10**6, 10**6)):
        M = np.array([[rng.randint(lo, hi) for _ in range(cols)] for _ in range(rows)], dtype=dt)
        a, c = clog2(rows), clog2(cols)
        for i in range(1 << a):
            for j in range(1 << c):
                got = oracle.mle_eval_bruteforce(M, bits_msb_first(i, a), bits_msb_first(j, c))
                want = int(M[i, j]) % P if (i < rows and j < cols) else 0
                assert got == want


def test_mle_random_points_against_bigint_and_tables(oracle):
    rng = random.Random(3)
    for rows, cols, dt in ((3, 5, np.int8), (6, 3, np.int32), (8, 8, np.int8), (5, 7, np.int32)):
        lo, hi = (-128, 127) if dt == np.int8 else (-2**31, 2**31 - 1)
        M = np.array([[rng.randint(lo, hi) for _ in range(cols)] for _ in range(rows)], dtype=dt)
        a, c = clog2(rows), clog2(cols)
        x, y = rand_fe(rng, a), rand_fe(rng, c)
        want = mle(M.tolist(), x, y)
        assert oracle.mle_eval_bruteforce(M, x, y) == want
        Er, Ec = oracle.eq_table(x), oracle.eq_table(y)
        assert oracle.mle_eval_point(M, Er, Ec) == want
        # partial evaluations, then finishing by hand, reach the same value
        rowbound = oracle.mle_partial_eval(M, oracle.BIND_ROWS, Er)      # length cols
        colbound = oracle.mle_partial_eval(M, oracle.BIND_COLS, Ec)      # length rows
        assert len(rowbound) == cols and len(colbound) == rows
        assert sum(int(v) * int(Ec[j]) for j, v in enumerate(rowbound)) % P == want
        assert sum(int(v) * int(Er[i]) for i, v in enumerate(colbound)) % P == want
        # each entry of a partial evaluation is itself an MLE value at a Boolean coordinate
        for j in range(cols):
            assert int(rowbound[j]) == mle(M.tolist(), x, bits_msb_first(j, c))
        for i in range(rows):
            assert int(colbound[i]) == mle(M.tolist(), bits_msb_first(i, a), y)


def test_mle_is_affine_in_each_variable(oracle):
    rng = random.Random(4)
    M = np.array([[rng.randint(-128, 127) for _ in range(8)] for _ in range(4)], dtype=np.int8)
    x, y = rand_fe(rng, 2), rand_fe(rng, 3)
    for var in range(5):
        def at(v):
            xx, yy = list(x), list(y)
            if var < 2:
                xx[var] = v
            else:
                yy[var - 2] = v
            return oracle.mle_eval_bruteforce(M, xx, yy)
        t = rng.randrange(P)
        assert at(t) == ((1 - t) * at(0) + t * at(1)) % P


def test_leading_dimension_and_special_matrices(oracle):
    rng = random.Random(5)
    wide = np.array([[rng.randint(-128, 127) for _ in range(11)] for _ in range(6)], dtype=np.int8)
    view = wide[:, :7]                                    # ld = 11, cols = 7
    x, y = rand_fe(rng, 3), rand_fe(rng, 3)
    Er, Ec = oracle.eq_table(x), oracle.eq_table(y)
    assert oracle.mle_eval_point(view, Er, Ec) == mle(view.tolist(), x, y)
    assert [int(v) for v in oracle.mle_partial_eval(view, oracle.BIND_ROWS, Er)] == \
        [int(v) for v in oracle.mle_partial_eval(np.ascontiguousarray(view), oracle.BIND_ROWS, Er)]
    # identity: binding the rows returns the eq table itself (truncated)
    I = np.eye(8, 5, dtype=np.int8)
    assert [int(v) for v in oracle.mle_partial_eval(I, oracle.BIND_ROWS, Er)] == [int(e) for e in Er[:5]]
    # all-ones: binding the columns gives the sum of the first `cols` eq entries (1 if a power of two)
    ones = np.ones((3, 8), dtype=np.int8)
    assert [int(v) for v in oracle.mle_partial_eval(ones, oracle.BIND_COLS, Ec)] == [1, 1, 1]
    ones7 = np.ones((3, 7), dtype=np.int8)
    s7 = sum(int(e) for e in Ec[:7]) % P
    assert [int(v) for v in oracle.mle_partial_eval(ones7, oracle.BIND_COLS, Ec)] == [s7] * 3
    # one extra leading padding variable r' scales every value by (1 - r')
    M = np.array([[rng.randint(-128, 127) for _ in range(4)] for _ in range(4)], dtype=np.int8)
    Mpad = np.zeros((5, 4), dtype=np.int8)               # 5 rows -> padded to 8: adds a top variable
    Mpad[:4] = M
    x2, y2, rp = rand_fe(rng, 2), rand_fe(rng, 2), rng.randrange(P)
    base = oracle.mle_eval_bruteforce(M, x2, y2)
    assert oracle.mle_eval_bruteforce(Mpad, [rp] + x2, y2) == (1 - rp) * base % P
