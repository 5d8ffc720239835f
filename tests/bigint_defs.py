"""Definition-level helpers in Python big integers, used only to pin the C oracle.

These are the textbook definitions evaluated the slowest possible way (sums over the whole
Boolean hypercube, ``%`` on unbounded ints).  They deliberately use a different algorithm from
the oracle's prover (no tables, no folding), so agreement is evidence and not a tautology.
"""
P = 2**64 - 2**32 + 1


def clog2(d):
    n = 0
    while (1 << n) < d:
        n += 1
    return n


def bits_msb_first(i, n):
    return [(i >> (n - 1 - t)) & 1 for t in range(n)]


def eq_point(r, z):
    """eq(r, z) for arbitrary field points r, z of equal length."""
    acc = 1
    for rt, zt in zip(r, z):
        acc = acc * ((rt * zt + (1 - rt) * (1 - zt)) % P) % P
    return acc


def mle(M, x, y):
    """M~(x, y) for a list-of-lists integer matrix, zero-padded to powers of two."""
    rows, cols = len(M), len(M[0])
    a, c = clog2(rows), clog2(cols)
    assert len(x) == a and len(y) == c
    acc = 0
    for i in range(rows):
        ei = eq_point(x, bits_msb_first(i, a))
        for j in range(cols):
            acc += ei * eq_point(y, bits_msb_first(j, c)) * M[i][j]
    return acc % P


def round_poly_by_definition(A, B, r_row, r_col, r_prev, X):
    """g_j(X) = sum over the free Boolean suffix z of A~(r_row,(r_prev,X,z)) * B~((r_prev,X,z),r_col)."""
    k = len(B)
    b = clog2(k)
    free = b - len(r_prev) - 1
    acc = 0
    for zi in range(1 << free):
        pt = list(r_prev) + [X] + bits_msb_first(zi, free)
        acc += mle(A, r_row, pt) * mle(B, pt, r_col)
    return acc % P


def interp_deg2(g0, g1, g2, r):
    """Value at r of the quadratic through (0,g0),(1,g1),(2,g2), via Newton forward differences."""
    d1 = g1 - g0
    d2 = g2 - 2 * g1 + g0
    inv2 = pow(2, P - 2, P)
    return (g0 + r * d1 + r * (r - 1) % P * inv2 % P * d2) % P
