"""Pins for the oracle's non-interactive (Fiat-Shamir) matmul proof (CPU only).

Challenges are re-derived here with the SHA-256 written from the standard in test_oracle_commit
(no hashlib); the field arithmetic is checked against exhaustive hypercube sums in Python big
integers at those challenges.
"""
import random

import numpy as np
import pytest

from bigint_defs import P, clog2, interp_deg2, mle, round_poly_by_definition
from test_oracle_commit import sha256_py
from test_oracle_sumcheck import rand_problem


def le(v, nbytes):
    return int(v).to_bytes(nbytes, "little")


def to_fe(digest):
    v = int.from_bytes(digest[:8], "big")
    return v % P


def coms_for(rng):
    return [rng.randbytes(32) for _ in range(3)]


def derive_independently(t, b, coms, m, k, n, pid):
    """(r_row, r_col, r_k) from the statement and the transcript, hashing with sha256_py."""
    s0 = sha256_py(b"\x10" + coms[0] + coms[1] + coms[2] + le(m, 8) + le(k, 8) + le(n, 8) + le(pid, 8))
    r_row = [to_fe(sha256_py(b"\x11" + s0 + le(1, 4) + le(i, 4))) for i in range(clog2(m))]
    r_col = [to_fe(sha256_py(b"\x11" + s0 + le(2, 4) + le(i, 4))) for i in range(clog2(n))]
    s = sha256_py(b"\x12" + s0 + le(t[0], 8))
    r_k = []
    for j in range(b):
        s = sha256_py(b"\x13" + s + le(t[1 + 3 * j], 8) + le(t[3 + 3 * j], 8))      # g_j(0), g_j(2); not g_j(1)
        r_k.append(to_fe(s))
    return r_row, r_col, r_k


@pytest.mark.parametrize("m,k,n", [(2, 4, 2), (3, 5, 2), (1, 8, 3), (4, 2, 1), (2, 1, 2), (3, 7, 4)])
def test_transcript_matches_definitions_at_hashed_challenges(oracle, m, k, n):
    rng = random.Random(1000 * m + 10 * k + n)
    A, B, C = rand_problem(rng, m, k, n)
    coms, pid = coms_for(rng), rng.getrandbits(40)
    t = oracle.fs.prove(A, B, C, coms, pid)
    b = clog2(k)
    assert len(t) == 3 * b + 3 and all(0 <= w < P for w in t)
    r_row, r_col, r_k = derive_independently(t, b, coms, m, k, n, pid)
    assert (r_row, r_col, r_k) == tuple(oracle.fs.challenges(t, b, coms, m, k, n, pid))
    Al, Bl, Cl = A.tolist(), B.tolist(), C.tolist()
    assert t[0] == mle(Cl, r_row, r_col)
    claim = t[0]
    for j in range(b):
        g = [round_poly_by_definition(Al, Bl, r_row, r_col, r_k[:j], X) for X in (0, 1, 2)]
        assert t[1 + 3 * j:4 + 3 * j] == g
        assert (g[0] + g[1]) % P == claim
        claim = interp_deg2(g[0], g[1], g[2], r_k[j])
    assert t[-2] == mle(Al, r_row, r_k) and t[-1] == mle(Bl, r_k, r_col)
    assert claim == t[-2] * t[-1] % P
    assert oracle.fs.verify(t, b, coms, m, k, n, pid) == (oracle.OK, -1)
    assert oracle.fs.verify(t, b, coms, m, k, n, pid, expect=(t[0], t[-2], t[-1])) == (oracle.OK, -1)


def test_field_mapping_of_a_digest(oracle):
    assert oracle.fs.fe(bytes(8) + b"x" * 24) == 0
    assert oracle.fs.fe(bytes.fromhex("ffffffff00000000") + bytes(24)) == P - 1
    assert oracle.fs.fe(bytes.fromhex("ffffffff00000001") + bytes(24)) == 0            # p itself wraps to 0
    assert oracle.fs.fe(bytes.fromhex("ffffffffffffffff") + bytes(24)) == 2**32 - 2
    assert oracle.fs.fe(bytes.fromhex("0102030405060708") + bytes(24)) == 0x0102030405060708


def test_every_challenge_depends_on_everything_before_it(oracle):
    rng = random.Random(5)
    m, k, n = 4, 8, 4
    A, B, C = rand_problem(rng, m, k, n)
    coms, pid = coms_for(rng), 77
    t = oracle.fs.prove(A, B, C, coms, pid)
    base = oracle.fs.challenges(t, 3, coms, m, k, n, pid)
    flat = lambda ch: ch[0] + ch[1] + ch[2]
    # statement: any commitment byte, any dimension (same padded sizes), the proof id
    for which in range(3):
        alt = list(coms)
        alt[which] = bytes([alt[which][0] ^ 1]) + alt[which][1:]
        other = oracle.fs.challenges(t, 3, alt, m, k, n, pid)
        assert all(x != y for x, y in zip(flat(base), flat(other)))
    for dims in ((3, 8, 4), (4, 7, 4), (4, 8, 3)):
        other = oracle.fs.challenges(t, 3, coms, *dims, pid)
        assert all(x != y for x, y in zip(flat(base), flat(other)))
    assert all(x != y for x, y in zip(flat(base), flat(oracle.fs.challenges(t, 3, coms, m, k, n, pid + 1))))
    # transcript: c0, g_j(0) and g_j(2) move every round challenge drawn after them and none before;
    # g_j(1) is not hashed (the sum check pins it to the claim)
    for pos in range(1 + 3 * 3):
        u = list(t)
        u[pos] = (u[pos] + 1) % P
        other = oracle.fs.challenges(u, 3, coms, m, k, n, pid)
        assert other[0] == base[0] and other[1] == base[1]
        if pos > 0 and (pos - 1) % 3 == 1:
            assert other == base
            assert oracle.fs.verify(u, 3, coms, m, k, n, pid) == (oracle.REJECT, (pos - 1) // 3)
            continue
        first = 0 if pos == 0 else (pos - 1) // 3
        assert other[2][:first] == base[2][:first]
        assert all(x != y for x, y in zip(other[2][first:], base[2][first:]))
    # the final words are sent after the last challenge
    u = list(t)
    u[-1] = (u[-1] + 1) % P
    assert oracle.fs.challenges(u, 3, coms, m, k, n, pid) == base


def test_verifier_rejects_every_single_word_change(oracle):
    rng = random.Random(6)
    m, k, n = 3, 16, 5
    A, B, C = rand_problem(rng, m, k, n)
    coms, pid = coms_for(rng), 3
    t = oracle.fs.prove(A, B, C, coms, pid)
    b = 4
    assert oracle.fs.verify(t, b, coms, m, k, n, pid) == (oracle.OK, -1)
    for pos in range(len(t)):
        u = list(t)
        u[pos] = (u[pos] + 1 + rng.randrange(P - 1)) % P
        status, where = oracle.fs.verify(u, b, coms, m, k, n, pid)
        assert status == oracle.REJECT
        if pos == 0:
            assert where == 0
        elif pos <= 3 * b:
            j, part = (pos - 1) // 3, (pos - 1) % 3
            # g_j(0), g_j(1) break round j's sum; g_j(2) moves r_j and the claim, caught one check later
            assert where == (j if part < 2 else j + 1)
        else:
            assert where == b
    # a transcript proved for other commitments does not verify against these
    other = coms_for(rng)
    assert oracle.fs.verify(oracle.fs.prove(A, B, C, other, pid), b, coms, m, k, n, pid)[0] == oracle.REJECT
    # the verifier's own evaluations
    assert oracle.fs.verify(t, b, coms, m, k, n, pid, expect=(t[0], (t[-2] + 1) % P, t[-1])) == (oracle.REJECT, b + 2)
    assert oracle.fs.verify(t[:3] + [P] + t[4:], b, coms, m, k, n, pid)[0] not in (oracle.OK, oracle.REJECT)


def test_wrong_product_is_rejected(oracle):
    rng = random.Random(8)
    A, B, C = rand_problem(rng, 4, 8, 4)
    C = C.copy()
    C[1, 2] += 1
    coms = coms_for(rng)
    t = oracle.fs.prove(A, B, C, coms, 0)
    assert oracle.fs.verify(t, 3, coms, 4, 8, 4, 0) == (oracle.REJECT, 0)


# ------------------------------------------------------------------ batched form

def levelwise_root_of(leaves, H):
    level = [H(b"\x00" + d) for d in leaves]
    while len(level) > 1:
        nxt = [H(b"\x01" + level[i] + level[i + 1]) for i in range(0, len(level) - 1, 2)]
        if len(level) % 2:
            nxt.append(level[-1])
        level = nxt
    return level[0]


def batch_problems(rng, shapes, first_id=50):
    out = []
    for i, (m, k, n) in enumerate(shapes):
        A, B, C = rand_problem(rng, m, k, n)
        out.append((A, B, C, coms_for(rng), first_id + 2 * i))
    return out


def padded_lists(A, B, kp):
    m, k = A.shape
    Ap = np.zeros((m, kp), dtype=np.int64)
    Ap[:, :k] = A
    Bp = np.zeros((kp, B.shape[1]), dtype=np.int64)
    Bp[:k] = B
    return Ap.tolist(), Bp.tolist()


@pytest.mark.parametrize("shapes", [[(2, 4, 2), (3, 4, 1)], [(1, 8, 3), (2, 3, 2), (3, 1, 1)], [(2, 2, 2)],
                                    [(1, 2, 1), (2, 2, 1), (1, 1, 2), (2, 2, 2), (1, 2, 2)]])
def test_batched_transcript_matches_definitions_at_hashed_coins(oracle, shapes):
    rng = random.Random(7 + sum(sum(x) for x in shapes))
    probs = batch_problems(rng, shapes)
    bid = rng.getrandbits(50)
    t = oracle.fs.prove_batched(probs, bid)
    count, b = len(probs), max(clog2(k) for (_, k, _) in shapes)
    assert len(t) == 1 + 3 * b + 3 * count
    # every coin re-derived without hashlib: statements, tree over them, T, rho, the chain
    stmts, pts = [], []
    for A, B, C, coms, pid in probs:
        m, k = A.shape
        n = B.shape[1]
        s0 = sha256_py(b"\x10" + coms[0] + coms[1] + coms[2] + le(m, 8) + le(k, 8) + le(n, 8) + le(pid, 8))
        stmts.append(s0)
        pts.append(([to_fe(sha256_py(b"\x11" + s0 + le(1, 4) + le(i, 4))) for i in range(clog2(m))],
                    [to_fe(sha256_py(b"\x11" + s0 + le(2, 4) + le(i, 4))) for i in range(clog2(n))]))
    T = sha256_py(b"\x14" + levelwise_root_of(stmts, sha256_py) + le(bid, 8) + le(count, 4))
    rho = [to_fe(sha256_py(b"\x15" + T + le(p, 4))) for p in range(count)]
    s = sha256_py(b"\x12" + T + le(t[0], 8))
    r_k = []
    for j in range(b):
        s = sha256_py(b"\x13" + s + le(t[1 + 3 * j], 8) + le(t[3 + 3 * j], 8))
        r_k.append(to_fe(s))
    assert (rho, r_k) == tuple(oracle.fs.challenges_batched(t, b, stmts, bid))
    assert stmts == [oracle.fs.statement(c, A.shape[0], A.shape[1], B.shape[1], pid) for A, B, C, c, pid in probs]
    # the words against exhaustive sums on explicitly padded matrices
    tail = [t[1 + 3 * b + 3 * p:4 + 3 * b + 3 * p] for p in range(count)]
    lists = [padded_lists(A, B, 1 << b) for A, B, _, _, _ in probs]
    for (A, B, C, _, _), (rr, rc), (Al, Bl), (c0, af, bf) in zip(probs, pts, lists, tail):
        assert c0 == mle(C.tolist(), rr, rc)
        assert af == mle(Al, rr, r_k) and bf == mle(Bl, r_k, rc)
    assert t[0] == sum(r * x[0] for r, x in zip(rho, tail)) % P
    claim = t[0]
    for j in range(b):
        g = [sum(r * round_poly_by_definition(Al, Bl, rr, rc, r_k[:j], X)
                 for r, (Al, Bl), (rr, rc) in zip(rho, lists, pts)) % P for X in (0, 1, 2)]
        assert t[1 + 3 * j:4 + 3 * j] == g and (g[0] + g[1]) % P == claim
        claim = interp_deg2(g[0], g[1], g[2], r_k[j])
    assert claim == sum(r * x[1] * x[2] for r, x in zip(rho, tail)) % P
    assert oracle.fs.verify_batched(t, b, stmts, bid) == (oracle.OK, -1)
    assert oracle.fs.verify_batched(t, b, stmts, bid, expect=[w for x in tail for w in x]) == (oracle.OK, -1)


def test_batched_coins_bind_every_member_and_the_verifier_locates_changes(oracle):
    rng = random.Random(77)
    shapes = [(2, 8, 2), (3, 5, 1), (1, 8, 4)]
    probs = batch_problems(rng, shapes)
    bid, b, count = 9, 3, 3
    t = oracle.fs.prove_batched(probs, bid)
    stmts = [oracle.fs.statement(c, A.shape[0], A.shape[1], B.shape[1], pid) for A, B, C, c, pid in probs]
    rho, r_k = oracle.fs.challenges_batched(t, b, stmts, bid)
    # any member's statement, the order of members, the batch id and the member count move every coin
    for alt in ([stmts[0], stmts[2], stmts[1]], [bytes([stmts[0][0] ^ 1]) + stmts[0][1:]] + stmts[1:], stmts[:2]):
        r2, k2 = oracle.fs.challenges_batched(t, b, alt, bid)
        assert all(x != y for x, y in zip(rho, r2)) and all(x != y for x, y in zip(r_k, k2))
    r2, k2 = oracle.fs.challenges_batched(t, b, stmts, bid + 1)
    assert all(x != y for x, y in zip(rho, r2)) and all(x != y for x, y in zip(r_k, k2))
    assert oracle.fs.verify_batched(t, b, stmts, bid) == (oracle.OK, -1)
    for pos in range(len(t)):
        u = list(t)
        u[pos] = (u[pos] + 1 + rng.randrange(P - 1)) % P
        status, where = oracle.fs.verify_batched(u, b, stmts, bid)
        assert status == oracle.REJECT
        if pos == 0:
            assert where == b + 1
        elif pos <= 3 * b:
            j, part = (pos - 1) // 3, (pos - 1) % 3
            assert where == (j if part < 2 else j + 1)
        else:
            assert where == (b + 1 if (pos - 1 - 3 * b) % 3 == 0 else b)
    exp = t[1 + 3 * b:]
    exp[4] = (exp[4] + 1) % P
    assert oracle.fs.verify_batched(t, b, stmts, bid, expect=exp) == (oracle.REJECT, b + 2 + 4)
    # one wrong member sinks the batch at round 0
    A, B, C, coms, pid = probs[1]
    C2 = C.copy()
    C2[0, 0] += 1
    bad = oracle.fs.prove_batched([probs[0], (A, B, C2, coms, pid), probs[2]], bid)
    assert oracle.fs.verify_batched(bad, b, stmts, bid) == (oracle.REJECT, 0)
