"""Pins for the oracle's batched (random-linear-combination) sumcheck prover and verifier (CPU only).

The expected values come from the definitions in Python big integers (exhaustive hypercube sums),
from the single-proof oracle under shared challenges, and from properties the protocol fixes.
"""
import random

import numpy as np
import pytest

from bigint_defs import P, clog2, interp_deg2, mle, round_poly_by_definition
from test_oracle_sumcheck import chal, rand_problem


def split(t, b, count):
    """(c0B, [g_j triple], [(c0_p, a_fin_p, b_fin_p)]) of a batched transcript."""
    t = [int(w) for w in t]
    assert len(t) == 1 + 3 * b + 3 * count
    rounds = [t[1 + 3 * j:4 + 3 * j] for j in range(b)]
    tail = [tuple(t[1 + 3 * b + 3 * p:4 + 3 * b + 3 * p]) for p in range(count)]
    return t[0], rounds, tail


def group(rng, shapes, first_id=10):
    return [rand_problem(rng, m, k, n) + (first_id + 3 * i,) for i, (m, k, n) in enumerate(shapes)]


@pytest.mark.parametrize("shapes", [
    [(2, 4, 2), (3, 4, 1)],
    [(1, 8, 3), (4, 5, 2), (2, 7, 2)],          # k = 8, 5, 7 all pad to three rounds
    [(3, 2, 3), (2, 2, 5), (1, 2, 1), (2, 2, 2)],
])
def test_batched_transcript_matches_exhaustive_definition(oracle, shapes):
    rng = random.Random(sum(sum(s) for s in shapes))
    probs = group(rng, shapes)
    seed, bid = 23, 77
    b = clog2(shapes[0][1])
    c0B, rounds, tail = split(oracle.sumcheck_matmul_prove_batched(probs, seed, bid), b, len(probs))
    rho = chal(oracle, seed, bid, 4, len(probs))
    r_k = chal(oracle, seed, bid, 3, b)
    pts = []
    for A, B, C, pid in probs:
        pts.append((chal(oracle, seed, pid, 1, clog2(A.shape[0])), chal(oracle, seed, pid, 2, clog2(B.shape[1]))))
    lists = [(A.tolist(), B.tolist(), C.tolist()) for A, B, C, _ in probs]
    # the per-proof tail is the three two-sided evaluations at the shared point
    for (Al, Bl, Cl), (r_row, r_col), (c0, af, bf) in zip(lists, pts, tail):
        assert c0 == mle(Cl, r_row, r_col)
        assert af == mle(Al, r_row, r_k) and bf == mle(Bl, r_k, r_col)
    assert c0B == sum(r * t[0] for r, t in zip(rho, tail)) % P
    claim = c0B
    for j in range(b):
        g = [sum(r * round_poly_by_definition(Al, Bl, rr, rc, r_k[:j], X)
                 for r, (Al, Bl, _), (rr, rc) in zip(rho, lists, pts)) % P for X in (0, 1, 2)]
        assert rounds[j] == g
        assert (g[0] + g[1]) % P == claim
        claim = interp_deg2(g[0], g[1], g[2], r_k[j])
    assert claim == sum(r * t[1] * t[2] for r, t in zip(rho, tail)) % P


def test_single_member_batch_is_the_single_proof_scaled(oracle):
    """With batch_id = proof_id the shared challenges are the single proof's, so the batched
    rounds are rho_0 times the single-proof rounds and the tail repeats its three words."""
    rng = random.Random(4)
    A, B, C = rand_problem(rng, 5, 11, 3)
    seed, pid = 9, 31
    single = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, seed, pid)]
    b = clog2(11)
    c0B, rounds, tail = split(oracle.sumcheck_matmul_prove_batched([(A, B, C, pid)], seed, pid), b, 1)
    rho = oracle.challenge(seed, pid, 4, 0)
    assert c0B == rho * single[0] % P
    assert [w for g in rounds for w in g] == [rho * w % P for w in single[1:1 + 3 * b]]
    assert tail == [(single[0], single[-2], single[-1])]


def test_combination_coefficients_are_their_own_domain(oracle):
    seed, bid = 5, 6
    rho = chal(oracle, seed, bid, 4, 8)
    assert len(set(rho)) == 8 and all(0 <= r < P for r in rho)
    for dom in (1, 2, 3):
        assert set(rho).isdisjoint(chal(oracle, seed, bid, dom, 8))


def test_batched_rounds_are_linear_in_the_members(oracle):
    """Proving the members one by one as single-member batches under the same batch_id gives
    rho_0-scaled rounds; dividing by rho_0 and recombining with rho_p reproduces the batch."""
    rng = random.Random(12)
    probs = group(rng, [(4, 16, 3), (2, 13, 6), (7, 9, 1)])
    seed, bid, b = 3, 1000, 4
    c0B, rounds, tail = split(oracle.sumcheck_matmul_prove_batched(probs, seed, bid), b, 3)
    rho = chal(oracle, seed, bid, 4, 3)
    inv0 = pow(rho[0], P - 2, P)
    acc = [0] * (1 + 3 * b)
    for p, prob in enumerate(probs):
        t = [int(w) for w in oracle.sumcheck_matmul_prove_batched([prob], seed, bid)]
        assert tuple(t[-3:]) == tail[p]
        for i in range(1 + 3 * b):
            acc[i] = (acc[i] + rho[p] * inv0 % P * t[i]) % P
    assert acc == [c0B] + [w for g in rounds for w in g]


def test_verifier_accepts_honest_and_locates_tampering(oracle):
    rng = random.Random(8)
    probs = group(rng, [(3, 8, 4), (2, 6, 2), (5, 8, 8)])
    seed, bid, b, count = 14, 2, 3, 3
    t = [int(w) for w in oracle.sumcheck_matmul_prove_batched(probs, seed, bid)]
    assert oracle.sumcheck_verify_batched(t, b, count, seed, bid) == (oracle.OK, -1)
    assert oracle.sumcheck_verify_batched(t, b, count, seed, bid, expect=t[-9:]) == (oracle.OK, -1)
    # other coins: the first thing to break is the combination of the c0_p
    assert oracle.sumcheck_verify_batched(t, b, count, seed + 1, bid) == (oracle.REJECT, b + 1)
    assert oracle.sumcheck_verify_batched(t, b, count, seed, bid + 1) == (oracle.REJECT, b + 1)

    def bump(i):
        u = list(t)
        u[i] = (u[i] + 1) % P
        return u
    assert oracle.sumcheck_verify_batched(bump(0), b, count, seed, bid) == (oracle.REJECT, b + 1)
    for j in range(b):
        # g_j(0) off by one breaks round j's sum; g_j(2) alone only shows at the next check
        assert oracle.sumcheck_verify_batched(bump(1 + 3 * j), b, count, seed, bid) == (oracle.REJECT, j)
        assert oracle.sumcheck_verify_batched(bump(3 + 3 * j), b, count, seed, bid) == (oracle.REJECT, j + 1)
    for p in range(count):
        base = 1 + 3 * b + 3 * p
        assert oracle.sumcheck_verify_batched(bump(base), b, count, seed, bid) == (oracle.REJECT, b + 1)
        assert oracle.sumcheck_verify_batched(bump(base + 1), b, count, seed, bid) == (oracle.REJECT, b)
        assert oracle.sumcheck_verify_batched(bump(base + 2), b, count, seed, bid) == (oracle.REJECT, b)
        # a tail that is self-consistent but not the verifier's own evaluation
        want = t[-9:]
        want[3 * p + 1] = (want[3 * p + 1] + 5) % P
        assert oracle.sumcheck_verify_batched(t, b, count, seed, bid, expect=want) == \
            (oracle.REJECT, b + 2 + 3 * p + 1)
    u = list(t)
    u[4] = P
    assert oracle.sumcheck_verify_batched(u, b, count, seed, bid)[0] not in (oracle.OK, oracle.REJECT)


@pytest.mark.parametrize("which", ["C", "A", "B"])
def test_one_wrong_member_sinks_the_batch(oracle, which):
    """A single altered entry in one member (so its C is no longer its A*B): the transcript of a
    prover that follows the procedure misses the round-0 sum, since sum_y a_p(y) b_p(y) is the MLE
    of A_p*B_p and not of the claimed C_p."""
    rng = random.Random(21)
    probs = group(rng, [(4, 8, 4), (4, 8, 4), (3, 7, 5)])
    seed, bid, b = 2, 9, 3
    A, B, C, pid = probs[1]
    A, B, C = A.copy(), B.copy(), C.copy()
    {"A": A, "B": B, "C": C}[which][2, 3] += 1
    bad = [int(w) for w in oracle.sumcheck_matmul_prove_batched([probs[0], (A, B, C, pid), probs[2]], seed, bid)]
    assert oracle.sumcheck_verify_batched(bad, b, 3, seed, bid) == (oracle.REJECT, 0)


def zero_padded(A, B, kp):
    """The same product with the inner dimension padded to kp by zero columns of A and zero rows of B."""
    m, k = A.shape
    Ap = np.zeros((m, kp), dtype=A.dtype)
    Ap[:, :k] = A
    Bp = np.zeros((kp, B.shape[1]), dtype=B.dtype)
    Bp[:k] = B
    return Ap, Bp


def test_members_of_different_inner_size_are_padded_to_the_largest(oracle):
    """k = 3, 16, 1, 6 in one batch: four rounds for everybody.  Against the exhaustive definition on
    explicitly padded matrices, and against the batch of those padded matrices itself."""
    rng = random.Random(31)
    shapes = [(2, 3, 3), (1, 16, 2), (3, 1, 1), (2, 6, 4)]
    probs = group(rng, shapes)
    seed, bid, b = 8, 15, 4
    t = oracle.sumcheck_matmul_prove_batched(probs, seed, bid)
    c0B, rounds, tail = split(t, b, 4)
    padded = [zero_padded(A, B, 16) + (C, pid) for A, B, C, pid in probs]
    assert [int(w) for w in oracle.sumcheck_matmul_prove_batched(padded, seed, bid)] == [int(w) for w in t]
    rho, r_k = chal(oracle, seed, bid, 4, 4), chal(oracle, seed, bid, 3, b)
    claim = c0B
    for j in range(b):
        g = [0, 0, 0]
        for r, (Ap, Bp, C, pid) in zip(rho, padded):
            rr = chal(oracle, seed, pid, 1, clog2(Ap.shape[0]))
            rc = chal(oracle, seed, pid, 2, clog2(Bp.shape[1]))
            for X in (0, 1, 2):
                g[X] = (g[X] + r * round_poly_by_definition(Ap.tolist(), Bp.tolist(), rr, rc, r_k[:j], X)) % P
        assert rounds[j] == g and (g[0] + g[1]) % P == claim
        claim = interp_deg2(g[0], g[1], g[2], r_k[j])
    assert claim == sum(r * x[1] * x[2] for r, x in zip(rho, tail)) % P
    assert oracle.sumcheck_verify_batched(t, b, 4, seed, bid) == (oracle.OK, -1)


def test_zero_round_batch(oracle):
    """k = 1 everywhere: no rounds, the claim is sum_p rho_p a_p b_p directly."""
    rng = random.Random(6)
    probs = group(rng, [(3, 1, 2), (1, 1, 1)])
    t = [int(w) for w in oracle.sumcheck_matmul_prove_batched(probs, 4, 4)]
    assert len(t) == 7
    rho = chal(oracle, 4, 4, 4, 2)
    assert t[0] == (rho[0] * t[1] + rho[1] * t[4]) % P == (rho[0] * t[2] * t[3] + rho[1] * t[5] * t[6]) % P
    assert oracle.sumcheck_verify_batched(t, 0, 2, 4, 4) == (oracle.OK, -1)
