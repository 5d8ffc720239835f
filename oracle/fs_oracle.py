"""CPU oracle of the non-interactive (Fiat-Shamir) matmul proof -- TEST INFRASTRUCTURE ONLY (nothing
on the product path may import this file; it shares no code or table with the CUDA library).

What it instantiates.  Algorithm 1 of the paper has the server send a proof pi with its response:
no verifier is on line to draw coins, so the public coins of the interactive sumcheck
(``imm_oracle.c``) are replaced by hashes of everything sent so far -- the Fiat-Shamir transform.
The paper fixes none of this; the readings below are this implementation's.

  H           SHA-256 (``hashlib``, a library step).  Integers are little-endian; a field element is
              the le64 of its canonical value.
  fe(d)       the first 8 bytes of a digest as a big-endian integer v, minus p if v >= p.
  s_0         H(0x10 || com_A || com_B || com_C || le64(m) || le64(k) || le64(n) || le64(proof_id)):
              the statement -- the three 32-byte commitments (``commit_oracle``) and the shape.
  points      r_row[t] = fe(H(0x11 || s_0 || le32(1) || le32(t))), r_col[t] likewise with le32(2).
  claim       c0 = C~(r_row, r_col);  s_1 = H(0x12 || s_0 || le64(c0)).
  round j     the prover sends g_j(0), g_j(1), g_j(2);
              s_{j+2} = H(0x13 || s_{j+1} || le64(g_j(0)) || le64(g_j(2)));
              r_j = fe(s_{j+2}); both tables fold with r_j.
              g_j(1) is not hashed: the verifier requires g_j(0) + g_j(1) = claim, and the claim is
              a function of what the state already binds, so g_j(1) carries nothing new -- and
              without it the message is 49 bytes, one SHA-256 block instead of two, on the one
              step of the proof that nothing can overlap.
  transcript  [c0, g_0(0..2), ..., g_{b-1}(0..2), a_fin, b_fin], as in the interactive proof.

The field arithmetic of the steps (eq tables, the two partial evaluations, the claim) is the C
oracle's, called through its binding; the rounds are written out here in Python integers.

Batched form (one non-interactive proof for P products, ``prove_batched``): the batched proof of
``imm_oracle.c`` (random linear combination, every k padded to the largest 2^b) with hashed coins:
  root        the Merkle tree hash of RFC 6962 (``commit_oracle.merkle_tree_hash``) over the list of
              member statements s_0^(0), ..., s_0^(P-1) (32-byte leaves)
  T           H(0x14 || root || le64(batch_id) || le32(P)): binds every member before any coin
  rho_p       fe(H(0x15 || T || le32(p)))
  claim       c0B = sum_p rho_p c0_p;  s_1 = H(0x12 || T || le64(c0B))
  round j     as above on the combined values G_j = sum_p rho_p g_j^(p)
  transcript  [c0B, G_0(0..2), ..., G_{b-1}(0..2), (c0_p, a_fin_p, b_fin_p) for every p].
The c0_p are not hashed: with binding commitments they are functions of the statements, and the
verifier compares them (and a_fin_p, b_fin_p) with its own evaluations.

Pins (tests/test_oracle_fs.py): every challenge re-derived with a SHA-256 written from the standard;
every round polynomial against exhaustive hypercube sums in big integers at those challenges;
g_j(0)+g_j(1) = running claim and the final product; each challenge depends on everything before it
(commitments, shape, proof id, c0, g(0) and g(2) of earlier rounds); the verifier accepts the honest transcript and
rejects every single-word change.
"""
from __future__ import annotations

import hashlib

import numpy as np

from . import imm_oracle as orc

P = orc.P


def _h(data: bytes) -> bytes:
    return hashlib.sha256(data).digest()


def _le64(v: int) -> bytes:
    return int(v).to_bytes(8, "little")


def _le32(v: int) -> bytes:
    return int(v).to_bytes(4, "little")


def fe(digest: bytes) -> int:
    v = int.from_bytes(digest[:8], "big")
    return v - P if v >= P else v


def statement(coms, m: int, k: int, n: int, proof_id: int) -> bytes:
    """s_0 from the three 32-byte commitments (com_A, com_B, com_C) and the shape."""
    com_a, com_b, com_c = (bytes(c) for c in coms)
    assert len(com_a) == len(com_b) == len(com_c) == 32
    return _h(b"\x10" + com_a + com_b + com_c + _le64(m) + _le64(k) + _le64(n) + _le64(proof_id))


def point(s0: bytes, domain: int, count: int):
    return [fe(_h(b"\x11" + s0 + _le32(domain) + _le32(t))) for t in range(count)]


def absorb_claim(s0: bytes, c0: int) -> bytes:
    return _h(b"\x12" + s0 + _le64(c0))


def absorb_round(s: bytes, g0: int, g1: int, g2: int) -> bytes:
    """g1 is part of the round's message but not of the hash (see the header)."""
    return _h(b"\x13" + s + _le64(g0) + _le64(g2))


def prove(A: np.ndarray, B: np.ndarray, C: np.ndarray, coms, proof_id: int):
    """Transcript (list of ints) of the non-interactive proof of the claim C = A*B (C used as given)."""
    m, k = A.shape
    n = B.shape[1]
    a, b, c = orc.ceil_log2(m), orc.ceil_log2(k), orc.ceil_log2(n)
    s0 = statement(coms, m, k, n, proof_id)
    e_row = orc.eq_table(point(s0, 1, a))
    e_col = orc.eq_table(point(s0, 2, c))
    av = [int(v) for v in orc.mle_partial_eval(A, orc.BIND_ROWS, e_row)] + [0] * ((1 << b) - k)
    bv = [int(v) for v in orc.mle_partial_eval(B, orc.BIND_COLS, e_col)] + [0] * ((1 << b) - k)
    c0 = orc.mle_eval_point(C, e_row, e_col)
    out = [c0]
    s = absorb_claim(s0, c0)
    for j in range(b):
        half = 1 << (b - 1 - j)
        g0 = g1 = g2 = 0
        for y in range(half):
            a0, a1, b0, b1 = av[y], av[y + half], bv[y], bv[y + half]
            g0 += a0 * b0
            g1 += a1 * b1
            g2 += (2 * a1 - a0) * (2 * b1 - b0)
        g0, g1, g2 = g0 % P, g1 % P, g2 % P
        out += [g0, g1, g2]
        s = absorb_round(s, g0, g1, g2)
        r = fe(s)
        av = [(av[y] + r * (av[y + half] - av[y])) % P for y in range(half)]
        bv = [(bv[y] + r * (bv[y + half] - bv[y])) % P for y in range(half)]
    return out + [av[0], bv[0]]


def challenges(transcript, nrounds: int, coms, m: int, k: int, n: int, proof_id: int):
    """(r_row, r_col, r_k) as the verifier derives them from the statement and the transcript."""
    s0 = statement(coms, m, k, n, proof_id)
    r_row, r_col = point(s0, 1, orc.ceil_log2(m)), point(s0, 2, orc.ceil_log2(n))
    s = absorb_claim(s0, transcript[0])
    r_k = []
    for j in range(nrounds):
        s = absorb_round(s, *transcript[1 + 3 * j:4 + 3 * j])
        r_k.append(fe(s))
    return r_row, r_col, r_k


def verify(transcript, nrounds: int, coms, m: int, k: int, n: int, proof_id: int, expect=None):
    """(status, fail_at) with the interactive verifier's meaning of fail_at; ``expect`` is the
    verifier's own (c0, a_fin, b_fin) or None."""
    t = [int(w) for w in transcript]
    if len(t) < 3 * nrounds + 3 or any(w >= P or w < 0 for w in t[:3 * nrounds + 3]):
        return -5, -2
    _, _, r_k = challenges(t, nrounds, coms, m, k, n, proof_id)
    claim = t[0]
    for j in range(nrounds):
        g0, g1, g2 = t[1 + 3 * j:4 + 3 * j]
        if (g0 + g1) % P != claim:
            return orc.REJECT, j
        claim = orc.interp_deg2(g0, g1, g2, r_k[j])
    a_fin, b_fin = t[3 * nrounds + 1], t[3 * nrounds + 2]
    if a_fin * b_fin % P != claim:
        return orc.REJECT, nrounds
    if expect is not None:
        for i, (want, got) in enumerate(zip(expect, (t[0], a_fin, b_fin))):
            if want is not None and want != got:
                return orc.REJECT, nrounds + 1 + i
    return orc.OK, -1


# ------------------------------------------------------------------ batched form


def batch_seed(statements, batch_id: int) -> bytes:
    """T from the member statements (list of 32-byte s_0) and the batch id."""
    from .commit_oracle import merkle_tree_hash
    root = merkle_tree_hash([bytes(x) for x in statements])
    return _h(b"\x14" + root + _le64(batch_id) + _le32(len(statements)))


def rho(T: bytes, count: int):
    return [fe(_h(b"\x15" + T + _le32(p))) for p in range(count)]


def prove_batched(problems, batch_id: int):
    """``problems``: list of (A, B, C, coms, proof_id).  Returns the batched transcript (list of ints)."""
    count = len(problems)
    b = max(orc.ceil_log2(A.shape[1]) for (A, _, _, _, _) in problems)
    stmts, tabs, c0s = [], [], []
    for A, B, C, coms, pid in problems:
        m, k = A.shape
        n = B.shape[1]
        s0 = statement(coms, m, k, n, pid)
        e_row = orc.eq_table(point(s0, 1, orc.ceil_log2(m)))
        e_col = orc.eq_table(point(s0, 2, orc.ceil_log2(n)))
        av = [int(v) for v in orc.mle_partial_eval(A, orc.BIND_ROWS, e_row)] + [0] * ((1 << b) - k)
        bv = [int(v) for v in orc.mle_partial_eval(B, orc.BIND_COLS, e_col)] + [0] * ((1 << b) - k)
        stmts.append(s0)
        tabs.append([av, bv])
        c0s.append(orc.mle_eval_point(C, e_row, e_col))
    T = batch_seed(stmts, batch_id)
    rh = rho(T, count)
    c0B = sum(r * c for r, c in zip(rh, c0s)) % P
    out = [c0B]
    s = absorb_claim(T, c0B)
    for j in range(b):
        half = 1 << (b - 1 - j)
        G = [0, 0, 0]
        for r, (av, bv) in zip(rh, tabs):
            g0 = g1 = g2 = 0
            for y in range(half):
                a0, a1, b0, b1 = av[y], av[y + half], bv[y], bv[y + half]
                g0 += a0 * b0
                g1 += a1 * b1
                g2 += (2 * a1 - a0) * (2 * b1 - b0)
            G[0] += r * (g0 % P)
            G[1] += r * (g1 % P)
            G[2] += r * (g2 % P)
        G = [g % P for g in G]
        out += G
        s = absorb_round(s, *G)
        rj = fe(s)
        for t in tabs:
            t[0] = [(t[0][y] + rj * (t[0][y + half] - t[0][y])) % P for y in range(half)]
            t[1] = [(t[1][y] + rj * (t[1][y + half] - t[1][y])) % P for y in range(half)]
    for c0, (av, bv) in zip(c0s, tabs):
        out += [c0, av[0], bv[0]]
    return out


def challenges_batched(transcript, nrounds: int, statements, batch_id: int):
    """(rho, r_k) as the verifier derives them from the member statements and the transcript."""
    T = batch_seed(statements, batch_id)
    s = absorb_claim(T, transcript[0])
    r_k = []
    for j in range(nrounds):
        s = absorb_round(s, *transcript[1 + 3 * j:4 + 3 * j])
        r_k.append(fe(s))
    return rho(T, len(statements)), r_k


def verify_batched(transcript, nrounds: int, statements, batch_id: int, expect=None):
    """(status, fail_at) with the meaning of ``orc_sumcheck_verify_batched``."""
    count = len(statements)
    t = [int(w) for w in transcript]
    total = 1 + 3 * nrounds + 3 * count
    if len(t) < total or any(w >= P or w < 0 for w in t[:total]):
        return -5, -2
    rh, r_k = challenges_batched(t, nrounds, statements, batch_id)
    tail = t[1 + 3 * nrounds:total]
    if t[0] != sum(r * tail[3 * p] for p, r in enumerate(rh)) % P:
        return orc.REJECT, nrounds + 1
    claim = t[0]
    for j in range(nrounds):
        g0, g1, g2 = t[1 + 3 * j:4 + 3 * j]
        if (g0 + g1) % P != claim:
            return orc.REJECT, j
        claim = orc.interp_deg2(g0, g1, g2, r_k[j])
    if claim != sum(r * tail[3 * p + 1] * tail[3 * p + 2] for p, r in enumerate(rh)) % P:
        return orc.REJECT, nrounds
    if expect is not None:
        for i, (want, got) in enumerate(zip(expect, tail)):
            if want != got:
                return orc.REJECT, nrounds + 2 + i
    return orc.OK, -1
