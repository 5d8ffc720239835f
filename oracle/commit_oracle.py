"""CPU oracle of the hash commitment -- TEST INFRASTRUCTURE ONLY (nothing on the product path may
import this file; it shares no code or table with the CUDA library).

What it instantiates.  The paper commits with a hash, c = Hash(m || r) (Section 2.1, cryptographic
commitment): the server's commitment to the model, psi_M = Hash(model), and to the logits of a
response under fresh randomness, psi = Hash(r, {l_1..l_N}) (Algorithm 1), which the auditor
recomputes (the auditing algorithm's first check).  The paper names no hash.  Readings fixed here:

  Hash        SHA-256 (FIPS 180-4), taken from ``hashlib`` as a library step.
  tree mode   a message of gigabytes cannot be hashed as one SHA-256 stream in parallel, so the
              message is cut into LEAF = 4096-byte chunks (the last may be shorter; an empty message
              is one empty chunk) and hashed as the Merkle tree of RFC 6962, Section 2.1:
                  MTH({d})      = SHA-256(0x00 || d)
                  MTH(D[0:n])   = SHA-256(0x01 || MTH(D[0:k]) || MTH(D[k:n])),  k the largest
                                  power of two smaller than n.
  commitment  c = SHA-256(0x02 || root || le64(len(m)) || r): the length fixes the tree's shape,
              the tag separates the final hash from leaves and nodes; r is 32 bytes of
              randomness, or empty for a commitment that hides nothing (the model's).
              (Section 2.1 writes m || r, Algorithm 1 writes (r, l): r enters last here, after the
              tree, so that the tree of m can be computed before r is drawn.)

``merkle_root`` is the recursive definition as printed in the RFC, not a level-by-level rewrite.

Pins (tests/test_oracle_commit.py): the SHA-256 example digests of FIPS 180-4 pin the library
routine; a pure-Python SHA-256 written from the standard (constants from cube and square roots of
primes) recomputes whole commitments without hashlib; a level-by-level tree with the odd node
promoted (a different algorithm) agrees on every leaf count up to 70; single-leaf and two-leaf
cases written out as nested hashes; length, tag and randomness separation properties.
"""
from __future__ import annotations

import hashlib

LEAF = 4096
DIGEST = 32


def sha256(data: bytes) -> bytes:
    return hashlib.sha256(data).digest()


def chunks(msg: bytes):
    """The leaf data d_0..d_{n-1}: consecutive LEAF-byte pieces, at least one."""
    return [msg[i:i + LEAF] for i in range(0, len(msg), LEAF)] or [b""]


def merkle_tree_hash(d) -> bytes:
    """MTH of RFC 6962, Section 2.1, for a non-empty list of byte strings."""
    n = len(d)
    if n == 1:
        return sha256(b"\x00" + d[0])
    k = 1
    while 2 * k < n:
        k *= 2
    return sha256(b"\x01" + merkle_tree_hash(d[:k]) + merkle_tree_hash(d[k:]))


def merkle_root(msg: bytes) -> bytes:
    return merkle_tree_hash(chunks(bytes(msg)))


def commit(msg: bytes, r: bytes = b"") -> bytes:
    """c = Hash(m || r) in the reading above; r is empty or 32 bytes."""
    if len(r) not in (0, DIGEST):
        raise ValueError("r must be empty or 32 bytes")
    msg = bytes(msg)
    return sha256(b"\x02" + merkle_root(msg) + len(msg).to_bytes(8, "little") + bytes(r))
