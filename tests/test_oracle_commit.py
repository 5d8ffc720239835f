"""Pins for the commitment oracle (CPU only).

The library SHA-256 is pinned by the example digests of FIPS 180-4; the tree and the final hash are
pinned by a SHA-256 written here from the standard (no hashlib), by a level-by-level tree (a
different algorithm from the oracle's recursion), by small cases written out as nested hashes and
by separation properties.
"""
import hashlib
import math
import random

import pytest


# ------------------------------------------------------------------ SHA-256 from FIPS 180-4

def _primes(count):
    out, c = [], 2
    while len(out) < count:
        if all(c % q for q in out if q * q <= c):
            out.append(c)
        c += 1
    return out


def _icbrt(v):
    x = 1 << ((v.bit_length() + 2) // 3)
    while True:
        y = (2 * x + v // (x * x)) // 3
        if y >= x:
            return x
        x = y


K = [_icbrt(p << 96) & 0xFFFFFFFF for p in _primes(64)]       # fractional parts of cube roots
H0 = [math.isqrt(p << 64) & 0xFFFFFFFF for p in _primes(8)]   # fractional parts of square roots
M32 = 0xFFFFFFFF


def _rotr(x, s):
    return ((x >> s) | (x << (32 - s))) & M32


def sha256_py(msg: bytes) -> bytes:
    bitlen = 8 * len(msg)
    msg = msg + b"\x80" + b"\x00" * ((55 - len(msg)) % 64) + bitlen.to_bytes(8, "big")
    h = list(H0)
    for off in range(0, len(msg), 64):
        w = [int.from_bytes(msg[off + 4 * t:off + 4 * t + 4], "big") for t in range(16)]
        for t in range(16, 64):
            s0 = _rotr(w[t - 15], 7) ^ _rotr(w[t - 15], 18) ^ (w[t - 15] >> 3)
            s1 = _rotr(w[t - 2], 17) ^ _rotr(w[t - 2], 19) ^ (w[t - 2] >> 10)
            w.append((w[t - 16] + s0 + w[t - 7] + s1) & M32)
        a, b, c, d, e, f, g, hh = h
        for t in range(64):
            t1 = (hh + (_rotr(e, 6) ^ _rotr(e, 11) ^ _rotr(e, 25)) + ((e & f) ^ (~e & M32 & g)) + K[t] + w[t]) & M32
            t2 = ((_rotr(a, 2) ^ _rotr(a, 13) ^ _rotr(a, 22)) + ((a & b) ^ (a & c) ^ (b & c))) & M32
            a, b, c, d, e, f, g, hh = (t1 + t2) & M32, a, b, c, (d + t1) & M32, e, f, g
        h = [(x + y) & M32 for x, y in zip(h, (a, b, c, d, e, f, g, hh))]
    return b"".join(x.to_bytes(4, "big") for x in h)


FIPS_EXAMPLES = [    # FIPS 180-4 / NIST example computations for SHA-256
    (b"abc", "ba7816bf8f01cfea414140de5dae2223b00361a396177a9cb410ff61f20015ad"),
    (b"", "e3b0c44298fc1c149afbf4c8996fb92427ae41e4649b934ca495991b7852b855"),
    (b"abcdbcdecdefdefgefghfghighijhijkijkljklmklmnlmnomnopnopq",
     "248d6a61d20638b8e5c026930c3e6039a33ce45964ff2167f6ecedd419db06c1"),
]


def test_standard_constants_and_examples():
    assert K[0] == 0x428A2F98 and K[63] == 0xC67178F2 and H0[0] == 0x6A09E667 and H0[7] == 0x5BE0CD19
    for msg, hexd in FIPS_EXAMPLES:
        assert sha256_py(msg).hex() == hexd
        assert hashlib.sha256(msg).hexdigest() == hexd


def test_library_routine_on_the_million_a_example(oracle):
    assert oracle.commitment.sha256(b"a" * 1000000).hex() == \
        "cdc76e5c9914fb9281a1c7e284d73e67f1809a48a497200e046d39ccc7112cd0"


# ------------------------------------------------------------------ the tree and the final hash

def levelwise_root(msg, leaf, H):
    """Pair neighbours level by level; an odd last node moves up unchanged."""
    level = [H(b"\x00" + msg[i:i + leaf]) for i in range(0, len(msg), leaf)] or [H(b"\x00")]
    while len(level) > 1:
        nxt = [H(b"\x01" + level[i] + level[i + 1]) for i in range(0, len(level) - 1, 2)]
        if len(level) % 2:
            nxt.append(level[-1])
        level = nxt
    return level[0]


def test_small_cases_written_out(oracle):
    C = oracle.commitment
    H = sha256_py
    assert C.LEAF == 4096
    r = bytes(range(32))
    for msg in (b"", b"x", b"q" * 4095, b"q" * 4096):
        root = H(b"\x00" + msg)
        assert C.merkle_root(msg) == root
        assert C.commit(msg, r) == H(b"\x02" + root + len(msg).to_bytes(8, "little") + r)
        assert C.commit(msg) == H(b"\x02" + root + len(msg).to_bytes(8, "little"))
    msg = bytes((7 * i + 3) & 255 for i in range(4097))
    root = H(b"\x01" + H(b"\x00" + msg[:4096]) + H(b"\x00" + msg[4096:]))
    assert C.merkle_root(msg) == root
    assert C.commit(msg, r) == H(b"\x02" + root + (4097).to_bytes(8, "little") + r)
    # three leaves: the left subtree is the complete pair, the third leaf hangs alone
    msg = bytes((5 * i + 1) & 255 for i in range(2 * 4096 + 10))
    l0, l1, l2 = (H(b"\x00" + msg[i:i + 4096]) for i in (0, 4096, 8192))
    assert C.merkle_root(msg) == H(b"\x01" + H(b"\x01" + l0 + l1) + l2)


def test_recursion_equals_levelwise_tree_for_every_leaf_count(oracle):
    C = oracle.commitment
    rng = random.Random(3)
    H = lambda b: hashlib.sha256(b).digest()
    for nleaves in range(1, 71):
        for tail in (1, 4096, rng.randrange(2, 4096)):
            msg = rng.randbytes((nleaves - 1) * 4096 + tail)
            assert len(C.chunks(msg)) == nleaves
            assert C.merkle_root(msg) == levelwise_root(msg, 4096, H)
    # the same once more without hashlib on a handful of counts
    for nleaves in (1, 2, 3, 5, 8, 9):
        msg = rng.randbytes(nleaves * 4096 - 17)
        assert C.merkle_root(msg) == levelwise_root(msg, 4096, sha256_py)


def test_separation_properties(oracle):
    C = oracle.commitment
    rng = random.Random(4)
    r = rng.randbytes(32)
    msg = rng.randbytes(3 * 4096 + 100)
    base = C.commit(msg, r)
    assert len(base) == 32
    # the length is bound: trailing zero bytes, or cutting at a leaf boundary, change c
    assert C.commit(msg + b"\x00", r) != base and C.commit(msg[:3 * 4096], r) != base
    # every leaf matters, and so does the randomness
    for pos in (0, 4095, 4096, 2 * 4096 + 7, len(msg) - 1):
        alt = bytearray(msg)
        alt[pos] ^= 1
        assert C.commit(bytes(alt), r) != base
    assert C.commit(msg, bytes(32)) != base and C.commit(msg) != base
    # an inner node's preimage is not a leaf's: 0x01 || left || right as a MESSAGE hashes differently
    left, right = C.merkle_root(msg[:4096]), C.merkle_root(msg[4096:8192])
    assert C.merkle_root(b"\x01" + left + right) != C.merkle_root(msg[:8192])
    # a root is not a commitment
    assert C.merkle_root(msg) != base
    with pytest.raises(ValueError):
        C.commit(msg, b"short")
