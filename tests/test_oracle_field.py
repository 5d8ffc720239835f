"""Pins for the oracle's field arithmetic and challenge generator (CPU only)."""
import random

import numpy as np

from bigint_defs import P

EDGE = [0, 1, 2, 2**32 - 2, 2**32 - 1, 2**32, 2**32 + 1, 2**63, 2**63 + 1, P - 2**32, P - 2, P - 1]


def test_modulus_and_identities(oracle):
    assert oracle.P == P == 0xFFFFFFFF00000001
    assert oracle.power(2, 64) == 2**32 - 1            # 2^64 = 2^32 - 1 (mod p)
    assert oracle.power(2, 96) == P - 1                # 2^96 = -1
    assert oracle.power(2, 192) == 1
    assert oracle.mul(P - 1, P - 1) == 1
    assert oracle.mul(2, 0x7FFFFFFF80000001) == 1      # inverse of two
    assert oracle.power(7, (P - 1) // 2) == P - 1      # 7 is a quadratic non-residue
    # the published 2^32-th root of unity of this field: 7^((p-1)/2^32)
    w = oracle.power(7, (P - 1) >> 32)
    assert w == 1753635133440165772
    assert oracle.power(w, 2**31) == P - 1 and oracle.power(w, 2**32) == 1


def test_edge_operands_against_python_ints(oracle):
    for x in EDGE:
        for y in EDGE:
            assert oracle.add(x, y) == (x + y) % P
            assert oracle.sub(x, y) == (x - y) % P
            assert oracle.mul(x, y) == (x * y) % P


def test_random_operands_and_fermat(oracle):
    rng = random.Random(7)
    for _ in range(2000):
        x, y = rng.randrange(P), rng.randrange(P)
        assert oracle.add(x, y) == (x + y) % P
        assert oracle.sub(x, y) == (x - y) % P
        assert oracle.mul(x, y) == (x * y) % P
    for _ in range(20):
        x = rng.randrange(1, P)
        assert oracle.power(x, P - 1) == 1
        assert oracle.mul(x, oracle.power(x, P - 2)) == 1


def test_lift(oracle):
    for v in (0, 1, 127, -1, -127, -128, 2**31 - 1, -2**31, 32385, -16129 * 4096):
        assert oracle.lift(v) == v % P


def test_splitmix64_published_outputs(oracle):
    # First three outputs of the reference SplitMix64 generator seeded with 0: state advances by
    # the golden-ratio increment, the mixer is applied to the state.
    G = 0x9E3779B97F4A7C15
    outs = [oracle.mix64((G * (i + 1)) % 2**64) for i in range(3)]
    assert outs == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert oracle.mix64(0) == 0


def test_stream_structure_and_challenge_range(oracle):
    G = 0x9E3779B97F4A7C15
    M = 2**64

    def mix(z):
        z %= M
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) % M
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) % M
        return z ^ (z >> 31)

    for seed, sid, ctr in ((1, 0, 0), (1, 0, 1), (5, 3, (3 << 32) | 2), (2**64 - 1, 2**40, 2**63)):
        key = mix(mix(seed + G) + G * (sid + 1))
        assert oracle.stream(seed, sid, ctr) == mix(key + G * (ctr + 1))
    # values derived independently with big-integer arithmetic from the definition
    assert oracle.mix64(1) == 0x5692161D100B05E5
    assert oracle.challenge(1, 0, 1, 0) == 0x0F583436CC1AB29E
    assert oracle.challenge(1, 0, 2, 0) == 0x85E63F2FB2B6C98D
    assert oracle.challenge(1, 0, 3, 0) == 0x217A22446F68AC28
    assert oracle.challenge(1, 0, 3, 1) == 0xFA1384ECCEAA4265
    seen = set()
    for pid in range(4):
        for dom in (1, 2, 3):
            for i in range(16):
                c = oracle.challenge(9, pid, dom, i)
                assert 0 <= c < P
                raw = oracle.stream(9, pid, (dom << 32) | i)
                assert c == (raw - P if raw >= P else raw)
                seen.add(c)
    assert len(seen) == 4 * 3 * 16


def test_synth_generator_matches_oracle_stream(oracle):
    import torch
    from paper_2602_22700_b200 import synth
    idx = torch.tensor([0, 1, 2, 1000, 2**33 + 5], dtype=torch.int64)
    got = synth.stream_u64(11, synth.tid(3, 1), idx).numpy().astype(np.uint64)
    want = [oracle.stream(11, synth.tid(3, 1), int(i)) for i in idx]
    assert [int(g) for g in got] == want


def test_synth_value_pins():
    # first entries derived independently from the recipe with big-integer arithmetic
    from paper_2602_22700_b200 import synth
    A = synth.uniform_i8(1, 0, 64, 64)
    assert A.view(-1)[:8].tolist() == [49, 120, -19, 78, -36, 88, 83, -54]
    assert int(A.to(int).sum()) == 14493
    assert int(A.min()) >= -127 and int(A.max()) <= 127
    assert synth.gauss_i8(1, 0, 1, 8, synth.Q_SIGMA20).view(-1).tolist() == [11, 26, -35, -11, -4, 1, 33, -22]
    assert synth.gauss_i8(1, 1, 1, 8, synth.Q_SIGMA8).view(-1).tolist() == [5, 12, 0, 2, -8, -8, 8, -8]
    g20 = synth.gauss_i8(3, 0, 512, 512, synth.Q_SIGMA20).float()
    g8 = synth.gauss_i8(3, 1, 512, 512, synth.Q_SIGMA8).float()
    assert abs(float(g20.std()) - 20.0) < 0.3 and abs(float(g20.mean())) < 0.2
    assert abs(float(g8.std()) - 8.0) < 0.15 and abs(float(g8.mean())) < 0.1
