"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared
symbol, and its host entry points (challenge generator, verifier, planners, argument
validation) agree with the oracle."""
import ctypes
import os
import random
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def imm():
    from paper_2602_22700_b200 import build, imm as binding
    build.build()
    return binding


def test_library_exports_every_declared_symbol(imm):
    header = open(os.path.join(ROOT, "include", "imm.h")).read()
    declared = set(re.findall(r"\b(imm_[a-z0-9_]+)\s*\(", header))
    declared -= {"imm_matmul_desc"}
    assert declared == set(imm.EXPORTS)
    L = imm.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert imm.version() >= 100


def test_challenges_match_oracle(imm, oracle):
    rng = random.Random(1)
    for _ in range(200):
        seed, pid = rng.getrandbits(64), rng.getrandbits(64)
        dom, idx = rng.choice((1, 2, 3, 4)), rng.randrange(0, 40)
        assert imm.challenge(seed, pid, dom, idx) == oracle.challenge(seed, pid, dom, idx)
    assert imm.challenge(1, 0, 1, 0) == 0x0F583436CC1AB29E


def test_host_verifier_matches_oracle_verifier(imm, oracle):
    rng = random.Random(2)
    for (m, k, n) in ((3, 8, 2), (2, 5, 4), (4, 1, 4), (1, 16, 1)):
        A = np.array([[rng.randint(-128, 127) for _ in range(k)] for _ in range(m)], dtype=np.int8)
        B = np.array([[rng.randint(-128, 127) for _ in range(n)] for _ in range(k)], dtype=np.int8)
        C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
        seed, pid = rng.getrandbits(64), rng.getrandbits(20)
        t = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, seed, pid)]
        b = oracle.ceil_log2(k)
        assert imm.sumcheck_verify(t, b, seed, pid) == (imm.OK, -1)
        assert imm.sumcheck_verify(t, b, seed, pid, t[0], t[-2], t[-1]) == (imm.OK, -1)
        for pos in range(len(t)):
            bad = list(t)
            bad[pos] = (bad[pos] + 1 + rng.randrange(oracle.P - 1)) % oracle.P
            assert imm.sumcheck_verify(bad, b, seed, pid) == oracle.sumcheck_verify(bad, b, seed, pid)
            assert imm.sumcheck_verify(bad, b, seed, pid)[0] == imm.REJECT
        for which in range(3):
            exp = [t[0], t[-2], t[-1]]
            exp[which] = (exp[which] + 1) % oracle.P
            assert imm.sumcheck_verify(t, b, seed, pid, *exp) == oracle.sumcheck_verify(t, b, seed, pid, *exp)
            assert imm.sumcheck_verify(t, b, seed, pid, *exp) == (imm.REJECT, b + 1 + which)
        assert imm.sumcheck_verify(t, b, seed + 1, pid)[0] == (imm.REJECT if b > 0 else imm.OK)
    with pytest.raises(imm.ImmError):
        imm.sumcheck_verify([oracle.P, 0, 0], 0, 1, 0)


def test_batched_host_verifier_matches_oracle_verifier(imm, oracle):
    rng = random.Random(3)
    for shapes in ([(3, 8, 2), (2, 5, 4), (1, 7, 1)], [(2, 1, 2), (1, 1, 3)], [(4, 16, 4)], [(2, 3, 2), (1, 9, 1)]):
        probs = []
        for i, (m, k, n) in enumerate(shapes):
            A = np.array([[rng.randint(-128, 127) for _ in range(k)] for _ in range(m)], dtype=np.int8)
            B = np.array([[rng.randint(-128, 127) for _ in range(n)] for _ in range(k)], dtype=np.int8)
            probs.append((A, B, (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32), 100 + i))
        seed, bid, count = rng.getrandbits(64), rng.getrandbits(30), len(shapes)
        b = max(oracle.ceil_log2(k) for (_, k, _) in shapes)
        t = [int(w) for w in oracle.sumcheck_matmul_prove_batched(probs, seed, bid)]
        assert len(t) == imm.batched_transcript_len(b, count)
        assert imm.sumcheck_verify_batched(t, b, count, seed, bid) == (imm.OK, -1)
        assert imm.sumcheck_verify_batched(t, b, count, seed, bid, t[-3 * count:]) == (imm.OK, -1)
        for pos in range(len(t)):
            bad = list(t)
            bad[pos] = (bad[pos] + 1 + rng.randrange(oracle.P - 1)) % oracle.P
            got = imm.sumcheck_verify_batched(bad, b, count, seed, bid)
            assert got == oracle.sumcheck_verify_batched(bad, b, count, seed, bid) and got[0] == imm.REJECT
        for pos in range(3 * count):
            exp = t[-3 * count:]
            exp[pos] = (exp[pos] + 1) % oracle.P
            got = imm.sumcheck_verify_batched(t, b, count, seed, bid, exp)
            assert got == oracle.sumcheck_verify_batched(t, b, count, seed, bid, exp) == (imm.REJECT, b + 2 + pos)
        assert imm.sumcheck_verify_batched(t, b, count, seed, bid + 1) == (imm.REJECT, b + 1)
    with pytest.raises(imm.ImmError):
        imm.sumcheck_verify_batched([oracle.P, 0, 0, 0], 0, 1, 1, 0)
    assert imm.batched_transcript_len(12, 96) == 1 + 36 + 288
    assert imm.batched_transcript_len(-1, 4) == 0 and imm.batched_transcript_len(3, 0) == 0


def test_fs_host_challenges_and_verifier_match_oracle(imm, oracle):
    rng = random.Random(4)
    for (m, k, n) in ((3, 8, 2), (2, 5, 4), (4, 1, 4), (1, 16, 1), (5, 33, 7)):
        A = np.array([[rng.randint(-128, 127) for _ in range(k)] for _ in range(m)], dtype=np.int8)
        B = np.array([[rng.randint(-128, 127) for _ in range(n)] for _ in range(k)], dtype=np.int8)
        C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
        coms, pid = [rng.randbytes(32) for _ in range(3)], rng.getrandbits(64)
        com96 = b"".join(coms)
        t = oracle.fs.prove(A, B, C, coms, pid)
        b = oracle.ceil_log2(k)
        want = oracle.fs.challenges(t, b, coms, m, k, n, pid)
        assert imm.fs_challenges(t, b, com96, m, k, n, pid) == tuple(want)
        assert imm.fs_challenges(None, b, com96, m, k, n, pid)[:2] == (want[0], want[1])
        assert imm.sumcheck_verify_fs(t, b, com96, m, k, n, pid) == (imm.OK, -1)
        assert imm.sumcheck_verify_fs(t, b, com96, m, k, n, pid, t[0], t[-2], t[-1]) == (imm.OK, -1)
        for pos in range(len(t)):
            bad = list(t)
            bad[pos] = (bad[pos] + 1 + rng.randrange(oracle.P - 1)) % oracle.P
            got = imm.sumcheck_verify_fs(bad, b, com96, m, k, n, pid)
            assert got == oracle.fs.verify(bad, b, coms, m, k, n, pid) and got[0] == imm.REJECT
        flipped = bytes([com96[40] ^ 4]) .join([com96[:40], com96[41:]])
        assert imm.sumcheck_verify_fs(t, b, flipped, m, k, n, pid)[0] == (imm.REJECT if b > 0 else imm.OK)
        assert imm.sumcheck_verify_fs(t, b, com96, m, k, n, pid, None, (t[-2] + 1) % oracle.P) == (imm.REJECT, b + 2)
        with pytest.raises(imm.ImmError):
            imm.sumcheck_verify_fs(t, b + 1, com96, m, k, n, pid)            # nrounds must be ceil(log2 k)
    with pytest.raises(imm.ImmError):
        imm.sumcheck_verify_fs([oracle.P, 0, 0], 0, bytes(96), 1, 1, 1, 0)


def test_fs_batched_host_coins_and_verifier_match_oracle(imm, oracle):
    rng = random.Random(5)
    for shapes in ([(3, 8, 2), (2, 5, 4), (1, 7, 1)], [(2, 1, 2), (1, 1, 3)], [(4, 16, 4)],
                   [(2, 3, 2), (1, 9, 1), (3, 2, 2), (2, 2, 2), (1, 1, 1)]):
        probs, meta = [], []
        for i, (m, k, n) in enumerate(shapes):
            A = np.array([[rng.randint(-128, 127) for _ in range(k)] for _ in range(m)], dtype=np.int8)
            B = np.array([[rng.randint(-128, 127) for _ in range(n)] for _ in range(k)], dtype=np.int8)
            C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
            coms, pid = [rng.randbytes(32) for _ in range(3)], rng.getrandbits(40)
            probs.append((A, B, C, coms, pid))
            meta.append((m, k, n, pid))
        bid, count = rng.getrandbits(64), len(shapes)
        b = max(oracle.ceil_log2(k) for (_, k, _) in shapes)
        t = oracle.fs.prove_batched(probs, bid)
        com = b"".join(b"".join(c) for (_, _, _, c, _) in probs)
        stmts = [oracle.fs.statement(c, m, k, n, pid) for (_, _, _, c, _), (m, k, n, pid) in zip(probs, meta)]
        want = oracle.fs.challenges_batched(t, b, stmts, bid)
        assert imm.fs_batched_challenges(t, b, meta, com, bid) == tuple(want)
        assert imm.sumcheck_verify_fs_batched(t, b, meta, com, bid) == (imm.OK, -1)
        assert imm.sumcheck_verify_fs_batched(t, b, meta, com, bid, t[-3 * count:]) == (imm.OK, -1)
        for pos in range(len(t)):
            bad = list(t)
            bad[pos] = (bad[pos] + 1 + rng.randrange(oracle.P - 1)) % oracle.P
            got = imm.sumcheck_verify_fs_batched(bad, b, meta, com, bid)
            assert got == oracle.fs.verify_batched(bad, b, stmts, bid)
            if got[0] != imm.REJECT:
                # only a factor whose partner is zero can change unnoticed by the rounds (the verifier's
                # own evaluations catch it): a_fin_p next to b_fin_p = 0, or the other way round
                off = pos - (1 + 3 * b)
                assert off >= 0 and off % 3 in (1, 2) and t[pos + (1 if off % 3 == 1 else -1)] == 0
        assert imm.sumcheck_verify_fs_batched(t, b, meta, com, bid + 1)[0] == imm.REJECT
        swapped = bytes([com[5] ^ 1]).join([com[:5], com[6:]])
        assert imm.sumcheck_verify_fs_batched(t, b, meta, swapped, bid)[0] == imm.REJECT
        with pytest.raises(imm.ImmError):
            imm.sumcheck_verify_fs_batched(t + [0] * 3, b + 1, meta, com, bid)       # nrounds is the largest ceil(log2 k)
    L = imm.lib()
    big = _desc_array(imm, [(2, 4, 2)] * 1025)
    assert L.imm_sumcheck_matmul_fs_batched_workspace(ctypes.addressof(big), 1025) == 0
    assert L.imm_sumcheck_matmul_prove_fs_batched(ctypes.addressof(big), 1025, 0x1000, 1, 0x1000, 0x1000, 0x1000,
                                                  1 << 30, None) == imm.ERR_LIMIT


def _desc_array(imm, shapes, base=0x10000):
    arr = (imm.MatmulDesc * len(shapes))()
    for i, (m, k, n) in enumerate(shapes):
        arr[i] = imm.MatmulDesc(base, base, base, m, k, n, k, n, n, i)
    return arr


def test_workspace_planner(imm):
    L = imm.lib()
    d = _desc_array(imm, [(64, 64, 64)])
    w1 = L.imm_sumcheck_matmul_workspace(ctypes.addressof(d), 1)
    assert w1 > 0 and w1 % 256 == 0
    d2 = _desc_array(imm, [(64, 64, 64), (512, 4096, 4096)])
    w2 = L.imm_sumcheck_matmul_workspace(ctypes.addressof(d2), 2)
    assert w2 > w1
    # eq tables + tables of the rounds are the floor
    assert w2 >= 8 * (512 + 4096 + 2 * 4096)
    for bad in ([(0, 4, 4)], [(4, 0, 4)], [(4, 4, 0)], [(4, (1 << 17) + 1, 4)], [((1 << 20) + 1, 4, 4)]):
        db = _desc_array(imm, bad)
        assert L.imm_sumcheck_matmul_workspace(ctypes.addressof(db), 1) == 0
    assert L.imm_sumcheck_matmul_workspace(None, 1) == 0
    assert L.imm_sumcheck_matmul_host_arena(ctypes.addressof(d2), 2) > w2 + 512 * 4096 + 4096 * 4096
    assert L.imm_mle_workspace(0, 100, 100, 0) > 0 and L.imm_mle_workspace(2, 100, 100, 0) == 0
    assert L.imm_mle_workspace(1, 0, 100, 1) == 0


def test_batched_workspace_and_validation(imm):
    L = imm.lib()
    d = _desc_array(imm, [(64, 4096, 64), (512, 3000, 4096)])         # both k pad to 2^12
    plain = L.imm_sumcheck_matmul_workspace(ctypes.addressof(d), 2)
    need = L.imm_sumcheck_matmul_batched_workspace(ctypes.addressof(d), 2)
    assert need >= plain + 2 * 39 * 8 and need % 256 == 0
    mixed = _desc_array(imm, [(64, 4096, 64), (64, 2048, 64)])                  # padded to twelve rounds each
    assert L.imm_sumcheck_matmul_batched_workspace(ctypes.addressof(mixed), 2) >= 2 * 39 * 8
    prove = L.imm_sumcheck_matmul_prove_batched
    assert prove(ctypes.addressof(d), 2, 1, 1, 0x1000, 0x1000, 0x1000, need - 1, None) == imm.ERR_WORKSPACE
    assert prove(ctypes.addressof(d), 2, 1, 1, 0x1000, 0x1000, 0x1010, need, None) == imm.ERR_ALIGN
    assert prove(ctypes.addressof(d), 2, 1, 1, None, 0x1000, 0x1000, need, None) == imm.ERR_ARG
    assert prove(ctypes.addressof(d), 0, 1, 1, 0x1000, 0x1000, 0x1000, need, None) == imm.ERR_ARG


def test_fs_and_commit_workspace_and_validation(imm):
    L = imm.lib()
    d = _desc_array(imm, [(64, 4096, 64), (512, 3000, 4096)])
    plain = L.imm_sumcheck_matmul_workspace(ctypes.addressof(d), 2)
    need = L.imm_sumcheck_matmul_fs_workspace(ctypes.addressof(d), 2)
    assert need >= plain + 2 * 2 * 4096 * 8 and need % 256 == 0             # two tables of 2^12 entries per proof
    prove = L.imm_sumcheck_matmul_prove_fs
    assert prove(ctypes.addressof(d), 2, None, 0x1000, 39, 0x1000, 0x1000, need, None) == imm.ERR_ARG
    assert prove(ctypes.addressof(d), 2, 0x1000, 0x1000, 39, 0x1000, 0x1000, need - 1, None) == imm.ERR_WORKSPACE
    assert prove(ctypes.addressof(d), 2, 0x1000, 0x1000, 38, 0x1000, 0x1000, need, None) == imm.ERR_SHAPE
    assert prove(ctypes.addressof(d), 2, 0x1000, 0x1000, 39, 0x1000, 0x1010, need, None) == imm.ERR_ALIGN
    c = (imm.CommitDesc * 2)()
    c[0].msg, c[0].nbytes = 0x1000, 5 << 20
    c[1].msg, c[1].nbytes, c[1].r_len = None, 0, 32
    w = L.imm_commit_workspace(ctypes.addressof(c), 2)
    assert w > 0 and w % 256 == 0 and w >= (10 + 1 + 1 + 1) * 32             # subtree roots of both, then the big one's root
    assert L.imm_commit_launches(ctypes.addressof(c), 2) == 3                # leaves, one node pass, final hashes
    assert L.imm_commit(ctypes.addressof(c), 2, 0x1000, None, 0x1000, w - 1, None) == imm.ERR_WORKSPACE
    assert L.imm_commit(ctypes.addressof(c), 2, None, None, 0x1000, w, None) == imm.ERR_ARG
    assert L.imm_commit(ctypes.addressof(c), 2, 0x1000, None, 0x1010, w, None) == imm.ERR_ALIGN
    c[1].r_len = 16
    assert L.imm_commit_workspace(ctypes.addressof(c), 2) == 0
    c[1].r_len, c[1].nbytes = 0, 100                                         # bytes without a pointer
    assert L.imm_commit_workspace(ctypes.addressof(c), 2) == 0
    c[1].nbytes, c[0].nbytes = 0, (1 << 40) + 1
    assert L.imm_commit(ctypes.addressof(c), 2, 0x1000, None, 0x1000, 1 << 30, None) == imm.ERR_LIMIT


def test_verifier_pass_workspace_and_validation(imm):
    L = imm.lib()
    d = _desc_array(imm, [(64, 4096, 64), (512, 3000, 4096), (8, 100, 8)])
    plain = L.imm_sumcheck_matmul_workspace(ctypes.addressof(d), 3)
    each = L.imm_sumcheck_expected_workspace(ctypes.addressof(d), 3, 0)
    shared = L.imm_sumcheck_expected_workspace(ctypes.addressof(d), 3, 1)
    assert each >= plain + 8 * (4096 + 4096 + 128) and each % 256 == 0      # one E_k table per proof
    assert shared >= plain + 8 * 3 * 4096 and shared > each                     # every table at the largest size
    assert L.imm_sumcheck_expected_workspace(None, 3, 0) == 0
    call = L.imm_sumcheck_expected
    assert call(ctypes.addressof(d), 3, 1, None, None, None, 0x1000, 0x1000, each, None) == imm.ERR_ARG
    assert call(ctypes.addressof(d), 3, 1, None, None, 0x1000, 0x1000, 0x1000, each - 1, None) == imm.ERR_WORKSPACE
    assert call(ctypes.addressof(d), 3, 1, None, None, 0x1000, 0x1000, 0x1010, each, None) == imm.ERR_ALIGN
    pts = (ctypes.c_uint64 * (96 * 3))()
    pts[100] = imm.P
    assert call(ctypes.addressof(d), 3, 1, None, ctypes.addressof(pts), 0x1000, 0x1000, 0x1000, each, None) == imm.ERR_NONCANONICAL
    bid = ctypes.c_uint64(5)
    assert call(ctypes.addressof(d), 3, 1, ctypes.addressof(bid), None, 0x1000, 0x1000, 0x1000, each, None) == imm.ERR_WORKSPACE


def test_argument_validation_happens_before_any_device_work(imm):
    L = imm.lib()
    r = (ctypes.c_uint64 * 4)(1, 2, 3, imm.P)
    assert L.imm_eq_table(ctypes.addressof(r), 21, 0x1000, None) == -2
    assert L.imm_eq_table(ctypes.addressof(r), 4, None, None) == -1
    assert L.imm_eq_table(ctypes.addressof(r), 4, 0x1008, None) == -3
    assert L.imm_eq_table(ctypes.addressof(r), 4, 0x1000, None) == -5
    assert L.imm_field_binop(7, 0x1000, 0x1000, 0x1000, 4, None) == -1
    assert L.imm_field_binop(0, None, None, None, 0, None) == 0
    assert L.imm_mle_partial_eval(0x1000, 0, 4, 8, 7, 0, 0x1000, 0x1000, 0x1000, 1 << 20, None) == -2
    assert L.imm_mle_partial_eval(0x1000, 5, 4, 8, 8, 0, 0x1000, 0x1000, 0x1000, 1 << 20, None) == -1
    assert L.imm_mle_partial_eval(0x1000, 0, 4, 8, 8, 0, 0x1000, 0x1000, 0x1000, 8, None) == -4
    assert L.imm_mle_eval_point(0x1000, 1, 4, 8, 8, 0x1000, 0x1000, 0x1000, 0x1004, 1 << 20, None) == -3
    d = _desc_array(imm, [(4, 8, 4)])
    assert L.imm_sumcheck_matmul_prove(ctypes.addressof(d), 1, 1, 0x1000, 11, 0x1000, 0x1000, 1 << 30, None) == -2
    assert L.imm_sumcheck_matmul_prove(ctypes.addressof(d), 1, 1, 0x1000, 12, 0x1000, 0x1000, 16, None) == -4
    assert L.imm_sumcheck_matmul_prove(ctypes.addressof(d), 0, 1, 0x1000, 12, 0x1000, 0x1000, 1 << 30, None) == -1
    d.__getitem__(0).lda = 7
    assert L.imm_sumcheck_matmul_prove(ctypes.addressof(d), 1, 1, 0x1000, 12, 0x1000, 0x1000, 1 << 30, None) == -2


def test_binding_refuses_cpu_tensors(imm):
    import torch
    A = torch.zeros((4, 4), dtype=torch.int8)
    with pytest.raises(ValueError):
        imm.make_descs([(A, A, A.to(torch.int32), 0)])
    with pytest.raises(ValueError):
        imm.mle_partial_eval(A, imm.BIND_ROWS, torch.zeros(4, dtype=torch.int64))


def test_launch_count_of_a_proving_pass(imm, monkeypatch):
    """Three launches where the batch takes the fused contraction launch (under 4 GiB, or under 16 GiB
    with proofs of 32 MiB or more on average), five otherwise; the integer-pipe back end always takes
    five; 0 on invalid input."""
    L = imm.lib()
    small = _desc_array(imm, [(512, 4096, 4096)])
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(small), 1) == 3
    experts = _desc_array(imm, [(8192, 4096, 14336)] * 8)                     # 4.5 GB, 562 MB per proof
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(experts), 8) == 3
    big = _desc_array(imm, [(8192, 4096, 14336)] * 40)                        # 22 GB
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(big), 40) == 5
    heads = _desc_array(imm, [(2048, 128, 2048)] * 300)                       # 5.2 GB of 17 MB proofs
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(heads), 300) == 5
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(heads), 160) == 3  # 2.8 GB: small enough whatever the proofs
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(big), 0) == 0
    assert L.imm_sumcheck_matmul_launches(None, 1) == 0
    monkeypatch.setenv("IMM_CONTRACT", "alu")
    assert L.imm_sumcheck_matmul_launches(ctypes.addressof(small), 1) == 5
