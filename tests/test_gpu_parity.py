"""GPU parity: every C-ABI device call against the CPU oracle, bit for bit (run with -m gpu)."""
import os
import random

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

P = 0xFFFFFFFF00000001
GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


@pytest.fixture(scope="module")
def imm():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2602_22700_b200 import imm as binding
    binding.lib()
    return binding


@pytest.fixture(params=["mma", "alu"])
def backend(request, monkeypatch):
    """Runs a prover test once per contraction back end (tensor-core limbs / integer pipe)."""
    monkeypatch.setenv("IMM_CONTRACT", request.param)
    return request.param


def u64_to_dev(vals):
    return torch.from_numpy(np.asarray(vals, dtype=np.uint64).view(np.int64)).cuda()


def dev_to_ints(t):
    return [int(v) for v in t.cpu().numpy().view(np.uint64)]


def rand_mat(rng, rows, cols, dtype, ld=None, offset=0, full_range=True):
    """numpy matrix view with leading dimension ld, starting `offset` elements into its buffer."""
    ld = ld or cols
    if dtype == np.int8:
        lo, hi = (-128, 127) if full_range else (-127, 127)
    else:
        lo, hi = -2**31, 2**31 - 1
    buf = rng.integers(lo, hi, size=rows * ld + offset, endpoint=True, dtype=np.int64).astype(dtype)
    return buf, buf[offset:offset + rows * ld].reshape(rows, ld)[:, :cols]


def to_dev_view(buf, rows, cols, ld, offset):
    d = torch.from_numpy(buf).cuda()
    return d[offset:offset + rows * ld].view(rows, ld)[:, :cols]


# ------------------------------------------------------------------ field arithmetic


def test_field_arithmetic_edge_and_random(imm):
    edge = [0, 1, 2, 2**32 - 2, 2**32 - 1, 2**32, 2**32 + 1, 2**63 - 1, 2**63, 2**63 + 1,
            0x7FFFFFFF7FFFFFFF, 0x7FFFFFFF80000000, P - 2**32, P - 2**32 - 1, P - 2, P - 1]
    xs = [x for x in edge for _ in edge]
    ys = [y for _ in edge for y in edge]
    rng = random.Random(5)
    for _ in range(200000):
        xs.append(rng.randrange(P)); ys.append(rng.randrange(P))
    # products whose high half stresses the borrow / carry corners of the reduction
    for _ in range(2000):
        xs.append(P - 1 - rng.randrange(1 << 33)); ys.append(P - 1 - rng.randrange(1 << 33))
        xs.append((rng.randrange(1 << 32) << 32) | 0xFFFFFFFF); ys.append(rng.randrange(1 << 32) << 32)
    xs = [x % P for x in xs]; ys = [y % P for y in ys]
    dx, dy = u64_to_dev(xs), u64_to_dev(ys)
    for op, fn in ((imm.FIELD_ADD, lambda a, b: (a + b) % P), (imm.FIELD_SUB, lambda a, b: (a - b) % P),
                   (imm.FIELD_MUL, lambda a, b: (a * b) % P)):
        got = dev_to_ints(imm.field_binop(op, dx, dy))
        want = [fn(a, b) for a, b in zip(xs, ys)]
        assert got == want


def test_field_arithmetic_matches_oracle_calls(imm, oracle):
    rng = random.Random(6)
    xs = [rng.randrange(P) for _ in range(3000)]
    ys = [rng.randrange(P) for _ in range(3000)]
    dx, dy = u64_to_dev(xs), u64_to_dev(ys)
    assert dev_to_ints(imm.field_binop(imm.FIELD_MUL, dx, dy)) == [oracle.mul(a, b) for a, b in zip(xs, ys)]
    assert dev_to_ints(imm.field_binop(imm.FIELD_ADD, dx, dy)) == [oracle.add(a, b) for a, b in zip(xs, ys)]
    assert dev_to_ints(imm.field_binop(imm.FIELD_SUB, dx, dy)) == [oracle.sub(a, b) for a, b in zip(xs, ys)]


# ------------------------------------------------------------------ eq tables


@pytest.mark.parametrize("nvars", [0, 1, 2, 3, 5, 8, 10, 11, 14, 17])
def test_eq_table(imm, oracle, nvars):
    rng = random.Random(nvars)
    r = [rng.randrange(P) for _ in range(nvars)]
    got = imm.eq_table(r).cpu().numpy().view(np.uint64)
    want = oracle.eq_table(r)
    assert got.shape == want.shape and (got == want).all()


def test_eq_table_boolean_and_edge_challenges(imm, oracle):
    for r in ([0, 1, 1, 0, 1], [P - 1, 1, 0, P - 1], [1] * 6, [0] * 7):
        got = imm.eq_table(r).cpu().numpy().view(np.uint64)
        assert (got == oracle.eq_table(r)).all()


# ------------------------------------------------------------------ partial evaluation / point evaluation

MAT_CASES = [
    # rows, cols, ld, offset
    (1, 1, None, 0), (1, 37, None, 0), (33, 1, None, 0), (5, 16, None, 0), (64, 64, None, 0),
    (7, 100, 112, 0), (130, 2049, 2064, 0), (70, 300, 300, 0), (40, 515, 528, 16),
    (9, 50, 67, 3), (300, 4100, 4112, 0), (1100, 600, 608, 0), (2100, 96, 96, 0),
]


@pytest.mark.parametrize("np_dtype", [np.int8, np.int32])
@pytest.mark.parametrize("rows,cols,ld,offset", MAT_CASES)
def test_partial_eval_and_point_eval(imm, oracle, np_dtype, rows, cols, ld, offset):
    rng = np.random.default_rng(rows * 131 + cols)
    prng = random.Random(rows * 7 + cols)
    ld = ld or cols
    buf, M = rand_mat(rng, rows, cols, np_dtype, ld, offset)
    dM = to_dev_view(buf, rows, cols, ld, offset)
    a, c = oracle.ceil_log2(rows), oracle.ceil_log2(cols)
    Er = oracle.eq_table([prng.randrange(P) for _ in range(a)])
    Ec = oracle.eq_table([prng.randrange(P) for _ in range(c)])
    dEr, dEc = u64_to_dev(Er), u64_to_dev(Ec)
    got_r = imm.mle_partial_eval(dM, imm.BIND_ROWS, dEr).cpu().numpy().view(np.uint64)
    assert (got_r == oracle.mle_partial_eval(M, oracle.BIND_ROWS, Er)).all()
    got_c = imm.mle_partial_eval(dM, imm.BIND_COLS, dEc).cpu().numpy().view(np.uint64)
    assert (got_c == oracle.mle_partial_eval(M, oracle.BIND_COLS, Ec)).all()
    got_p = dev_to_ints(imm.mle_eval_point(dM, dEr, dEc))[0]
    assert got_p == oracle.mle_eval_point(M, Er, Ec)


def test_partial_eval_extreme_values(imm, oracle):
    """All entries at the extremes with extreme eq weights: the lazy accumulators' worst case."""
    for np_dtype, lo, hi in ((np.int8, -128, 127), (np.int32, -2**31, 2**31 - 1)):
        for val in (lo, hi):
            rows, cols = 1024, 160
            M = np.full((rows, cols), val, dtype=np_dtype)
            for w in (P - 1, 0x7FFFFFFF7FFFFFFF, 0x7FFFFFFF80000000, 0xFFFFFFFF, 0x80000000, 0xFFFFFFFE00000000):
                Er = np.full(rows, w, dtype=np.uint64)
                Ec = np.full(256, w, dtype=np.uint64)
                dM = torch.from_numpy(M).cuda()
                got = imm.mle_partial_eval(dM, imm.BIND_ROWS, u64_to_dev(Er)).cpu().numpy().view(np.uint64)
                assert (got == oracle.mle_partial_eval(M, oracle.BIND_ROWS, Er)).all()
                got = imm.mle_partial_eval(dM, imm.BIND_COLS, u64_to_dev(Ec)).cpu().numpy().view(np.uint64)
                assert (got == oracle.mle_partial_eval(M, oracle.BIND_COLS, Ec)).all()
                assert dev_to_ints(imm.mle_eval_point(dM, u64_to_dev(Er), u64_to_dev(Ec)))[0] == \
                    oracle.mle_eval_point(M, Er, Ec)


# ------------------------------------------------------------------ prover


def np_problem(rng, m, k, n, tamper=None):
    A = rng.integers(-128, 127, size=(m, k), endpoint=True, dtype=np.int64).astype(np.int8)
    B = rng.integers(-128, 127, size=(k, n), endpoint=True, dtype=np.int64).astype(np.int8)
    C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
    return A, B, C


def gpu_prove(imm, probs, seed):
    dev = [(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C).cuda(), pid)
           for (A, B, C, pid) in probs]
    return imm.sumcheck_matmul_prove(dev, seed)


def read_golden(name):
    with open(os.path.join(GOLD, name + ".txt")) as f:
        return [int(line, 16) for line in f if line.strip() and not line.startswith("#")]


def test_golden_transcripts(imm, backend):
    from paper_2602_22700_b200 import synth
    A = np.array([[1, -2, 3, -4], [5, 6, -7, 8]], dtype=np.int8)
    B = np.array([[1, 2], [-3, 4], [5, -6], [7, 8]], dtype=np.int8)
    C = np.array([[-6, -56], [8, 140]], dtype=np.int32)
    assert gpu_prove(imm, [(A, B, C, 0)], 1)[0] == read_golden("example_2x4x2")
    p = synth.single_small(1, 64, 64, 64, device="cuda")[0]
    assert imm.sumcheck_matmul_prove([(p.A, p.B, p.C, 0)], 1)[0] == read_golden("uniform_64x64x64")
    p = synth.qkv_projection(1, 24, 100, 72, device="cuda")[0]
    assert imm.sumcheck_matmul_prove([(p.A, p.B, p.C, 3)], 5)[0] == read_golden("gauss_24x100x72")


SHAPES = [(1, 1, 1), (1, 2, 1), (3, 1, 5), (2, 4, 2), (1, 8, 1), (5, 3, 7), (17, 33, 9), (64, 64, 64),
          (100, 257, 50), (33, 2048, 40), (40, 2049, 33), (130, 700, 515), (1030, 96, 2050),
          (300, 1100, 4100), (31, 1025, 1030), (1056, 130, 65), (65, 4200, 1000)]


@pytest.mark.parametrize("m,k,n", SHAPES)
def test_prove_single_matches_oracle(imm, oracle, backend, m, k, n):
    rng = np.random.default_rng(m * 10007 + k * 101 + n)
    A, B, C = np_problem(rng, m, k, n)
    seed, pid = 1000 + m, k
    got = gpu_prove(imm, [(A, B, C, pid)], seed)[0]
    want = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, seed, pid)]
    assert got == want
    b = oracle.ceil_log2(k)
    assert imm.sumcheck_verify(got, b, seed, pid) == (imm.OK, -1)


@pytest.mark.parametrize("m,k,n", [(4, 20000, 5), (3, 40000, 2), (2, 70000, 3), (2, 131072, 2)])
def test_prove_many_rounds(imm, oracle, m, k, n):
    """15 to 17 rounds: the round kernel spreads one proof over the blocks of a cluster (16 blocks,
    an opt-in cluster size, from 2^16 < k on)."""
    rng = np.random.default_rng(k)
    A, B, C = np_problem(rng, m, k, n)
    got = gpu_prove(imm, [(A, B, C, 7)], 11)[0]
    assert got == [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 11, 7)]
    assert imm.sumcheck_verify(got, oracle.ceil_log2(k), 11, 7) == (imm.OK, -1)


@pytest.mark.parametrize("cluster", ["1", "2", "4", "8"])
def test_round_kernel_cluster_sizes_give_the_same_words(imm, oracle, monkeypatch, cluster):
    """A batch mixing short proofs (one block each) and long ones, for every cluster size."""
    monkeypatch.setenv("IMM_SC_CLUSTER", cluster)
    rng = np.random.default_rng(91)
    shapes = [(5, 5000, 7), (3, 8, 2), (9, 2049, 4), (2, 1024, 3), (6, 8192, 2), (1, 1, 1), (4, 1025, 33)]
    probs = [np_problem(rng, *s) + (20 + i,) for i, s in enumerate(shapes)]
    got = gpu_prove(imm, probs, 17)
    for (A, B, C, pid), t in zip(probs, got):
        assert t == [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 17, pid)]


def test_prove_unaligned_leading_dimensions(imm, oracle, backend):
    """Rows that are not 16-byte aligned take the element-wise loads; same transcript."""
    rng = np.random.default_rng(78)
    m, k, n = 70, 333, 130
    A, B, C = np_problem(rng, m, k, n)
    want = [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 5, 9)]

    def odd_view(M, ld, off):
        buf = torch.zeros(M.shape[0] * ld + off + 8, dtype=torch.from_numpy(M).dtype, device="cuda")
        v = buf[off:off + M.shape[0] * ld].view(M.shape[0], ld)[:, :M.shape[1]]
        v.copy_(torch.from_numpy(M).cuda())
        return v

    dA, dB, dC = odd_view(A, k + 3, 1), odd_view(B, n + 5, 3), odd_view(C, n + 1, 1)
    assert imm.sumcheck_matmul_prove([(dA, dB, dC, 9)], 5)[0] == want


def test_prove_ragged_batch_matches_oracle(imm, oracle, backend):
    rng = np.random.default_rng(77)
    shapes = [(37, 300, 41), (1, 1, 1), (250, 64, 513), (64, 1000, 64), (5, 4097, 3), (129, 2, 2049)]
    probs = [np_problem(rng, *s) + (10 + i,) for i, s in enumerate(shapes)]
    got = gpu_prove(imm, probs, 99)
    for (A, B, C, pid), t in zip(probs, got):
        assert t == [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 99, pid)]
    # the same proofs one by one (different tile geometry) give the same words
    for prob, t in zip(probs, got):
        assert gpu_prove(imm, [prob], 99)[0] == t


def test_transcript_rows_are_zero_padded_and_status_ok(imm, backend):
    rng = np.random.default_rng(5)
    probs = [np_problem(rng, 4, 2, 4) + (0,), np_problem(rng, 4, 64, 4) + (1,)]
    dev = [(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C).cuda(), pid)
           for (A, B, C, pid) in probs]
    pr = imm.Prover(dev)
    pr.transcripts.fill_(-1)
    pr.prove(3)
    torch.cuda.synchronize()
    assert pr.stride == 21 and pr.lengths() == [6, 21]
    assert (pr.transcripts[0, 6:] == 0).all() and (pr.status == 0).all()
    # a second pass with the same buffers reproduces the transcripts exactly
    first = pr.transcripts.clone()
    pr.prove(3)
    torch.cuda.synchronize()
    assert (pr.transcripts == first).all()


def test_tampering_is_rejected(imm, oracle, backend):
    rng = np.random.default_rng(21)
    A, B, C = np_problem(rng, 48, 200, 36)
    seed, pid, b = 4, 2, 8
    good = gpu_prove(imm, [(A, B, C, pid)], seed)[0]
    assert imm.sumcheck_verify(good, b, seed, pid) == (imm.OK, -1)
    C2 = C.copy(); C2[11, 7] += 1
    bad = gpu_prove(imm, [(A, B, C2, pid)], seed)[0]
    assert bad == [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C2, seed, pid)]
    assert imm.sumcheck_verify(bad, b, seed, pid) == (imm.REJECT, 0)
    for delta in (1, -1):
        B2 = B.copy()
        B2[150, 20] = np.int8(max(-128, min(127, int(B2[150, 20]) + delta)) if abs(int(B2[150, 20])) < 127 else int(B2[150, 20]) - delta)
        assert (B2 != B).sum() == 1
        bad = gpu_prove(imm, [(A, B2, C, pid)], seed)[0]
        assert imm.sumcheck_verify(bad, b, seed, pid) == (imm.REJECT, 0)
        # a prover consistent with the altered weight passes the rounds but not the verifier's own B~
        C3 = (A.astype(np.int64) @ B2.astype(np.int64)).astype(np.int32)
        sneaky = gpu_prove(imm, [(A, B2, C3, pid)], seed)[0]
        assert imm.sumcheck_verify(sneaky, b, seed, pid) == (imm.OK, -1)
        r_k = imm.challenges(seed, pid, 3, b)
        r_col = imm.challenges(seed, pid, 2, oracle.ceil_log2(36))
        true_b = dev_to_ints(imm.mle_eval_point(torch.from_numpy(B).cuda(), imm.eq_table(r_k), imm.eq_table(r_col)))[0]
        assert true_b == oracle.mle_eval_point(B, oracle.eq_table(r_k), oracle.eq_table(r_col))
        assert imm.sumcheck_verify(sneaky, b, seed, pid, None, None, true_b) == (imm.REJECT, b + 3)


def test_implicit_padding_equals_explicit_padding_on_gpu(imm, backend):
    rng = np.random.default_rng(31)
    for (m, k, n) in ((5, 14, 6), (100, 300, 70), (33, 1500, 20)):
        A, B, C = np_problem(rng, m, k, n)
        mp, kp, np_ = (1 << (x - 1).bit_length() for x in (m, k, n))
        Ap = np.zeros((mp, kp), np.int8); Ap[:m, :k] = A
        Bp = np.zeros((kp, np_), np.int8); Bp[:k, :n] = B
        Cp = np.zeros((mp, np_), np.int32); Cp[:m, :n] = C
        assert gpu_prove(imm, [(A, B, C, 4)], 6) == gpu_prove(imm, [(Ap, Bp, Cp, 4)], 6)


def test_finals_match_point_evaluations(imm, backend):
    """c0, a_fin, b_fin are C~(r_row,r_col), A~(r_row,r_k), B~(r_k,r_col) by the point-evaluation call."""
    rng = np.random.default_rng(41)
    m, k, n = 70, 500, 90
    A, B, C = np_problem(rng, m, k, n)
    seed, pid = 12, 7
    t = gpu_prove(imm, [(A, B, C, pid)], seed)[0]
    a, b, c = 7, 9, 7
    Er = imm.eq_table(imm.challenges(seed, pid, 1, a))
    Ec = imm.eq_table(imm.challenges(seed, pid, 2, c))
    Ek = imm.eq_table(imm.challenges(seed, pid, 3, b))
    dA, dB, dC = (torch.from_numpy(x).cuda() for x in (A, B, C))
    assert dev_to_ints(imm.mle_eval_point(dC, Er, Ec))[0] == t[0]
    assert dev_to_ints(imm.mle_eval_point(dA, Er, Ek))[0] == t[-2]
    assert dev_to_ints(imm.mle_eval_point(dB, Ek, Ec))[0] == t[-1]
    assert imm.sumcheck_verify(t, b, seed, pid, t[0], t[-2], t[-1]) == (imm.OK, -1)


def test_host_buffer_entry_point_matches_device_entry_point(imm, backend):
    rng = np.random.default_rng(51)
    shapes = [(37, 300, 41), (64, 100, 130)]
    probs = [np_problem(rng, *s) + (i,) for i, s in enumerate(shapes)]
    want = gpu_prove(imm, probs, 8)
    host = [(torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory(),
             torch.from_numpy(C).pin_memory(), pid) for (A, B, C, pid) in probs]
    hp = imm.HostProver(host)
    for _ in range(2):
        t = hp.prove(8)
        got = [[int(v) & 0xFFFFFFFFFFFFFFFF for v in t[i, :n]] for i, n in enumerate([30, 24])]
        assert got == want and (hp.status == 0).all()
