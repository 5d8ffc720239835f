"""GPU parity of the non-interactive (Fiat-Shamir) proof against the CPU oracle, word for word (run
with -m gpu): commitments from the GPU hash kernels feed the GPU prover; the oracle recomputes both."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def imm():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2602_22700_b200 import imm as binding
    binding.lib()
    return binding


@pytest.fixture(params=["mma", "alu"])
def backend(request, monkeypatch):
    monkeypatch.setenv("IMM_CONTRACT", request.param)
    return request.param


def make(rng, shapes, first_id=0, honest=True):
    out = []
    for i, (m, k, n) in enumerate(shapes):
        A = rng.integers(-128, 127, size=(m, k), endpoint=True).astype(np.int8)
        B = rng.integers(-128, 127, size=(k, n), endpoint=True).astype(np.int8)
        C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
        if not honest:
            C[m // 2, n // 2] += 1
        out.append((A, B, C, first_id + 5 * i))
    return out


def on_gpu(group):
    return [(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C).cuda(), pid)
            for A, B, C, pid in group]


def oracle_coms(oracle, group, rs=None):
    """Per problem the three commitments, from the commitment oracle."""
    out = []
    for i, (A, B, C, _) in enumerate(group):
        r = [b"", b"", b""] if rs is None else rs[3 * i:3 * i + 3]
        out.append([oracle.commitment.commit(M.tobytes(), rr or b"") for M, rr in zip((A, B, C), r)])
    return out


def check_batch(imm, oracle, group, rs=None):
    dev = on_gpu(group)
    coms = imm.commit_matrices(dev, rs)
    want_coms = oracle_coms(oracle, group, rs)
    host_coms = coms.cpu().numpy()
    for i in range(len(group)):
        assert bytes(host_coms[i]) == b"".join(want_coms[i])
    got = imm.sumcheck_matmul_prove_fs(dev, coms)
    for (A, B, C, pid), t, cm in zip(group, got, want_coms):
        assert t == oracle.fs.prove(A, B, C, cm, pid)
    return got, want_coms


@pytest.mark.parametrize("shapes", [
    [(3, 8, 2), (2, 5, 4), (1, 7, 1)],
    [(2, 1, 2), (4, 2, 1)],                                          # no rounds; one round
    [(33, 300, 17), (64, 512, 64), (1, 257, 129), (130, 511, 3)],
    [(100, 1000, 40), (7, 4096, 9), (300, 33, 700)],                 # mixed round counts in one batch
])
def test_transcripts_equal_oracle(imm, oracle, backend, shapes):
    rng = np.random.default_rng(sum(sum(s) for s in shapes))
    group = make(rng, shapes, first_id=3)
    got, coms = check_batch(imm, oracle, group)
    for (A, B, C, pid), t, cm in zip(group, got, coms):
        m, k = A.shape
        n = B.shape[1]
        b = oracle.ceil_log2(k)
        assert imm.sumcheck_verify_fs(t, b, b"".join(cm), m, k, n, pid) == (imm.OK, -1)
        # the verifier's own evaluations at the hashed points
        r_row, r_col, r_k = imm.fs_challenges(t, b, b"".join(cm), m, k, n, pid)
        e_row, e_col, e_k = oracle.eq_table(r_row), oracle.eq_table(r_col), oracle.eq_table(r_k)
        assert t[0] == oracle.mle_eval_point(C, e_row, e_col)
        assert t[-2] == oracle.mle_eval_point(A, e_row, e_k) and t[-1] == oracle.mle_eval_point(B, e_k, e_col)


def test_hidden_commitments_and_long_tables(imm, oracle):
    """Commitments under randomness; k up to 2^17 (tables of 128 Ki entries in the round kernel)."""
    rng = np.random.default_rng(11)
    group = make(rng, [(2, 131072, 3), (5, 70000, 2), (3, 16384, 4), (1, 9000, 1)], first_id=100)
    rs = [bytes(rng.integers(0, 255, size=32, endpoint=True, dtype=np.uint8)) for _ in range(12)]
    check_batch(imm, oracle, group, rs)


def test_wrong_product_is_rejected_and_statement_is_bound(imm, oracle):
    rng = np.random.default_rng(12)
    group = make(rng, [(8, 64, 8)], honest=False)
    got, coms = check_batch(imm, oracle, group)
    com96 = b"".join(coms[0])
    assert imm.sumcheck_verify_fs(got[0], 6, com96, 8, 64, 8, 0) == (imm.REJECT, 0)
    good = make(rng, [(8, 64, 8)])
    got, coms = check_batch(imm, oracle, good)
    com96 = b"".join(coms[0])
    assert imm.sumcheck_verify_fs(got[0], 6, com96, 8, 64, 8, 0) == (imm.OK, -1)
    # the same transcript under another statement: other matrices' commitments, shape or id
    other = bytes([com96[0] ^ 1]) + com96[1:]
    assert imm.sumcheck_verify_fs(got[0], 6, other, 8, 64, 8, 0)[0] == imm.REJECT
    assert imm.sumcheck_verify_fs(got[0], 6, com96, 7, 64, 8, 0)[0] == imm.REJECT
    assert imm.sumcheck_verify_fs(got[0], 6, com96, 8, 64, 8, 1)[0] == imm.REJECT


def test_ffn_pair_full_size(imm, oracle):
    """2048 x 4096 x 14336 and 2048 x 14336 x 4096 (twelve and fourteen rounds), commitments included."""
    from paper_2602_22700_b200 import synth
    probs = synth.ffn_pair(1, device="cuda")
    dev = [(p.A, p.B, p.C, p.proof_id) for p in probs]
    coms = imm.commit_matrices(dev)
    got = imm.sumcheck_matmul_prove_fs(dev, coms)
    host_coms = coms.cpu().numpy()
    for p, t, c in zip(probs, got, host_coms):
        A, B, C = p.A.cpu().numpy(), p.B.cpu().numpy(), p.C.cpu().numpy()
        cm = [oracle.commitment.commit(M.tobytes()) for M in (A, B, C)]
        assert bytes(c) == b"".join(cm)
        assert t == oracle.fs.prove(A, B, C, cm, p.proof_id)
        m, k, n = p.mkn
        assert imm.sumcheck_verify_fs(t, oracle.ceil_log2(k), bytes(c), m, k, n, p.proof_id) == (imm.OK, -1)


def test_repeated_calls_and_interleaving_with_the_interactive_prover(imm, oracle):
    rng = np.random.default_rng(13)
    group = make(rng, [(40, 700, 9), (3, 513, 200)])
    dev = on_gpu(group)
    coms = imm.commit_matrices(dev)
    fp = imm.FsProver(dev, coms)
    first = fp.prove().clone()
    plain = imm.sumcheck_matmul_prove(dev, 5)
    again = fp.prove().clone()
    torch.cuda.synchronize()
    assert torch.equal(first, again) and int(fp.status.abs().max()) == 0
    for (A, B, C, pid), t in zip(group, plain):
        assert t == [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 5, pid)]


# ------------------------------------------------------------------ batched non-interactive proof

def batched_case(imm, oracle, group, bid, rs=None):
    dev = on_gpu(group)
    coms = imm.commit_matrices(dev, rs)
    want_coms = oracle_coms(oracle, group, rs)
    got = imm.sumcheck_matmul_prove_fs_batched(dev, coms, bid)
    want = oracle.fs.prove_batched([(A, B, C, cm, pid) for (A, B, C, pid), cm in zip(group, want_coms)], bid)
    assert got == want
    meta = [(A.shape[0], A.shape[1], B.shape[1], pid) for A, B, C, pid in group]
    com = b"".join(b"".join(c) for c in want_coms)
    b = max(oracle.ceil_log2(k) for (_, k, _, _) in meta)
    assert imm.sumcheck_verify_fs_batched(got, b, meta, com, bid) == (imm.OK, -1)
    return dev, got, meta, com, b


@pytest.mark.parametrize("shapes", [
    [(3, 8, 2), (2, 5, 4), (1, 7, 1)],
    [(2, 1, 2), (1, 1, 3)],                                          # no rounds
    [(5, 2, 5)],                                                     # one member, one round
    [(33, 300, 17), (64, 512, 64), (1, 257, 129), (130, 511, 3), (9, 1, 3)],
    [(4, 100 + 37 * i, 3 + i % 4) for i in range(37)],               # 37 members: odd tree levels over the statements
])
def test_batched_transcripts_equal_oracle(imm, oracle, backend, shapes):
    rng = np.random.default_rng(sum(sum(s) for s in shapes) + 1)
    group = make(rng, shapes, first_id=8)
    batched_case(imm, oracle, group, bid=2**63 + 11)


def test_batched_full_loop_with_the_verifiers_pass(imm, oracle):
    """Prove, derive the coins on the host, evaluate the opened matrices on the GPU, verify."""
    rng = np.random.default_rng(21)
    group = make(rng, [(40, 700, 9), (3, 513, 200), (64, 64, 64), (7, 5000, 2)], first_id=1)
    dev, got, meta, com, b = batched_case(imm, oracle, group, bid=5)
    _, r_k = imm.fs_batched_challenges(got, b, meta, com, 5)
    points = []
    for i, (m, k, n, pid) in enumerate(meta):
        r_row, r_col, _ = imm.fs_challenges(None, oracle.ceil_log2(k), com[96 * i:96 * i + 96], m, k, n, pid)
        points.append((r_row, r_col, r_k))
    own = imm.sumcheck_expected(dev, batch_id=5, points=points)
    flat = [w for vals in own for w in vals]
    assert got[1 + 3 * b:] == flat
    assert imm.sumcheck_verify_fs_batched(got, b, meta, com, 5, expect=flat) == (imm.OK, -1)
    # an opened matrix that differs from the committed one: other statement, other coins, rejected
    A, B, C, pid = group[2]
    C2 = C.copy()
    C2[1, 1] += 1
    bad = [group[0], group[1], (A, B, C2, pid), group[3]]
    com2 = imm.commit_matrices(on_gpu(bad)).cpu().numpy().tobytes()
    assert imm.sumcheck_verify_fs_batched(got, b, meta, com2, 5)[0] == imm.REJECT


def test_batched_many_members_and_limit(imm, oracle):
    rng = np.random.default_rng(22)
    shapes = [(1 + i % 3, 40 + i % 50, 1 + i % 4) for i in range(1024)]
    group = make(rng, shapes, first_id=0)
    batched_case(imm, oracle, group, bid=1)
    dev = on_gpu(make(rng, [(2, 4, 2)] * 1025))
    coms = torch.zeros((1025, 96), dtype=torch.uint8, device="cuda")
    with pytest.raises(imm.ImmError) as e:
        imm.FsBatchedProver(dev, coms)
    assert e.value.code == imm.ERR_LIMIT


def test_batched_decoder_layers_full_size(imm, oracle):
    """Four layers of the decoder block at 8192 tokens (16 products, k = 4096 and 14336) as one
    non-interactive proof of fourteen rounds, against the oracle."""
    from paper_2602_22700_b200 import synth
    probs = synth.decoder_block(1, 4, 8192, device="cuda")
    dev = [(p.A, p.B, p.C, p.proof_id) for p in probs]
    coms = imm.commit_matrices(dev)
    got = imm.sumcheck_matmul_prove_fs_batched(dev, coms, 99)
    host_coms = coms.cpu().numpy()
    members = []
    for p, c in zip(probs, host_coms):
        members.append((p.A.cpu().numpy(), p.B.cpu().numpy(), p.C.cpu().numpy(),
                        [bytes(c[0:32]), bytes(c[32:64]), bytes(c[64:96])], p.proof_id))
    assert got == oracle.fs.prove_batched(members, 99)
    assert len(got) == 1 + 42 + 48


def test_weight_commitments_computed_once_serve_every_request(imm, oracle):
    """The weights belong to the model commitment: hashed once, their digests are reused while the
    activations and outputs of each audited request are hashed afresh.  Statement and proof must equal
    the oracle's (which hashes all three matrices of every request), request after request."""
    rng = np.random.default_rng(41)
    shapes = [(33, 300, 17), (64, 512, 64), (5, 129, 130)]
    weights = [rng.integers(-128, 127, size=(k, n), endpoint=True).astype(np.int8) for (_, k, n) in shapes]
    dev_w = [torch.from_numpy(B).cuda() for B in weights]
    com_w = imm.Committer(dev_w)
    com_w.commit()                                             # once
    cached = com_w.digests.view(len(shapes), 32).clone()
    n = len(shapes)
    for request in range(3):
        group = []
        for i, (m, k, _) in enumerate(shapes):
            A = rng.integers(-128, 127, size=(m, k), endpoint=True).astype(np.int8)
            C = (A.astype(np.int64) @ weights[i].astype(np.int64)).astype(np.int32)
            group.append((A, weights[i], C, 100 * request + i))
        dev = [(torch.from_numpy(A).cuda(), dev_w[i], torch.from_numpy(C).cuda(), pid) for i, (A, _, C, pid) in enumerate(group)]
        fresh = imm.Committer([t for (A, _, C, _) in dev for t in (A, C)])
        fresh.commit()
        stmt = torch.empty((n, 96), dtype=torch.uint8, device="cuda")
        stmt.view(n, 3, 32)[:, 0].copy_(fresh.digests.view(n, 2, 32)[:, 0])
        stmt.view(n, 3, 32)[:, 1].copy_(cached)
        stmt.view(n, 3, 32)[:, 2].copy_(fresh.digests.view(n, 2, 32)[:, 1])
        want = oracle_coms(oracle, group)
        host = stmt.cpu().numpy()
        for i in range(n):
            assert bytes(host[i]) == b"".join(want[i])
        assert bytes(imm.commit_matrices(dev).cpu().numpy().tobytes()) == host.tobytes()
        got = imm.sumcheck_matmul_prove_fs(dev, stmt)
        for (A, B, C, pid), t, cm in zip(group, got, want):
            assert t == oracle.fs.prove(A, B, C, cm, pid)
            assert imm.sumcheck_verify_fs(t, oracle.ceil_log2(A.shape[1]), b"".join(cm), A.shape[0], A.shape[1], B.shape[1], pid) == (imm.OK, -1)
