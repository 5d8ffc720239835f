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
