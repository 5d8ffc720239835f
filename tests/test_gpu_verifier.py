"""GPU parity of the verifier's pass: its own (c0, a_fin, b_fin) per proof against the oracle's
two-sided evaluations, and the full Prove -> Vrfy loop on the GPU for all three proof forms (run
with -m gpu)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

P = 0xFFFFFFFF00000001


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


def make(rng, shapes, first_id=0):
    out = []
    for i, (m, k, n) in enumerate(shapes):
        A = rng.integers(-128, 127, size=(m, k), endpoint=True).astype(np.int8)
        B = rng.integers(-128, 127, size=(k, n), endpoint=True).astype(np.int8)
        C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
        out.append((A, B, C, first_id + 3 * i))
    return out


def on_gpu(group):
    return [(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C).cuda(), pid)
            for A, B, C, pid in group]


def oracle_expected(oracle, A, B, C, r_row, r_col, r_k):
    e_row, e_col, e_k = oracle.eq_table(r_row), oracle.eq_table(r_col), oracle.eq_table(r_k)
    return (oracle.mle_eval_point(C, e_row, e_col), oracle.mle_eval_point(A, e_row, e_k),
            oracle.mle_eval_point(B, e_k, e_col))


SHAPES = [(3, 8, 2), (2, 1, 2), (33, 300, 17), (64, 512, 64), (1, 257, 129), (130, 4100, 3), (700, 33, 900)]


def test_interactive_proofs(imm, oracle, backend):
    rng = np.random.default_rng(1)
    group = make(rng, SHAPES, first_id=9)
    dev = on_gpu(group)
    seed = 21
    got = imm.sumcheck_expected(dev, seed)
    transcripts = imm.sumcheck_matmul_prove(dev, seed)
    for (A, B, C, pid), vals, t in zip(group, got, transcripts):
        m, k = A.shape
        a, b, c = (oracle.ceil_log2(d) for d in (m, k, B.shape[1]))
        want = oracle_expected(oracle, A, B, C, oracle.challenges(seed, pid, 1, a), oracle.challenges(seed, pid, 2, c),
                               oracle.challenges(seed, pid, 3, b))
        assert vals == want
        assert (t[0], t[-2], t[-1]) == vals                      # an honest prover's words are the verifier's values
        assert imm.sumcheck_verify(t, b, seed, pid, *vals) == (imm.OK, -1)


def test_a_false_claim_meets_the_verifiers_own_value(imm, oracle):
    """C altered in one entry, and a prover that lies consistently: it sends the c0 of the TRUE product so
    that every round checks out; only the verifier's own evaluation of the opened C gives it away."""
    rng = np.random.default_rng(2)
    (A, B, C, pid), = make(rng, [(16, 64, 16)])
    Cbad = C.copy()
    Cbad[3, 5] += 1
    seed = 4
    t = imm.sumcheck_matmul_prove(on_gpu([(A, B, C, pid)]), seed)[0]            # transcript of the true product
    assert imm.sumcheck_verify(t, 6, seed, pid) == (imm.OK, -1)                  # self-consistent
    vals = imm.sumcheck_expected(on_gpu([(A, B, Cbad, pid)]), seed)[0]           # verifier reads the claimed C
    assert vals[1:] == (t[-2], t[-1]) and vals[0] != t[0]
    assert imm.sumcheck_verify(t, 6, seed, pid, *vals) == (imm.REJECT, 6 + 1)


def test_batched_proof_members(imm, oracle, backend):
    rng = np.random.default_rng(3)
    group = make(rng, SHAPES, first_id=100)
    dev = on_gpu(group)
    seed, bid = 8, 77
    got = imm.sumcheck_expected(dev, seed, batch_id=bid)
    b = max(oracle.ceil_log2(k) for (_, k, _) in SHAPES)
    r_k = oracle.challenges(seed, bid, 3, b)
    for (A, B, C, pid), vals in zip(group, got):
        a, c = oracle.ceil_log2(A.shape[0]), oracle.ceil_log2(B.shape[1])
        assert vals == oracle_expected(oracle, A, B, C, oracle.challenges(seed, pid, 1, a),
                                       oracle.challenges(seed, pid, 2, c), r_k)
    bt = imm.sumcheck_matmul_prove_batched(dev, seed, bid)
    flat = [w for vals in got for w in vals]
    assert bt[1 + 3 * b:] == flat
    assert imm.sumcheck_verify_batched(bt, b, len(group), seed, bid, expect=flat) == (imm.OK, -1)


def test_non_interactive_proofs(imm, oracle, backend):
    rng = np.random.default_rng(4)
    group = make(rng, SHAPES[:5], first_id=5)
    dev = on_gpu(group)
    coms = imm.commit_matrices(dev)
    transcripts = imm.sumcheck_matmul_prove_fs(dev, coms)
    host_coms = coms.cpu().numpy()
    points = []
    for (A, B, C, pid), t, c in zip(group, transcripts, host_coms):
        m, k = A.shape
        points.append(imm.fs_challenges(t, oracle.ceil_log2(k), bytes(c), m, k, B.shape[1], pid))
    got = imm.sumcheck_expected(dev, points=points)
    for (A, B, C, pid), t, c, pts, vals in zip(group, transcripts, host_coms, points, got):
        assert vals == oracle_expected(oracle, A, B, C, *pts)
        m, k = A.shape
        assert imm.sumcheck_verify_fs(t, oracle.ceil_log2(k), bytes(c), m, k, B.shape[1], pid, *vals) == (imm.OK, -1)


def test_decoder_block_in_bench_geometry(imm, oracle):
    """The verifier's pass over all 128 proofs of the benchmark workload: equal to the honest prover's
    words everywhere, and to the oracle's evaluations on sampled proofs."""
    from paper_2602_22700_b200 import synth
    free, _ = torch.cuda.mem_get_info()
    if free < 60 << 30:
        pytest.fail("the full decoder-block batch needs 60 GB of free device memory")
    probs = synth.decoder_block(1, 32, 8192, device="cuda")
    dev = [(p.A, p.B, p.C, p.proof_id) for p in probs]
    v = imm.Verifier(dev)
    vals = v.expected(1).cpu().numpy().view(np.uint64)
    assert int(v.status.abs().max()) == 0
    del v
    pr = imm.Prover(dev)
    t = pr.prove(1).cpu().numpy().view(np.uint64)
    for i, n in enumerate(pr.lengths()):
        assert (int(t[i, 0]), int(t[i, n - 2]), int(t[i, n - 1])) == tuple(int(x) for x in vals[i])
    rng = np.random.default_rng(6)
    for i in sorted(int(x) for x in rng.choice(128, size=2, replace=False)):
        p = probs[i]
        m, k, n = p.mkn
        want = oracle_expected(oracle, p.A.cpu().numpy(), p.B.cpu().numpy(), p.C.cpu().numpy(),
                               oracle.challenges(1, p.proof_id, 1, oracle.ceil_log2(m)),
                               oracle.challenges(1, p.proof_id, 2, oracle.ceil_log2(n)),
                               oracle.challenges(1, p.proof_id, 3, oracle.ceil_log2(k)))
        assert tuple(int(x) for x in vals[i]) == want
