"""GPU parity of the batched (random-linear-combination) proof against the CPU oracle, word for
word (run with -m gpu)."""
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


def make_group(rng, shapes, first_id=0, honest=True):
    """[(A, B, C, proof_id)] as numpy arrays; C = A*B exactly unless honest is False (random C)."""
    out = []
    for i, (m, k, n) in enumerate(shapes):
        A = rng.integers(-128, 127, size=(m, k), endpoint=True).astype(np.int8)
        B = rng.integers(-128, 127, size=(k, n), endpoint=True).astype(np.int8)
        if honest:
            C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
        else:
            C = rng.integers(-2**31, 2**31 - 1, size=(m, n), endpoint=True).astype(np.int32)
        out.append((A, B, C, first_id + 7 * i))
    return out


def on_gpu(group):
    return [(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C).cuda(), pid)
            for A, B, C, pid in group]


@pytest.mark.parametrize("shapes", [
    [(3, 8, 2), (2, 5, 4), (1, 7, 1)],                              # tiny, ragged, k pads to 8
    [(2, 1, 2), (1, 1, 3)],                                         # no rounds at all
    [(5, 2, 5)],                                                    # a batch of one
    [(33, 300, 17), (64, 512, 64), (1, 257, 129), (130, 511, 3)],   # nine rounds, several tiles
    [(100, 1000 - 3 * i, 40 + i) for i in range(9)],                # ten rounds, nine members
])
def test_batched_transcript_equals_oracle(imm, oracle, backend, shapes):
    rng = np.random.default_rng(len(shapes) * 1000 + shapes[0][1])
    group = make_group(rng, shapes, first_id=11)
    seed, bid = 77, 123456789
    want = [int(w) for w in oracle.sumcheck_matmul_prove_batched(group, seed, bid)]
    got = imm.sumcheck_matmul_prove_batched(on_gpu(group), seed, bid)
    assert got == want
    b = max(oracle.ceil_log2(k) for (_, k, _) in shapes)
    assert imm.sumcheck_verify_batched(got, b, len(shapes), seed, bid) == (imm.OK, -1)


def test_claimed_matrices_are_used_as_given(imm, oracle):
    """Random C (not A*B): the transcript still equals the oracle's, and the verifier rejects at
    round 0 because the combined round-0 sum is that of the true products."""
    rng = np.random.default_rng(5)
    group = make_group(rng, [(16, 64, 16), (8, 40, 24)], honest=False)
    got = imm.sumcheck_matmul_prove_batched(on_gpu(group), 3, 4)
    assert got == [int(w) for w in oracle.sumcheck_matmul_prove_batched(group, 3, 4)]
    assert imm.sumcheck_verify_batched(got, 6, 2, 3, 4) == (imm.REJECT, 0)


def test_many_members_cluster_rounds_and_strided_views(imm, oracle):
    """300 members (more than one block of the combining kernel's member loop and tail copy) of
    thirteen rounds (tables split over a cluster), some read through strided views."""
    rng = np.random.default_rng(8)
    shapes = [(1 + i % 5, 8192 - 11 * i, 1 + (i * 7) % 9) for i in range(300)]
    group = make_group(rng, shapes, first_id=5000)
    dev = on_gpu(group)
    # every third member lives in a wider buffer (leading dimensions larger than the extents)
    for i in range(0, 300, 3):
        A, B, C, pid = dev[i]
        wa = torch.zeros((A.shape[0], A.shape[1] + 16), dtype=torch.int8, device="cuda")
        wa[:, :A.shape[1]] = A
        wc = torch.zeros((C.shape[0], C.shape[1] + 4), dtype=torch.int32, device="cuda")
        wc[:, :C.shape[1]] = C
        dev[i] = (wa[:, :A.shape[1]], B, wc[:, :C.shape[1]], pid)
    seed, bid = 2**63 + 5, 2**64 - 1
    got = imm.sumcheck_matmul_prove_batched(dev, seed, bid)
    assert got == [int(w) for w in oracle.sumcheck_matmul_prove_batched(group, seed, bid)]
    assert len(got) == 1 + 39 + 900


def test_batched_is_the_combination_of_shared_challenge_proofs(imm, oracle):
    """Structure check through the ABI alone: single-member batches under the same batch id,
    rescaled by rho_p / rho_0, add up to the batch."""
    rng = np.random.default_rng(9)
    group = make_group(rng, [(20, 128, 12), (7, 100, 30), (64, 65, 64)])
    dev = on_gpu(group)
    seed, bid, b = 10, 20, 7
    whole = imm.sumcheck_matmul_prove_batched(dev, seed, bid)
    rho = [imm.challenge(seed, bid, 4, p) for p in range(3)]
    inv0 = pow(rho[0], P - 2, P)
    acc = [0] * (1 + 3 * b)
    for p in range(3):
        t = imm.sumcheck_matmul_prove_batched([dev[p]], seed, bid)
        assert t[-3:] == whole[1 + 3 * b + 3 * p:4 + 3 * b + 3 * p]
        for i in range(1 + 3 * b):
            acc[i] = (acc[i] + rho[p] * inv0 % P * t[i]) % P
    assert acc == whole[:1 + 3 * b]


def test_moe_expert_group_full_size(imm, oracle):
    """The eight ragged expert products (k = 4096) as one twelve-round batched proof."""
    from paper_2602_22700_b200 import synth
    probs = synth.moe_experts(1, device="cuda")
    assert len(probs) == 8 and all(p.mkn[1] == 4096 for p in probs)
    dev = [(p.A, p.B, p.C, p.proof_id) for p in probs]
    host = [(p.A.cpu().numpy(), p.B.cpu().numpy(), p.C.cpu().numpy(), p.proof_id) for p in probs]
    got = imm.sumcheck_matmul_prove_batched(dev, 1, 900)
    assert got == [int(w) for w in oracle.sumcheck_matmul_prove_batched(host, 1, 900)]
    assert len(got) == 1 + 36 + 24                        # against 8 * 39 words proof by proof
    assert imm.sumcheck_verify_batched(got, 12, 8, 1, 900, expect=got[-24:]) == (imm.OK, -1)


def test_repeated_and_interleaved_calls_reuse_buffers(imm, oracle):
    """A BatchedProver proves twice under different ids, with a plain batch proved in between on
    the same stream: no state leaks between calls."""
    rng = np.random.default_rng(12)
    group = make_group(rng, [(40, 700, 9), (3, 513, 200)])
    dev = on_gpu(group)
    bp = imm.BatchedProver(dev)
    first = bp.prove(5, 1).clone()
    plain = imm.sumcheck_matmul_prove(dev, 5)
    second = bp.prove(5, 2).clone()
    again = bp.prove(5, 1).clone()
    torch.cuda.synchronize()
    assert int(bp.status.abs().max()) == 0
    as_ints = lambda t: [int(v) for v in t.cpu().numpy().view(np.uint64)]
    assert as_ints(first) == as_ints(again) == [int(w) for w in oracle.sumcheck_matmul_prove_batched(group, 5, 1)]
    assert as_ints(second) == [int(w) for w in oracle.sumcheck_matmul_prove_batched(group, 5, 2)]
    for (A, B, C, pid), t in zip(group, plain):
        assert t == [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, 5, pid)]


def test_members_of_different_inner_size_share_the_longest_round_count(imm, oracle, backend):
    """k from 1 to 5000 in one batch: thirteen rounds for every member (tables zero beyond each k)."""
    rng = np.random.default_rng(1)
    shapes = [(4, 64, 4), (4, 65, 4), (9, 1, 3), (2, 5000, 7), (130, 300, 2), (1, 4096, 1)]
    group = make_group(rng, shapes, first_id=40)
    got = imm.sumcheck_matmul_prove_batched(on_gpu(group), 6, 7)
    assert got == [int(w) for w in oracle.sumcheck_matmul_prove_batched(group, 6, 7)]
    assert len(got) == 1 + 39 + 18
    assert imm.sumcheck_verify_batched(got, 13, 6, 6, 7) == (imm.OK, -1)
