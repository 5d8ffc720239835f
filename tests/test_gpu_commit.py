"""GPU parity of the hash commitments against the CPU oracle, byte for byte (run with -m gpu)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

LEAF = 4096


@pytest.fixture(scope="module")
def imm():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2602_22700_b200 import imm as binding
    binding.lib()
    return binding


def rand_bytes(rng, n):
    return torch.from_numpy(rng.integers(0, 255, size=n, endpoint=True, dtype=np.uint8))


def check(imm, oracle, msgs, rs):
    """Commit on the GPU, compare digests and roots with the oracle."""
    C = oracle.commitment
    dev = [m.cuda() for m in msgs]
    c = imm.Committer(dev, rs)
    got = c.commit().cpu().numpy()
    roots = c.roots.cpu().numpy()
    for i, (m, r) in enumerate(zip(msgs, rs)):
        data = m.numpy().tobytes()
        assert bytes(roots[i]) == C.merkle_root(data), f"root of message {i} ({len(data)} bytes)"
        assert bytes(got[i]) == C.commit(data, r or b""), f"commitment of message {i} ({len(data)} bytes)"
    return c


def test_padding_and_leaf_boundaries(imm, oracle):
    """Lengths around the SHA-256 padding boundary of the tagged leaf (54/55/56, 118..120), the leaf
    size, and two and three leaves; with and without randomness."""
    rng = np.random.default_rng(1)
    sizes = [0, 1, 2, 3, 54, 55, 56, 63, 64, 65, 118, 119, 120, 1000, LEAF - 1, LEAF, LEAF + 1,
             2 * LEAF - 1, 2 * LEAF, 2 * LEAF + 1, 3 * LEAF, 3 * LEAF + 62]
    msgs = [rand_bytes(rng, n) for n in sizes]
    rs = [bytes(rng.integers(0, 255, size=32, endpoint=True, dtype=np.uint8)) if i % 2 else None
          for i in range(len(sizes))]
    check(imm, oracle, msgs, rs)


def test_subtree_and_pass_boundaries(imm, oracle):
    """Leaf counts around one block's subtree (128 leaves), odd counts at several levels (an unpaired
    node moves up), and more than 1024 subtree roots (a second node pass)."""
    rng = np.random.default_rng(2)
    counts = [127, 128, 129, 130, 255, 256, 257, 383, 1000, 128 * 3 + 1, 128 * 1024 + 5]
    tails = [1, LEAF, 17, LEAF, 4095, LEAF, 100, LEAF, 3000, 1, 2]
    msgs = [rand_bytes(rng, (n - 1) * LEAF + t) for n, t in zip(counts, tails)]
    rs = [None] * len(msgs)
    rs[3] = bytes(range(32))
    rs[-1] = bytes(range(32, 64))
    check(imm, oracle, msgs, rs)


def test_every_leaf_count_up_to_140(imm, oracle):
    rng = np.random.default_rng(3)
    msgs = [rand_bytes(rng, (n - 1) * LEAF + int(rng.integers(1, LEAF, endpoint=True))) for n in range(1, 141)]
    check(imm, oracle, msgs, [None] * len(msgs))


def test_unaligned_messages_and_typed_tensors(imm, oracle):
    C = oracle.commitment
    rng = np.random.default_rng(4)
    buf = rand_bytes(rng, 5 * LEAF + 100).cuda()
    views = [buf[1:], buf[3:3 + 2 * LEAF], buf[8:], buf[16:16 + LEAF]]           # offsets 1, 3, 8 (slow), 16 (fast)
    got = imm.commit(views)
    host = buf.cpu().numpy().tobytes()
    want = [C.commit(host[1:]), C.commit(host[3:3 + 2 * LEAF]), C.commit(host[8:]), C.commit(host[16:16 + LEAF])]
    assert got == want
    # the bytes of typed tensors: float32 logits, int8 and int32 matrices
    logits = torch.from_numpy(rng.standard_normal((37, 1001)).astype(np.float32))
    A = torch.from_numpy(rng.integers(-128, 127, size=(300, 77), endpoint=True).astype(np.int8))
    Cm = torch.from_numpy(rng.integers(-2**31, 2**31 - 1, size=(65, 129), endpoint=True).astype(np.int32))
    r = bytes(range(100, 132))
    got = imm.commit([logits.cuda(), A.cuda(), Cm.cuda()], [r, None, r])
    assert got == [C.commit(logits.numpy().tobytes(), r), C.commit(A.numpy().tobytes()),
                   C.commit(Cm.numpy().tobytes(), r)]
    with pytest.raises(ValueError):
        imm.Committer([A.cuda()[:, :5]])                                          # not contiguous


def test_change_detection_and_repeatability(imm, oracle):
    rng = np.random.default_rng(5)
    m = rand_bytes(rng, 300 * LEAF + 9).cuda()
    r = bytes(range(32))
    c = imm.Committer([m], [r])
    first = c.commit().clone()
    again = c.commit().clone()
    assert torch.equal(first, again)
    for pos in (0, LEAF - 1, 128 * LEAF, 300 * LEAF + 8):
        old = int(m[pos])
        m[pos] = old ^ 0x80
        assert not torch.equal(c.commit(), first)
        m[pos] = old
    assert torch.equal(c.commit(), first)
    assert bytes(first.cpu().numpy()[0]) == oracle.commitment.commit(m.cpu().numpy().tobytes(), r)


def test_response_logits_of_the_benchmark_workload(imm, oracle):
    """The commitments bench.py times: every audited request's block of float32 logits (8192 steps x
    128256 entries over 64 requests of uneven length, 4.2 GB), each under its own randomness."""
    from paper_2602_22700_b200 import synth
    steps, vocab, requests = 8192, 128256, 64
    ref = synth.reference_logits(1, steps, vocab, device="cuda")
    dep = synth.deployed_logits(ref, 1, synth.NOISE_BENIGN)
    del ref
    off = synth.request_offsets(1, steps, requests, device="cpu").tolist()
    msgs = [dep[off[i]:off[i + 1]] for i in range(requests)]
    rs = [bytes((7 * i + j) & 255 for j in range(32)) for i in range(requests)]
    got = imm.commit(msgs, rs)
    C = oracle.commitment
    host = dep.cpu().numpy()
    for i in range(requests):
        assert got[i] == C.commit(host[off[i]:off[i + 1]].tobytes(), rs[i])
    assert len(set(got)) == requests


def test_message_beyond_four_gibibytes(imm, oracle):
    """Byte offsets above 2^32 and three levels of launches (1.18 M leaves -> 9217 -> 10 -> 1)."""
    n = (9 << 29) + 4096 * 3 + 5                       # 4.5 GiB and a bit
    g = torch.Generator(device="cuda").manual_seed(7)
    m = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda", generator=g)
    r = bytes(range(64, 96))
    c = imm.Committer([m], [r])
    assert c.launches == 4
    got = bytes(c.commit().cpu().numpy()[0])
    assert got == oracle.commitment.commit(m.cpu().numpy().tobytes(), r)
