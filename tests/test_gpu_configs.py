"""GPU parity at the full sizes of the benchmark configurations (run with -m gpu).

The smaller configurations are compared with the CPU oracle word for word on every proof.  The
decoder block (128 proofs; 9 GiB at 1024 tokens, 39 GiB at 8192, 74 GiB at 16384) is proved in the
batch geometry bench.py times -- the planner picks tile heights and chunk widths from the batch's
bytes, so each token count of the sweep runs its own tile shapes; there the oracle proves the proofs
of one layer in full, and for proofs sampled from the rest it recomputes the three values that pin
a transcript to its inputs (c0, a_fin, b_fin as two-sided MLE evaluations) while the verifier
checks every proof's rounds.
"""
import gc
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

SEED = 1


@pytest.fixture(scope="module")
def imm():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2602_22700_b200 import imm as binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def synth():
    from paper_2602_22700_b200 import synth as s
    return s


def host(p):
    return p.A.cpu().numpy(), p.B.cpu().numpy(), p.C.cpu().numpy()


def oracle_transcripts(oracle, problems, seed):
    """Oracle transcripts of several proofs, one proof per thread (the C oracle releases the GIL)."""
    def one(p):
        A, B, C = host(p)
        return [int(w) for w in oracle.sumcheck_matmul_prove(A, B, C, seed, p.proof_id)]
    with ThreadPoolExecutor(max_workers=8) as ex:
        return list(ex.map(one, problems))


def gpu_transcripts(imm, problems, seed):
    return imm.sumcheck_matmul_prove([(p.A, p.B, p.C, p.proof_id) for p in problems], seed)


def check_sampled_entries_of_C(p, rng, count=64):
    """The claimed C came from a library GEMM on the GPU: recompute sampled entries exactly."""
    A, B = p.A.cpu().numpy().astype(np.int64), p.B.cpu().numpy().astype(np.int64)
    C = p.C.cpu().numpy()
    for _ in range(count):
        i, j = int(rng.integers(A.shape[0])), int(rng.integers(B.shape[1]))
        assert int(C[i, j]) == int(A[i] @ B[:, j])


def test_qkv_projection_512x4096x4096(imm, oracle, synth):
    probs = synth.qkv_projection(SEED, device="cuda")
    assert probs[0].mkn == (512, 4096, 4096)
    check_sampled_entries_of_C(probs[0], np.random.default_rng(2))
    got = gpu_transcripts(imm, probs, SEED)
    assert got == oracle_transcripts(oracle, probs, SEED)
    assert len(got[0]) == 39
    assert imm.sumcheck_verify(got[0], 12, SEED, 0) == (imm.OK, -1)


def test_ffn_pair_full_size_and_padding_invariance(imm, oracle, synth):
    up, down = synth.ffn_pair(SEED, device="cuda")
    assert up.mkn == (2048, 4096, 14336) and down.mkn == (2048, 14336, 4096)
    rng = np.random.default_rng(3)
    check_sampled_entries_of_C(up, rng, 16)
    check_sampled_entries_of_C(down, rng, 16)
    got = gpu_transcripts(imm, [up, down], SEED)
    want = oracle_transcripts(oracle, [up, down], SEED)
    assert got == want
    assert len(got[1]) == 3 * 14 + 3                     # k = 14336 pads to 2^14: 14 rounds
    # explicit zero padding of k to 16384 gives the identical 45 words
    Hp = torch.zeros((2048, 16384), dtype=torch.int8, device="cuda")
    Hp[:, :14336] = down.A
    Wp = torch.zeros((16384, 4096), dtype=torch.int8, device="cuda")
    Wp[:14336] = down.B
    padded = imm.sumcheck_matmul_prove([(Hp, Wp, down.C, down.proof_id)], SEED)[0]
    assert padded == got[1]
    for t, p in zip(got, (up, down)):
        assert imm.sumcheck_verify(t, 12 if p is up else 14, SEED, p.proof_id) == (imm.OK, -1)


def test_moe_expert_batch_ragged(imm, oracle, synth):
    probs = synth.moe_experts(SEED, device="cuda")
    assert len(probs) == 8
    rows = [p.mkn[0] for p in probs]
    assert sum(rows) == 2 * 4096 and len(set(rows)) > 1          # top-2 routing, ragged counts
    # the routing on the GPU is the routing on the CPU
    cpu_rows = [int(r.numel()) for r in synth.moe_routing(SEED, 4096, 8, 2, "cpu")]
    assert rows == cpu_rows
    check_sampled_entries_of_C(probs[5], np.random.default_rng(4), 16)
    got = gpu_transcripts(imm, probs, SEED)                        # one launch sequence for all experts
    assert got == oracle_transcripts(oracle, probs, SEED)
    for t, p in zip(got, probs):
        assert imm.sumcheck_verify(t, 12, SEED, p.proof_id) == (imm.OK, -1)


def test_attention_products_many_small_proofs(imm, oracle, synth):
    """Scores (k = head_dim: few rounds, a large claimed matrix) and outputs (k = tokens) of 2 layers x
    4 heads in one batch: 16 proofs, every transcript against the oracle."""
    probs = synth.attention_block(SEED, layers=2, tokens=640, heads=4, head_dim=128, device="cuda")
    assert len(probs) == 16 and probs[0].mkn == (640, 128, 640) and probs[1].mkn == (640, 640, 128)
    check_sampled_entries_of_C(probs[3], np.random.default_rng(6), 16)
    got = gpu_transcripts(imm, probs, SEED)
    assert got == oracle_transcripts(oracle, probs, SEED)
    assert len(got[0]) == 3 * 7 + 3 and len(got[1]) == 3 * 10 + 3
    for t, p in zip(got, probs):
        assert imm.sumcheck_verify(t, oracle.ceil_log2(p.mkn[1]), SEED, p.proof_id) == (imm.OK, -1)


def test_narrow_left_factors_share_rows_among_warps(imm, oracle):
    """Left factors with fewer columns than the 1024 a block covers (an attention head's Q has 128): the
    warps without columns take rows instead and their partial sums are merged.  Widths of one, two,
    three and five warps, ragged last columns, tiles of several and of one group of 32 rows, rows that
    do not fill the last group; every transcript against the oracle."""
    from collections import namedtuple
    P = namedtuple("P", "A B C proof_id mkn")
    rng = np.random.default_rng(77)
    probs = []
    for pid, (m, k, n) in enumerate([(2048, 128, 2048), (1500, 64, 700), (1100, 200, 300), (3000, 384, 128),
                                     (2500, 520, 64), (33, 100, 40), (31, 129, 17), (1024, 1, 5)]):
        A = rng.integers(-128, 128, size=(m, k), dtype=np.int64).astype(np.int8)
        B = rng.integers(-128, 128, size=(k, n), dtype=np.int64).astype(np.int8)
        C = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.int32)
        probs.append(P(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C).cuda(), 900 + pid, (m, k, n)))
    got = gpu_transcripts(imm, probs, SEED)
    assert got == oracle_transcripts(oracle, probs, SEED)
    # and one at a time (other tile heights: the partition follows the batch)
    for p in probs[:4]:
        assert gpu_transcripts(imm, [p], SEED + 1) == oracle_transcripts(oracle, [p], SEED + 1)


def two_sided(oracle, M, r_row, r_col):
    return oracle.mle_eval_point(M, oracle.eq_table(r_row), oracle.eq_table(r_col))


@pytest.mark.parametrize("tokens", [1024, 8192, 16384])
def test_decoder_block_in_bench_geometry(imm, oracle, synth, tokens):
    """All 128 proofs in one batch, as bench.py launches them, at the ends and the middle of the
    token sweep (each runs a different tile geometry)."""
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    # inputs (4.75 GiB of weights + 4.31 MiB per token) + the two workspaces + generator temporaries
    need = int(1.3 * ((4.75 * 2**30) + tokens * 4.32 * 2**20)) + (4 << 30)
    if free < need:
        pytest.fail(f"the decoder-block batch at {tokens} tokens needs {need >> 30} GiB of free device memory")
    probs = synth.decoder_block(SEED, 32, tokens, device="cuda")
    assert len(probs) == 128
    prover = imm.Prover([(p.A, p.B, p.C, p.proof_id) for p in probs])
    t = prover.prove(SEED)
    torch.cuda.synchronize()
    assert int(prover.status.abs().max()) == 0
    hostt = t.cpu().numpy().view(np.uint64)
    lens = prover.lengths()
    got = [[int(w) for w in hostt[i, :n]] for i, n in enumerate(lens)]
    # rows are zero beyond each transcript
    for i, n in enumerate(lens):
        assert not hostt[i, n:].any()
    # every proof's rounds check out
    for tr, p in zip(got, probs):
        b = imm.ceil_log2(p.mkn[1])
        assert imm.sumcheck_verify(tr, b, SEED, p.proof_id) == (imm.OK, -1)
    # layer 17 in full against the oracle
    layer = probs[4 * 17:4 * 17 + 4]
    assert got[4 * 17:4 * 17 + 4] == oracle_transcripts(oracle, layer, SEED)
    # sampled proofs elsewhere: the three words that tie the transcript to A, B and C
    rng = np.random.default_rng(5)
    for i in sorted(int(v) for v in rng.choice(128, size=3, replace=False)):
        p = probs[i]
        m, k, n = p.mkn
        a, b, c = (oracle.ceil_log2(d) for d in (m, k, n))
        r_row = oracle.challenges(SEED, p.proof_id, 1, a)
        r_col = oracle.challenges(SEED, p.proof_id, 2, c)
        r_k = oracle.challenges(SEED, p.proof_id, 3, b)
        A, B, C = host(p)
        assert got[i][0] == two_sided(oracle, C, r_row, r_col)
        assert got[i][-2] == two_sided(oracle, A, r_row, r_k)
        assert got[i][-1] == two_sided(oracle, B, r_k, r_col)
        check_sampled_entries_of_C(p, rng, 8)

    # The same products as ONE batched proof (every k padded to 2^14): the verifier accepts it; every
    # member's c0 is the one of its own proof above; for sampled members a_fin and b_fin are the
    # oracle's evaluations at the batch's shared point.
    del prover
    b, count, bid = 14, 128, 4242
    bt = imm.sumcheck_matmul_prove_batched([(p.A, p.B, p.C, p.proof_id) for p in probs], SEED, bid)
    assert len(bt) == 1 + 3 * b + 3 * count
    assert imm.sumcheck_verify_batched(bt, b, count, SEED, bid) == (imm.OK, -1)
    tail = bt[1 + 3 * b:]
    assert [tail[3 * j] for j in range(count)] == [got[i][0] for i in range(count)]
    r_k = oracle.challenges(SEED, bid, 3, b)
    e_k = oracle.eq_table(r_k)
    for j in sorted(int(v) for v in rng.choice(count, size=3, replace=False)):
        p = probs[j]
        m, k, n = p.mkn
        e_row = oracle.eq_table(oracle.challenges(SEED, p.proof_id, 1, oracle.ceil_log2(m)))
        e_col = oracle.eq_table(oracle.challenges(SEED, p.proof_id, 2, oracle.ceil_log2(n)))
        A, B, _ = host(p)
        # (the first k entries of the 2^14-entry table weigh the real inner indices; the rest meet zero padding)
        assert tail[3 * j + 1] == oracle.mle_eval_point(A, e_row, e_k)
        assert tail[3 * j + 2] == oracle.mle_eval_point(B, e_k, e_col)
