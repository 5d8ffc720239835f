"""Guard bands around every caller-owned buffer of the device calls (run with -m gpu).

The library writes only into buffers its caller hands it: a workspace of exactly the size the query
call returned, and the outputs.  Each case here places those buffers between two 4 KiB bands filled
with a pattern, gives the call exactly the bytes it asked for, and afterwards requires (a) both bands
untouched and (b) the result still equal to the CPU oracle's.  A workspace 16 bytes short must be
refused with IMM_ERR_WORKSPACE before anything is launched.  (An out-of-bounds write by a kernel
would otherwise go unseen unless it happened to hit a compared word.)
"""
import ctypes
import random
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

SEED = 5
GUARD = 4096
PATTERN = 0xA5
P = 0xFFFFFFFF00000001


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


class Guarded:
    """`nbytes` bytes of device memory between two guard bands."""

    def __init__(self, nbytes, fill=0xEE):
        self.nbytes = int(nbytes)
        self.buf = torch.full((self.nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.bytes = self.buf[GUARD:GUARD + self.nbytes]
        self.bytes.fill_(fill)                       # stale contents the call must not rely on

    def typed(self, dtype, shape):
        return self.bytes.view(dtype).view(shape)

    def ptr(self):
        return self.bytes.data_ptr() if self.nbytes else self.buf.data_ptr() + GUARD

    def intact(self):
        return bool((self.buf[:GUARD] == PATTERN).all()) and bool((self.buf[GUARD + self.nbytes:] == PATTERN).all())


def all_intact(*guards):
    torch.cuda.synchronize()
    return all(g.intact() for g in guards)


def strided(t, pad, offset_elems=0):
    """The same matrix as a view with a leading dimension of cols + pad, starting offset_elems into its buffer."""
    rows, cols = t.shape
    buf = torch.zeros(rows * (cols + pad) + offset_elems + 16, dtype=t.dtype, device=t.device)
    v = buf[offset_elems:offset_elems + rows * (cols + pad)].view(rows, cols + pad)[:, :cols]
    v.copy_(t)
    return v


def random_problem(rng, m, k, n, pid, odd=False):
    A = torch.from_numpy(rng.integers(-128, 128, size=(m, k), dtype=np.int64).astype(np.int8)).cuda()
    B = torch.from_numpy(rng.integers(-128, 128, size=(k, n), dtype=np.int64).astype(np.int8)).cuda()
    C = torch.from_numpy((A.cpu().numpy().astype(np.int64) @ B.cpu().numpy().astype(np.int64)).astype(np.int32)).cuda()
    if odd:                                          # rows that are not 16-byte aligned: the element-wise paths
        A, B, C = strided(A, 3, 1), strided(B, 5, 3), strided(C, 1, 1)
    return (A, B, C, pid)


def small_batches(rng):
    """Ragged, unaligned and full-tile batches."""
    return {
        "ragged": [random_problem(rng, 300, 1000, 700, 0), random_problem(rng, 37, 129, 1031, 1),
                   random_problem(rng, 1, 1, 5, 2), random_problem(rng, 1500, 257, 33, 3)],
        "unaligned": [random_problem(rng, 130, 517, 263, 7, odd=True), random_problem(rng, 65, 2049, 100, 8, odd=True)],
        "full_tiles": [random_problem(rng, 512, 4096, 1024, 11), random_problem(rng, 1024, 2048, 512, 12)],
    }


def oracle_transcripts(oracle, problems, seed):
    def one(p):
        A, B, C, pid = p
        return [int(w) for w in oracle.sumcheck_matmul_prove(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy(), seed, pid)]
    with ThreadPoolExecutor(max_workers=8) as ex:
        return list(ex.map(one, problems))


def guard_object(obj, names):
    """Replace the device buffers `names` of a prover-like object by guarded ones of the same size."""
    guards = []
    for name in names:
        old = getattr(obj, name)
        g = Guarded(old.numel() * old.element_size())
        setattr(obj, name, g.typed(old.dtype, tuple(old.shape)))
        guards.append(g)
    return guards


def coms3(row96):
    """96 statement bytes -> the three 32-byte commitments."""
    b = bytes(row96)
    return [b[0:32], b[32:64], b[64:96]]


def words(t, n):
    return [int(v) & (2**64 - 1) for v in t[:n]]


# ------------------------------------------------------------------ the interactive prover and its relatives


@pytest.mark.parametrize("batch", ["ragged", "unaligned", "full_tiles"])
def test_prover_stays_inside_its_buffers(imm, oracle, batch):
    probs = small_batches(np.random.default_rng(31))[batch]
    want = oracle_transcripts(oracle, probs, SEED)
    pr = imm.Prover(probs)
    guards = guard_object(pr, ["ws", "transcripts", "status"])
    for _ in range(2):
        pr.prove(SEED)
    assert all_intact(*guards)
    assert int(pr.status.abs().max()) == 0
    host = pr.transcripts.cpu()
    assert [words(host[i], n) for i, n in enumerate(pr.lengths())] == want
    # a workspace 16 bytes short is refused
    L = imm.lib()
    rc = L.imm_sumcheck_matmul_prove(ctypes.addressof(pr.descs), pr.nproofs, SEED, pr.transcripts.data_ptr(), pr.stride,
                                     pr.status.data_ptr(), pr.ws.data_ptr(), pr.ws.numel() - 16, None)
    assert rc == imm.ERR_WORKSPACE


def test_prover_on_the_expert_batch_stays_inside_its_buffers(imm, oracle, synth):
    probs = [(p.A, p.B, p.C, p.proof_id) for p in synth.moe_experts(1, device="cuda")]
    pr = imm.Prover(probs)
    guards = guard_object(pr, ["ws", "transcripts", "status"])
    pr.prove(1)
    assert all_intact(*guards)
    host = pr.transcripts.cpu()
    assert [words(host[i], n) for i, n in enumerate(pr.lengths())] == oracle_transcripts(oracle, probs, 1)


@pytest.mark.parametrize("batch", ["ragged", "unaligned", "full_tiles"])
def test_batched_prover_stays_inside_its_buffers(imm, oracle, batch):
    probs = small_batches(np.random.default_rng(32))[batch]
    host = [(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy(), pid) for (A, B, C, pid) in probs]
    want = [int(w) for w in oracle.sumcheck_matmul_prove_batched(host, SEED, 77)]
    bp = imm.BatchedProver(probs)
    guards = guard_object(bp, ["ws", "transcript", "status"])
    bp.prove(SEED, 77)
    assert all_intact(*guards)
    assert words(bp.transcript.cpu(), bp.length) == want
    L = imm.lib()
    rc = L.imm_sumcheck_matmul_prove_batched(ctypes.addressof(bp.descs), bp.nproofs, SEED, 77, bp.transcript.data_ptr(),
                                             bp.status.data_ptr(), bp.ws.data_ptr(), bp.ws.numel() - 16, None)
    assert rc == imm.ERR_WORKSPACE


@pytest.mark.parametrize("batch", ["ragged", "unaligned"])
def test_verifier_pass_stays_inside_its_buffers(imm, oracle, batch):
    probs = small_batches(np.random.default_rng(33))[batch]
    ver = imm.Verifier(probs)
    guards = guard_object(ver, ["ws", "values", "status"])
    ver.expected(SEED)
    assert all_intact(*guards)
    vals = ver.values.cpu()
    for i, (A, B, C, pid) in enumerate(probs):
        m, k = A.shape
        n = B.shape[1]
        e_row = oracle.eq_table(oracle.challenges(SEED, pid, 1, oracle.ceil_log2(m)))
        e_col = oracle.eq_table(oracle.challenges(SEED, pid, 2, oracle.ceil_log2(n)))
        e_k = oracle.eq_table(oracle.challenges(SEED, pid, 3, oracle.ceil_log2(k)))
        assert words(vals[i], 3) == [oracle.mle_eval_point(C.cpu().numpy(), e_row, e_col),
                                     oracle.mle_eval_point(A.cpu().numpy(), e_row, e_k),
                                     oracle.mle_eval_point(B.cpu().numpy(), e_k, e_col)]
    L = imm.lib()
    rc = L.imm_sumcheck_expected(ctypes.addressof(ver.descs), ver.nproofs, SEED, None, None, ver.values.data_ptr(),
                                 ver.status.data_ptr(), ver.ws.data_ptr(), ver.ws.numel() - 16, None)
    assert rc == imm.ERR_WORKSPACE


@pytest.mark.parametrize("batch", ["ragged", "unaligned"])
def test_noninteractive_provers_stay_inside_their_buffers(imm, oracle, batch):
    probs = small_batches(np.random.default_rng(34))[batch]
    msgs = [t.contiguous() for (A, B, C, _) in probs for t in (A, B, C)]
    com = imm.Committer(msgs)
    cguards = guard_object(com, ["ws", "digests", "roots"])
    com.commit()
    assert all_intact(*cguards)
    digests = com.digests.cpu().numpy()
    for i, t in enumerate(msgs):
        assert bytes(digests[i]) == oracle.commitment.commit(t.cpu().numpy().tobytes(), b"")
    L = imm.lib()
    rc = L.imm_commit(ctypes.addressof(com.descs), com.n, com.digests.data_ptr(), com.roots.data_ptr(),
                      com.ws.data_ptr(), com.ws.numel() - 16, None)
    assert rc == imm.ERR_WORKSPACE

    contiguous = [(A.contiguous(), B.contiguous(), C.contiguous(), pid) for (A, B, C, pid) in probs]
    statement = com.digests.clone().view(len(probs), 96)
    fp = imm.FsProver(contiguous, statement)
    guards = guard_object(fp, ["ws", "transcripts", "status"])
    fp.prove()
    assert all_intact(*guards)
    host_t = fp.transcripts.cpu()
    host_c = statement.cpu().numpy()
    for i, (A, B, C, pid) in enumerate(contiguous):
        want = oracle.fs.prove(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy(), coms3(host_c[i]), pid)
        assert words(host_t[i], len(want)) == [int(w) for w in want]
    rc = L.imm_sumcheck_matmul_prove_fs(ctypes.addressof(fp.descs), fp.nproofs, fp.commitments.data_ptr(),
                                        fp.transcripts.data_ptr(), fp.stride, fp.status.data_ptr(), fp.ws.data_ptr(),
                                        fp.ws.numel() - 16, None)
    assert rc == imm.ERR_WORKSPACE

    fb = imm.FsBatchedProver(contiguous, statement)
    guards = guard_object(fb, ["ws", "transcript", "status"])
    fb.prove(91)
    assert all_intact(*guards)
    members = [(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy(), coms3(host_c[i]), pid)
               for i, (A, B, C, pid) in enumerate(contiguous)]
    want = oracle.fs.prove_batched(members, 91)
    assert words(fb.transcript.cpu(), fb.length) == [int(w) for w in want]
    rc = L.imm_sumcheck_matmul_prove_fs_batched(ctypes.addressof(fb.descs), fb.nproofs, fb.commitments.data_ptr(), 91,
                                                fb.transcript.data_ptr(), fb.status.data_ptr(), fb.ws.data_ptr(),
                                                fb.ws.numel() - 16, None)
    assert rc == imm.ERR_WORKSPACE


# ------------------------------------------------------------------ single-matrix calls


@pytest.mark.parametrize("rows,cols,dtype,odd", [(300, 1000, np.int8, False), (1027, 4100, np.int8, False),
                                                 (129, 517, np.int8, True), (700, 1300, np.int32, False),
                                                 (2048, 4096, np.int32, False), (65, 263, np.int32, True),
                                                 (1, 1, np.int8, False), (4096, 64, np.int32, False)])
def test_single_matrix_calls_stay_inside_their_buffers(imm, oracle, rows, cols, dtype, odd):
    rng = np.random.default_rng(rows * 31 + cols)
    prng = random.Random(rows * 31 + cols)
    lo, hi = (-128, 127) if dtype == np.int8 else (-2**31, 2**31 - 1)
    Mh = rng.integers(lo, hi, size=(rows, cols), endpoint=True, dtype=np.int64).astype(dtype)
    M = torch.from_numpy(Mh).cuda()
    if odd:
        M = strided(M, 3, 1)
    r_row = [prng.randrange(P) for _ in range(imm.ceil_log2(rows))]
    r_col = [prng.randrange(P) for _ in range(imm.ceil_log2(cols))]
    er, ec = imm.eq_table(r_row), imm.eq_table(r_col)
    oer, oec = oracle.eq_table(r_row), oracle.eq_table(r_col)
    L = imm.lib()
    ptr, code, _, _, ld = imm._matrix(M, "M")
    for bind, eq, count, want in ((imm.BIND_ROWS, er, cols, oracle.mle_partial_eval(Mh, oracle.BIND_ROWS, oer)),
                                  (imm.BIND_COLS, ec, rows, oracle.mle_partial_eval(Mh, oracle.BIND_COLS, oec))):
        need = L.imm_mle_workspace(code, rows, cols, bind)
        ws, out = Guarded(need), Guarded(8 * count)
        rc = L.imm_mle_partial_eval(ptr, code, rows, cols, ld, bind, eq.data_ptr(), out.ptr(), ws.ptr(), need, None)
        assert rc == 0
        assert all_intact(ws, out)
        assert words(out.typed(torch.int64, (count,)).cpu(), count) == [int(v) for v in want]
        if need > 16:
            assert L.imm_mle_partial_eval(ptr, code, rows, cols, ld, bind, eq.data_ptr(), out.ptr(), ws.ptr(), need - 16,
                                          None) == imm.ERR_WORKSPACE
    need = L.imm_mle_workspace(code, rows, cols, imm.BIND_ROWS)
    ws, out = Guarded(need), Guarded(8)
    assert L.imm_mle_eval_point(ptr, code, rows, cols, ld, er.data_ptr(), ec.data_ptr(), out.ptr(), ws.ptr(), need, None) == 0
    assert all_intact(ws, out)
    assert words(out.typed(torch.int64, (1,)).cpu(), 1) == [oracle.mle_eval_point(Mh, oer, oec)]
    # eq tables themselves: exactly 2^n words
    for r in (r_row, r_col):
        g = Guarded(8 << len(r))
        arr = (ctypes.c_uint64 * max(len(r), 1))(*r)
        assert L.imm_eq_table(ctypes.addressof(arr), len(r), g.ptr(), None) == 0
        assert all_intact(g)
        assert words(g.typed(torch.int64, (1 << len(r),)).cpu(), 1 << len(r)) == [int(v) for v in oracle.eq_table(r)]


# ------------------------------------------------------------------ logit distances


@pytest.mark.parametrize("steps,n,k", [(5, 100, 4), (7, 1000, 20), (3, 40003, 20), (2, 128256, 64)])
def test_logit_distance_calls_stay_inside_their_buffers(imm, synth, steps, n, k):
    from oracle import ldd
    ref = synth.reference_logits(41, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 41, synth.NOISE_QUANTISED)
    top = torch.topk(dep, k, dim=1).indices.to(torch.int32).contiguous()
    L = imm.lib()
    tv, kl = Guarded(8 * steps), Guarded(8 * steps)
    assert L.imm_ldd_tv_kl(dep.data_ptr(), ref.data_ptr(), steps, n, n, tv.ptr(), kl.ptr(), None) == 0
    need = L.imm_ldd_topk_workspace(steps, n, k)
    ws, dist, status = Guarded(need), Guarded(8 * steps), Guarded(4 * steps)
    assert L.imm_ldd_topk_distance(ref.data_ptr(), steps, n, n, top.data_ptr(), k, dist.ptr(), status.ptr(), ws.ptr(), need,
                                   None) == 0
    offsets = torch.tensor([0, steps // 2, steps], dtype=torch.int64, device="cuda")
    p, flag = Guarded(16), Guarded(8)
    assert L.imm_ldd_tail_fraction(tv.ptr(), offsets.data_ptr(), 2, 0.05, 0.3, p.ptr(), flag.ptr(), None) == 0
    assert all_intact(tv, kl, ws, dist, status, p, flag)
    x, y, idx = dep.cpu().numpy(), ref.cpu().numpy(), top.cpu().numpy()
    gtv, gkl = tv.typed(torch.float64, (steps,)).cpu().numpy(), kl.typed(torch.float64, (steps,)).cpu().numpy()
    gd = dist.typed(torch.float64, (steps,)).cpu().numpy()
    assert int(status.typed(torch.int32, (steps,)).abs().max()) == 0
    for i in range(steps):
        assert abs(gtv[i] - ldd.tv_distance(x[i], y[i])) <= 2e-5
        want_kl = ldd.kl_divergence(x[i], y[i])
        assert abs(gkl[i] - want_kl) <= 2e-5 + 2e-4 * abs(want_kl)
        want_d = ldd.topk_distance(y[i], idx[i])
        assert abs(gd[i] - want_d) <= 1e-9 * max(1.0, abs(want_d))
    want_p = ldd.request_tail_fractions(gtv, [0, steps // 2, steps], 0.05)
    assert (p.typed(torch.float64, (2,)).cpu().numpy() == want_p).all()
    if need > 256:
        assert L.imm_ldd_topk_distance(ref.data_ptr(), steps, n, n, top.data_ptr(), k, dist.ptr(), status.ptr(), ws.ptr(),
                                       need - 16, None) == imm.ERR_WORKSPACE
