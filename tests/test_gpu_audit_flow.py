"""One audited request end to end on the GPU (run with -m gpu): the server commits to its logits and
attaches non-interactive proofs of its matrix products; the auditor re-derives the commitments from
what was opened, measures the logit distances against the reference execution, runs the verifier's
pass and checks the proofs.  Every number is compared with the CPU oracles."""
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


def serve(imm, synth, seed, steps, vocab, topk, noise, tokens):
    """What a server sends for one request: commitments, committed top-K sets, proofs; and what it opens on audit."""
    ref = synth.reference_logits(seed, steps, vocab, device="cuda")
    logits = synth.deployed_logits(ref, seed, noise)                      # what the deployed model computed
    r = bytes((11 * i + 3) & 255 for i in range(32))
    psi = imm.commit([logits], [r])[0]
    top = torch.topk(logits, topk, dim=1).indices.to(torch.int32).contiguous()
    probs = synth.ffn_pair(seed, tokens, 512, 1408, device="cuda")        # the products of one (small) layer
    mats = [(p.A, p.B, p.C, p.proof_id) for p in probs]
    coms = imm.commit_matrices(mats)
    proofs = imm.sumcheck_matmul_prove_fs(mats, coms)
    return dict(ref=ref, logits=logits, r=r, psi=psi, top=top, mats=mats, coms=coms.cpu().numpy(), proofs=proofs)


def audit(imm, sent, opened_logits, opened_mats, t1, t2, offsets):
    """The auditor's checks on the GPU; returns a dict of findings."""
    out = {}
    out["commitment_ok"] = imm.commit([opened_logits], [sent["r"]])[0] == sent["psi"]
    tv, kl = imm.ldd_tv_kl(opened_logits, sent["ref"])
    dist, status = imm.ldd_topk_distance(sent["ref"], sent["top"])
    assert int(status.abs().max()) == 0
    p, flag = imm.ldd_tail_fraction(tv, offsets, t1, t2)
    out.update(tv=tv, kl=kl, topk=dist, p=p, flag=flag)
    # statements are re-derived from the opened matrices; then the verifier's pass and the checks
    coms = imm.commit_matrices(opened_mats).cpu().numpy()
    verdicts, points = [], []
    for (A, B, C, pid), t, c in zip(opened_mats, sent["proofs"], coms):
        m, k = A.shape
        points.append(imm.fs_challenges(t, imm.ceil_log2(k), bytes(c), m, k, B.shape[1], pid))
    own = imm.sumcheck_expected(opened_mats, points=points)
    for (A, B, C, pid), t, c, vals in zip(opened_mats, sent["proofs"], coms, own):
        m, k = A.shape
        verdicts.append(imm.sumcheck_verify_fs(t, imm.ceil_log2(k), bytes(c), m, k, B.shape[1], pid, *vals))
    out["proofs"] = verdicts
    out["statement_ok"] = [bytes(a) == bytes(b) for a, b in zip(coms, sent["coms"])]
    return out


def test_honest_server_passes_and_numbers_match_the_oracles(imm, oracle):
    from paper_2602_22700_b200 import synth
    steps, vocab, topk = 96, 32000, 20
    sent = serve(imm, synth, 3, steps, vocab, topk, synth.NOISE_BENIGN, 128)
    offsets = torch.tensor([0, 40, 96], dtype=torch.int64, device="cuda")
    got = audit(imm, sent, sent["logits"], sent["mats"], 0.1, 0.02, offsets)
    assert got["commitment_ok"] and all(got["statement_ok"])
    assert got["proofs"] == [(imm.OK, -1)] * 2
    assert int(got["flag"].sum()) == 0                                     # benign numerical noise is not flagged
    x, y, idx = sent["logits"].cpu().numpy(), sent["ref"].cpu().numpy(), sent["top"].cpu().numpy()
    assert sent["psi"] == oracle.commitment.commit(x.tobytes(), sent["r"])
    tv = [oracle.ldd.tv_distance(x[i], y[i]) for i in range(steps)]
    for i in (0, 41, 95):
        assert abs(float(got["tv"][i]) - tv[i]) <= 2e-5
        want_kl = oracle.ldd.kl_divergence(x[i], y[i])
        assert abs(float(got["kl"][i]) - want_kl) <= 2e-5 + 2e-4 * abs(want_kl)
        want_d = oracle.ldd.topk_distance(y[i], idx[i])
        assert abs(float(got["topk"][i]) - want_d) <= 1e-9 * max(1.0, abs(want_d))
    want_p = oracle.ldd.request_tail_fractions(np.array(tv), [0, 40, 96], 0.1)
    assert np.allclose(got["p"].cpu().numpy(), want_p, atol=1e-12)
    for (A, B, C, pid), t, c in zip(sent["mats"], sent["proofs"], sent["coms"]):
        cm = [bytes(c[0:32]), bytes(c[32:64]), bytes(c[64:96])]
        assert t == oracle.fs.prove(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy(), cm, pid)


def test_cheating_is_caught_where_the_paper_says(imm, oracle):
    from paper_2602_22700_b200 import synth
    steps, vocab, topk = 96, 32000, 20
    offsets = torch.tensor([0, 40, 96], dtype=torch.int64, device="cuda")
    # (1) a server that ran a degraded model: its committed logits sit far from the reference -> flagged
    sent = serve(imm, synth, 4, steps, vocab, topk, synth.NOISE_QUANTISED, 128)
    got = audit(imm, sent, sent["logits"], sent["mats"], 0.1, 0.02, offsets)
    assert got["commitment_ok"] and got["proofs"] == [(imm.OK, -1)] * 2
    assert int(got["flag"].sum()) == 2
    # (2) a server that opens other logits than it committed to -> the commitment does not match
    other = sent["ref"].clone()
    got = audit(imm, sent, other, sent["mats"], 0.1, 0.02, offsets)
    assert not got["commitment_ok"]
    # (3) a server that opens another claimed product than the one its proof was made for
    A, B, C, pid = sent["mats"][1]
    C2 = C.clone()
    C2[5, 7] += 1
    got = audit(imm, sent, sent["logits"], [sent["mats"][0], (A, B, C2, pid)], 0.1, 0.02, offsets)
    assert got["statement_ok"] == [True, False]
    assert got["proofs"][0] == (imm.OK, -1) and got["proofs"][1][0] == imm.REJECT
    # (4) a proof made for a wrong product from the start (committed as such): the rounds break at once
    bad = [sent["mats"][0], (A, B, C2, pid)]
    coms = imm.commit_matrices(bad)
    proofs = imm.sumcheck_matmul_prove_fs(bad, coms)
    c = coms.cpu().numpy()[1]
    m, k = A.shape
    assert imm.sumcheck_verify_fs(proofs[1], imm.ceil_log2(k), bytes(c), m, k, B.shape[1], pid) == (imm.REJECT, 0)
