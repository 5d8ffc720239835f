"""GPU parity of the logit-distance-distribution calls against the float64 oracle (run with -m gpu).

Tolerances.  TV and KL are sums of float32 terms (exp2-based softmax, about 2e-6 relative per term,
plus about 3e-6 from the float32 log-sum-exp that scales every term), so the absolute error of TV is
below 1e-5 and that of KL below 1e-5 + 1e-4 * KL; the tests allow 2e-5 (+ 2e-4 relative for KL).
The Top-K distance is selected exactly and evaluated in float64 on the float32 inputs: 1e-9 relative.
The tail statistic is a count: exact.
"""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

TV_TOL = 2e-5
KL_ABS, KL_REL = 2e-5, 2e-4


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


@pytest.fixture(scope="module")
def ldd():
    from oracle import ldd as o
    return o


def check_tv_kl(imm, ldd, x, y):
    tv, kl = imm.ldd_tv_kl(x, y)
    tv, kl = tv.cpu().numpy(), kl.cpu().numpy()
    xs, ys = x.cpu().numpy(), y.cpu().numpy()
    for i in range(xs.shape[0]):
        want_tv, want_kl = ldd.tv_distance(xs[i], ys[i]), ldd.kl_divergence(xs[i], ys[i])
        if math.isnan(want_tv):                               # a row without a finite entry
            assert math.isnan(tv[i]) and math.isnan(kl[i]) and math.isnan(want_kl), (i, tv[i], kl[i])
            continue
        assert abs(tv[i] - want_tv) <= TV_TOL, (i, tv[i], want_tv)
        if math.isinf(want_kl):                               # reference mass on an entry the deployed row masks
            assert kl[i] == want_kl, (i, kl[i], want_kl)
        else:
            assert abs(kl[i] - want_kl) <= KL_ABS + KL_REL * abs(want_kl), (i, kl[i], want_kl)


@pytest.mark.parametrize("steps,n", [(7, 1), (5, 3), (9, 100), (19, 64), (9, 128), (5, 256), (4, 1000), (3, 1024), (3, 1025),
                                     (1003, 100), (515, 200), (66, 257),
                                     (4, 4097), (3, 16384), (3, 16388), (3, 40003),
                                     (2, 128256), (2, 151936), (1, 300000)])
@pytest.mark.parametrize("noise", ["benign", "quantised", "substituted"])
def test_tv_kl_matches_oracle(imm, ldd, synth, steps, n, noise):
    ref = synth.reference_logits(3, steps, n, device="cuda")
    if noise == "substituted":
        dep = synth.reference_logits(4, steps, n, device="cuda")
    else:
        dep = synth.deployed_logits(ref, 3, synth.NOISE_BENIGN if noise == "benign" else synth.NOISE_QUANTISED)
    check_tv_kl(imm, ldd, dep, ref)


def test_tv_kl_identical_rows_and_far_rows(imm, ldd, synth):
    ref = synth.reference_logits(5, 4, 50000, device="cuda")
    tv, kl = imm.ldd_tv_kl(ref, ref)
    assert float(tv.abs().max()) <= 1e-6 and float(kl.abs().max()) <= 1e-6
    far = ref.clone()
    far[:, 123] += 60.0                                   # all mass on one entry
    check_tv_kl(imm, ldd, far, ref)
    check_tv_kl(imm, ldd, ref + 1000.0, ref - 500.0)      # shifts cancel: large magnitudes must not overflow


@pytest.mark.parametrize("n", [40, 200, 700, 5000, 40003, 128256])
def test_tv_kl_masked_logits(imm, ldd, synth, n):
    """-inf entries (masked vocabulary): one, many, a whole slice, all but one, and all of a row; in
    both rows, in the reference only (those entries add nothing to KL) and in the deployed row only
    (KL = +inf when the reference keeps mass there).  Every kernel family by row length."""
    steps = 8
    ref = synth.reference_logits(21, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 21, synth.NOISE_QUANTISED)
    g = torch.Generator().manual_seed(n)
    many = (torch.rand(n, generator=g) < 0.5).cuda()
    one = torch.zeros(n, dtype=torch.bool, device="cuda"); one[n // 3] = True
    head = torch.zeros(n, dtype=torch.bool, device="cuda"); head[:min(n - 1, 20000)] = True     # whole slices of a long row
    but_one = torch.ones(n, dtype=torch.bool, device="cuda"); but_one[n - 2] = False
    everything = torch.ones(n, dtype=torch.bool, device="cuda")
    masks = [one, many, head, but_one, everything, many, many, one]
    both_r, both_d = ref.clone(), dep.clone()
    for i in range(5):
        both_r[i, masks[i]] = -math.inf
        both_d[i, masks[i]] = -math.inf
    both_r[5, masks[5]] = -math.inf                        # reference only
    both_d[6, masks[6]] = -math.inf                        # deployed only: infinite divergence
    both_d[7, :] = -math.inf                               # deployed row dead, reference alive
    check_tv_kl(imm, ldd, both_d, both_r)
    tv, kl = imm.ldd_tv_kl(both_d, both_r)
    assert math.isnan(float(tv[4])) and math.isnan(float(kl[7])) and float(kl[6]) == math.inf
    assert float(tv[3]) <= TV_TOL                           # one live entry on both sides: identical distributions


def test_tv_kl_unaligned_rows_take_the_element_path(imm, ldd, synth):
    steps, n = 5, 20001
    ref = synth.reference_logits(6, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 6, synth.NOISE_QUANTISED)

    def odd(t, ld, off):
        buf = torch.zeros(steps * ld + off + 8, dtype=torch.float32, device="cuda")
        v = buf[off:off + steps * ld].view(steps, ld)[:, :n]
        v.copy_(t)
        return v

    check_tv_kl(imm, ldd, odd(dep, n + 3, 1), odd(ref, n + 3, 1))
    check_tv_kl(imm, ldd, odd(dep, n + 7, 0), odd(ref, n + 7, 0))      # aligned base, unaligned pitch


def test_short_rows_with_a_row_pitch(imm, ldd, synth):
    """Expert-routing shapes (one warp per row), rows not contiguous in memory."""
    steps, n, k = 37, 128, 8
    ref = synth.reference_logits(11, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 11, synth.NOISE_QUANTISED)
    buf_r = torch.zeros((steps, n + 5), dtype=torch.float32, device="cuda")
    buf_d = torch.zeros((steps, n + 5), dtype=torch.float32, device="cuda")
    buf_r[:, :n] = ref
    buf_d[:, :n] = dep
    check_tv_kl(imm, ldd, buf_d[:, :n], buf_r[:, :n])
    top = torch.topk(dep, k, dim=1).indices.to(torch.int32).contiguous()
    check_topk(imm, ldd, buf_r[:, :n], top)


def check_topk(imm, ldd, ref, topk, rel=1e-9):
    dist, status = imm.ldd_topk_distance(ref, topk)
    dist, status = dist.cpu().numpy(), status.cpu().numpy()
    ys, idx = ref.cpu().numpy(), topk.cpu().numpy()
    assert (status == 0).all(), status
    for i in range(ys.shape[0]):
        want = ldd.topk_distance(ys[i], idx[i])
        assert abs(dist[i] - want) <= rel * max(1.0, abs(want)), (i, dist[i], want)
    return dist


@pytest.mark.parametrize("steps,n,k", [(6, 5, 2), (21, 64, 6), (5, 128, 8), (4, 256, 8), (4, 1000, 20), (3, 1024, 64), (3, 1025, 8),
                                        (1003, 100, 5), (515, 200, 16), (67, 129, 2), (9, 256, 17),      # several rows per warp; K past that path

                                        (3, 16384, 20),
                                        (3, 40003, 20), (3, 128256, 20), (2, 151936, 20), (2, 128256, 64),
                                        (2, 300000, 1)])
def test_topk_distance_matches_oracle(imm, ldd, synth, steps, n, k):
    ref = synth.reference_logits(7, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 7, synth.NOISE_QUANTISED)
    claimed = torch.topk(dep, k, dim=1).indices.to(torch.int32).contiguous()      # what the server committed to
    check_topk(imm, ldd, ref, claimed)
    valid = torch.topk(ref, k, dim=1).indices.to(torch.int32).contiguous()
    assert (check_topk(imm, ldd, ref, valid) == 0.0).all()                        # a valid top-K set costs nothing
    rnd = torch.stack([torch.randperm(n, generator=torch.Generator().manual_seed(i))[:k] for i in range(steps)])
    far = check_topk(imm, ldd, ref, rnd.to(torch.int32).cuda().contiguous())
    if n > 4 * k:
        assert (far > 0.0).all()


def test_topk_distance_ties_and_adversarial_rows(imm, ldd):
    n, k = 131072, 20
    rows = [
        torch.zeros(n),                                              # every entry ties
        torch.arange(n, dtype=torch.float32),                        # ascending: thousands of entries above the first bound
        torch.arange(n, 0, -1, dtype=torch.float32),                 # descending
        torch.round(torch.randn(n, generator=torch.Generator().manual_seed(1)) * 2) / 2,   # heavy ties
        torch.cat([torch.full((3000,), 5.0), torch.zeros(n - 3000)]),                      # a plateau above the rest
    ]
    ref = torch.stack(rows).cuda().contiguous()
    g = torch.Generator().manual_seed(2)
    sets = [torch.randperm(n, generator=g)[:k] for _ in rows]
    sets[1] = torch.arange(k)                                        # the K smallest of the ascending row
    topk = torch.stack(sets).to(torch.int32).cuda().contiguous()
    check_topk(imm, ldd, ref, topk, rel=1e-12)


def test_topk_distance_whole_row_inside_and_bad_indices(imm, ldd):
    ref = torch.tensor([[3.0, 1.0, 2.0, 5.0], [0.5, 0.25, 4.0, -1.0]], device="cuda")
    everything = torch.tensor([[0, 1, 2, 3], [3, 2, 1, 0]], dtype=torch.int32, device="cuda")
    assert (check_topk(imm, ldd, ref, everything) == 0.0).all()
    bad = torch.tensor([[0, 0], [1, 7]], dtype=torch.int32, device="cuda")          # repeated; out of range
    dist, status = imm.ldd_topk_distance(ref, bad)
    assert status.cpu().tolist() == [imm.ERR_ARG, imm.ERR_ARG]
    assert all(math.isnan(v) for v in dist.cpu().tolist())
    good_and_bad = torch.tensor([[3, 0], [2, -1]], dtype=torch.int32, device="cuda")
    dist, status = imm.ldd_topk_distance(ref, good_and_bad)
    assert status.cpu().tolist() == [0, imm.ERR_ARG] and float(dist[0]) == 0.0


@pytest.mark.parametrize("n,k", [(100, 4), (256, 8), (1000, 20), (40003, 20), (128256, 20)])
def test_topk_distance_masked_logits(imm, ldd, synth, n, k):
    """Masked entries outside I cost nothing; a masked member of I makes the distance +inf; a row
    with no finite entry likewise.  Checked against the oracle on every kernel family."""
    steps = 6
    ref = synth.reference_logits(22, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 22, synth.NOISE_QUANTISED)
    top = torch.topk(dep, k, dim=1).indices.to(torch.int32).contiguous()
    g = torch.Generator().manual_seed(n + k)
    for i in range(steps):
        mask = (torch.rand(n, generator=g) < (0.5 if i < 3 else 0.95)).cuda()
        mask[top[i].long()] = False
        ref[i, mask] = -math.inf
    ref[2, :min(n, 9000)] = -math.inf                      # a whole slice of a long row, members of I included or not
    ref[4, int(top[4, 1])] = -math.inf                     # a masked member of I
    ref[5, :] = -math.inf                                  # nothing finite
    dist, status = imm.ldd_topk_distance(ref, top)
    dist, status = dist.cpu().numpy(), status.cpu().numpy()
    ys, idx = ref.cpu().numpy(), top.cpu().numpy()
    assert (status == 0).all()
    for i in range(steps):
        want = ldd.topk_distance(ys[i], idx[i])
        if math.isinf(want):
            assert dist[i] == want, (i, dist[i])
        else:
            assert abs(dist[i] - want) <= 1e-9 * max(1.0, abs(want)), (i, dist[i], want)
    assert dist[4] == math.inf and dist[5] == math.inf


def test_malformed_index_sets_cannot_lower_the_tail_statistic(imm, ldd):
    """A committed index set that is repeated or out of range gives a NaN distance, and the tail
    statistic counts NaN as exceeding t1 -- the oracle's rule -- so garbage never lowers p(t1)."""
    rng = np.random.default_rng(23)
    steps, n, k = 40, 300, 5
    ref = torch.from_numpy(rng.normal(0, 2, (steps, n)).astype(np.float32)).cuda()
    top = torch.topk(ref, k, dim=1).indices.to(torch.int32).contiguous()           # valid sets: distance 0
    top[3, 1] = top[3, 0]                                                            # repeated
    top[17, 2] = n + 5                                                               # out of range
    top[18, 0] = -1
    top[30] = torch.topk(-ref[30], k).indices.to(torch.int32)                        # a wrong but well-formed set
    dist, status = imm.ldd_topk_distance(ref, top)
    assert status.cpu().tolist().count(imm.ERR_ARG) == 3
    d = dist.cpu().numpy()
    assert np.isnan(d[[3, 17, 18]]).all() and d[30] > 0 and np.nansum(d) == d[30]
    offsets = np.array([0, 10, 20, 40], dtype=np.int64)
    t1, t2 = 0.5, 0.09
    p, flag = imm.ldd_tail_fraction(dist, torch.from_numpy(offsets).cuda(), t1, t2)
    want = ldd.request_tail_fractions(d, offsets, t1)
    assert want.tolist() == [1 / 10, 2 / 10, 1 / 20]
    assert (p.cpu().numpy() == want).all()
    assert flag.cpu().tolist() == [1, 1, 0] and ldd.flag_requests(d, offsets, t1, t2).tolist() == [True, True, False]
    # a NaN from the TV/KL call (a dead row) counts the same way
    x = ref.clone(); x[7, :] = -math.inf
    tv, _ = imm.ldd_tv_kl(x, ref)
    p2, _ = imm.ldd_tail_fraction(tv, torch.from_numpy(offsets).cuda(), 0.9, 0.0)
    assert p2.cpu().tolist() == [1 / 10, 0.0, 0.0]


def test_tail_fraction_is_exact(imm, ldd, synth):
    steps, requests = 5000, 37
    rng = np.random.default_rng(8)
    d = rng.uniform(0, 0.3, steps)
    d[::17] = 0.1                                                   # entries equal to the threshold do not count
    offsets = synth.request_offsets(8, steps, requests).numpy()
    offsets[5] = offsets[4]                                         # an empty request
    offsets.sort()
    p, flag = imm.ldd_tail_fraction(torch.from_numpy(d).cuda(), torch.from_numpy(offsets).cuda(), 0.1, 0.65)
    want = np.array([ldd.tail_fraction(d[offsets[r]:offsets[r + 1]], 0.1) if offsets[r + 1] > offsets[r] else 0.0
                     for r in range(requests)])
    assert (p.cpu().numpy() == want).all()
    assert (flag.cpu().numpy() == (want > 0.65)).all()


def test_audit_statistic_end_to_end(imm, ldd, synth):
    """Distances on the GPU, then the per-request decision, against the oracle chain.  Steps whose TV
    lies within the TV tolerance of t1 are left out of the count on both sides."""
    steps, n, requests, t1, t2 = 96, 128256, 6, 0.05, 0.2
    ref = synth.reference_logits(9, steps, n, device="cuda")
    dep = synth.deployed_logits(ref, 9, synth.NOISE_QUANTISED)
    tv, _ = imm.ldd_tv_kl(dep, ref)
    offsets = synth.request_offsets(9, steps, requests)
    p, flag = imm.ldd_tail_fraction(tv, offsets.cuda(), t1, t2)
    xs, ys = dep.cpu().numpy(), ref.cpu().numpy()
    want_tv = np.array([ldd.tv_distance(xs[i], ys[i]) for i in range(steps)])
    assert np.abs(tv.cpu().numpy() - want_tv).max() <= TV_TOL
    clear = np.abs(want_tv - t1) > TV_TOL
    assert clear.all(), "pick another seed: a step sits on the threshold"
    off = offsets.numpy()
    want_p = ldd.request_tail_fractions(want_tv, off, t1)
    assert (p.cpu().numpy() == want_p).all()
    assert (flag.cpu().numpy().astype(bool) == ldd.flag_requests(want_tv, off, t1, t2)).all()
    assert 0 < want_p.max() and want_p.min() < 1


def test_topk_workspace_is_checked_and_reusable(imm, ldd, synth):
    steps, n, k = 6, 40000, 20
    ref = synth.reference_logits(12, steps, n, device="cuda")
    top = torch.topk(ref, k, dim=1).indices.to(torch.int32).contiguous()
    need = imm.lib().imm_ldd_topk_workspace(steps, n, k)
    assert need > 0 and imm.lib().imm_ldd_topk_workspace(steps, n, 65) == 0
    with pytest.raises(imm.ImmError) as err:
        imm.ldd_topk_distance(ref, top, workspace=torch.empty(need - 256, dtype=torch.uint8, device="cuda"))
    assert err.value.code == imm.ERR_WORKSPACE
    ws = torch.full((need,), 0xAB, dtype=torch.uint8, device="cuda")          # stale contents must not matter
    d1, s1 = imm.ldd_topk_distance(ref, top, workspace=ws)
    d2, s2 = imm.ldd_topk_distance(ref, top, workspace=ws)
    assert (d1 == 0).all() and (d2 == 0).all() and int(s1.abs().max()) == 0 and int(s2.abs().max()) == 0


def test_ldd_calls_refuse_bad_arguments(imm, synth):
    ref = synth.reference_logits(1, 2, 64, device="cuda")
    with pytest.raises(ValueError):
        imm.ldd_tv_kl(ref.cpu(), ref.cpu())
    with pytest.raises(ValueError):
        imm.ldd_tv_kl(ref, ref[:, :32].contiguous())
    with pytest.raises(imm.ImmError):
        imm.ldd_topk_distance(ref, torch.zeros((2, 65), dtype=torch.int32, device="cuda"))     # K beyond the limit
    with pytest.raises(imm.ImmError):
        imm.ldd_topk_distance(ref[:, :3].contiguous(), torch.zeros((2, 4), dtype=torch.int32, device="cuda"))  # K > n
