"""Pins of the LDD oracle (oracle/ldd_oracle.py) against closed forms, library routines, brute force
and a linear-programme solver.  CPU only."""
import math

import numpy as np
import pytest

from oracle import ldd


def sigmoid(x):
    return 1.0 / (1.0 + math.exp(-x))


def bernoulli_kl(q, p):
    return q * math.log(q / p) + (1 - q) * math.log((1 - q) / (1 - p))


# ------------------------------------------------------------------ TV / KL


@pytest.mark.parametrize("a,b", [(0.0, 0.0), (1.5, -0.25), (-3.0, 4.0), (10.0, 9.0)])
def test_two_entry_closed_forms(a, b):
    """n = 2: softmax([x, 0]) = (sigmoid(x), 1 - sigmoid(x)); TV = |sigmoid(a) - sigmoid(b)|."""
    l, ls = np.array([a, 0.0]), np.array([b, 0.0])
    assert ldd.tv_distance(l, ls) == pytest.approx(abs(sigmoid(a) - sigmoid(b)), abs=1e-15)
    assert ldd.kl_divergence(l, ls) == pytest.approx(bernoulli_kl(sigmoid(b), sigmoid(a)), abs=1e-14)


def test_kl_direction_is_reference_first():
    """KL(q || p) with q from the reference logits: not symmetric, so the order is observable."""
    l, ls = np.array([2.0, 0.0]), np.array([-1.0, 0.0])
    forward = bernoulli_kl(sigmoid(-1.0), sigmoid(2.0))
    backward = bernoulli_kl(sigmoid(2.0), sigmoid(-1.0))
    assert abs(forward - backward) > 0.1
    assert ldd.kl_divergence(l, ls) == pytest.approx(forward, abs=1e-14)


def test_tv_kl_basic_properties():
    rng = np.random.default_rng(1)
    for n in (3, 17, 1000):
        l, ls = rng.normal(0, 3, n), rng.normal(0, 3, n)
        tv, kl = ldd.tv_distance(l, ls), ldd.kl_divergence(l, ls)
        assert 0.0 < tv < 1.0 and kl > 0.0
        assert ldd.tv_distance(l, l) == 0.0 and abs(ldd.kl_divergence(l, l)) < 1e-15
        assert ldd.tv_distance(ls, l) == pytest.approx(tv, abs=1e-15)               # symmetric
        assert ldd.tv_distance(l + 7.25, ls - 3.5) == pytest.approx(tv, abs=1e-13)  # shift invariant
        assert ldd.kl_divergence(l + 7.25, ls - 3.5) == pytest.approx(kl, abs=1e-12)
        assert tv <= math.sqrt(kl / 2) + 1e-15                                       # Pinsker
        # TV = 1 - sum min(p, q) = sum max(p - q, 0)
        p, q = ldd.softmax(l), ldd.softmax(ls)
        assert tv == pytest.approx(1.0 - np.minimum(p, q).sum(), abs=1e-14)


def test_disjoint_peaks_give_distance_one():
    l = np.full(50, -1000.0); l[3] = 0.0
    ls = np.full(50, -1000.0); ls[40] = 0.0
    assert ldd.tv_distance(l, ls) == pytest.approx(1.0, abs=1e-300)
    assert ldd.softmax(l)[3] == 1.0


def test_against_scipy_routines():
    from scipy.special import softmax as sp_softmax
    from scipy.stats import entropy
    rng = np.random.default_rng(2)
    for n in (5, 300, 5000):
        l, ls = rng.normal(0, 4, n), rng.normal(0, 4, n)
        p, q = sp_softmax(l), sp_softmax(ls)
        assert np.allclose(ldd.softmax(l), p, rtol=1e-13, atol=0)
        assert ldd.tv_distance(l, ls) == pytest.approx(0.5 * np.abs(p - q).sum(), abs=1e-14)
        assert ldd.kl_divergence(l, ls) == pytest.approx(entropy(q, p), rel=1e-11)


def test_large_logits_do_not_overflow():
    l = np.array([1e4, 1e4 - 1.0, -1e4]); ls = np.array([1e4 - 1.0, 1e4, -1e4])
    assert ldd.tv_distance(l, ls) == pytest.approx(abs(sigmoid(1.0) - sigmoid(-1.0)), abs=1e-12)


def test_masked_entries_have_probability_zero():
    """-inf logits: the distances are those of the rows with the masked entries removed, where both
    rows mask the same entries; scipy's entropy (which treats 0 log 0 as 0 and q > 0 = p as inf) as a
    second opinion where they differ."""
    from scipy.stats import entropy
    rng = np.random.default_rng(11)
    n = 40
    l, ls = rng.normal(0, 3, n), rng.normal(0, 3, n)
    mask = rng.random(n) < 0.3
    lm, lsm = np.where(mask, -np.inf, l), np.where(mask, -np.inf, ls)
    assert ldd.softmax(lm)[mask].tolist() == [0.0] * int(mask.sum())
    assert ldd.softmax(lm).sum() == pytest.approx(1.0, abs=1e-15)
    assert ldd.tv_distance(lm, lsm) == pytest.approx(ldd.tv_distance(l[~mask], ls[~mask]), abs=1e-15)
    assert ldd.kl_divergence(lm, lsm) == pytest.approx(ldd.kl_divergence(l[~mask], ls[~mask]), abs=1e-14)
    # only the reference masks: those entries add nothing to KL(q || p); TV sees p's mass there
    p, q = ldd.softmax(l), ldd.softmax(lsm)
    assert ldd.kl_divergence(l, lsm) == pytest.approx(entropy(q, p), rel=1e-12)
    assert ldd.tv_distance(l, lsm) == pytest.approx(0.5 * np.abs(p - q).sum(), abs=1e-15)
    assert math.isfinite(ldd.kl_divergence(l, lsm))
    # only the deployed row masks an entry the reference gives mass: infinite divergence, finite TV
    assert ldd.kl_divergence(lm, ls) == math.inf and entropy(ldd.softmax(ls), ldd.softmax(lm)) == math.inf
    assert 0.0 < ldd.tv_distance(lm, ls) <= 1.0
    # two-entry closed form with a third, masked entry
    a, b = 1.5, -0.25
    assert ldd.tv_distance([a, 0.0, -np.inf], [b, 0.0, -np.inf]) == pytest.approx(abs(sigmoid(a) - sigmoid(b)), abs=1e-15)
    assert ldd.kl_divergence([a, -np.inf, 0.0], [b, -np.inf, 0.0]) == pytest.approx(bernoulli_kl(sigmoid(b), sigmoid(a)), abs=1e-14)
    # no finite entry: no distribution
    dead = np.full(5, -np.inf)
    assert math.isnan(ldd.tv_distance(dead, l[:5])) and math.isnan(ldd.kl_divergence(l[:5], dead))


# ------------------------------------------------------------------ tail statistic


def test_tail_fraction_and_flags():
    d = np.array([0.05, 0.2, 0.1, 0.100001, 0.0, 0.3, 0.3, 0.01])
    assert ldd.tail_fraction(d, 0.1) == 4 / 8                      # strict: the entry equal to t1 does not count
    offsets = [0, 3, 8]
    p = ldd.request_tail_fractions(d, offsets, 0.1)
    assert p.tolist() == [1 / 3, 3 / 5]
    assert ldd.flag_requests(d, offsets, 0.1, 0.5).tolist() == [False, True]
    assert ldd.flag_requests(d, offsets, 0.1, 0.6).tolist() == [False, False]   # strict in t2 as well


def test_tail_fraction_counts_what_is_not_known_to_be_below():
    """NaN (a malformed index set, a row without a distribution) and +inf count as exceeding t1; for
    ordinary numbers the rule is the strict comparison."""
    d = np.array([0.05, np.nan, 0.1, np.inf, 0.2, np.nan])
    assert ldd.tail_fraction(d, 0.1) == 4 / 6
    assert ldd.tail_fraction(np.array([np.nan]), 1e9) == 1.0
    assert ldd.flag_requests(d, [0, 3, 6], 0.1, 0.5).tolist() == [False, True]
    rng = np.random.default_rng(12)
    x = rng.uniform(0, 1, 1000)
    assert ldd.tail_fraction(x, 0.4) == float((x > 0.4).sum()) / 1000


# ------------------------------------------------------------------ Top-K distance


def test_topk_distance_zero_iff_valid_topk():
    rng = np.random.default_rng(3)
    for n, k in ((10, 3), (64, 6), (500, 20)):
        l = rng.normal(0, 2, n)
        good = ldd.top_k(l, k)
        assert ldd.topk_distance(l, good) == 0.0
        bad = good.copy()
        bad[0] = np.argsort(-l)[k + 4]                           # replace one member by a smaller entry
        assert ldd.topk_distance(l, bad) > 0.0
    # ties: any K-subset containing everything above the tie value is valid
    l = np.array([5.0, 3.0, 3.0, 3.0, 1.0])
    for I in ([0, 1], [0, 2], [0, 3]):
        assert ldd.topk_distance(l, I) == 0.0
    assert ldd.topk_distance(l, [1, 2]) == 2.0                    # 5 has to come down to 3


def test_topk_distance_closed_forms():
    # n = 2, K = 1: choosing the smaller entry costs the gap
    assert ldd.topk_distance([4.0, 1.5], [1]) == 2.5
    assert ldd.topk_distance([4.0, 1.5], [0]) == 0.0
    # true top-K with its smallest member swapped for the next entry: the gap between the two
    l = np.array([9.0, 7.0, 6.5, 4.0, 3.0, -1.0])
    assert ldd.topk_distance(l, [0, 1, 3]) == pytest.approx(6.5 - 4.0)
    # the worst K entries of a strictly decreasing vector with K = 1: everything above has to meet it
    l = np.array([3.0, 2.0, 1.0])
    # I = {2}: t in [1, 3]; cost(t) = (3 - t)+ + (2 - t)+ + (t - 1); minimum 2 at t = 2
    assert ldd.topk_distance(l, [2]) == 2.0


def test_topk_distance_matches_every_threshold_evaluation():
    rng = np.random.default_rng(4)
    for trial in range(40):
        n = int(rng.integers(2, 60))
        k = int(rng.integers(1, n + 1))
        l = np.round(rng.normal(0, 2, n), 1 if trial % 2 else 6)   # rounded values give ties
        I = rng.choice(n, size=k, replace=False)
        assert ldd.topk_distance(l, I) == pytest.approx(ldd.topk_distance_all_thresholds(l, I), abs=1e-12)


def test_topk_distance_with_masked_entries():
    """-inf entries outside I cost nothing (the distance is that of the row without them); a masked
    member of I cannot be raised to any finite threshold."""
    rng = np.random.default_rng(13)
    for trial in range(30):
        n = int(rng.integers(6, 50))
        k = int(rng.integers(1, 5))
        l = np.round(rng.normal(0, 2, n), 1 if trial % 2 else 6)
        I = rng.choice(n, size=k, replace=False)
        inside = np.zeros(n, dtype=bool); inside[I] = True
        mask = (rng.random(n) < 0.4) & ~inside
        lm = np.where(mask, -np.inf, l)
        keep = np.flatnonzero(~mask)
        I_kept = [int(np.flatnonzero(keep == i)[0]) for i in I]
        want = ldd.topk_distance(l[keep], I_kept)
        assert ldd.topk_distance(lm, I) == pytest.approx(want, abs=1e-12)
        assert ldd.topk_distance_all_thresholds(lm, I) == pytest.approx(want, abs=1e-12)
        lm2 = lm.copy(); lm2[I[0]] = -np.inf
        assert ldd.topk_distance(lm2, I) == math.inf and ldd.topk_distance_all_thresholds(lm2, I) == math.inf
    assert ldd.topk_distance(np.full(4, -np.inf), [1]) == math.inf
    # a masked entry is a valid non-member: the true top-K of the finite part still costs nothing
    assert ldd.topk_distance([3.0, -np.inf, 2.0, 1.0], [0, 2]) == 0.0


def test_topk_distance_is_the_l1_minimum_linear_programme():
    """min sum |l' - l| s.t. l'_i >= t (i in I), l'_j <= t (j not in I), solved by scipy's LP solver."""
    from scipy.optimize import linprog
    rng = np.random.default_rng(5)
    for trial in range(12):
        n = int(rng.integers(3, 14))
        k = int(rng.integers(1, n))
        l = rng.normal(0, 2, n)
        I = rng.choice(n, size=k, replace=False)
        inside = np.zeros(n, dtype=bool); inside[I] = True
        # variables: up_i >= 0 (raise), down_i >= 0 (lower), t free; l' = l + up - down
        c = np.concatenate([np.ones(2 * n), [0.0]])
        A, b = [], []
        for i in range(n):
            row = np.zeros(2 * n + 1)
            if inside[i]:          # l_i + up_i - down_i >= t   ->  -up_i + down_i + t <= l_i
                row[i], row[n + i], row[2 * n] = -1.0, 1.0, 1.0
                A.append(row); b.append(l[i])
            else:                  # l_i + up_i - down_i <= t   ->   up_i - down_i - t <= -l_i
                row[i], row[n + i], row[2 * n] = 1.0, -1.0, -1.0
                A.append(row); b.append(-l[i])
        res = linprog(c, A_ub=np.array(A), b_ub=np.array(b), bounds=[(0, None)] * (2 * n) + [(None, None)])
        assert res.status == 0
        assert ldd.topk_distance(l, I) == pytest.approx(res.fun, abs=1e-8)


def test_topk_distance_is_one_lipschitz():
    rng = np.random.default_rng(6)
    for _ in range(50):
        n, k = 80, 7
        l = rng.normal(0, 2, n)
        I = rng.choice(n, size=k, replace=False)
        noise = rng.normal(0, 0.05, n)
        d0, d1 = ldd.topk_distance(l, I), ldd.topk_distance(l + noise, I)
        assert abs(d0 - d1) <= np.abs(noise).sum() + 1e-12


def test_topk_distance_only_depends_on_the_top_k_outside_values():
    """Lowering entries outside I that are not among the K largest outside I changes nothing:
    the minimising threshold never lies below the K-th largest outside entry."""
    rng = np.random.default_rng(7)
    for _ in range(30):
        n, k = 200, 5
        l = rng.normal(0, 2, n)
        I = rng.choice(n, size=k, replace=False)
        inside = np.zeros(n, dtype=bool); inside[I] = True
        outside_sorted = np.argsort(-np.where(inside, -np.inf, l))
        rest = outside_sorted[k:n - k]                              # outside entries below the K largest
        l2 = l.copy()
        l2[rest] -= rng.uniform(0, 5, rest.size)
        assert ldd.topk_distance(l2, I) == pytest.approx(ldd.topk_distance(l, I), abs=1e-12)
