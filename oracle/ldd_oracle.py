"""CPU oracle for the logit distance distribution (LDD) -- TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, one decision step at a time; no blocking, no fusion.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it; it shares no code with the CUDA
library.

What it follows
  * Definition of the logit distance distribution (Section 4.2): the distances Dis(l_i, l*_i)
    between the logits a deployed execution produced and the reference logits, with Dis the total
    variation distance or the KL divergence between the two vectors.
  * The per-request statistic of Section 5.3: p(t1) = |{i : TV(l_i, l*_i) > t1}| / T, and the
    decision "flag the response if p(t1) > t2".
  * The Top-K distance of the appendix on Top-K verification:
    Delta(l, I) = min over l' with Top_K(l') = I of ||l' - l||_1, evaluated the way that appendix
    does: sort the logits, and for every candidate threshold t = l_(u) add what the entries
    outside I above t have to be lowered and the entries of I below t have to be raised.

Readings (the paper leaves these open)
  * "Distance between two logit vectors" is taken between the softmax distributions of the two
    vectors at temperature 1:  TV = 1/2 * sum_v |p_v - q_v|.
  * The direction of the KL divergence is not stated.  Here KL = KL(q || p) with q = softmax(l*),
    the reference, first:  sum_v q_v (log q_v - log p_v).
  * The comparison in p(t1) is strict (">"), as printed.
  * I is a set of K distinct indices; ties in the logits need no rule because entries equal to the
    threshold cost nothing on either side.
  * Masked entries.  A logit of -inf (a vocabulary entry the sampler has masked out) is a legal
    input: its softmax probability is exactly 0.  The KL sum uses the usual convention
    0 * log(0 / x) = 0, so an entry the reference gives no mass adds nothing, and KL = +inf when
    the reference gives mass to an entry the deployed row masks.  The Top-K cost is minimised over
    finite thresholds; raising a masked member of I to a finite threshold costs +inf, lowering a
    masked outside entry costs nothing.  A row with no finite entry has no softmax: TV and KL are
    NaN (its Top-K distance is +inf, like that of any row whose I has a masked member).
  * A distance that is not a number (such a row, or a malformed committed index set) must not
    help the server: p(t1) counts a step unless its distance is known to be <= t1, so NaN counts
    as exceeding the threshold.  For ordinary numbers this is the printed strict comparison.

Pins (tests/test_oracle_ldd.py): closed forms for two-entry vectors; TV of a vector with itself,
of disjoint peaks, bounds, symmetry, shift invariance; Pinsker's inequality; scipy's softmax /
entropy routines as a second opinion; Top-K distance zero iff I is a valid top-K set, the
swap-one-neighbour closed form, 1-Lipschitz in l, the O(n^2) evaluation of every threshold
straight from the cost definition, and the minimisation solved as a linear programme by scipy on
small cases; masked (-inf) entries against the same functions on the row with those entries
removed, scipy's entropy on distributions with zeros, and the every-threshold evaluation; NaN
distances in the tail count.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


def log_softmax(logits) -> np.ndarray:
    """log softmax(l) in float64: l - max - log(sum exp(l - max)); -inf entries stay -inf
    (probability 0); a row without a finite entry gives NaN throughout."""
    x = np.asarray(logits, dtype=np.float64)
    if not np.isfinite(x).any():
        return np.full(x.shape, np.nan)
    z = x - x.max()
    return z - np.log(np.exp(z).sum())


def softmax(logits) -> np.ndarray:
    return np.exp(log_softmax(logits))


def tv_distance(logits, ref_logits) -> float:
    """Total variation distance between softmax(l) and softmax(l*) (Section 4.2)."""
    p, q = softmax(logits), softmax(ref_logits)
    return 0.5 * float(np.abs(p - q).sum())


def kl_divergence(logits, ref_logits) -> float:
    """KL(softmax(l*) || softmax(l)): the reference distribution first (a reading, see the header)."""
    lp, lq = log_softmax(logits), log_softmax(ref_logits)
    if np.isnan(lp).any() or np.isnan(lq).any():
        return float("nan")
    q = np.exp(lq)
    live = q > 0.0                                             # 0 * log(0 / x) = 0
    with np.errstate(invalid="ignore"):
        return float((q[live] * (lq[live] - lp[live])).sum())


def tail_fraction(distances, t1: float) -> float:
    """p(t1) of Section 5.3 for one request: the share of its steps whose distance exceeds t1.
    A step counts unless its distance is known to be <= t1 (NaN counts: see the header)."""
    d = np.asarray(distances, dtype=np.float64)
    return float((~(d <= t1)).sum()) / float(d.size)


def request_tail_fractions(distances, offsets, t1: float) -> np.ndarray:
    """p(t1) for each request; request r owns the steps offsets[r] .. offsets[r+1]-1."""
    return np.array([tail_fraction(distances[offsets[r]:offsets[r + 1]], t1) for r in range(len(offsets) - 1)],
                    dtype=np.float64)


def flag_requests(distances, offsets, t1: float, t2: float) -> np.ndarray:
    """Section 5.3: a response is flagged when p(t1) > t2."""
    return request_tail_fractions(distances, offsets, t1) > t2


def topk_cost(logits, index_set, t: float) -> float:
    """L1 cost of making `index_set` the top-K set with threshold t: entries of I are raised to
    max(l_i, t), the others lowered to min(l_j, t) (the greedy choice of the appendix)."""
    x = np.asarray(logits, dtype=np.float64)
    inside = np.zeros(x.size, dtype=bool)
    inside[np.asarray(index_set, dtype=np.int64)] = True
    return float(np.maximum(x[~inside] - t, 0.0).sum() + np.maximum(t - x[inside], 0.0).sum())


def topk_distance_all_thresholds(logits, index_set) -> float:
    """Delta(l, I) by trying every finite entry of l as the threshold: O(n^2), small inputs only."""
    x = np.asarray(logits, dtype=np.float64)
    finite = x[np.isfinite(x)]
    if finite.size == 0:
        return float("inf")
    return min(topk_cost(x, index_set, float(t)) for t in finite)


def topk_distance(logits, index_set) -> float:
    """Delta(l, I) the way the appendix computes it: sort the logits in descending order; with
    the threshold at the u-th largest entry, the entries outside I among the first u are lowered
    to it and the entries of I after the u-th are raised to it; take the best u."""
    x = np.asarray(logits, dtype=np.float64)
    idx = np.asarray(index_set, dtype=np.int64)
    assert idx.size == np.unique(idx).size and idx.size <= x.size
    inside = np.zeros(x.size, dtype=bool)
    inside[idx] = True
    order = np.argsort(-x, kind="stable")
    xs, ins = x[order], inside[order]
    nfin = int(np.isfinite(xs).sum())                          # masked (-inf) entries sort last
    if ins[nfin:].any():                                       # a masked member of I cannot be raised
        return float("inf")
    xs, ins = xs[:nfin], ins[:nfin]                            # masked outside entries cost nothing
    out_cnt = np.cumsum(~ins)                                  # entries outside I among the first u
    out_sum = np.cumsum(np.where(ins, 0.0, xs))
    in_cnt_after = ins.sum() - np.cumsum(ins)                  # entries of I after the u-th
    in_sum_after = np.where(ins, xs, 0.0).sum() - np.cumsum(np.where(ins, xs, 0.0))
    cost = (out_sum - out_cnt * xs) + (in_cnt_after * xs - in_sum_after)
    return float(cost.min())


def top_k(logits, k: int) -> np.ndarray:
    """Indices of the k largest entries (ties to the lower index), the operator Top_K."""
    x = np.asarray(logits, dtype=np.float64)
    return np.argsort(-x, kind="stable")[:k]
