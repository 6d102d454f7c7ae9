"""Pins for the CPU oracle's top-k / top-p truncation (oracle/warp.py).  CPU only.

Checked against things other than the oracle's own code path: rows worked by hand (dyadic
values, so every sum is exact), numpy's sort and fp64 cumulative sums on rows without
near-ties, nesting and switch-off identities, the tie order, and the law of the emitted
token when the truncated rows go through the speculative-sampling rule (it must be the
truncated target row, which is what makes truncation compatible with the method).
"""
import numpy as np
import pytest

from oracle import sampling as S
from oracle import warp

F32 = np.float32


def test_hand_worked_dyadic_rows():
    w = np.array([0.125, 0.5, 0.125, 0.25], dtype=F32)           # order: 1, 3, 0, 2
    np.testing.assert_array_equal(warp.kept_set(w, top_k=2), [False, True, False, True])
    np.testing.assert_array_equal(warp.warp_row(w, top_k=2), np.array([0, 2 / 3, 0, 1 / 3], dtype=F32))
    # cumulative mass along the order: 0.5, 0.75, 0.875, 1.0
    np.testing.assert_array_equal(warp.kept_set(w, top_p=0.7), [False, True, False, True])
    np.testing.assert_array_equal(warp.kept_set(w, top_p=0.75), [False, True, False, True])   # reached exactly
    np.testing.assert_array_equal(warp.kept_set(w, top_p=0.76), [True, True, False, True])    # tie 0 before 2
    np.testing.assert_array_equal(warp.kept_set(w, top_p=0.9), [True, True, True, True])
    np.testing.assert_array_equal(warp.kept_set(w, top_p=0.5), [False, True, False, False])
    np.testing.assert_array_equal(warp.kept_set(w, top_p=0.01), [False, True, False, False])
    # top-k first, top-p relative to what top-k kept: k = 3 keeps {1, 3, 0} with mass 0.875;
    # 0.8 * 0.875 = 0.7 <= 0.75 -> {1, 3}; 0.9 * 0.875 = 0.7875 > 0.75 -> {1, 3, 0}
    np.testing.assert_array_equal(warp.kept_set(w, top_k=3, top_p=0.8), [False, True, False, True])
    np.testing.assert_array_equal(warp.kept_set(w, top_k=3, top_p=0.9), [True, True, False, True])
    out = warp.warp_row(w, top_k=3, top_p=0.9)
    np.testing.assert_array_equal(out, (w / F32(0.875)) * np.array([1, 1, 0, 1], dtype=F32))


def test_ties_go_to_the_lowest_index():
    w = np.full(8, 0.125, dtype=F32)
    np.testing.assert_array_equal(np.flatnonzero(warp.kept_set(w, top_k=3)), [0, 1, 2])
    np.testing.assert_array_equal(np.flatnonzero(warp.kept_set(w, top_p=0.5)), [0, 1, 2, 3])
    np.testing.assert_array_equal(np.flatnonzero(warp.kept_set(w, top_p=0.51)), [0, 1, 2, 3, 4])


def _rows(n, V, seed, scale=3.0):
    g = np.random.default_rng(seed)
    return S.softmax_t(g.standard_normal((n, V)).astype(F32) * F32(scale), 1.0)


@pytest.mark.parametrize("k", [1, 5, 50])
def test_top_k_against_numpy_sort(k):
    for w in _rows(20, 300, 1):
        assert len(np.unique(w)) == len(w)          # no ties: the answer is unique
        keep = warp.kept_set(w, top_k=k)
        assert set(np.flatnonzero(keep)) == set(np.argsort(w)[-k:])
        out = warp.warp_row(w, top_k=k)
        ref = np.where(keep, w.astype(np.float64), 0.0)
        np.testing.assert_allclose(out, ref / ref.sum(), rtol=3e-7, atol=0)
        assert abs(float(out.astype(np.float64).sum()) - 1.0) < 1e-5


@pytest.mark.parametrize("top_p", [0.3, 0.9, 0.99])
def test_top_p_against_fp64_cumulative_sum(top_p):
    checked = 0
    for w in _rows(40, 300, 2):
        order = np.argsort(-w.astype(np.float64), kind="stable")
        cum = np.cumsum(w[order].astype(np.float64))
        n = int(np.searchsorted(cum, top_p * cum[-1], side="left")) + 1
        if min(abs(cum[n - 1] - top_p * cum[-1]), abs(cum[n - 2] - top_p * cum[-1]) if n > 1 else 1.0) < 1e-5:
            continue                                  # too close to the cut for fp64 to decide
        keep = warp.kept_set(w, top_p=top_p)
        assert set(np.flatnonzero(keep)) == set(order[:n])
        # minimality and sufficiency of the nucleus
        assert w[keep].astype(np.float64).sum() >= top_p * cum[-1] - 1e-6
        assert w[keep].astype(np.float64).sum() - w[keep].min() < top_p * cum[-1] + 1e-6
        checked += 1
    assert checked >= 30


def test_nesting_and_switch_off():
    for w in _rows(10, 200, 3):
        prev = np.zeros(len(w), dtype=bool)
        for k in (1, 2, 7, 40, 199):
            keep = warp.kept_set(w, top_k=k)
            assert keep.sum() == k and (keep | prev).sum() == k    # supersets as k grows
            prev = keep
        prev = np.zeros(len(w), dtype=bool)
        for top_p in (0.05, 0.4, 0.8, 0.95, 0.999):
            keep = warp.kept_set(w, top_p=top_p)
            assert (keep | prev).sum() == keep.sum()
            prev = keep
        # switched off: everything is kept and the row changes by the renormalisation only
        for k, top_p in ((0, 1.0), (len(w), 1.0), (-3, 2.0)):
            assert warp.kept_set(w, k, top_p).all()
            np.testing.assert_allclose(warp.warp_row(w, k, top_p), w, rtol=3e-7, atol=0)
        # top-1 and a tiny nucleus are the argmax, with probability one
        for out in (warp.warp_row(w, top_k=1), warp.warp_row(w, top_p=1e-6)):
            assert np.flatnonzero(out).tolist() == [int(np.argmax(w))]
            assert abs(float(out.max()) - 1.0) < 1e-6


def test_truncated_rows_through_the_rule_emit_the_truncated_target_row():
    """Exact law of the first emitted token (sum over draft tokens of the rule's branches) equals
    p' when both rows are truncated -- and differs from the untruncated p."""
    g = np.random.default_rng(4)
    V = 6
    for _ in range(20):
        p = S.softmax_t(g.standard_normal(V).astype(F32) * 2, 1.0)
        q = S.softmax_t(g.standard_normal(V).astype(F32) * 2, 1.0)
        pp, qq = warp.warp_row(p, top_k=4, top_p=0.9), warp.warp_row(q, top_k=4, top_p=0.9)
        P, Q = pp.astype(np.float64), qq.astype(np.float64)
        res = np.maximum(0.0, P - Q)
        res = res / res.sum() if res.sum() > 0 else P
        law = np.zeros(V)
        for x in range(V):
            if Q[x] == 0:
                continue
            a = min(1.0, P[x] / Q[x])
            law[x] += Q[x] * a
            law += Q[x] * (1 - a) * res
        np.testing.assert_allclose(law, P / P.sum(), atol=2e-6)
        assert np.abs(law - p).max() > 1e-3
    # and the sampler itself follows it: 200000 blocks with gamma = 1 on one fixed pair
    n = 200000
    u = g.random((n, 3)).astype(F32)
    counts = np.zeros(V)
    for i in range(n):
        x = S.sample_fixed_point(qq, u[i, 0])
        a, tok = S.reject_sample(np.stack([pp, pp]), qq[None], [x], u[i, 1:])
        counts[x if a == 1 else tok] += 1        # first emitted token: the draft's if accepted
    expect = P / P.sum() * n
    mask = expect > 0
    assert counts[~mask].sum() == 0
    chi2 = float(((counts[mask] - expect[mask]) ** 2 / expect[mask]).sum())
    assert chi2 < 25.0          # 3 degrees of freedom: P(chi2 > 25) ~ 1.5e-5
