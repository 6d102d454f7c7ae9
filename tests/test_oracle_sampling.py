"""Pins for the CPU oracle's rejection-sampling rule (oracle/sampling.py).  CPU only.

Checked against what the paper and the mathematics fix: the output law equals the target's
(Sec. 2.1), the acceptance rate equals sum min(p, q), block efficiency follows the
geometric closed form and never exceeds gamma + 1 (Sec. 4 "Metrics"), a hand-worked dyadic
example enumerated exactly (tests/golden/reject_rule_dyadic.json), the degenerate cases,
and an fp64 library inverse-CDF for the integer sampler.
"""
import json
import os

import numpy as np
import pytest
from scipy import stats

import synth
from oracle import sampling as S
from oracle.spd import block_efficiency_closed_form, mbsu

F32 = np.float32
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "reject_rule_dyadic.json")


def rand_dist(g, V, conc=1.0):
    return S.softmax_t(g.standard_normal(V).astype(F32) * conc, 1.0)


# ------------------------------------------------------------------ exact enumeration

def test_dyadic_example_enumerated_exactly():
    gold = json.load(open(GOLDEN))
    p1 = np.array(gold["p"], F32)
    q1 = np.array(gold["q"], F32)
    p = np.stack([p1, p1])
    q = q1[None]
    grid = (np.arange(64) + 0.5) / 64
    counts = np.zeros(4)
    accepted = 0
    for ud in grid:
        d = S.sample_fixed_point(q1, ud)
        for ua in grid:
            a, _ = S.reject_sample(p, q, [d], [ua, 0.0])
            accepted += a * 64
            for ur in grid:
                a2, nxt = S.reject_sample(p, q, [d], [ua, ur])
                assert a2 == a
                counts[d if a else nxt] += 1
    total = 64 ** 3
    assert np.array_equal(counts / total, gold["first_token_law"])
    assert accepted / total == gold["accept_rate"]
    for x in range(4):
        assert float(S.accept_prob(p1[x], q1[x])) == gold["accept_prob_per_token"][x]


def test_exact_law_by_formula_small_vocab():
    """For random p, q on V <= 4 the law implied by the rule,
    sum_d q(d) [a(d) 1{x=d} + (1 - a(d)) res(x)], equals p (to rounding)."""
    g = np.random.default_rng(0)
    for V in (2, 3, 4):
        for _ in range(20):
            p, q = rand_dist(g, V, 2.0), rand_dist(g, V, 2.0)
            a = np.array([float(S.accept_prob(p[x], q[x])) for x in range(V)])
            res = np.maximum(0, p.astype(np.float64) - q)
            res = res / res.sum() if res.sum() > 0 else res
            law = q * a + (q * (1 - a)).sum() * res
            assert np.abs(law - p).max() < 1e-6


# ------------------------------------------------------------------ statistics, 10^6 trials

@pytest.fixture(scope="module")
def million_trials():
    """gamma = 2, V = 8, the same (p, q) at every position, 10^6 blocks through the
    oracle's own functions."""
    g = np.random.default_rng(1)
    V, gamma, N = 8, 2, 1_000_000
    p1, q1 = rand_dist(g, V, 1.5), rand_dist(g, V, 1.5)
    p = np.stack([p1] * (gamma + 1))
    q = np.stack([q1] * gamma)
    ud = synth.uniforms(31, "chi.draft", (N, gamma))
    uv = synth.uniforms(32, "chi.verify", (N, gamma + 1))
    first = np.zeros(V, np.int64)
    second_given_acc = np.zeros(V, np.int64)
    bonus = np.zeros(V, np.int64)
    n_acc_hist = np.zeros(gamma + 1, np.int64)
    for t in range(N):
        ids = [S.sample_fixed_point(q1, ud[t, 0]), S.sample_fixed_point(q1, ud[t, 1])]
        a, nxt = S.reject_sample(p, q, ids, uv[t])
        emitted = ids[:a] + [nxt]
        n_acc_hist[a] += 1
        first[emitted[0]] += 1
        if a >= 1:
            second_given_acc[emitted[1]] += 1
        if a == gamma:
            bonus[nxt] += 1
    return dict(p=p1, q=q1, first=first, second=second_given_acc, bonus=bonus,
                hist=n_acc_hist, N=N, gamma=gamma)


def test_output_law_equals_target_chi_squared(million_trials):
    r = million_trials
    for counts in (r["first"], r["second"], r["bonus"]):
        e = r["p"].astype(np.float64)
        chi2, pval = stats.chisquare(counts, e / e.sum() * counts.sum())
        assert pval > 1e-4, (chi2, pval)
    # the draft's law q is NOT what comes out (the test has power)
    e = r["q"].astype(np.float64)
    _, pval_q = stats.chisquare(r["first"], e / e.sum() * r["N"])
    assert pval_q < 1e-12


def test_acceptance_rate_is_sum_min(million_trials):
    r = million_trials
    alpha = float(np.minimum(r["p"], r["q"]).sum())
    rate = 1.0 - r["hist"][0] / r["N"]
    sigma = np.sqrt(alpha * (1 - alpha) / r["N"])
    assert abs(rate - alpha) < 4 * sigma


def test_block_efficiency_closed_form(million_trials):
    r = million_trials
    gamma, N = r["gamma"], r["N"]
    tau = (r["hist"] * (np.arange(gamma + 1) + 1)).sum() / N
    alpha = 1.0 - r["hist"][0] / N                     # measured per-token acceptance
    assert tau <= gamma + 1
    assert abs(tau - block_efficiency_closed_form(alpha, gamma)) < 5e-3
    assert block_efficiency_closed_form(1.0, 5) == 6.0
    assert abs(block_efficiency_closed_form(0.5, 2) - 1.75) < 1e-12


# ------------------------------------------------------------------ degenerate cases

def test_identical_models_accept_everything():
    g = np.random.default_rng(2)
    p = np.stack([rand_dist(g, 16) for _ in range(5)])
    u = synth.uniforms(1, "same", (200, 5))
    for t in range(200):
        ids = [S.sample_fixed_point(p[j], u[t, j]) for j in range(4)]
        a, nxt = S.reject_sample(p, p[:4], ids, [0.999999] * 4 + [u[t, 4]])
        assert a == 4 and nxt == S.sample_fixed_point(p[4], u[t, 4])


def test_disjoint_supports_reject_first_and_resample_from_target():
    p1 = np.array([0.5, 0.5, 0, 0], F32)
    q1 = np.array([0, 0, 0.25, 0.75], F32)
    for u in (0.0, 0.3, 0.7, 0.99):
        a, nxt = S.reject_sample(np.stack([p1, p1]), q1[None], [3], [0.0, u])
        assert a == 0 and nxt == (0 if u < 0.5 else 1)


def test_gamma_zero_is_plain_sampling():
    p = np.array([[0.125, 0.5, 0.375]], F32)
    for u, want in ((0.0, 0), (0.124, 0), (0.125, 1), (0.62, 1), (0.625, 2), (0.999, 2)):
        assert S.reject_sample(p, np.zeros((0, 3), F32), [], [u]) == (0, want)


def test_greedy_rule():
    p = np.array([[0.1, 0.7, 0.2], [0.4, 0.4, 0.2], [0.3, 0.3, 0.4]], F32)
    assert S.reject_sample(p, None, [1, 0], None, greedy=True) == (2, 2)   # all match; bonus argmax
    assert S.reject_sample(p, None, [1, 1], None, greedy=True) == (1, 0)   # tie -> lowest index
    assert S.reject_sample(p, None, [0, 0], None, greedy=True) == (0, 1)


def test_zero_draft_probability_edge():
    assert S.accept_prob(0.2, 0.0) == 1.0 and S.accept_prob(0.0, 0.0) == 0.0
    assert S.accept_prob(0.1, 0.4) == F32(0.1) / F32(0.4)
    assert S.accept_prob(0.4, 0.1) == 1.0


# ------------------------------------------------------------------ the integer inverse CDF

def test_fixed_point_sampler_vs_fp64_library_inverse_cdf():
    g = np.random.default_rng(3)
    V = 2000
    w = rand_dist(g, V, 3.0)
    cdf = np.cumsum(w.astype(np.float64))
    Z = cdf[-1]
    us = synth.uniforms(5, "cdf", 3000)
    near = 0
    for u in us:
        k = S.sample_fixed_point(w, u)
        ref = int(np.searchsorted(cdf, float(u) * Z, side="right"))
        if k != ref:
            # only allowed when u*Z is within 2^-20 * Z of a CDF step
            assert abs(k - ref) == 1 and np.min(np.abs(cdf - float(u) * Z)) < 2.0 ** -20 * Z
            near += 1
    assert near < 30
    # integer sums do not depend on order
    W = S.fixed_point(w)
    assert int(W.sum()) == int(W[::-1].sum()) == int(W[g.permutation(V)].sum())
    # scaling by 2^32 and truncation are exact
    assert int(S.fixed_point(np.array([0.5], F32))[0]) == 1 << 31
    assert int(S.fixed_point(np.array([1.0], F32))[0]) == 1 << 32
    assert int(S.fixed_point(np.array([2.0 ** -33], F32))[0]) == 0


def test_unnormalised_weights_and_zero_mass_fallback():
    w = np.array([0.0, 0.02, 0.0, 0.06], F32)            # mass 1/4 and 3/4 after normalising
    picks = [S.sample_fixed_point(w, u) for u in synth.uniforms(6, "un", 4000)]
    frac = np.mean(np.array(picks) == 1)
    assert set(picks) == {1, 3} and abs(frac - 0.25) < 0.03
    assert S.sample_fixed_point(np.array([0.0, 1e-12, 0.0], F32), 0.7) == 1   # Z == 0 -> argmax


def test_softmax_temperature():
    l = np.array([1.0, 2.0, 3.0], F32)
    p = S.softmax_t(l, 1.0)
    assert abs(p.sum() - 1) < 1e-6 and np.allclose(p[1] / p[0], np.e, rtol=1e-5)
    p2 = S.softmax_t(l, 2.0)
    assert np.allclose(p2[1] / p2[0], np.exp(0.5), rtol=1e-5)
    assert np.allclose(S.softmax_t(l + 100, 1.0), p, atol=1e-6)               # shift invariance


def test_mbsu_reading():
    # with the parameter ratio of a 115M draft to a 7B target, the paper's 2.37x needs a
    # block efficiency near 2.5; the formula as printed would give ~0.04 instead
    c = 115e6 / 6.74e9
    assert 2.3 < mbsu(2.5, c, 3) < 2.4
    assert c * 2.5 / (c * 3 + 1) < 0.05


def test_batch_form_is_the_rule_applied_to_each_sequence():
    """reject_sample_batch (the expected value of the bit-exact device tests) must be nothing but
    reject_sample per sequence: checked on sequences whose outcome is known in closed form --
    identical rows accept everything, disjoint supports reject at once, and a dyadic pair whose
    accept probability 1/2 is decided by the uniform -- stacked in one batch, sampling and greedy."""
    V, gamma = 8, 2
    e = lambda k: np.eye(V, dtype=F32)[k]
    half = (e(0) + e(1)) * F32(0.5)
    p = np.stack([np.stack([half] * 3), np.stack([e(3)] * 3), np.stack([e(0), e(0), e(0)]),
                  np.stack([(e(0) + e(2)) * F32(0.5)] * 3)])
    q = np.stack([np.stack([half] * 2), np.stack([e(4)] * 2), np.stack([e(0), e(0)]), np.stack([e(0)] * 2)])
    ids = np.array([[0, 1], [4, 4], [0, 0], [0, 0]], np.int32)
    u = np.array([[0.9, 0.9, 0.75], [0.0, 0.0, 0.5], [0.5, 0.5, 0.1], [0.25, 0.75, 0.3]], F32)
    a, n = S.reject_sample_batch(p, q, ids, u)
    # seq 0: p == q, all accepted, bonus from (1/2, 1/2) at u = .75 -> token 1
    # seq 1: p(x) = 0 -> rejected at once, residual = p -> token 3
    # seq 2: p == q point masses -> all accepted, bonus token 0
    # seq 3: p/q = 1/2: u = .25 accepts, u = .75 rejects; residual = (0, 0, 1/2) -> token 2
    assert a.tolist() == [2, 0, 2, 1] and n.tolist() == [1, 3, 0, 2]
    for b in range(4):
        assert (a[b], n[b]) == S.reject_sample(p[b], q[b], ids[b], u[b])
    ag, ng = S.reject_sample_batch(p, None, ids, None, greedy=True)
    assert ag.tolist() == [1, 0, 2, 2] and ng.tolist() == [0, 3, 0, 0]
    assert a.dtype == np.int32 and n.dtype == np.int32
