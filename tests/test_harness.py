"""The tolerance helpers of the GPU parity harness, checked on the CPU against hand-worked cases
(they decide whether a difference between the CUDA path and the oracle is inside the stated
tolerance, so a mistake here would silently widen it)."""
import numpy as np

import harness as H
from oracle import sampling as S

F32 = np.float32


def test_safe_uniforms_keep_the_stated_distance_and_plain_uniforms_skip_nothing():
    su = H.SafeUniforms(5, "t")
    for p_x, q_x in ((0.3, 0.6), (0.125, 0.5), (0.2, 0.21)):
        for _ in range(200):
            u = su.for_accept(F32(p_x), F32(q_x))
            assert H.accept_distance(F32(p_x), F32(q_x), u) > H.ACCEPT_TOL
    pu = H.PlainUniforms(5, "t")
    first = [pu.for_accept(F32(0.3), F32(0.6)) for _ in range(50)]
    assert np.array_equal(np.asarray(first, F32), pu.pool[:50]) and pu.skipped == 0
    w = np.full(1000, 1e-3, F32)
    assert pu.for_cdf(w) == pu.pool[50]
    # accept probability 1: every uniform in [0, 1) accepts, none is skipped
    n0 = su.skipped
    for _ in range(50):
        su.for_accept(F32(0.7), F32(0.5))
    assert su.skipped == n0


def test_accept_distance_and_cdf_band():
    assert abs(H.accept_distance(F32(0.25), F32(0.5), 0.5 + 3e-5) - 3e-5) < 1e-7
    assert H.accept_distance(F32(0.6), F32(0.5), 0.25) == 0.75          # min(1, p/q) = 1
    assert H.cdf_band(True, 1e-3) == 2.0 ** -20                          # fp32 models: fixed
    assert abs(H.cdf_band(False, 1e-3) - (2e-3 + 1e-6)) < 1e-12
    assert abs(H.cdf_band(False, 1e-3, 5e-4, 0.25) - (2 * 1.5e-3 / 0.25 + 1e-6)) < 1e-12


def test_token_within_cdf_band_on_a_four_token_row():
    w = np.array([0.25, 0.25, 0.25, 0.25], F32)
    # u = 0.5 + 1e-4: token 2 is the draw; token 1 is allowed only by a band wider than 1e-4
    u = 0.5 + 1e-4
    assert S.sample_fixed_point(w, u) == 2
    assert H.token_within_cdf_band(w, u, 2, 0.0)
    assert not H.token_within_cdf_band(w, u, 1, 5e-5)
    assert H.token_within_cdf_band(w, u, 1, 2e-4)
    assert not H.token_within_cdf_band(w, u, 3, 2e-4) and not H.token_within_cdf_band(w, u, 0, 2e-4)


def test_cut_zone_brackets_every_admissible_kept_set():
    """Perturb the logits of a row by up to eps many times: the kept set of the perturbed row must
    contain `sure`, be contained in `maybe`, and every renormalised probability of a sure token
    must stay within the relative uncertainty rho."""
    from oracle import warp as W
    g = np.random.default_rng(0)
    V, eps = 400, 1e-3
    for top_k, top_p in ((0, 0.9), (25, 1.0), (40, 0.7)):
        logits = (g.standard_normal(V) * 1.5).astype(F32)
        p = S.softmax_t(logits, 1.0)
        z = H.cut_zone(p, top_k, top_p, eps)
        base = W.warp_row(p, top_k, top_p)
        assert z["sure"].sum() > 0 and np.all(z["maybe"][z["sure"]])
        assert np.all(z["maybe"][base > 0]) and np.all(base[z["sure"]] > 0)
        for _ in range(200):
            pert = S.softmax_t(logits + g.uniform(-eps, eps, V).astype(F32), 1.0)
            row = W.warp_row(pert, top_k, top_p)
            kept = row > 0
            assert np.all(kept[z["sure"]]) and not np.any(kept & ~z["maybe"])
            rel = np.abs(row[z["sure"]] / base[z["sure"]] - 1.0)
            assert rel.max() <= z["rho"] + 1e-6
