"""Pins for the CPU oracle's image adapter (oracle/adapter.py).  CPU only.

GELU is checked against things that do not go through the oracle's own erf call: tabulated
values of the normal CDF, a numerical integral of the normal density, torch's GELU and
scipy's normal CDF in fp64, and the identities of x * Phi(x).  The two-layer map is checked
against a triple loop on small non-square shapes and against its linear limit.
"""
import math

import numpy as np
import torch
from scipy.stats import norm

from oracle import adapter


def test_gelu_tabulated_values_of_the_normal_cdf():
    # Phi(1) = 0.8413447460685429, Phi(2) = 0.9772498680518208 (standard tables)
    got = adapter.gelu(np.array([0.0, 1.0, -1.0, 2.0, -2.0]))
    want = np.array([0.0, 0.8413447460685429, -(1.0 - 0.8413447460685429), 2 * 0.9772498680518208,
                     -2 * (1.0 - 0.9772498680518208)])
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-14)
    # the tanh approximation gives 0.84119 at x = 1: the exact form must not be confused with it
    assert abs(got[1] - 0.841192) > 1e-4


def test_gelu_against_a_numerical_integral_of_the_normal_density():
    xs = np.array([-3.0, -0.7, 0.3, 1.9])
    for x in xs:
        t = np.linspace(-12.0, x, 400001)
        pdf = np.exp(-0.5 * t * t) / math.sqrt(2 * math.pi)
        cdf = np.sum((pdf[1:] + pdf[:-1]) * 0.5 * np.diff(t))
        assert abs(adapter.gelu(np.array([x]))[0] - x * cdf) < 1e-9


def test_gelu_matches_library_routines_in_fp64():
    x = np.random.default_rng(0).standard_normal(5000) * 3
    np.testing.assert_allclose(adapter.gelu(x), torch.nn.functional.gelu(torch.from_numpy(x)).numpy(),
                               rtol=0, atol=1e-14)
    np.testing.assert_allclose(adapter.gelu(x), x * norm.cdf(x), rtol=0, atol=1e-14)


def test_gelu_identities():
    x = np.random.default_rng(1).standard_normal(1000) * 4
    # x Phi(x) - (-x) Phi(-x) = x (Phi(x) + Phi(-x)) = x
    np.testing.assert_allclose(adapter.gelu(x) - adapter.gelu(-x), x, rtol=0, atol=1e-13)
    big = np.array([12.0, 30.0])
    np.testing.assert_allclose(adapter.gelu(big), big, rtol=0, atol=1e-12)
    np.testing.assert_allclose(adapter.gelu(-big), 0.0, rtol=0, atol=1e-12)
    h = 1e-6   # slope 1/2 at the origin
    assert abs(adapter.gelu(np.array([h]))[0] / h - 0.5) < 1e-6
    # curvature at the origin is 2 * phi(0) = sqrt(2 / pi)
    second = (adapter.gelu(np.array([h * 1e3]))[0] + adapter.gelu(np.array([-h * 1e3]))[0]) / (h * 1e3) ** 2
    assert abs(second - math.sqrt(2 / math.pi)) < 1e-6


def test_adapter_against_triple_loop_on_non_square_shapes():
    g = np.random.default_rng(2)
    m, d_in, d_hid, d_out = 3, 5, 7, 4
    H, W1, W2 = g.standard_normal((m, d_in)), g.standard_normal((d_hid, d_in)), g.standard_normal((d_out, d_hid))
    want = np.zeros((m, d_out))
    for i in range(m):
        hid = [sum(H[i, k] * W1[j, k] for k in range(d_in)) for j in range(d_hid)]
        act = [h * 0.5 * (1.0 + math.erf(h / math.sqrt(2.0))) for h in hid]
        for o in range(d_out):
            want[i, o] = sum(act[j] * W2[o, j] for j in range(d_hid))
    got = adapter.image_adapter(H, W1, W2)
    assert got.shape == (m, d_out)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def test_adapter_linear_limit_and_row_independence():
    g = np.random.default_rng(3)
    H = g.uniform(1.0, 2.0, (4, 6))
    W1 = g.uniform(4.0, 5.0, (8, 6))    # hidden values >= 24: GELU is the identity there to 1e-100
    W2 = g.standard_normal((5, 8))
    np.testing.assert_allclose(adapter.image_adapter(H, W1, W2), H @ W1.T @ W2.T, rtol=1e-13, atol=0)
    # each output row depends on its own feature row only
    W1n = g.standard_normal((8, 6))
    full = adapter.image_adapter(H, W1n, W2)
    for i in range(4):
        np.testing.assert_allclose(adapter.image_adapter(H[i:i + 1], W1n, W2)[0], full[i], rtol=0, atol=1e-13)
    # zero features give zero embeddings (no bias)
    assert np.all(adapter.image_adapter(np.zeros((2, 6)), W1n, W2) == 0.0)
