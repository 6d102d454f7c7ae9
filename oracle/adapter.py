"""CPU oracle: the image adapter g_theta that turns vision-encoder features into image
embeddings, V_i = g_theta(H_i) (Sec. 2.2), in fp64.

TEST INFRASTRUCTURE ONLY -- see oracle/llama.py.  Shares no code with the CUDA path.

What the paper fixes: the adapter is "a small multi-layer perceptron" (Sec. 2.2) with two
linear layers, 1024 -> 4096 -> 4096 for the LLaVA-7B target and 1024 -> 1024 -> 1024 for a
draft that has its own adapter (Appendix A.1).  Readings the paper leaves open:

* the non-linearity between the two layers is not named; LLaVA's projector is
  Linear - GELU - Linear, so GELU in its exact form x * Phi(x) is used (not the tanh
  approximation);
* biases are not mentioned; none are used, as everywhere else in this model family here;
* the features are used as given (the vision encoder is outside the method's hot path).

Each function is the definition written out; `@` (BLAS dgemm) and `math.erf` are the
library primitives.  Pinned by tests/test_oracle_adapter.py (closed forms and identities
of GELU, torch's GELU in fp64, a triple-loop product on small shapes, shape/transposition
cases).
"""
from __future__ import annotations

import math

import numpy as np

F64 = np.float64
_erf = np.vectorize(math.erf, otypes=[F64])


def gelu(x: np.ndarray) -> np.ndarray:
    """x * Phi(x) with Phi the standard normal CDF, Phi(x) = (1 + erf(x / sqrt 2)) / 2."""
    x = np.asarray(x, dtype=F64)
    return x * (0.5 * (1.0 + _erf(x / math.sqrt(2.0))))


def image_adapter(H: np.ndarray, W1: np.ndarray, W2: np.ndarray) -> np.ndarray:
    """V = GELU(H W1^T) W2^T.

    H [m, d_in] features, W1 [d_hid, d_in], W2 [d_out, d_hid] (row-major [out, in] like every
    matrix of the model).  Returns V [m, d_out] in fp64.
    """
    H, W1, W2 = (np.asarray(a, dtype=F64) for a in (H, W1, W2))
    assert H.shape[1] == W1.shape[1] and W1.shape[0] == W2.shape[1]
    hidden = H @ W1.T
    return gelu(hidden) @ W2.T
