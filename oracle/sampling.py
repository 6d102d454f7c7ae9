"""CPU oracle: the speculative (rejection) sampling rule.

TEST INFRASTRUCTURE ONLY -- see oracle/llama.py.  Shares no code with the CUDA path.

Letters.  The paper writes p for the draft and q for the target (Sec. 2.1).  This code
uses the opposite, more common letters: **p = target, q = draft**.  In these letters the
paper's rule (Sec. 2.1 and Sec. 3) reads: draft token j is accepted with probability
min{1, p_j(x_j) / q_j(x_j)}; at the first rejection a replacement is drawn from the
residual max(0, p_j - q_j).  Readings the paper leaves open:

* the residual is printed un-normalised; it is divided by its sum, which the claim "same
  output token distribution as the target" (Sec. 2.1) requires;
* when every draft token is accepted one more token is drawn from the target's next row
  (Sec. 4 "Metrics": block efficiency can reach gamma + 1);
* greedy decoding (Sec. 4 "Decoding"): a draft token is accepted iff it is the argmax of
  the target's row, and the emitted replacement / bonus token is that row's argmax, so
  the output equals the target's own greedy continuation;
* argmax ties go to the lowest index;
* "accepted with probability a" is realised as `u < a` with a supplied uniform u in
  [0, 1), a = min(1, p/q) evaluated with one fp32 division; q == 0 accepts iff p > 0;
* drawing from a weight vector w with a uniform u is an inverse-CDF lookup carried out
  in integers so that the result does not depend on summation order:
  W_k = trunc(w_k * 2^32) (exact), Z = sum W_k, t = floor(Z * floor(u * 2^24) / 2^24),
  result = the smallest k whose inclusive prefix sum exceeds t; if Z == 0, argmax(w).

Uniform layout per block: u[0..gamma-1] are the accept tests, u[gamma] is the single
replacement / bonus draw.

Pinned by tests/test_oracle_sampling.py (chi-squared against p on a small vocabulary,
acceptance rate == sum min(p, q), block-efficiency closed form, exact law by brute
force, special cases, fp64 searchsorted cross-check).
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
TWO32 = F32(4294967296.0)


def softmax_t(logits: np.ndarray, temperature: float) -> np.ndarray:
    """softmax(logits / T) along the last axis, fp32."""
    s = np.asarray(logits, dtype=F32) / F32(temperature)
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m, dtype=F32)
    return e / np.sum(e, axis=-1, keepdims=True, dtype=F32)


def argmax_lowest(x: np.ndarray) -> int:
    return int(np.argmax(x))  # numpy returns the first maximal index


def fixed_point(w: np.ndarray) -> np.ndarray:
    """W_k = trunc(w_k * 2^32) as exact integers (w_k fp32 in [0, 1])."""
    return np.trunc(np.asarray(w, dtype=F32) * TWO32).astype(np.uint64)


def sample_fixed_point(w: np.ndarray, u: float) -> int:
    """Inverse CDF of the weights w (need not sum to 1) at uniform u, in integers."""
    W = fixed_point(w)
    Z = int(W.sum(dtype=np.uint64))
    if Z == 0:
        return argmax_lowest(w)
    u24 = int(np.trunc(F32(u) * F32(16777216.0)))
    t = (Z * u24) >> 24
    cum = np.cumsum(W, dtype=np.uint64)
    return int(np.searchsorted(cum, np.uint64(t), side="right"))


def accept_prob(p_x: float, q_x: float) -> float:
    """min(1, p/q) with one fp32 division; q == 0 -> 1 if p > 0 else 0."""
    p_x, q_x = F32(p_x), F32(q_x)
    if q_x == F32(0.0):
        return F32(1.0) if p_x > F32(0.0) else F32(0.0)
    return min(F32(1.0), p_x / q_x)


def reject_sample(p: np.ndarray, q, ids, u, greedy: bool = False):
    """One block of verification.

    p [gamma+1, V]: target rows (row j scores draft token j+1; row gamma is the bonus row).
    q [gamma, V]:   draft rows the tokens were drawn from (unused when greedy).
    ids [gamma], u [gamma+1].  Returns (n_accepted, next_token).
    """
    gamma = len(ids)
    assert p.shape[0] == gamma + 1
    if greedy:
        for j in range(gamma):
            top = argmax_lowest(p[j])
            if top != int(ids[j]):
                return j, top
        return gamma, argmax_lowest(p[gamma])
    for j in range(gamma):
        x = int(ids[j])
        if not (F32(u[j]) < accept_prob(p[j, x], q[j, x])):
            residual = np.maximum(F32(0.0), p[j].astype(F32) - q[j].astype(F32))
            return j, sample_fixed_point(residual, u[gamma])
    return gamma, sample_fixed_point(p[gamma], u[gamma])


def reject_sample_batch(p, q, ids, u, greedy: bool = False):
    """p [B, gamma+1, V], q [B, gamma, V], ids [B, gamma], u [B, gamma+1]."""
    B = p.shape[0]
    n_acc = np.zeros(B, dtype=np.int32)
    nxt = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n_acc[b], nxt[b] = reject_sample(p[b], None if q is None else q[b], ids[b],
                                         None if u is None else u[b], greedy)
    return n_acc, nxt
