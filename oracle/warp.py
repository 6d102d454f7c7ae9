"""CPU oracle: top-k / top-p (nucleus) truncation of a probability row before the
speculative-sampling rule.

TEST INFRASTRUCTURE ONLY -- see oracle/llama.py.  Shares no code with the CUDA path.

The paper evaluates greedy decoding only and leaves "sampling-based decoding (varying
temperature, varying top-p, top-k)" to future work (Sec. 4 "Decoding").  The standard way
to combine truncated sampling with speculative decoding, used here, is to truncate and
renormalise BOTH distributions, p' = trunc(p) for the target and q' = trunc(q) for the
draft, draw the draft tokens from q' and apply the unchanged rule of oracle/sampling.py to
(p', q'): the output is then distributed as p'.

Definitions (the usual ones, made exact so that two implementations agree bit for bit):

* order: tokens are ranked by probability, larger first; equal probabilities rank by
  index, lower first (fp32 comparisons are exact, so the order has no rounding);
* mass: the mass of token i is the integer W_i = trunc(w_i * 2^32) of oracle/sampling.py,
  sums of masses are integer sums;
* top-k (k >= 1): keep the first k tokens of the order;
* top-p (0 < top_p < 1): among the tokens still kept, with total mass Z, keep the shortest
  prefix of the order whose mass reaches T = ceil(Z * trunc(top_p * 2^24) / 2^24), at least
  one token;
* top-k is applied first, then top-p on what it kept (top_p is relative to the kept mass);
  k <= 0 or k >= V switches top-k off, top_p >= 1 switches top-p off;
* renormalisation: with Z' the integer mass of the kept set and S = fp32(Z') * 2^-32 (one
  round-to-nearest conversion), p'_i = w_i / S (one fp32 division) for kept tokens and 0
  for the others; if Z' == 0 (underflow only) the kept values stay as they are.

Pinned by tests/test_oracle_warp.py (hand-worked dyadic rows, numpy sort / cumsum in fp64,
nesting and switch-off identities, tie order, the emitted-token law of the full rule).
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
TWO32 = F32(4294967296.0)


def _mass(w: np.ndarray) -> np.ndarray:
    return np.trunc(np.asarray(w, dtype=F32) * TWO32).astype(np.uint64)


def kept_set(w: np.ndarray, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """Boolean mask of the tokens that survive top-k followed by top-p."""
    w = np.asarray(w, dtype=F32)
    V = w.shape[0]
    # rank: larger probability first, lower index first among equals (stable sort on -w)
    order = np.argsort(-w.astype(np.float64), kind="stable")
    n = V
    if 1 <= top_k < V:
        n = top_k
    order = order[:n]
    if 0.0 < top_p < 1.0:
        W = _mass(w[order])
        Z = int(W.sum(dtype=np.uint64))
        if Z > 0:
            p24 = int(np.trunc(F32(top_p) * F32(16777216.0)))
            T = max(1, (Z * p24 + (1 << 24) - 1) >> 24)
            cum = np.cumsum(W, dtype=np.uint64)
            n = int(np.searchsorted(cum, np.uint64(T), side="left")) + 1   # first prefix with cum >= T
            order = order[:n]
    keep = np.zeros(V, dtype=bool)
    keep[order] = True
    return keep


def warp_row(w: np.ndarray, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """Truncated, renormalised row p' (fp32)."""
    w = np.asarray(w, dtype=F32)
    keep = kept_set(w, top_k, top_p)
    Zk = int(_mass(w[keep]).sum(dtype=np.uint64))
    out = np.zeros_like(w)
    if Zk == 0:
        out[keep] = w[keep]
        return out
    S = F32(np.uint64(Zk)) * F32(2.0 ** -32)
    out[keep] = w[keep] / S
    return out


def warp_rows(p: np.ndarray, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """Every row along the last axis."""
    p = np.asarray(p, dtype=F32)
    flat = p.reshape(-1, p.shape[-1])
    return np.stack([warp_row(r, top_k, top_p) for r in flat]).reshape(p.shape)
