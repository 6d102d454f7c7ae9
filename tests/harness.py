"""Shared helpers of the GPU parity tests: build the CUDA context and the CPU oracle from
the same seeded inputs, and drive both in lock-step.

Sampling decisions compare a floating-point quantity with a uniform.  The two sides agree
bit for bit only when that quantity is not within rounding distance of the uniform.  Two
uniform sources exist:

* SafeUniforms: the ORACLE chooses each uniform from a seeded stream and skips candidates that
  fall inside the stated tolerance of a decision boundary: |u - min(1, p/q)| <= 1e-4 for an
  accept test (the tolerance this path is held to), 2e-6 * Z around a CDF step for a draw.
  Inputs depend on the oracle and the seed only, never on the CUDA path, and every compared
  decision then has exactly one answer inside the tolerance.
* PlainUniforms: the seeded stream taken as it is.  A differing decision must then lie inside
  the tolerance (checked by the caller with the helpers below) and is counted.
"""
from __future__ import annotations

import numpy as np

import synth
from oracle import llama, sampling as S, warp as W
from oracle.spd import SpdOracle

F32 = np.float32
ACCEPT_TOL = 1e-4          # accept/reject decisions may differ only where |u - min(1, p/q)| < 1e-4
CDF_TOL_FP32 = 2.0 ** -20  # fp32 models: a drawn token may differ only if u*Z is this close (x Z) to a CDF step


def build_weights(wl, std=0.02):
    tw = synth.Weights(wl.target, wl.seeds["weights"], "target", std=std)
    dw = synth.Weights(wl.draft, wl.seeds["weights"], "draft", adapter_in=0 if wl.draft_mlp else wl.adapter_in,
                       std=std)
    return tw, dw


def make_oracle(wl, tw, dw, max_seq, temperature=1.0, greedy=False, top_k=0, top_p=1.0):
    t = llama.Model(wl.target, tw, max_seq)
    d = llama.Model(wl.draft, dw, max_seq)
    ad = dw.f32("adapter") if wl.adapter_in and not wl.draft_mlp else None
    return SpdOracle(t, d, temperature, greedy, adapter_w=ad, top_k=top_k, top_p=top_p)


def make_gpu(wl, tw, dw, max_seq, temperature=1.0, greedy=False, gamma_max=7, grid_mode=0, top_k=0, top_p=0.0):
    import paper_2404_08856_b200 as spd
    return spd.Spd(wl.target, wl.draft, tw.stored, dw.stored, max_seq, gamma_max, temperature, greedy,
                   adapter_in=wl.draft.d_model if wl.draft_mlp else wl.adapter_in, grid_mode=grid_mode,
                   top_k=top_k, top_p=top_p)


class SafeUniforms:
    """Seeded stream of uniforms on the 2^-24 grid from which the oracle side picks the
    first candidate that keeps a decision away from its boundary."""

    def __init__(self, seed, tag, accept_margin=ACCEPT_TOL, cdf_margin=2e-6, n=1 << 16):
        self.pool = synth.uniforms(seed, tag, n)
        self.i = 0
        self.skipped = 0
        self.accept_margin, self.cdf_margin = accept_margin, cdf_margin

    def _next(self):
        u = self.pool[self.i]
        self.i += 1
        return F32(u)

    def for_cdf(self, w):
        """u whose inverse-CDF threshold is at least cdf_margin * Z from both ends of the
        selected token's interval."""
        W = S.fixed_point(w).astype(np.float64)
        cum = np.cumsum(W)
        Z = cum[-1]
        while True:
            u = self._next()
            t = Z * float(u)
            k = int(np.searchsorted(cum, t, side="right"))
            lo = cum[k - 1] if k else 0.0
            if t - lo > self.cdf_margin * Z and cum[k] - t > self.cdf_margin * Z:
                return u
            self.skipped += 1

    def for_accept(self, p_x, q_x):
        a = float(S.accept_prob(p_x, q_x))
        while True:
            u = self._next()
            if abs(float(u) - a) > self.accept_margin or (a >= 1.0):
                return u
            self.skipped += 1

    # hooks for SpdOracle.draft / SpdOracle.verify
    def draft_hook(self, j, prob):
        return self.for_cdf(prob)

    def verify_hook(self, p, q, ids):
        gamma = len(ids)
        u = np.zeros(gamma + 1, dtype=F32)
        r = gamma
        for j in range(gamma):
            x = int(ids[j])
            u[j] = self.for_accept(p[j, x], q[j, x])
            if r == gamma and not (u[j] < S.accept_prob(p[j, x], q[j, x])):
                r = j
        w = p[gamma] if r == gamma else np.maximum(F32(0), p[r] - q[r])
        u[gamma] = self.for_cdf(w)
        return u


class PlainUniforms(SafeUniforms):
    """The seeded stream as it is: no candidate is skipped."""

    def for_cdf(self, w):
        return self._next()

    def for_accept(self, p_x, q_x):
        return self._next()


def accept_distance(p_x, q_x, u):
    """|u - min(1, p/q)| with the oracle's values: how far a uniform is from flipping the test."""
    return abs(float(u) - float(S.accept_prob(p_x, q_x)))


def cdf_band(fp32_model, err_p, err_q=0.0, residual_mass=1.0):
    """Relative half-width (in units of Z) of the region around a CDF step in which the two sides
    may draw neighbouring tokens.  A logit error eps moves every probability by a factor within
    exp(+-2 eps), so a normalised prefix sum of a softmax row moves by at most 2 eps; for the
    residual max(0, p - q) the weights move by 2 eps_p p + 2 eps_q q and are normalised by the
    residual's own mass, which gives 2 (eps_p + eps_q) / mass.  fp32 models are held to the fixed
    2^-20 instead (their logit error is ~1e-5, below the skip margin of SafeUniforms)."""
    if fp32_model:
        return CDF_TOL_FP32
    return 2.0 * (err_p + err_q) / max(residual_mass, 1e-6) + 1e-6


def cut_zone(w_raw, top_k, top_p, eps):
    """What a logit error of at most `eps` leaves open about the top-k / top-p cut of a row.

    w_raw: the oracle's un-truncated probabilities.  The other side's probabilities lie within a
    factor exp(+-2 eps) of them, so (i) two tokens can swap places in the order only if their
    probabilities are within exp(4 eps) of each other: a token of the top k is surely kept if it
    exceeds the (k+1)-th probability by that factor, a token outside is surely dropped if it is
    below the k-th by that factor; (ii) every prefix mass relative to the total moves by at most
    exp(+-4 eps), so the nucleus ends somewhere between the cuts for top_p * exp(-10 eps) and
    top_p * exp(+10 eps) (the extra 2 eps covers (i) changing the total).  Returns
    `sure` (kept on both sides), `maybe` (kept on at least one side, a superset of `sure`),
    `rho` (relative uncertainty of any renormalised probability of a `sure` token: its own factor
    exp(2 eps) times that of the kept mass) and `amb` (mass of maybe-but-not-sure tokens relative
    to the sure mass)."""
    w = np.asarray(w_raw, dtype=F32)
    V = w.shape[0]
    w64 = w.astype(np.float64)
    sure_k = np.ones(V, dtype=bool)
    maybe_k = np.ones(V, dtype=bool)
    if 1 <= top_k < V:
        srt = np.sort(w64)[::-1]
        sure_k = w64 > srt[top_k] * np.exp(4 * eps)
        maybe_k = w64 >= srt[top_k - 1] * np.exp(-4 * eps)
    in_p = 0.0 < top_p < 1.0
    lo = W.kept_set(w, top_k, top_p * np.exp(-10 * eps) if in_p else top_p)
    mid = W.kept_set(w, top_k, top_p)
    hi = W.kept_set(w, top_k, top_p * np.exp(10 * eps) if in_p else top_p)
    sure = lo & sure_k
    maybe = hi | mid | (maybe_k & ~sure_k & (w64 >= (w64[mid].min() if mid.any() else 0.0) * np.exp(-4 * eps)))
    maybe |= sure
    s_sure, s_mid, s_maybe = w64[sure].sum(), w64[mid].sum(), w64[maybe].sum()
    rho = float(np.exp(4 * eps) * max(s_mid / max(s_sure, 1e-30), s_maybe / max(s_mid, 1e-30)) - 1.0)
    amb = float((s_maybe - s_sure) / max(s_sure, 1e-30))
    return {"sure": sure, "maybe": maybe, "rho": rho, "amb": amb}


def top2_gap(row):
    part = np.partition(row, -2)[-2:]
    return float(part[1] - part[0])


def token_within_cdf_band(w, u, token, delta):
    """True if `token` is what the inverse-CDF draw returns for SOME weight vector within a
    relative perturbation `delta` of w: the threshold u*Z lies within delta*Z of the token's
    CDF interval.  Used where logits differ by a known bound eps between the two sides: a
    logit error eps changes every probability by at most a factor e^(2 eps), hence any prefix
    sum of the CDF by at most about 2 eps."""
    W = S.fixed_point(w).astype(np.float64)
    cum = np.cumsum(W)
    Z = cum[-1]
    t = Z * float(u)
    lo = cum[token - 1] if token else 0.0
    return lo - delta * Z <= t <= cum[token] + delta * Z
