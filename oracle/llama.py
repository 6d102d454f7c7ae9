"""CPU oracle: LLaMA-style decoder forward with a KV cache, in fp32.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package; it exists
so that tests, the smoke check and the benchmark's CPU-baseline leg can compare the CUDA
path with a slow, plain statement of what the paper's method computes.  It shares no code
with the CUDA path.

What it follows.  The target generates X_{n+1} ~ q(. | V_{1:m}, X_{1:n}) (paper Eq. 1,
Sec. 2.2): a decoder-only language model whose input rows are the m projected image
embeddings followed by the token embeddings of the text.  The draft is the same
architecture at a smaller size and sees the text rows only (Sec. 3).  "Follows the LLaMA
architecture" (Sec. 4 and Table 1: SiLU activation, 32 layers / 32 heads / intermediate
11008 for the target) is read as: pre-norm residual blocks with RMSNorm, rotary position
embedding on q and k (rotate-half pairing (i, i + d_h/2), theta = 10000), multi-head
causal self-attention with 1/sqrt(d_h) scaling, SwiGLU feed-forward, no biases, final
RMSNorm, linear LM head.

Arithmetic is fp32 throughout (numpy), with `@` (BLAS sgemm) as the one library
primitive.  No blocking, fusion or reordering: each line below is one step of the
definition.  Weights are whatever fp32 values the caller hands in (for a bf16 model: the
bf16-rounded values widened to fp32).  The KV cache keeps K and V either as fp32 or
rounded to bfloat16 (round-to-nearest-even) at the moment a row is appended, matching
the storage format of the model (`kv_dtype`).

Pinned by tests/test_oracle_forward.py: primitives against closed forms and fp64 library
routines, the whole stack against an independent library LLaMA in fp64, cached block
forward == cache-free recompute, one M-row call == M one-row calls, rollback == never
having fed the rejected rows, RoPE norm preservation and relative-position property;
`forward_tree` (tests/test_oracle_tree.py): a chain-shaped tree == `forward`, and every
root-to-leaf path of a branching tree == that path fed alone as a chain.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32


def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bfloat16 (ties to even) -> fp32."""
    u = np.ascontiguousarray(x, dtype=F32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return (((u + r) >> np.uint32(16)) << np.uint32(16)).view(F32)


def rope_table(n_pos: int, d_head: int, theta: float):
    """cos/sin of pos * theta^(-2i/d_head), i < d_head/2; computed in fp64, stored fp32."""
    i = np.arange(d_head // 2, dtype=np.float64)
    inv_freq = np.power(float(theta), -2.0 * i / float(d_head))
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang).astype(F32), np.sin(ang).astype(F32)


def apply_rope(x: np.ndarray, pos: np.ndarray, cos: np.ndarray, sin: np.ndarray, n_heads: int):
    """x [M, n_heads*d_h]; element pair (i, i + d_h/2) of each head is rotated by the angle
    of its position: a' = a cos - b sin, b' = b cos + a sin."""
    M, d = x.shape
    dh = d // n_heads
    xh = x.reshape(M, n_heads, dh)
    a, b = xh[..., : dh // 2], xh[..., dh // 2:]
    c, s = cos[pos][:, None, :], sin[pos][:, None, :]
    out = np.empty_like(xh)
    out[..., : dh // 2] = a * c - b * s
    out[..., dh // 2:] = b * c + a * s
    return out.reshape(M, d)


def rmsnorm(x: np.ndarray, w: np.ndarray, eps: float) -> np.ndarray:
    """x * w / sqrt(mean(x^2) + eps), row-wise, fp32."""
    ms = np.mean(x * x, axis=-1, keepdims=True, dtype=F32)
    inv = F32(1.0) / np.sqrt(ms + F32(eps), dtype=F32)
    return (x * inv) * w


def silu(x: np.ndarray) -> np.ndarray:
    return x / (F32(1.0) + np.exp(-x, dtype=F32))


def softmax_rows(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m, dtype=F32)
    return e / np.sum(e, axis=-1, keepdims=True, dtype=F32)


class KVCache:
    """K and V rows per layer: [n_layers, max_seq, d_model]; `length` rows are valid."""

    def __init__(self, n_layers: int, max_seq: int, d_model: int, kv_dtype: str = "fp32"):
        self.k = np.zeros((n_layers, max_seq, d_model), dtype=F32)
        self.v = np.zeros((n_layers, max_seq, d_model), dtype=F32)
        self.length = 0
        self.kv_dtype = kv_dtype

    def store(self, layer: int, pos0: int, k: np.ndarray, v: np.ndarray):
        if self.kv_dtype == "bf16":
            k, v = round_bf16(k), round_bf16(v)
        self.k[layer, pos0: pos0 + k.shape[0]] = k
        self.v[layer, pos0: pos0 + v.shape[0]] = v


class Model:
    """`cfg` needs n_layers, d_model, n_heads, d_ffn, vocab, rms_eps, rope_theta;
    `weights.f32(name, layer=None)` returns fp32 arrays, matrices row-major [out, in]."""

    def __init__(self, cfg, weights, max_seq: int):
        self.cfg, self.w, self.max_seq = cfg, weights, max_seq
        self.cos, self.sin = rope_table(max_seq, cfg.d_model // cfg.n_heads, cfg.rope_theta)

    def new_cache(self) -> KVCache:
        c = self.cfg
        return KVCache(c.n_layers, self.max_seq, c.d_model,
                       "bf16" if getattr(c, "dtype", "fp32") == "bf16" else "fp32")

    def embed(self, ids) -> np.ndarray:
        return self.w.f32("tok_embed")[np.asarray(ids, dtype=np.int64)].astype(F32)

    # -- one decoder layer on M new rows at positions pos0 .. pos0+M-1 -----------------
    def _layer(self, l: int, x: np.ndarray, cache: KVCache, pos0: int) -> np.ndarray:
        c, w = self.cfg, self.w
        M, H = x.shape[0], c.n_heads
        dh = c.d_model // H
        pos = np.arange(pos0, pos0 + M)

        h = rmsnorm(x, w.f32("attn_norm", l), c.rms_eps)
        q = h @ w.f32("wq", l).T
        k = h @ w.f32("wk", l).T
        v = h @ w.f32("wv", l).T
        q = apply_rope(q, pos, self.cos, self.sin, H)
        k = apply_rope(k, pos, self.cos, self.sin, H)
        cache.store(l, pos0, k, v)

        # query row j (position pos0+j) sees cache rows 0 .. pos0+j
        n_ctx = pos0 + M
        visible = np.arange(n_ctx)[None, :] <= pos[:, None]
        scale = F32(1.0 / np.sqrt(float(dh)))
        o = np.empty((M, c.d_model), dtype=F32)
        for hd in range(H):
            sl = slice(hd * dh, (hd + 1) * dh)
            s = (q[:, sl] @ cache.k[l, :n_ctx, sl].T) * scale
            s = np.where(visible, s, F32(-np.inf))
            o[:, sl] = softmax_rows(s) @ cache.v[l, :n_ctx, sl]
        x = x + o @ w.f32("wo", l).T

        h = rmsnorm(x, w.f32("ffn_norm", l), c.rms_eps)
        g = h @ w.f32("w_gate", l).T
        u = h @ w.f32("w_up", l).T
        return x + (silu(g) * u) @ w.f32("w_down", l).T

    def forward(self, cache: KVCache, rows: np.ndarray, pos0: int) -> np.ndarray:
        """Feed M input rows (already embeddings) at positions pos0.., append their K/V,
        return logits [M, vocab].  Sets cache.length = pos0 + M (rows beyond are stale)."""
        x = np.ascontiguousarray(rows, dtype=F32)
        assert pos0 + x.shape[0] <= self.max_seq
        for l in range(self.cfg.n_layers):
            x = self._layer(l, x, cache, pos0)
        cache.length = pos0 + x.shape[0]
        h = rmsnorm(x, self.w.f32("final_norm"), self.cfg.rms_eps)
        return h @ self.w.f32("lm_head").T

    # -- draft TREE: rows are nodes of a token tree hanging off the last committed token ----
    def forward_tree(self, cache: KVCache, rows: np.ndarray, origin: int, slots, depths, sees) -> np.ndarray:
        """Tree-based speculative decoding (the paper's Sec. 5 names it as the next step and
        cites SpecInfer / Medusa-style token trees): the M input rows are nodes of a tree whose
        root sits at sequence position `origin`.  Row i is a node at depth depths[i] below the
        root (the root itself has depth 0), so its rotary position is origin + depths[i]; its K/V
        go to cache row origin + slots[i] (every node has its own row, siblings share a position
        but not a row); it attends every cache row below `origin` (the committed prefix) and, of
        the rows from `origin` on, exactly those whose slot is in sees[i] (its ancestors and
        itself).  A chain (slots = depths = 0..M-1, sees[i] = {0..i}) is `forward`.  Returns
        logits [M, vocab]; cache.length is left to the caller (which rows survive is decided by
        the verification)."""
        c, w = self.cfg, self.w
        x = np.ascontiguousarray(rows, dtype=F32)
        M, H = x.shape[0], c.n_heads
        dh = c.d_model // H
        slots = [int(s) for s in slots]
        pos = np.asarray([origin + int(d) for d in depths])
        n_slots = max(max(slots), max((max(s) for s in sees if len(s)), default=0)) + 1
        n_ctx = origin + n_slots
        assert n_ctx <= self.max_seq and min(slots) >= 0
        visible = np.zeros((M, n_ctx), dtype=bool)
        visible[:, :origin] = True
        for i in range(M):
            for s_ in sees[i]:
                visible[i, origin + int(s_)] = True
        scale = F32(1.0 / np.sqrt(float(dh)))
        for l in range(c.n_layers):
            h = rmsnorm(x, w.f32("attn_norm", l), c.rms_eps)
            q = apply_rope(h @ w.f32("wq", l).T, pos, self.cos, self.sin, H)
            k = apply_rope(h @ w.f32("wk", l).T, pos, self.cos, self.sin, H)
            v = h @ w.f32("wv", l).T
            for i in range(M):
                cache.store(l, origin + slots[i], k[i:i + 1], v[i:i + 1])
            o = np.empty((M, c.d_model), dtype=F32)
            for hd in range(H):
                sl = slice(hd * dh, (hd + 1) * dh)
                s = (q[:, sl] @ cache.k[l, :n_ctx, sl].T) * scale
                s = np.where(visible, s, F32(-np.inf))
                o[:, sl] = softmax_rows(s) @ cache.v[l, :n_ctx, sl]
            x = x + o @ w.f32("wo", l).T
            h = rmsnorm(x, w.f32("ffn_norm", l), c.rms_eps)
            x = x + (silu(h @ w.f32("w_gate", l).T) * (h @ w.f32("w_up", l).T)) @ w.f32("w_down", l).T
        h = rmsnorm(x, self.w.f32("final_norm"), self.cfg.rms_eps)
        return h @ self.w.f32("lm_head").T

    # -- cache-free statement of the same function, written independently (loops) -----
    def forward_full(self, rows_all: np.ndarray, kv_dtype: str = "fp32") -> np.ndarray:
        """Logits for every row of a whole sequence, no cache: row t attends rows 0..t."""
        c, w = self.cfg, self.w
        x = np.ascontiguousarray(rows_all, dtype=F32)
        T, H = x.shape[0], c.n_heads
        dh = c.d_model // H
        pos = np.arange(T)
        for l in range(c.n_layers):
            h = rmsnorm(x, w.f32("attn_norm", l), c.rms_eps)
            q = apply_rope(h @ w.f32("wq", l).T, pos, self.cos, self.sin, H)
            k = apply_rope(h @ w.f32("wk", l).T, pos, self.cos, self.sin, H)
            v = h @ w.f32("wv", l).T
            if kv_dtype == "bf16":
                k, v = round_bf16(k), round_bf16(v)
            o = np.zeros_like(x)
            for t in range(T):
                for hd in range(H):
                    sl = slice(hd * dh, (hd + 1) * dh)
                    s = (k[: t + 1, sl] @ q[t, sl]) / F32(np.sqrt(float(dh)))
                    e = np.exp(s - s.max(), dtype=F32)
                    o[t, sl] = (e / e.sum(dtype=F32)) @ v[: t + 1, sl]
            x = x + o @ w.f32("wo", l).T
            h = rmsnorm(x, w.f32("ffn_norm", l), c.rms_eps)
            x = x + (silu(h @ w.f32("w_gate", l).T) * (h @ w.f32("w_up", l).T)) @ w.f32("w_down", l).T
        return rmsnorm(x, w.f32("final_norm"), c.rms_eps) @ w.f32("lm_head").T
