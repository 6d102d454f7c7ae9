"""Pins for the CPU oracle's forward pass (oracle/llama.py).  CPU only.

The oracle is checked against things other than itself: closed forms and identities for
each primitive, library routines in fp64 (torch's bf16 cast, rms_norm, silu), an
independent library implementation of the LLaMA architecture (HuggingFace transformers,
fp64) for the whole stack, and invariants of the cache (cached == recomputed, block ==
row by row, rollback == never fed).
"""
import math

import numpy as np
import pytest
import torch

import synth
from oracle import llama

F32 = np.float32


def small_cfg(dtype="fp32"):
    return synth.ModelCfg(2, 64, 4, 88, 96, False, dtype=dtype)


def small_model(dtype="fp32", seed=11, std=0.08, max_seq=48):
    cfg = small_cfg(dtype)
    w = synth.Weights(cfg, seed, "t", std=std)
    # non-trivial norm gains so that a dropped gain is visible
    g = np.random.default_rng(5)
    for l in range(cfg.n_layers):
        w.stored["attn_norm"][l] = g.uniform(0.5, 1.5, cfg.d_model).astype(F32)
        w.stored["ffn_norm"][l] = g.uniform(0.5, 1.5, cfg.d_model).astype(F32)
    w.stored["final_norm"] = g.uniform(0.5, 1.5, cfg.d_model).astype(F32)
    return llama.Model(cfg, w, max_seq), w


# ------------------------------------------------------------------ primitives

def test_round_bf16_matches_library_cast_and_ties_to_even():
    x = np.random.default_rng(0).standard_normal(20000).astype(F32) * 3
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(llama.round_bf16(x), want)
    # 1 + 2^-8 is exactly half-way between 1 and 1 + 2^-7: ties go to the even mantissa
    assert llama.round_bf16(np.array([1 + 2.0 ** -8], F32))[0] == F32(1.0)
    assert llama.round_bf16(np.array([1 + 3 * 2.0 ** -8], F32))[0] == F32(1 + 2.0 ** -6)
    assert np.array_equal(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x)), want)


def test_rmsnorm_closed_form_and_library():
    x = np.array([[3.0, -4.0, 0.0, 0.0]], F32)           # mean square = 25/4
    w = np.array([1.0, 2.0, 3.0, 4.0], F32)
    got = llama.rmsnorm(x, w, 0.0)
    assert np.allclose(got, [[3 / 2.5, -8 / 2.5, 0, 0]], atol=1e-6)
    g = np.random.default_rng(1)
    x = g.standard_normal((5, 64)).astype(F32)
    w = g.uniform(0.5, 2, 64).astype(F32)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (64,),
                                        torch.from_numpy(w).double(), 1e-5).numpy()
    assert np.allclose(llama.rmsnorm(x, w, 1e-5), want, atol=2e-6)
    # unit gain => unit mean square
    y = llama.rmsnorm(x, np.ones(64, F32), 0.0)
    assert np.allclose((y.astype(np.float64) ** 2).mean(-1), 1.0, atol=1e-5)


def test_silu_identities():
    x = np.linspace(-12, 12, 97).astype(F32)
    s = llama.silu(x)
    assert s[48] == 0.0                                   # silu(0) = 0
    assert np.allclose(s - llama.silu(-x), x, atol=1e-5)  # x*sig(x) + x*sig(-x) = x
    assert abs(llama.silu(np.array([1.0], F32))[0] - 1 / (1 + math.exp(-1))) < 1e-6
    want = torch.nn.functional.silu(torch.from_numpy(x).double()).numpy()
    assert np.allclose(s, want, atol=1e-5)


def test_rope_pairing_frequency_norm_and_relativity():
    dh, H, theta = 16, 2, 10000.0
    cos, sin = llama.rope_table(64, dh, theta)
    # a unit vector in element i of head 1 at position 7 becomes (cos, sin) in (i, i + dh/2)
    i, pos = 3, 7
    x = np.zeros((1, H * dh), F32)
    x[0, dh + i] = 1.0
    y = llama.apply_rope(x, np.array([pos]), cos, sin, H)
    ang = pos * theta ** (-2.0 * i / dh)
    want = np.zeros_like(x)
    want[0, dh + i], want[0, dh + i + dh // 2] = math.cos(ang), math.sin(ang)
    assert np.allclose(y, want, atol=1e-6)
    # position 0 is the identity; rotation preserves norms
    g = np.random.default_rng(2)
    q = g.standard_normal((1, H * dh)).astype(F32)
    k = g.standard_normal((1, H * dh)).astype(F32)
    assert np.array_equal(llama.apply_rope(q, np.array([0]), cos, sin, H), q)
    assert abs(np.linalg.norm(llama.apply_rope(q, np.array([33]), cos, sin, H)) - np.linalg.norm(q)) < 1e-5

    # per-head q.k depends on the position difference only
    def dots(a, b):
        qa = llama.apply_rope(q, np.array([a]), cos, sin, H).reshape(H, dh)
        kb = llama.apply_rope(k, np.array([b]), cos, sin, H).reshape(H, dh)
        return (qa * kb).sum(-1)
    assert np.allclose(dots(9, 4), dots(25, 20), atol=1e-4)
    assert not np.allclose(dots(9, 4), dots(9, 5), atol=1e-3)


# ------------------------------------------------------------------ whole stack vs a library

def hf_llama(cfg, w):
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
                     num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                     num_key_value_heads=cfg.n_heads, rms_norm_eps=cfg.rms_eps,
                     rope_theta=cfg.rope_theta, max_position_embeddings=256,
                     tie_word_embeddings=False, attention_bias=False, mlp_bias=False,
                     hidden_act="silu")
    hc._attn_implementation = "eager"
    m = LlamaForCausalLM(hc).double().eval()
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    sd = {"model.embed_tokens.weight": t(w.f32("tok_embed")), "lm_head.weight": t(w.f32("lm_head")),
          "model.norm.weight": t(w.f32("final_norm"))}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj",
             "w_down": "mlp.down_proj", "attn_norm": "input_layernorm",
             "ffn_norm": "post_attention_layernorm"}
    for l in range(cfg.n_layers):
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}.weight"] = t(w.f32(k, l))
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not [k for k in missing if "rotary" not in k] and not unexpected
    return m


def test_forward_matches_library_llama_with_image_prefix():
    """Rows = [image embeddings ; token embeddings] (paper Eq. 1) through the oracle in
    fp32 vs an independent fp64 LLaMA implementation fed the same rows as inputs_embeds."""
    model, w = small_model()
    g = np.random.default_rng(3)
    img = g.standard_normal((5, 64)).astype(F32)
    ids = g.integers(0, 96, 9)
    rows = np.concatenate([img, model.embed(ids)], 0)
    got = model.forward(model.new_cache(), rows, 0)
    hf = hf_llama(model.cfg, w)
    with torch.no_grad():
        want = hf(inputs_embeds=torch.from_numpy(rows).double()[None]).logits[0].numpy()
    assert got.shape == want.shape == (14, 96)
    assert np.abs(got - want).max() < 2e-5 * max(1.0, np.abs(want).max())
    # ... and a planted mistake is caught: swapping gate and up projections
    w.stored["w_gate"], w.stored["w_up"] = w.stored["w_up"], w.stored["w_gate"]
    bad = model.forward(model.new_cache(), rows, 0)
    assert np.abs(bad - want).max() > 1e-3


# ------------------------------------------------------------------ cache invariants

@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_cached_block_equals_recompute_and_row_by_row(dtype):
    model, _ = small_model(dtype)
    g = np.random.default_rng(6)
    rows = g.standard_normal((20, 64)).astype(F32) * 0.5
    full = model.forward_full(rows, kv_dtype="bf16" if dtype == "bf16" else "fp32")
    # prefix of 12 rows, then a block of 5, then 3 single rows
    c = model.new_cache()
    a = model.forward(c, rows[:12], 0)
    b = model.forward(c, rows[12:17], 12)
    singles = [model.forward(c, rows[t:t + 1], t) for t in range(17, 20)]
    got = np.concatenate([a, b] + singles, 0)
    assert np.abs(got - full).max() < 2e-5
    # the 5-row block equals five one-row calls (block-causal mask)
    c2 = model.new_cache()
    model.forward(c2, rows[:12], 0)
    one = np.concatenate([model.forward(c2, rows[t:t + 1], t) for t in range(12, 17)], 0)
    assert np.abs(one - b).max() < 2e-5


def test_rollback_equals_never_fed():
    model, _ = small_model()
    g = np.random.default_rng(7)
    rows = g.standard_normal((16, 64)).astype(F32) * 0.5
    junk = g.standard_normal((4, 64)).astype(F32) * 0.5
    c = model.new_cache()
    model.forward(c, rows[:10], 0)
    model.forward(c, np.concatenate([rows[10:12], junk]), 10)   # 2 kept, 4 rejected
    got = model.forward(c, rows[12:16], 12)                      # overwrite from row 12
    clean = model.new_cache()
    model.forward(clean, rows[:12], 0)
    want = model.forward(clean, rows[12:16], 12)
    assert np.abs(got - want).max() < 2e-5   # BLAS blocks 2-row and 6-row calls differently
    stale = model.forward(c, rows[12:16], 13)                   # off by one row: junk row 12 leaks
    assert np.abs(stale - want).max() > 1e-3
