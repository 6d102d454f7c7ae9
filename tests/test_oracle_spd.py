"""Pins for the CPU oracle's block loop (oracle/spd.py) on the tiny workload.  CPU only.

The paper fixes one exact behaviour: with greedy decoding the speculative output is
identical to the target's own auto-regressive output (Sec. 4 "Decoding"), for any draft
and any block size.  Beyond that: block efficiency <= gamma + 1 (Sec. 4 "Metrics"), the
caches after a rejection hold exactly the emitted tokens, and with the draft equal to the
target every token is accepted.
"""
import numpy as np
import pytest

import synth
from oracle import llama
from oracle.spd import SpdOracle

F32 = np.float32


def build(wl, temperature=1.0, greedy=False, same_draft=False, std=0.02):
    tw = synth.Weights(wl.target, wl.seeds["weights"], "target", std=std)
    dw = tw if same_draft else synth.Weights(wl.draft, wl.seeds["weights"], "draft",
                                             adapter_in=wl.adapter_in, std=std)
    t = llama.Model(wl.target, tw, 128)
    d = llama.Model(wl.target if same_draft else wl.draft, dw, 128)
    ad = dw.f32("adapter") if wl.adapter_in and not same_draft else None
    return SpdOracle(t, d, temperature, greedy, adapter_w=ad)


@pytest.mark.parametrize("gamma", [1, 3, 4])
def test_greedy_speculative_equals_target_only(gamma):
    # std 0.2 so that logits are well separated and the draft agrees with the target now
    # and then (both accept and reject paths run)
    wl = synth.tiny_workload(gamma)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    a = build(wl, greedy=True, std=0.2)
    a.prefill(img, ids)
    spd, st = a.generate(wl.n_new, gamma, None)
    b = build(wl, greedy=True, std=0.2)
    b.prefill(img, ids)
    ar = b.generate_target_only(wl.n_new)
    assert np.array_equal(spd, ar)
    assert 1.0 <= st["tau"] <= gamma + 1
    assert st["blocks"] <= wl.n_new


def test_identical_draft_accepts_all_and_tau_is_gamma_plus_one():
    wl = synth.Workload("same", synth.TINY_TARGET, synth.TINY_TARGET, 0, 16, 3, 24)
    ids = synth.prompt_ids(wl)
    for greedy in (True, False):
        o = build(wl, greedy=greedy, same_draft=True, std=0.2)
        o.prefill(None, ids, u0=0.3)
        u = synth.uniforms(3, "same.spd", (wl.n_new, 2 * 3 + 1))
        out, st = o.generate(wl.n_new, 3, None if greedy else u)
        assert st["accepted"] == 3 * st["blocks"]
        assert st["tau"] == 4.0


def test_sampling_loop_caches_hold_exactly_the_emitted_tokens():
    wl = synth.tiny_workload(4)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    o = build(wl, temperature=1.0, std=0.1)
    o.prefill(img, ids, u0=0.5)
    u = synth.uniforms(3, "loop", (wl.n_new, 9))
    out, st = o.generate(20, 4, u)
    assert st["tau"] <= 5 and len(out) == 20
    assert st["accepted"] > 0                      # accept path exercised
    assert st["accepted"] < 4 * st["blocks"]       # reject path exercised
    # the target's next logits equal those of a fresh model fed only the emitted tokens
    seq = list(o.seq)
    nxt_logits = o.t.forward(o.tc, o.t.embed([seq[-1]]), o.m + len(seq) - 1)[0]
    fresh = build(wl, std=0.1)
    rows = np.concatenate([img, fresh.t.embed(seq)], 0)
    want = fresh.t.forward(fresh.t.new_cache(), rows, 0)[-1]
    assert np.abs(nxt_logits - want).max() < 2e-5
    # same for the draft (text rows only)
    dl = o.d.forward(o.dc, o.d.embed(seq[o.d_fed:]), o.off + o.d_fed)[-1]
    dwant = fresh.d.forward(fresh.d.new_cache(), fresh.d.embed(seq), 0)[-1]
    assert np.abs(dl - dwant).max() < 2e-5


def test_draft_with_image_adapter_sees_projected_features():
    wl = synth.tiny_workload(4, adapter=True)
    img, ids, feats = synth.image_embeds(wl), synth.prompt_ids(wl), synth.image_features(wl)
    o = build(wl, greedy=True, std=0.2)
    o.prefill(img, ids, draft_image_feats=feats)
    assert o.off == wl.n_image and o.dc.length == wl.n_image + wl.n_prompt
    d_ids, _ = o.draft(4, None)
    # the draft's first logits equal a cache-free pass over [H W_a^T ; embed(text)]
    rows = np.concatenate([feats @ o.adapter_w.T, o.d.embed(o.seq)], 0)
    want = o.d.forward_full(rows)[-1]
    assert np.abs(o.last_draft_logits[0] - want).max() < 2e-5
    # and differ from a text-only draft's (the image rows matter)
    t = build(synth.tiny_workload(4), greedy=True, std=0.2)
    t.prefill(img, ids)
    t.draft(4, None)
    assert np.abs(t.last_draft_logits[0] - want).max() > 1e-3


def test_draft_rows_given_in_its_own_space_equal_the_linear_adapter_applied_outside():
    """The draft's image rows may be handed in already projected (the output of its own
    two-layer adapter): with rows = H W_a^T that must reproduce the run in which the loop
    applies the linear adapter W_a itself, and the rows must matter (a text-only draft
    proposes other tokens)."""
    wl = synth.tiny_workload(4, adapter=True)
    img, ids, feats = synth.image_embeds(wl), synth.prompt_ids(wl), synth.image_features(wl)
    u = synth.uniforms(3, "rows.given", (12, 2 * 4 + 1))
    a = build(wl, std=0.2)
    a.prefill(img, ids, u0=0.3, draft_image_feats=feats)
    out_a, st_a = a.generate(12, 4, u)
    b = build(wl, std=0.2)
    rows = feats.astype(F32) @ b.adapter_w.T
    b.adapter_w = None
    b.prefill(img, ids, u0=0.3, draft_image_feats=rows)
    out_b, st_b = b.generate(12, 4, u)
    assert np.array_equal(out_a, out_b) and st_a == st_b
    assert b.off == wl.n_image
    c = build(wl, std=0.2)
    c.adapter_w = None
    c.prefill(img, ids, u0=0.3)
    assert c.off == 0
    qa = build(wl, std=0.2)
    qa.prefill(img, ids, u0=0.3, draft_image_feats=feats)
    _, q_with = qa.draft(4, u[0, :4])
    _, q_without = c.draft(4, u[0, :4])
    assert np.abs(np.asarray(q_with[0]) - np.asarray(q_without[0])).max() > 1e-6


def test_top_k_one_sampling_equals_greedy_decoding():
    """top_k = 1 leaves a point mass at the arg-max of every row of both models, so the sampling
    rule accepts a draft token iff it is the target's arg-max and otherwise emits that arg-max:
    the whole loop must reproduce greedy speculative decoding (hence the target's own greedy
    continuation, Sec. 4 "Decoding") whatever the uniforms are."""
    wl = synth.tiny_workload(4)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    g = build(wl, greedy=True, std=0.2)
    g.prefill(img, ids)
    want = g.generate_target_only(wl.n_new)
    o = build(wl, greedy=False, std=0.2)
    o.top_k, o.truncate = 1, True
    o.prefill(img, ids, u0=0.77)
    u = synth.uniforms(11, "topk1", (wl.n_new, 9))
    got, st = o.generate(wl.n_new, 4, u)
    assert np.array_equal(got, want)


def test_truncated_loop_emits_only_tokens_of_the_targets_kept_sets():
    """With top-k / top-p on, every emitted token has non-zero probability in the target's
    truncated row at its position (the rule's output law is the truncated target row), the
    draft's rows handed to the rule are truncated rows (at most k non-zeros, sum 1), and
    switching truncation off with k >= V and top_p = 1 changes nothing."""
    from oracle import warp as W, sampling as S
    wl = synth.tiny_workload(4)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    o = build(wl, greedy=False, std=0.1)
    o.top_k, o.top_p, o.truncate = 20, 0.8, True
    o.prefill(img, ids, u0=0.4)
    u = synth.uniforms(12, "trunc.loop", (16, 9))
    for b in range(8):
        n0 = len(o.seq)
        d_ids, q = o.draft(4, u[b, :4])
        assert np.all((q > 0).sum(axis=1) <= 20) and np.allclose(q.sum(axis=1), 1.0, atol=1e-5)
        assert all(q[j, d_ids[j]] > 0 for j in range(4))
        a, nxt = o.verify(d_ids, q, u[b, 4:])
        kept = W.warp_rows(S.softmax_t(o.last_logits, 1.0), 20, 0.8) > 0
        assert np.array_equal(kept, o.last_p > 0)
        emitted = o.seq[n0:]
        assert all(kept[j, tok] for j, tok in enumerate(emitted))
    full = build(wl, greedy=False, std=0.1)
    off = build(wl, greedy=False, std=0.1)
    off.top_k, off.top_p, off.truncate = wl.target.vocab, 1.0, True
    for m in (full, off):
        m.prefill(img, ids, u0=0.4)
    a1, _ = full.generate(12, 4, u)
    a2, _ = off.generate(12, 4, u)
    assert np.array_equal(a1, a2)
