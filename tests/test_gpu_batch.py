"""Several sequences through one pass over the weights (spd_batch_*) against the oracle, which
decodes every sequence on its own (the method is stated per sequence, Sec. 2.1: a batch must give
each sequence exactly what it would get alone).  Tolerances as in tests/test_gpu_spd.py."""
import numpy as np
import pytest

import synth
from oracle import sampling as S

import harness as H
from test_gpu_spd import _lib

F32 = np.float32


def _inputs(wl, k, extra_prompt):
    w2 = synth.Workload(wl.name, wl.target, wl.draft, wl.n_image, wl.n_prompt + extra_prompt * k, wl.gamma, wl.n_new,
                        seeds={"weights": 1, "inputs": 40 + k, "uniforms": 3})
    return synth.image_embeds(w2), synth.prompt_ids(w2)


def run_batch_lockstep(wl, B, gamma, n_blocks, greedy, logit_tol, std, extra_prompt=3, max_seq=None, top_k=0):
    """top_k = 1 (sampling mode): every row is a point mass at its arg-max, so the sampling kernels of
    the batched path must reproduce greedy decoding whatever the uniforms are; the oracle then runs
    greedy."""
    spd = _lib()
    tw, dw = H.build_weights(wl, std)
    max_seq = max_seq or (wl.n_image + wl.n_prompt + extra_prompt * B + 8 * (n_blocks + 2) + 16)
    seqs = [H.make_gpu(wl, tw, dw, max_seq, 1.0, greedy and not top_k, top_k=top_k)]
    seqs += [seqs[0].fork() for _ in range(B - 1)]
    inputs = [_inputs(wl, k, extra_prompt) for k in range(B)]
    orcs = [H.make_oracle(wl, tw, dw, max_seq, 1.0, greedy) for _ in range(B)]
    su = H.SafeUniforms(7, f"batch.{wl.name}.{greedy}")
    rep = {"blocks": 0, "accepted": [0] * B, "tolerated": 0, "max_logit_err": 0.0, "max_draft_logit_err": 0.0}
    for k in range(B):
        img, ids = inputs[k]
        if greedy:
            x0 = orcs[k].prefill(img, ids)
            g0 = seqs[k].prefill(img, ids, u0=0.37 if top_k else None)
        else:
            probe = H.make_oracle(wl, tw, dw, max_seq, 1.0, greedy)
            probe.prefill(img, ids, u0=0.5)
            u0 = su.for_cdf(S.softmax_t(probe.prefill_logits, 1.0))
            x0 = orcs[k].prefill(img, ids, u0=u0)
            g0 = seqs[k].prefill(img, ids, u0=u0)
        if g0 != x0:
            seqs[k].rollback(len(ids), int(ids[-1]), x0)
            rep["tolerated"] += 1
    bt = spd.SpdBatch(seqs)
    V = wl.target.vocab
    for blk in range(n_blocks):
        # oracle: every sequence alone
        d_all, q_all, u_d = [], [], []
        for k in range(B):
            d_ids, q = orcs[k].draft(gamma, None if greedy else su.draft_hook)
            d_all.append(d_ids); q_all.append(q); u_d.append(orcs[k].last_draft_u)
        any_u = synth.uniforms(8, f"batch.any.{blk}", (B, 2 * gamma + 1))     # top_k = 1: the values do not matter
        g_ids = bt.draft(gamma, (any_u[:, :gamma].copy() if top_k else None) if greedy else np.stack(u_d))
        dl = bt.get_logits(2 * B).reshape(B, 2, V)[:, 1]          # last draft step's rows
        for k in range(B):
            derr = float(np.abs(dl[k] - orcs[k].last_draft_logits[gamma - 1]).max()) \
                if np.array_equal(g_ids[k], d_all[k]) else 0.0
            rep["max_draft_logit_err"] = max(rep["max_draft_logit_err"], derr)
            assert derr < logit_tol
        same = [np.array_equal(g_ids[k], d_all[k]) for k in range(B)]
        res, u_v = [], []
        for k in range(B):
            res.append(orcs[k].verify(d_all[k], q_all[k], None if greedy else su.verify_hook))
            u_v.append(None if greedy else orcs[k].last_u)
        if not all(same):
            # a draft token inside the tolerance band: the whole batch is put back on the oracle's text
            for k in range(B):
                if not same[k]:
                    j = int(np.argmax(g_ids[k] != d_all[k]))
                    if greedy:
                        assert H.top2_gap(orcs[k].last_draft_logits[j]) < 1e-2
                    else:
                        assert H.token_within_cdf_band(q_all[k][j], u_d[k][j], int(g_ids[k][j]), H.cdf_band(False, 2e-3))
            rep["tolerated"] += 1
        else:
            ga, gn = bt.verify(gamma, (any_u[:, gamma:].copy() if top_k else None) if greedy else np.stack(u_v))
            lg = bt.get_logits(B * (gamma + 1)).reshape(B, gamma + 1, V)
            for k in range(B):
                verr = float(np.abs(lg[k] - orcs[k].last_logits).max())
                rep["max_logit_err"] = max(rep["max_logit_err"], verr)
                assert verr < logit_tol, f"block {blk} sequence {k}: logits differ by {verr}"
                a, nxt = res[k]
                rep["accepted"][k] += a
                if (int(ga[k]), int(gn[k])) != (a, nxt):
                    if greedy:
                        gaps = [H.top2_gap(orcs[k].last_logits[j]) for j in range(gamma + 1)]
                        assert min(gaps[: min(a, int(ga[k])) + 1]) < 1e-2, f"block {blk} sequence {k}"
                    else:
                        assert int(ga[k]) == a, f"block {blk} sequence {k}: accepted {ga[k]} vs {a}"
                        p_o = orcs[k].last_p
                        w = p_o[gamma] if a == gamma else np.maximum(F32(0), p_o[a] - q_all[k][a])
                        band = H.cdf_band(False, verr, 2e-3, float(w.sum(dtype=np.float64)))
                        assert H.token_within_cdf_band(w, u_v[k][gamma], int(gn[k]), band)
                    same[k] = False
                    rep["tolerated"] += 1
                else:
                    assert seqs[k].get_state() == (len(orcs[k].seq) - 1, orcs[k].seq[-1])
        for k in range(B):
            if not same[k] or not all(same):
                img, _ = inputs[k]
                seqs[k].prefill(img, np.asarray(orcs[k].seq[:-1], dtype=np.int32),
                                u0=0.5 if (top_k or not greedy) else None)
                seqs[k].rollback(len(orcs[k].seq) - 1, orcs[k].seq[-2], orcs[k].seq[-1])
        rep["blocks"] += 1
    bt.close()
    for g in seqs[1:]:
        g.close()
    seqs[0].close()
    return rep


@pytest.mark.gpu
@pytest.mark.parametrize("greedy", [True, False])
def test_three_ragged_sequences_small_bf16(greedy):
    """B = 3 sequences with prompts of different lengths at the small bf16 shapes (d 256 / 128,
    ragged ffn widths): per-sequence positions, caches, accepted counts and commits."""
    t = synth.ModelCfg(2, 256, 4, 688, 1024, False, dtype="bf16")
    d = synth.ModelCfg(1, 128, 2, 344, 1024, False, dtype="bf16")
    wl = synth.Workload("tiny-bf16-batch", t, d, 16, 16, 4, 32)
    r = run_batch_lockstep(wl, 3, 4, 8, greedy, 5e-2, 0.08 if not greedy else 0.15, extra_prompt=5)
    print("batch of 3", greedy, r)
    assert r["blocks"] == 8
    if not greedy:
        assert sum(r["accepted"]) > 0 and len(set(r["accepted"])) > 1      # sequences advance at their own pace


@pytest.mark.gpu
def test_batched_sampling_kernels_with_top_k_one_reproduce_greedy():
    """The probability-row path of the batched steps (softmax rows, truncation, per-sequence draw
    and rule) with top_k = 1: the output must be the greedy one for any uniforms."""
    t = synth.ModelCfg(2, 256, 4, 688, 1024, False, dtype="bf16")
    d = synth.ModelCfg(1, 128, 2, 344, 1024, False, dtype="bf16")
    wl = synth.Workload("tiny-bf16-batch", t, d, 16, 16, 4, 32)
    r = run_batch_lockstep(wl, 3, 4, 6, True, 5e-2, 0.15, extra_prompt=5, top_k=1)
    print("batch of 3, top_k = 1", r)
    assert r["blocks"] == 6


@pytest.mark.gpu
def test_sixteen_sequences_with_1600_cached_rows_two_layers():
    """The batched KV-heavy shape on the 2-layer truncation: 16 sequences, each with 576 image
    rows + 1024 prompt ids in its bf16 cache, gamma 5, temperature 1: 96 target rows per step in
    one weight pass, every sequence against the oracle decoding it alone."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2, n_prompt=1024)
    r = run_batch_lockstep(wl, 16, 5, 2, False, 5e-2, 0.02, extra_prompt=1)
    print("batch of 16", r)
    assert r["blocks"] == 2 and r["max_logit_err"] < 2e-2


@pytest.mark.gpu
def test_batch_argument_errors_and_mixing_with_single_calls():
    spd = _lib()
    t = synth.ModelCfg(2, 256, 4, 688, 1024, False, dtype="bf16")
    d = synth.ModelCfg(1, 128, 2, 344, 1024, False, dtype="bf16")
    wl = synth.Workload("tiny-bf16-batch", t, d, 16, 16, 4, 32)
    tw, dw = H.build_weights(wl, 0.15)
    a = H.make_gpu(wl, tw, dw, 128, 1.0, True)
    b = a.fork()
    other = H.make_gpu(wl, tw, dw, 128, 1.0, True)
    with pytest.raises(spd.SpdError):
        spd.SpdBatch([a, other])                     # not forks of one context
    with pytest.raises(spd.SpdError):
        spd.SpdBatch([a, a])
    bt = spd.SpdBatch([a, b])
    with pytest.raises(spd.SpdError) as e:
        bt.draft(4)                                  # nothing prefilled yet
    assert e.value.status == spd.SPD_ESTATE
    (img0, ids0), (img1, ids1) = _inputs(wl, 0, 3), _inputs(wl, 1, 3)
    a.prefill(img0, ids0)
    b.prefill(img1, ids1)
    with pytest.raises(spd.SpdError) as e:
        bt.verify(4)                                 # no batched draft with gamma 4
    assert e.value.status == spd.SPD_ESTATE
    # greedy: a block done by the batch and a block done by single calls give the same tokens
    # (greedy speculative output is the target's own continuation, whatever path computed it)
    want = []
    for g, (img, ids) in ((a, (img0, ids0)), (b, (img1, ids1))):
        first = g.prefill(img, ids)
        out, _ = g.generate(12, 4)
        want.append(out.tolist())
        g.prefill(img, ids)
    got = [[want[0][0]], [want[1][0]]]
    for blk in range(12):
        if blk % 2 == 0:
            ids = bt.draft(4)
            acc, nxt = bt.verify(4)
            for k in range(2):
                got[k] += [int(x) for x in ids[k][: acc[k]]] + [int(nxt[k])]
        else:
            for k, g in enumerate((a, b)):
                d_ids = g.draft(4)
                acc1, nxt1 = g.verify(4)
                got[k] += [int(x) for x in d_ids[:acc1]] + [nxt1]
    for k in range(2):
        n = min(len(got[k]), 12)
        assert got[k][:n] == want[k][:n]
    bt.close()
    b.close(); a.close(); other.close()
