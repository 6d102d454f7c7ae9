"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element on the
same seeded inputs.  Tolerances (stated by the benchmark spec for this path): logits within 5e-2
max-abs; greedy tokens identical unless the oracle's top-2 logit gap is below 1e-2;
accept/reject decisions identical except where |u - p/q| < 1e-4; the rejection rule on given
fp32 probabilities bit-exact.  fp32 models are held to 2e-4 on logits.
"""
import ctypes as C
import os
import re

import numpy as np
import pytest

import synth
from oracle import sampling as S

import harness as H

F32 = np.float32
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _lib():
    from paper_2404_08856_b200 import build
    build.build()
    import paper_2404_08856_b200 as spd
    return spd


# ------------------------------------------------------------------ no GPU needed

def test_library_exports_every_declared_symbol():
    spd = _lib()
    header = open(os.path.join(ROOT, "include", "spd.h")).read()
    declared = set(re.findall(r"\b(spd_[a-z_]+)\s*\(", header))
    assert declared == set(spd.EXPORTS)
    lib = spd.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_argument_errors_before_any_device_work():
    spd = _lib()
    lib = spd.lib()
    ctx = C.c_void_p(0)
    assert lib.spd_create(None, None, None, C.byref(ctx)) == spd.SPD_EINVAL and not ctx.value
    assert lib.spd_reject_sample(None, None, None, None, 1, 1, 8, 0, None, None, None) == spd.SPD_EINVAL
    assert lib.spd_skinny_gemm(None, None, 1, 1, 8, 8, None, None) == spd.SPD_EINVAL
    x = np.zeros(8, F32)
    p = C.c_void_p(x.ctypes.data)
    assert lib.spd_skinny_gemm(p, p, 1, 9, 8, 8, p, None) == spd.SPD_EINVAL      # M > 8
    assert lib.spd_skinny_gemm(p, p, 1, 1, 8, 12, p, None) == spd.SPD_EINVAL     # K % 8
    assert lib.spd_prefill(None, None, 0, None, None, 1, None, None) == spd.SPD_EINVAL
    assert lib.spd_last_error(None) == b"null context"


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    import paper_2404_08856_b200 as spd
    monkeypatch.setattr(spd, "_lib", None)
    monkeypatch.setattr(spd, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        spd.lib()


# ------------------------------------------------------------------ kernels alone

@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K,dtype", [(6, 4096 + 40, 4096, 1), (8, 1000, 11008, 1), (1, 33, 8, 1),
                                         (2, 32000, 768, 1), (3, 100, 688, 0), (5, 260, 4104, 0),
                                         (7, 64, 256, 1), (4, 12288, 4096, 1)])
def test_skinny_gemm_matches_matmul(M, N, K, dtype):
    import torch
    spd = _lib()
    g = np.random.default_rng(M * 1000 + N)
    x = g.standard_normal((M, K)).astype(F32)
    w = (g.standard_normal((N, K)) * 0.05).astype(F32)
    if dtype == 1:
        bits = synth.f32_to_bf16_bits(w)
        w = synth.bf16_bits_to_f32(bits)
        wd = torch.from_numpy(bits.view(np.int16)).cuda()
    else:
        wd = torch.from_numpy(w).cuda()
    xd = torch.from_numpy(x).cuda()
    yd = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    spd.skinny_gemm(xd, wd, yd, dtype)
    torch.cuda.synchronize()
    want = x.astype(np.float64) @ w.astype(np.float64).T
    got = yd.cpu().numpy()
    scale = np.sqrt(K) * 0.05
    assert np.abs(got - want).max() < 2e-5 * scale * 10


@pytest.mark.gpu
@pytest.mark.parametrize("B", [1, 8, 32])
@pytest.mark.parametrize("sigma", [0.1, 0.5, 1.0])
def test_reject_sample_bit_exact_microbench(B, sigma):
    """Rejection-sampling microbench: V = 32000, gamma = 5, target logits N(0, 3^2), draft
    logits = target + sigma N(0,1); p, q are the oracle's softmaxes, handed to both sides."""
    import torch
    spd = _lib()
    gamma, V = 5, 32000
    tl, dl = synth.microbench_logits(B, gamma, V, sigma)
    p, q = S.softmax_t(tl, 1.0), S.softmax_t(dl, 1.0)
    ud = synth.uniforms(9, f"mb.d.{B}.{sigma}", (B, gamma))
    ids = np.array([[S.sample_fixed_point(q[b, j], ud[b, j]) for j in range(gamma)] for b in range(B)], np.int32)
    u = synth.uniforms(9, f"mb.v.{B}.{sigma}", (B, gamma + 1))
    for greedy in (False, True):
        want_a, want_n = S.reject_sample_batch(p, q, ids, u, greedy)
        pd, qd = torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda()
        idd, udv = torch.from_numpy(ids).cuda(), torch.from_numpy(u).cuda()
        a = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        spd.reject_sample(pd, qd, idd, udv, gamma, greedy, a, n)
        torch.cuda.synchronize()
        assert np.array_equal(a.cpu().numpy(), want_a)
        assert np.array_equal(n.cpu().numpy(), want_n)
    if sigma == 0.1 and B == 32:
        assert want_a.mean() > 0  # the sweep reaches the accept path


@pytest.mark.gpu
def test_reject_sample_distribution_small_vocab():
    """V = 8, 10^6 blocks on the device: the first emitted token follows the target's p
    (chi-squared), and a 20000-block sample is bit-identical to the oracle."""
    import torch
    from scipy import stats
    spd = _lib()
    V, gamma, N = 8, 2, 1_000_000
    g = np.random.default_rng(1)
    p1 = S.softmax_t(g.standard_normal(V).astype(F32) * 1.5, 1.0)
    q1 = S.softmax_t(g.standard_normal(V).astype(F32) * 1.5, 1.0)
    cq = np.cumsum(S.fixed_point(q1))
    ud = synth.uniforms(41, "gpu.chi.d", (N, gamma))
    t = ((int(cq[-1]) * (ud.astype(np.float64) * (1 << 24)).astype(np.int64)) >> 24)
    ids = np.searchsorted(cq, t.astype(np.uint64), side="right").astype(np.int32)
    u = synth.uniforms(42, "gpu.chi.v", (N, gamma + 1))
    p = np.broadcast_to(p1, (N, gamma + 1, V)).copy()
    q = np.broadcast_to(q1, (N, gamma, V)).copy()
    a = torch.zeros(N, dtype=torch.int32, device="cuda")
    n = torch.zeros(N, dtype=torch.int32, device="cuda")
    spd.reject_sample(torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(), torch.from_numpy(ids).cuda(),
                      torch.from_numpy(u).cuda(), gamma, False, a, n)
    torch.cuda.synchronize()
    a, n = a.cpu().numpy(), n.cpu().numpy()
    sub = slice(0, 20000)
    wa, wn = S.reject_sample_batch(p[sub], q[sub], ids[sub], u[sub], False)
    assert np.array_equal(a[sub], wa) and np.array_equal(n[sub], wn)
    first = np.where(a >= 1, ids[:, 0], n)
    counts = np.bincount(first, minlength=V)
    e = p1.astype(np.float64)
    _, pval = stats.chisquare(counts, e / e.sum() * N)
    assert pval > 1e-4
    alpha = float(np.minimum(p1, q1).sum())
    assert abs((a >= 1).mean() - alpha) < 4 * np.sqrt(alpha * (1 - alpha) / N)


# ------------------------------------------------------------------ whole path, lock-step

def lockstep(wl, greedy, temperature, n_blocks, logit_tol, std=0.02, gammas=None, max_seq=None, gain_seed=None,
             image_from=None, uniforms="safe", grid_mode=0, top_k=0, top_p=0.0):
    """Drives the CUDA context and the oracle block by block on the same inputs and compares
    logits, draft tokens, accept decisions and drawn tokens.

    What may differ, and how far (anything else fails):
    * logits by `logit_tol`;
    * greedy tokens where the oracle's top-2 logit gap is below 1e-2;
    * an accept/reject decision where |u - min(1, p/q)| < 1e-4 (oracle's p, q).  On bf16 models a
      decision further out is accepted only inside what the measured logit errors explain
      (p/q moves by a factor exp(+-2 (err_p + err_q))) and is counted in `accept_beyond_tol`;
    * a drawn token inside the CDF band of H.cdf_band (2^-20 * Z on fp32 models).
    After any tolerated difference the device is put back on the oracle's sequence: by
    spd_rollback when its caches hold the right rows, by a fresh spd_prefill over the emitted
    text when the device's draft was fed a token that the oracle's was not.  The comparison
    always runs all `n_blocks`.

    `image_from(gpu_ctx) -> (device image rows, oracle image rows[, device draft rows, oracle
    draft rows])` replaces the generated image embeddings (and the draft's image rows); used to
    put the image adapters in front of the prefill.  `uniforms`: "safe" (the oracle skips
    candidates inside the tolerance of a boundary) or "plain" (the seeded stream as it is).
    `grid_mode`: launch shape (spd_cfg.grid_mode; 2 = one thread-block cluster per model).

    `top_k`, `top_p`: truncated sampling on both sides.  The two sides may then also disagree on
    which tokens survive the cut when a token's probability is within the logit error of it
    (H.cut_zone): a decision that involves such a token is exempt (`cut_ambiguous`), and every
    other probability of a truncated row is uncertain by the relative amount `rho` of its zone,
    which widens the accept tolerance to 1e-4 + (p/q) * ((1 + rho_p)(1 + rho_q) - 1) and the CDF
    band to (rho_p + rho_q + ambiguous mass) / (mass of the weights drawn from)."""
    spd = _lib()
    tw, dw = H.build_weights(wl, std)
    if gain_seed is not None:
        # non-trivial RMSNorm gains (the generated ones are all 1): a gain taken from the wrong
        # norm or layer, or dropped, then shows up in the logits
        g = np.random.default_rng(gain_seed)
        for w, cfg in ((tw, wl.target), (dw, wl.draft)):
            for l in range(cfg.n_layers):
                w.stored["attn_norm"][l] = g.uniform(0.5, 1.5, cfg.d_model).astype(np.float32)
                w.stored["ffn_norm"][l] = g.uniform(0.5, 1.5, cfg.d_model).astype(np.float32)
            w.stored["final_norm"] = g.uniform(0.5, 1.5, cfg.d_model).astype(np.float32)
    max_seq = max_seq or (wl.n_image + wl.n_prompt + 8 * (n_blocks + 2) + 16)
    fp32 = wl.target.dtype == "fp32"
    trunc = (not greedy) and (top_k >= 1 or 0.0 < top_p < 1.0)
    okp = top_p if 0.0 < top_p < 1.0 else 1.0
    orc = H.make_oracle(wl, tw, dw, max_seq, temperature, greedy, top_k, okp)
    gpu = H.make_gpu(wl, tw, dw, max_seq, temperature, greedy, grid_mode=grid_mode, top_k=top_k, top_p=top_p)

    def zone(logits_row, eps):
        return H.cut_zone(S.softmax_t(logits_row, temperature), top_k, okp, eps)
    img = synth.image_embeds(wl) if wl.n_image else None
    gpu_img = img
    feats = synth.image_features(wl) if wl.adapter_in else None
    gpu_feats = feats
    if image_from is not None:
        got = image_from(gpu)
        gpu_img, img = got[0], got[1]
        if len(got) == 4:
            gpu_feats, feats = got[2], got[3]
    ids = synth.prompt_ids(wl)
    su = (H.SafeUniforms if uniforms == "safe" else H.PlainUniforms)(wl.seeds["uniforms"], f"lock.{wl.name}.{greedy}")
    report = {"max_logit_err": 0.0, "max_draft_logit_err": 0.0, "tolerated": 0, "blocks": 0, "accepted": 0,
              "accept_within_tol": 0, "accept_beyond_tol": 0, "cdf_band_tokens": 0, "greedy_near_ties": 0,
              "reprefills": 0, "decisions": 0, "draws": 0, "cut_ambiguous": 0}

    # prefill: first token from the target's last row (Eq. 1)
    x0 = orc.prefill(img, ids, u0=None, draft_image_feats=feats) if greedy else None
    if not greedy:
        # choose u0 on the oracle side after seeing the row: run the target once to get it
        probe = H.make_oracle(wl, tw, dw, max_seq, temperature, greedy, top_k, okp)
        probe.prefill(img, ids, u0=0.5, draft_image_feats=feats)
        u0 = su.for_cdf(probe._probs(probe.prefill_logits))
        del probe
        x0 = orc.prefill(img, ids, u0=u0, draft_image_feats=feats)
    g0 = gpu.prefill(gpu_img, ids, u0=None if greedy else u0, draft_image_feats=gpu_feats)
    err = float(np.abs(gpu.get_logits(1)[0] - orc.prefill_logits).max())
    report["prefill_logit_err"] = err
    report["max_logit_err"] = max(report["max_logit_err"], err)
    assert err < logit_tol, f"prefill logits differ by {err}"
    if g0 != x0:
        if greedy:
            assert H.top2_gap(orc.prefill_logits) < 1e-2, "first token differs"
            report["greedy_near_ties"] += 1
        elif trunc:
            z = zone(orc.prefill_logits, err)
            amb = z["maybe"] & ~z["sure"]
            assert amb[g0] or amb[x0] or H.token_within_cdf_band(orc._probs(orc.prefill_logits), u0, g0,
                                                                 z["rho"] + z["amb"] + 1e-6), "first token"
            report["cut_ambiguous" if (amb[g0] or amb[x0]) else "cdf_band_tokens"] += 1
        else:
            assert H.token_within_cdf_band(S.softmax_t(orc.prefill_logits, temperature), u0, g0,
                                           H.cdf_band(fp32, err)), "first token outside the CDF band"
            report["cdf_band_tokens"] += 1
        gpu.rollback(len(ids), int(ids[-1]), x0)
        report["tolerated"] += 1

    for b in range(n_blocks):
        gamma = (gammas or [wl.gamma])[b % len(gammas or [wl.gamma])]
        seq_before = list(orc.seq)
        d_ids, q = orc.draft(gamma, None if greedy else su.draft_hook)
        g_ids = gpu.draft(gamma, None if greedy else orc.last_draft_u)
        rows = min(gamma, 6)
        derr = 0.0
        gl = gpu.get_draft_logits(rows)
        same = True
        for j in range(rows):
            if not same:
                break
            derr = max(derr, float(np.abs(gl[j] - orc.last_draft_logits[j]).max()))
            same = g_ids[j] == d_ids[j]
        report["max_draft_logit_err"] = max(report["max_draft_logit_err"], derr)
        assert derr < logit_tol, f"block {b}: draft logits differ by {derr}"
        draft_same = np.array_equal(g_ids, d_ids)
        first_diff = gamma if draft_same else int(np.argmax(g_ids != d_ids))
        report["draws"] += 0 if greedy else first_diff + (0 if draft_same else 1)
        if not draft_same:
            j = first_diff
            if greedy:
                assert H.top2_gap(orc.last_draft_logits[j]) < 1e-2, f"block {b}: draft token {j} differs"
                report["greedy_near_ties"] += 1
            elif trunc:
                z = zone(orc.last_draft_logits[j], derr)
                amb = z["maybe"] & ~z["sure"]
                if amb[int(g_ids[j])] or amb[int(d_ids[j])]:
                    report["cut_ambiguous"] += 1
                else:
                    assert H.token_within_cdf_band(q[j], orc.last_draft_u[j], int(g_ids[j]),
                                                   z["rho"] + z["amb"] + 1e-6), \
                        f"block {b}: draft token {j} = {g_ids[j]} outside the CDF band of {d_ids[j]}"
                    report["cdf_band_tokens"] += 1
            else:
                assert H.token_within_cdf_band(q[j], orc.last_draft_u[j], int(g_ids[j]), H.cdf_band(fp32, derr)), \
                    f"block {b}: draft token {j} = {g_ids[j]} outside the CDF band of {d_ids[j]}"
                report["cdf_band_tokens"] += 1
            report["tolerated"] += 1
        a, nxt = orc.verify(d_ids, q, None if greedy else su.verify_hook)
        if draft_same:
            ga, gn = gpu.verify(gamma, None if greedy else orc.last_u)
        else:  # keep going on the oracle's tokens; the device draft cache is put right below
            import torch
            qd = None if greedy else torch.from_numpy(q).cuda()
            ga, gn = gpu.verify(gamma, None if greedy else orc.last_u, draft_ids=d_ids, draft_probs=qd)
        verr = float(np.abs(gpu.get_logits(gamma + 1) - orc.last_logits).max())
        report["max_logit_err"] = max(report["max_logit_err"], verr)
        assert verr < logit_tol, f"block {b}: verify logits differ by {verr}"
        report["decisions"] += min(a + 1, gamma)
        report["draws"] += 0 if greedy else 1
        if (ga, gn) != (a, nxt):
            if greedy:
                gaps = [H.top2_gap(orc.last_logits[j]) for j in range(gamma + 1)]
                assert min(gaps[: min(a, ga) + 1]) < 1e-2, f"block {b}: ({ga},{gn}) vs oracle ({a},{nxt})"
                report["greedy_near_ties"] += 1
            elif ga != a:
                # the first test the two sides decide differently
                j = min(a, ga)
                x = int(d_ids[j])
                p_x, q_x = orc.last_p[j, x], q[j, x]
                dist = H.accept_distance(p_x, q_x, orc.last_u[j])
                if dist < H.ACCEPT_TOL:
                    report["accept_within_tol"] += 1
                elif trunc:
                    zp, zq = zone(orc.last_logits[j], verr), zone(orc.last_draft_logits[j], derr)
                    if (zp["maybe"][x] and not zp["sure"][x]) or (zq["maybe"][x] and not zq["sure"][x]):
                        report["cut_ambiguous"] += 1
                    else:
                        ratio = float(S.accept_prob(p_x, q_x))
                        explained = ratio * ((1 + zp["rho"]) * (1 + zq["rho"]) - 1) + H.ACCEPT_TOL
                        assert dist <= explained, \
                            f"block {b}: accepted {ga} vs oracle {a}; |u - p/q| = {dist:.3e} at test {j} " \
                            f"(cut zones explain {explained:.3e})"
                        report["accept_beyond_tol"] += 1
                else:
                    ratio = float(S.accept_prob(p_x, q_x))
                    explained = ratio * float(np.expm1(2.0 * (verr + derr))) + H.ACCEPT_TOL
                    assert not fp32 and dist <= explained, \
                        f"block {b}: accepted {ga} vs oracle {a}; |u - p/q| = {dist:.3e} at test {j} " \
                        f"(logit errors {verr:.2e} / {derr:.2e} explain {explained:.3e})"
                    report["accept_beyond_tol"] += 1
            else:
                # same accept decisions; the drawn token may move to a neighbour of the oracle's
                # when the logits differ: it must stay inside the CDF band
                p_o = orc.last_p
                ambiguous = False
                if a == gamma:
                    w, band = p_o[gamma], H.cdf_band(fp32, verr)
                    if trunc:
                        zp = zone(orc.last_logits[gamma], verr)
                        band = zp["rho"] + zp["amb"] + 1e-6
                        ambiguous = bool((zp["maybe"] & ~zp["sure"])[[gn, nxt]].any())
                else:
                    w = np.maximum(F32(0), p_o[a] - q[a])
                    mass = float(w.sum(dtype=np.float64))
                    band = H.cdf_band(fp32, verr, derr, mass)
                    if trunc:
                        zp, zq = zone(orc.last_logits[a], verr), zone(orc.last_draft_logits[a], derr)
                        band = (zp["rho"] + zp["amb"] + zq["rho"] + zq["amb"]) / max(mass, 1e-6) + 1e-6
                        ambiguous = bool(((zp["maybe"] & ~zp["sure"]) | (zq["maybe"] & ~zq["sure"]))[[gn, nxt]].any())
                if ambiguous:
                    report["cut_ambiguous"] += 1
                else:
                    assert H.token_within_cdf_band(w, orc.last_u[gamma], gn, band), \
                        f"block {b}: token {gn} outside the CDF band of the oracle's draw {nxt} (logit err {verr})"
                    report["cdf_band_tokens"] += 1
            report["tolerated"] += 1
        report["blocks"] += 1
        report["accepted"] += a
        n_text, pend = gpu.get_state()
        if (ga, gn) == (a, nxt) and draft_same:
            assert (n_text, pend) == (len(orc.seq) - 1, orc.seq[-1])
        elif not draft_same and a > first_diff:
            # the device's draft was fed a token the oracle's draft was not and rows computed from it
            # would stay in its cache: rebuild both caches from the emitted text
            gpu.prefill(gpu_img, np.asarray(orc.seq[:-1], dtype=np.int32), u0=None if greedy else 0.5,
                        draft_image_feats=gpu_feats)
            gpu.rollback(len(orc.seq) - 1, orc.seq[-2], orc.seq[-1])
            report["reprefills"] += 1
        else:
            gpu.rollback(len(orc.seq) - 1, orc.seq[-2], orc.seq[-1])
        assert orc.seq[: len(seq_before)] == seq_before
    report["skipped_uniforms"] = su.skipped
    gpu.close()
    return report


@pytest.mark.gpu
@pytest.mark.parametrize("grid_mode", [1, 2])
@pytest.mark.parametrize("greedy", [True, False])
def test_tiny_lockstep(greedy, grid_mode):
    """grid_mode 1: one CTA per SM and the barrier in global memory; 2: one 16-CTA cluster."""
    wl = synth.tiny_workload(4)
    r = lockstep(wl, greedy, 1.0, 10, 2e-4, std=0.2 if greedy else 0.1, gammas=[4, 1, 7, 3, 2, 5, 6],
                 grid_mode=grid_mode)
    assert r["blocks"] == 10
    assert r["accept_within_tol"] == 0 and r["accept_beyond_tol"] == 0 and r["cdf_band_tokens"] == 0
    if not greedy:
        assert r["accepted"] > 0, "accept path not exercised"


@pytest.mark.gpu
@pytest.mark.parametrize("greedy", [True, False])
def test_tiny_identical_draft_accepts_everything(greedy):
    """Draft == target and no image: every draft token is accepted, tau = gamma + 1."""
    spd = _lib()
    wl = synth.Workload("same", synth.TINY_TARGET, synth.TINY_TARGET, 0, 16, 3, 24)
    tw = synth.Weights(wl.target, 1, "target", std=0.2)
    gpu = spd.Spd(wl.target, wl.target, tw.stored, tw.stored, 128, 7, 1.0, greedy)
    ids = synth.prompt_ids(wl)
    gpu.prefill(None, ids, u0=0.3)
    u = synth.uniforms(3, "same.gpu", (24, 7))
    out, st = gpu.generate(24, 3, None if greedy else u)
    assert st["accepted"] == 3 * st["blocks"] and st["tau"] == 4.0
    orc = H.make_oracle(wl, tw, tw, 128, 1.0, greedy)
    orc.prefill(None, ids, u0=0.3)
    want, _ = orc.generate(24, 3, None if greedy else u)
    if greedy:
        assert np.array_equal(out, want)
    gpu.close()


@pytest.mark.gpu
def test_tiny_lockstep_with_draft_adapter():
    wl = synth.tiny_workload(4, adapter=True)
    r = lockstep(wl, False, 1.0, 6, 2e-4, std=0.1)
    assert r["blocks"] == 6


@pytest.mark.gpu
def test_tiny_temperature_and_no_image():
    wl = synth.Workload("tiny-noimg", synth.TINY_TARGET, synth.TINY_DRAFT, 0, 19, 3, 16)
    r = lockstep(wl, False, 0.7, 6, 2e-4, std=0.1)
    assert r["blocks"] == 6


@pytest.mark.gpu
@pytest.mark.parametrize("gamma", [3, 5, 7])
def test_llava7b_shaped_two_layer_lockstep(gamma):
    """Per-layer shapes of the LLaVA-7B target (d 4096, 32 heads, ffn 11008, vocab 32000,
    bf16 weights and KV cache) and of the 115M draft, truncated to 2 layers each so that the
    CPU oracle finishes in seconds; 576 image rows + 64 prompt ids."""
    wl = synth.llava7b_workload(gamma=gamma, n_layers=2, draft_layers=2)
    r = lockstep(wl, False, 1.0, 3, 5e-2)
    print("two-layer report", r)
    assert r["blocks"] == 3
    assert r["max_logit_err"] < 1e-2   # far inside the 5e-2 allowance
    assert r["accept_beyond_tol"] == 0


@pytest.mark.gpu
@pytest.mark.parametrize("shape", ["tiny", "llava7b-3L"])
def test_lockstep_with_random_norm_gains(shape):
    """Every RMSNorm gain differs (per layer, per norm, per column): covers the gains that the
    residual epilogue multiplies in for the NEXT norm on bf16 models (attention norm of the next
    layer, FFN norm of the same layer, final norm after the last layer) and the on-load path."""
    if shape == "tiny":
        r = lockstep(synth.tiny_workload(gamma=4), False, 1.0, 4, 2e-4, gain_seed=7)
    else:
        wl = synth.llava7b_workload(gamma=5, n_layers=3, draft_layers=3, n_image=64, n_prompt=24)
        r = lockstep(wl, False, 1.0, 3, 3e-2, gain_seed=8)   # gains up to 1.5 scale the logits and their error
    assert r["blocks"] == (4 if shape == "tiny" else 3)


@pytest.mark.gpu
def test_small_bf16_models_where_most_ctas_own_no_rows():
    """bf16 weights at the tiny shapes (d 256 / 128): most of the 148 CTAs get no row of a
    projection, the ragged K = 688 and 344 need zero padding, heads are 64 wide; exercises the
    empty-CTA branches (residual copy, zero partial sums) and the dense prefill at odd sizes."""
    t = synth.ModelCfg(2, 256, 4, 688, 1024, False, dtype="bf16")
    d = synth.ModelCfg(1, 128, 2, 344, 1024, False, dtype="bf16")
    wl = synth.Workload("tiny-bf16", t, d, 16, 16, 4, 32)
    r = lockstep(wl, False, 1.0, 4, 2e-2, std=0.08, gain_seed=9, grid_mode=1)
    assert r["blocks"] == 4
    r = lockstep(wl, False, 1.0, 4, 2e-2, std=0.08, gain_seed=9, grid_mode=2)
    assert r["blocks"] == 4


@pytest.mark.gpu
def test_llava7b_shaped_two_layer_greedy():
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2)
    r = lockstep(wl, True, 1.0, 3, 5e-2)
    assert r["blocks"] == 3


@pytest.mark.gpu
@pytest.mark.parametrize("grid_mode", [1, 2])
def test_llava7b_shaped_two_layer_forced_launch_shapes(grid_mode):
    """Both launch shapes at the 7B / 115M layer shapes: one CTA per SM (1, the default) and one
    16-CTA cluster per model (2)."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2)
    r = lockstep(wl, False, 1.0, 2, 5e-2, grid_mode=grid_mode)
    assert r["blocks"] == 2 and r["max_logit_err"] < 1e-2


@pytest.mark.gpu
@pytest.mark.parametrize("shape", ["tiny", "llava7b-2L"])
def test_lockstep_on_unfiltered_uniforms(shape):
    """The seeded uniform stream taken as it is (no candidate skipped near a boundary): decisions
    may differ only inside the stated tolerance -- |u - min(1, p/q)| < 1e-4 for an accept test,
    the CDF band for a draw -- and every such case is counted; the device is put back on the
    oracle's sequence afterwards and the comparison goes on."""
    if shape == "tiny":
        r = lockstep(synth.tiny_workload(4), False, 1.0, 24, 2e-4, std=0.1, gammas=[4, 7, 2, 5], uniforms="plain")
        assert r["blocks"] == 24 and r["accept_beyond_tol"] == 0
    else:
        wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2)
        r = lockstep(wl, False, 1.0, 6, 5e-2, uniforms="plain")
        assert r["blocks"] == 6
    print("unfiltered uniforms", shape, r)
    assert r["skipped_uniforms"] == 0 and r["decisions"] > 0 and r["draws"] > r["blocks"]


@pytest.mark.gpu
@pytest.mark.parametrize("shape,top_k,top_p", [("tiny", 40, 0.0), ("tiny", 0, 0.9), ("tiny", 64, 0.8),
                                               ("llava7b-2L", 50, 0.9)])
def test_lockstep_with_top_k_top_p(shape, top_k, top_p):
    """Truncated sampling inside spd_prefill / spd_draft / spd_verify (spd_cfg.top_k, top_p): both
    models' rows truncated and renormalised, draft tokens drawn from the truncated rows, the rule
    on truncated rows -- block by block against the oracle running the same mode."""
    if shape == "tiny":
        r = lockstep(synth.tiny_workload(4), False, 1.0, 12, 2e-4, std=0.1, gammas=[4, 7, 2, 5], top_k=top_k,
                     top_p=top_p)
        assert r["blocks"] == 12 and r["accepted"] > 0
    else:
        wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2)
        r = lockstep(wl, False, 1.0, 4, 5e-2, top_k=top_k, top_p=top_p)
        assert r["blocks"] == 4
    print("top-k/top-p", shape, top_k, top_p, r)
    assert r["decisions"] >= r["blocks"]   # (unrelated 32000-token models share few of their top 50: few accepts)


@pytest.mark.gpu
def test_top_k_one_sampling_reproduces_greedy_decoding():
    """top_k = 1 leaves a point mass on every row of both models: the sampling path must then emit
    exactly what greedy speculative decoding emits (which is the target's own greedy continuation,
    Sec. 4 "Decoding"), through spd_generate's graph replay, for any uniforms."""
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.2)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    g = H.make_gpu(wl, tw, dw, 128, 1.0, True)
    g.prefill(img, ids)
    want, _ = g.generate(wl.n_new, 4)
    g.close()
    t = H.make_gpu(wl, tw, dw, 128, 1.0, False, top_k=1)
    t.prefill(img, ids, u0=0.6)
    got, st = t.generate(wl.n_new, 4, synth.uniforms(13, "topk1.gpu", (wl.n_new, 9)))
    t.close()
    assert np.array_equal(got, want)


# ------------------------------------------------------------------ block loop

@pytest.mark.gpu
@pytest.mark.parametrize("gamma", [0, 4])
def test_tiny_generate_greedy_equals_oracle_and_target_only(gamma):
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.2)
    orc = H.make_oracle(wl, tw, dw, 128, 1.0, True)
    gpu = H.make_gpu(wl, tw, dw, 128, 1.0, True)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    orc.prefill(img, ids)
    want = orc.generate_target_only(wl.n_new)     # Sec. 4 "Decoding": greedy SPD == target AR
    gpu.prefill(img, ids)
    got, st = gpu.generate(wl.n_new, gamma)
    if not np.array_equal(got, want):
        k = int(np.argmax(got != want))
        # allowed only at a near-tie of the oracle's logits; replay the oracle up to there
        o2 = H.make_oracle(wl, tw, dw, 128, 1.0, True)
        o2.prefill(img, ids)
        o2.generate_target_only(k) if k > 0 else None
        row = o2.prefill_logits if k == 0 else o2.last_logits[-1]
        assert H.top2_gap(row) < 1e-2
    assert st["tokens"] == wl.n_new and 1.0 <= st["tau"] <= gamma + 1
    gpu.close()


@pytest.mark.gpu
def test_tiny_generate_sampling_follows_oracle():
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.1)
    orc = H.make_oracle(wl, tw, dw, 128, 1.0, False)
    gpu = H.make_gpu(wl, tw, dw, 128, 1.0, False)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    u = synth.uniforms(3, "gen.tiny", (wl.n_new, 9))
    orc.prefill(img, ids, u0=0.25)
    want, ost = orc.generate(wl.n_new, 4, u)
    gpu.prefill(img, ids, u0=0.25)
    got, st = gpu.generate(wl.n_new, 4, u)
    assert st["tau"] <= 5 and got.min() >= 0 and got.max() < wl.target.vocab
    same = int(np.argmax(np.append(got != want, True)))
    # fp32 on both sides: a divergence needs a uniform within ~1e-6 of a boundary
    assert same >= wl.n_new // 2, f"diverged after {same} tokens"
    if same == wl.n_new:
        assert st["blocks"] == ost["blocks"] and st["accepted"] == ost["accepted"]
    gpu.close()


# ------------------------------------------------------------------ host-side errors

@pytest.mark.gpu
def test_state_and_overflow_errors():
    spd = _lib()
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl)
    gpu = H.make_gpu(wl, tw, dw, 48, 1.0, True, gamma_max=4)
    with pytest.raises(spd.SpdError) as e:
        gpu.draft(2)
    assert e.value.status == spd.SPD_ESTATE
    with pytest.raises(spd.SpdError) as e:
        gpu.prefill(synth.image_embeds(wl), np.zeros(40, np.int32))
    assert e.value.status == spd.SPD_EOVERFLOW
    with pytest.raises(spd.SpdError) as e:
        gpu.prefill(synth.image_embeds(wl), np.array([5, 99999], np.int32))
    assert e.value.status == spd.SPD_EINVAL
    gpu.prefill(synth.image_embeds(wl), synth.prompt_ids(wl))
    with pytest.raises(spd.SpdError) as e:
        gpu.draft(5)                      # gamma > gamma_max
    assert e.value.status == spd.SPD_EINVAL
    with pytest.raises(spd.SpdError) as e:
        gpu.verify(3)                     # no draft with gamma 3
    assert e.value.status == spd.SPD_ESTATE
    with pytest.raises(spd.SpdError) as e:
        gpu.generate(64, 4)               # 16 + 16 + 64 > max_seq 48
    assert e.value.status == spd.SPD_EOVERFLOW
    out, st = gpu.generate(8, 4)          # still usable afterwards
    assert len(out) == 8
    gpu.close()
    bad = synth.ModelCfg(2, 100, 3, 64, 64, dtype="fp32")   # d_model not divisible by heads
    with pytest.raises(spd.SpdError):
        H.make_gpu(synth.Workload("bad", bad, bad, 0, 4, 1, 4), tw, tw, 48)
    # bf16 with d_head 32: the tensor-core attention tiles need rows of at least 128 bytes
    narrow = synth.ModelCfg(1, 128, 4, 344, 1024, False, dtype="bf16")
    nw = synth.Weights(narrow, 3, "narrow")
    with pytest.raises(spd.SpdError) as e:
        H.make_gpu(synth.Workload("narrow", narrow, narrow, 0, 4, 1, 4), nw, nw, 48)
    assert e.value.status == spd.SPD_EINVAL


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_out_of_range_ids_in_device_memory_are_reported_not_dereferenced(dtype):
    """Ids handed over in device memory cannot be checked by the host.  The kernels read an
    offender as token 0 (so no access leaves the tables) and report it: spd_prefill returns
    SPD_EINVAL and leaves the context un-prefilled, spd_verify returns SPD_EINVAL, and
    spd_reject_sample marks the sequence with n_acc = next = -1.  The context stays usable."""
    import torch
    spd = _lib()
    t = synth.ModelCfg(2, 256, 4, 688, 1024, False, dtype=dtype)
    d = synth.ModelCfg(1, 128, 2, 344, 1024, False, dtype=dtype)
    wl = synth.Workload("tiny-badid", t, d, 16, 16, 4, 32)
    tw, dw = H.build_weights(wl, 0.1)
    gpu = H.make_gpu(wl, tw, dw, 96, 1.0, True)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    bad = ids.copy()
    bad[5] = 1 << 20
    with pytest.raises(spd.SpdError) as e:
        gpu.prefill(img, torch.from_numpy(bad).cuda())
    assert e.value.status == spd.SPD_EINVAL
    with pytest.raises(spd.SpdError) as e:
        gpu.draft(4)
    assert e.value.status == spd.SPD_ESTATE          # the failed prefill left no sequence
    first = gpu.prefill(img, torch.from_numpy(ids).cuda())
    assert first == gpu.prefill(img, ids)            # device ids == host ids
    gpu.draft(4)
    with pytest.raises(spd.SpdError) as e:
        gpu.verify(4, None, draft_ids=torch.tensor([3, -1, 7, 9], dtype=torch.int32, device="cuda"))
    assert e.value.status == spd.SPD_EINVAL
    gpu.prefill(img, ids)
    out, _ = gpu.generate(8, 4)
    assert len(out) == 8 and out.min() >= 0
    gpu.close()
    # the rule alone
    V, gamma, B = 64, 2, 3
    g = np.random.default_rng(3)
    p = S.softmax_t(g.standard_normal((B, gamma + 1, V)).astype(F32), 1.0)
    q = S.softmax_t(g.standard_normal((B, gamma, V)).astype(F32), 1.0)
    idv = np.array([[1, 2], [5, V], [3, 4]], np.int32)
    u = synth.uniforms(5, "badid", (B, gamma + 1))
    a = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    for greedy in (False, True):
        spd.reject_sample(torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(), torch.from_numpy(idv).cuda(),
                          torch.from_numpy(u).cuda(), gamma, greedy, a, n)
        torch.cuda.synchronize()
        wa, wn = S.reject_sample_batch(p[[0, 2]], q[[0, 2]], idv[[0, 2]], u[[0, 2]], greedy)
        assert a.cpu().tolist() == [wa[0], -1, wa[1]] and n.cpu().tolist() == [wn[0], -1, wn[1]]


@pytest.mark.gpu
def test_bounded_device_waits_give_up_and_the_context_stays_usable():
    """A wait that can never succeed (a shared-memory barrier nobody arrives at; a grid barrier
    whose target is one arrival beyond the grid) runs out of its poll limit, the kernel returns
    normally and the library reports SPD_ETIMEOUT; the same context then decodes as before."""
    spd = _lib()
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.2)
    gpu = H.make_gpu(wl, tw, dw, 96, 1.0, True)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    gpu.prefill(img, ids)
    want, _ = gpu.generate(12, 4)
    for which in (0, 1):
        assert gpu.wait_selftest(which, 3000) == spd.SPD_ETIMEOUT
        assert b"wait ran out" in spd.lib().spd_last_error(gpu._ctx)
        gpu.prefill(img, ids)
        got, _ = gpu.generate(12, 4)
        assert np.array_equal(got, want)
    assert gpu.wait_selftest(2, 100) == spd.SPD_EINVAL
    gpu.close()


# ------------------------------------------------------------------ full size

@pytest.mark.gpu
def test_llava7b_full_size_sampling_properties():
    """Speculative sampling in the benchmark's configuration (all 32 target layers, 12 draft
    layers, gamma 5, temperature 1), checked by properties that hold at any size: the block loop
    through spd_generate (CUDA-graph replay) emits exactly what step-by-step spd_draft /
    spd_verify calls emit for the same uniforms; a second run from the same state reproduces it;
    the statistics add up (every block emits its accepted tokens plus one, at most gamma + 1); the
    draft rows q_j handed to the rule are probability rows; each emitted draft token is one the
    draft proposed."""
    import torch
    spd = _lib()
    wl = synth.llava7b_workload(gamma=5)
    tw, dw = H.build_weights(wl)
    gamma, n_new = 5, 24
    gpu = H.make_gpu(wl, tw, dw, wl.n_image + wl.n_prompt + 8 * n_new + 64, 1.0, False)
    del tw, dw
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    u = synth.uniforms(7, "full.sampling", (n_new, 2 * gamma + 1))
    first = gpu.prefill(img, ids, u0=0.375)
    n_text0, pend0 = gpu.get_state()
    assert pend0 == first and n_text0 == len(ids)
    out1, st1 = gpu.generate(n_new, gamma, u)
    assert out1[0] == first and out1.min() >= 0 and out1.max() < wl.target.vocab
    assert st1["tokens"] == n_new and st1["blocks"] >= 1
    assert st1["blocks"] + st1["accepted"] >= n_new - 1 and st1["accepted"] <= gamma * st1["blocks"]
    assert 1.0 <= st1["tau"] <= gamma + 1
    # same state, same uniforms: identical output
    gpu.rollback(n_text0, int(ids[-1]), pend0)
    out2, st2 = gpu.generate(n_new, gamma, u)
    assert np.array_equal(out1, out2) and st2["blocks"] == st1["blocks"] and st2["accepted"] == st1["accepted"]
    # step by step through spd_draft / spd_verify
    gpu.rollback(n_text0, int(ids[-1]), pend0)
    q = torch.empty((gamma, wl.target.vocab), device="cuda", dtype=torch.float32)
    emitted, blocks, accepted = [first], 0, 0
    while len(emitted) < n_new:
        d_ids = gpu.draft(gamma, u[blocks, :gamma], probs_out=q)
        sums = q.sum(dim=1).cpu().numpy()
        assert np.all(np.abs(sums - 1.0) < 1e-3) and float(q.min()) >= 0.0
        assert all(float(q[j, int(d_ids[j])]) > 0.0 for j in range(gamma))
        a, nxt = gpu.verify(gamma, u[blocks, gamma:])
        assert 0 <= a <= gamma and 0 <= nxt < wl.target.vocab
        emitted += [int(x) for x in d_ids[:a]] + [nxt]
        blocks += 1
        accepted += a
    assert emitted[:n_new] == out1.tolist()
    assert blocks == st1["blocks"] and accepted == st1["accepted"]
    n_text, pend = gpu.get_state()
    assert n_text == len(ids) + len(emitted) - 1 and pend == emitted[-1]
    gpu.close()


@pytest.mark.gpu
def test_llava7b_full_size_greedy_blocks_match_oracle():
    """The benchmark's own configuration: all 32 layers of the LLaVA-7B-shaped target and the
    12-layer draft, 576 image rows + 64 prompt ids, gamma 5, greedy acceptance.  Prefill
    logits, two drafted blocks and two verify steps against the oracle (about a minute of CPU).
    Sampling decisions at this depth are covered on the 2-layer truncation: with 32000 nearly
    equiprobable tokens a draw flips on logit differences far below the 5e-2 allowance."""
    wl = synth.llava7b_workload(gamma=5)
    r = lockstep(wl, True, 1.0, 3, 5e-2, gammas=[5, 3, 7])
    assert r["blocks"] == 3
    assert r["max_logit_err"] < 4e-2 and r["max_draft_logit_err"] < 2e-2
    print("full-size greedy report", r)


@pytest.mark.gpu
def test_llava7b_full_size_sampling_blocks_match_oracle():
    """Temperature-1 speculative sampling at full depth (32 target layers, 12 draft layers) against
    the oracle: prefill row and first drawn token, then blocks with gamma = 5, 5, 3, 7 -- draft
    logits and drawn draft tokens, verify logits, every accept/reject decision, and the
    replacement / bonus draw.  Accept tests are held to |u - p/q| < 1e-4; a decision outside
    that would be reported in `accept_beyond_tol` (and must then be explained by the measured
    logit error)."""
    wl = synth.llava7b_workload(gamma=5)
    r = lockstep(wl, False, 1.0, 4, 5e-2, gammas=[5, 5, 3, 7])
    print("full-size sampling report", r)
    assert r["blocks"] == 4
    assert r["max_logit_err"] < 4e-2 and r["max_draft_logit_err"] < 2e-2
    assert r["accept_beyond_tol"] == 0


@pytest.mark.gpu
def test_llava7b_full_size_top_k_top_p_blocks_match_oracle():
    """Truncated sampling (top-k 50, top-p 0.9) at full depth against the oracle running the same
    mode: 3 blocks with gamma = 5, 3, 7."""
    wl = synth.llava7b_workload(gamma=5)
    r = lockstep(wl, False, 1.0, 3, 5e-2, gammas=[5, 3, 7], top_k=50, top_p=0.9)
    print("full-size top-k/top-p report", r)
    assert r["blocks"] == 3 and r["max_logit_err"] < 4e-2


@pytest.mark.gpu
def test_llava7b_shaped_two_layer_with_draft_adapter():
    """The draft with an image adapter at LLaVA-7B shapes: 576 features of width 1024 projected
    by one linear layer to the draft's width and prepended to its input (bf16, tensor-core
    prefill path)."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2, adapter=True)
    r = lockstep(wl, False, 1.0, 2, 5e-2)
    print("adapter report", r)
    assert r["blocks"] == 2 and r["max_draft_logit_err"] < 1e-2


# ------------------------------------------------------------------ more edges

@pytest.mark.gpu
def test_llava7b_shaped_long_context_uses_attention_sub_chunks():
    """576 image rows + 300 prompt ids: each KV split of the target now exceeds the attention
    scratch, so the running softmax across sub-chunks is exercised (bf16 tensor-core attention),
    as is a multi-split draft context."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2, n_prompt=300)
    r = lockstep(wl, False, 1.0, 2, 5e-2)
    print("long-context report", r)
    assert r["blocks"] == 2 and r["max_logit_err"] < 1e-2


@pytest.mark.gpu
def test_llava7b_shaped_1600_cached_rows():
    """The cache length of the batched KV-heavy workload (576 image rows + 1024 text rows) on the
    2-layer truncation: the target's KV splits reach their cap and each split spans 400 rows
    in several sub-chunks; the draft attends over 1024 rows."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2, n_prompt=1024)
    r = lockstep(wl, False, 1.0, 2, 5e-2)
    print("1600-row report", r)
    assert r["blocks"] == 2 and r["max_logit_err"] < 1e-2


@pytest.mark.gpu
def test_tiny_long_prompt_fp32_attention_splits():
    wl = synth.Workload("tiny-long", synth.TINY_TARGET, synth.TINY_DRAFT, 16, 400, 4, 16)
    r = lockstep(wl, False, 1.0, 3, 2e-4, std=0.1)
    assert r["blocks"] == 3


@pytest.mark.gpu
def test_rollback_replays_identically_and_cache_overflow_is_reported():
    spd = _lib()
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.1)
    max_seq = 16 + 16 + 40
    gpu = H.make_gpu(wl, tw, dw, max_seq, 1.0, False, gamma_max=4)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    first = gpu.prefill(img, ids, u0=0.25)
    u = synth.uniforms(3, "rollback", (12, 9))
    a, sa = gpu.generate(12, 4, u)
    # roll back to the state right after prefill and run the same loop again
    gpu.rollback(len(ids), int(ids[-1]), first)
    b, sb = gpu.generate(12, 4, u)
    assert np.array_equal(a, b) and sa["blocks"] == sb["blocks"] and sa["accepted"] == sb["accepted"]
    # fill the cache: verify steps until the library refuses
    gpu.rollback(len(ids), int(ids[-1]), first)
    seen = None
    for _ in range(64):
        try:
            gpu.draft(4, u[0, :4])
            gpu.verify(4, u[0, 4:])
        except spd.SpdError as e:
            seen = e.status
            break
    assert seen == spd.SPD_EOVERFLOW
    n_text, _ = gpu.get_state()
    assert 16 + n_text + 4 + 1 > max_seq - 5      # it stopped at the end of the cache, not before
    gpu.close()


@pytest.mark.gpu
def test_device_resident_ids_and_probabilities():
    """spd_draft writing ids / probabilities to device buffers and spd_verify reading them back
    from there gives the same result as the internal hand-over."""
    import torch
    wl = synth.tiny_workload(4)
    tw, dw = H.build_weights(wl, 0.1)
    img, ids = synth.image_embeds(wl), synth.prompt_ids(wl)
    u = synth.uniforms(3, "devptr", 9)
    res = []
    for external in (False, True):
        gpu = H.make_gpu(wl, tw, dw, 96, 1.0, False)
        gpu.prefill(img, ids, u0=0.5)
        if external:
            probs = torch.zeros(4, wl.target.vocab, device="cuda")
            d = gpu.draft(4, u[:4], probs_out=probs)
            assert abs(float(probs.sum()) - 4.0) < 1e-3
            res.append(gpu.verify(4, u[4:], draft_ids=d, draft_probs=probs))
        else:
            gpu.draft(4, u[:4])
            res.append(gpu.verify(4, u[4:]))
        gpu.close()
    assert res[0] == res[1]


def _prompt_variant(wl, k):
    """k-th prompt / image of a multi-sequence case: same shapes, different seeded draws."""
    w2 = synth.Workload(wl.name, wl.target, wl.draft, wl.n_image, wl.n_prompt + 3 * k, wl.gamma, wl.n_new,
                        adapter_in=wl.adapter_in, seeds={"weights": 1, "inputs": 20 + k, "uniforms": 3})
    return synth.image_embeds(w2), synth.prompt_ids(w2)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_forked_sequences_share_weights_and_keep_their_own_state(dtype):
    """Three sequences on one set of weights (spd_fork), driven block by block in an interleaved
    order with per-sequence rollback: each must produce what the oracle produces for that
    sequence alone (greedy speculative decoding == target-only greedy decoding, Sec. 4), so
    neither KV caches nor device state leak between sequences."""
    t = synth.ModelCfg(2, 256, 4, 688, 1024, False, dtype=dtype)
    d = synth.ModelCfg(1, 128, 2, 344, 1024, False, dtype=dtype)
    wl = synth.Workload("tiny-fork", t, d, 16, 16, 4, 32)
    # std 0.2 saturates the softmaxes: fine in fp32, but with a bf16 KV cache one rounding flip
    # then moves a whole attention row, so the bf16 case uses a gentler scale
    tw, dw = H.build_weights(wl, 0.2 if dtype == "fp32" else 0.05)
    max_seq = 160
    seqs = [H.make_gpu(wl, tw, dw, max_seq, 1.0, True)]
    seqs += [seqs[0].fork(), seqs[0].fork()]
    inputs = [_prompt_variant(wl, k) for k in range(3)]
    want = []
    for img, ids in inputs:
        o = H.make_oracle(wl, tw, dw, max_seq, 1.0, True)
        o.prefill(img, ids)
        want.append(np.asarray(o.generate_target_only(24)))
    firsts = [g.prefill(img, ids) for g, (img, ids) in zip(seqs, inputs)]
    got = [[f] for f in firsts]
    # sequence 1 runs two blocks that are thrown away again (rollback to the state after prefill)
    seqs[1].draft(4, None); seqs[1].verify(4, None)
    seqs[1].draft(4, None); seqs[1].verify(4, None)
    seqs[1].rollback(len(inputs[1][1]), int(inputs[1][1][-1]), firsts[1])
    for blk in range(40):
        order = [(blk + k) % 3 for k in range(3)]
        for k in order:
            if len(got[k]) >= 24:
                continue
            ids_k = seqs[k].draft(4, None)
            a, nxt = seqs[k].verify(4, None)
            got[k] += [int(x) for x in ids_k[:a]] + [int(nxt)]
        if all(len(g) >= 24 for g in got):
            break
    # the origin may go first: the weights live as long as a fork does
    seqs[0].close()
    extra = seqs[2].draft(4, None)
    assert len(extra) == 4
    for k in range(3):
        g = np.asarray(got[k][:24])
        if not np.array_equal(g, want[k]):
            j = int(np.argmax(g != want[k]))
            o2 = H.make_oracle(wl, tw, dw, max_seq, 1.0, True)
            o2.prefill(*inputs[k])
            if j > 0:
                o2.generate_target_only(j)
            row = o2.prefill_logits if j == 0 else o2.last_logits[-1]
            assert H.top2_gap(row) < 1e-2, f"sequence {k} differs at token {j}"
    seqs[1].close()
    seqs[2].close()
