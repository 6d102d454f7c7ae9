"""Parity of the image adapter V = g_theta(H) (spd_image_adapter, tensor-core GEMMs with the
GELU in the first GEMM's epilogue) with the fp64 CPU oracle, alone and in front of the
prefill.

Tolerance on the adapter's output.  Features and the hidden layer are carried as bf16 hi + lo
pairs (relative error 2^-17 per element) and accumulated in fp32 over K <= 4096 terms; with
|V| of order 1 both error sources stay below 1e-5, erff adds a few ulp.  The bound used is
1e-4 absolute + 1e-4 relative.
"""
import ctypes as C

import numpy as np
import pytest

import synth
from oracle import adapter as OA

import harness as H
from test_gpu_spd import _lib, lockstep

F32 = np.float32


def _tiny_ctx():
    wl = synth.tiny_workload()
    tw, dw = H.build_weights(wl)
    return H.make_gpu(wl, tw, dw, 64)


def _run(gpu, feats, w1_bits, w2_bits, host_feats):
    import torch
    w1 = torch.from_numpy(w1_bits.view(np.int16)).cuda().view(torch.bfloat16)
    w2 = torch.from_numpy(w2_bits.view(np.int16)).cuda().view(torch.bfloat16)
    out = torch.full((feats.shape[0], w2.shape[0]), float("nan"), device="cuda", dtype=torch.float32)
    f = np.ascontiguousarray(feats) if host_feats else torch.from_numpy(feats).cuda()
    gpu.image_adapter(f, w1, w2, out)
    return out.cpu().numpy()


@pytest.mark.gpu
@pytest.mark.parametrize("m,d_in,d_hid,d_out,host_feats", [
    (576, 1024, 4096, 4096, True),     # the 7B target's adapter (Appendix A.1)
    (576, 1024, 1024, 1024, False),    # a draft's own adapter (Appendix A.1)
    (100, 72, 200, 52, False),         # ragged: partial row tile, K tails, odd output width
    (1, 8, 8, 1, True),
])
def test_image_adapter_matches_oracle(m, d_in, d_hid, d_out, host_feats):
    _lib()
    gpu = _tiny_ctx()
    feats = synth.vision_features(2, m, d_in)
    w1, w2 = synth.adapter_mlp(1, "target", d_in, d_hid, d_out, std=0.02 if d_in >= 1024 else 0.2)
    want = OA.image_adapter(feats, synth.bf16_bits_to_f32(w1), synth.bf16_bits_to_f32(w2))
    for _ in range(2):   # second call reuses the context's scratch
        got = _run(gpu, feats, w1, w2, host_feats)
        assert got.shape == want.shape and np.isfinite(got).all()
        err = np.abs(got - want)
        assert (err <= 1e-4 + 1e-4 * np.abs(want)).all(), f"max error {err.max()} at scale {np.abs(want).max()}"
    assert np.abs(want).max() > 0.05   # the comparison is not vacuous
    gpu.close()


@pytest.mark.gpu
def test_image_adapter_argument_errors():
    import torch
    spd = _lib()
    gpu = _tiny_ctx()
    lib = spd.lib()
    feats = np.zeros((4, 16), F32)
    w = torch.zeros((16, 16), device="cuda", dtype=torch.bfloat16)
    out = torch.zeros((4, 16), device="cuda", dtype=torch.float32)
    host_w = np.zeros((16, 16), np.uint16)
    p = lambda a: C.c_void_p(a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data)
    call = lambda f, m, di, w1, dh, w2, do, o: lib.spd_image_adapter(gpu._ctx, f, m, di, w1, dh, w2, do, o)
    assert call(p(feats), 4, 16, p(w), 16, p(w), 16, p(out)) == spd.SPD_OK
    assert call(p(feats), 4, 12, p(w), 16, p(w), 16, p(out)) == spd.SPD_EINVAL      # d_in % 8
    assert call(p(feats), 0, 16, p(w), 16, p(w), 16, p(out)) == spd.SPD_EINVAL      # no rows
    assert call(p(feats), 4, 16, p(host_w), 16, p(w), 16, p(out)) == spd.SPD_EINVAL  # host weights
    assert call(None, 4, 16, p(w), 16, p(w), 16, p(out)) == spd.SPD_EINVAL
    assert lib.spd_image_adapter(None, p(feats), 4, 16, p(w), 16, p(w), 16, p(out)) == spd.SPD_EINVAL
    assert b"adapter" in lib.spd_last_error(gpu._ctx)
    gpu.close()


@pytest.mark.gpu
@pytest.mark.parametrize("greedy", [True, False])
def test_adapter_in_front_of_the_prefill_two_layer_llava7b_shape(greedy):
    """H [576, 1024] -> g_theta (1024 -> 4096 -> 4096) -> V -> prefill -> speculative blocks,
    device result handed from the adapter to the prefill without leaving the GPU."""
    import torch
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=2)
    feats = synth.vision_features(wl.seeds["inputs"], wl.n_image, 1024)
    w1, w2 = synth.adapter_mlp(wl.seeds["weights"], "target", 1024, 4096, 4096)

    def image_from(gpu):
        out = torch.empty((wl.n_image, 4096), device="cuda", dtype=torch.float32)
        gpu.image_adapter(feats, torch.from_numpy(w1.view(np.int16)).cuda().view(torch.bfloat16),
                          torch.from_numpy(w2.view(np.int16)).cuda().view(torch.bfloat16), out)
        want = OA.image_adapter(feats, synth.bf16_bits_to_f32(w1), synth.bf16_bits_to_f32(w2)).astype(F32)
        return out, want

    rep = lockstep(wl, greedy=greedy, temperature=1.0, n_blocks=2, logit_tol=5e-2, image_from=image_from)
    assert rep["blocks"] == 2 and rep["max_logit_err"] < 1e-2


@pytest.mark.gpu
def test_table1_draft_with_its_own_two_layer_adapter():
    """The paper's own draft column (Table 1: 4 layers, hidden 1024, 8 heads, intermediate 2816;
    2 layers here) with the draft-side adapter 1024 -> 1024 -> 1024 of Appendix A.1: both
    adapters run on the GPU, their outputs go to the prefill as device rows, then speculative
    blocks follow in lock-step with the oracle."""
    import torch
    wl = synth.llava7b_workload(gamma=3, n_layers=2, draft_layers=2, draft="table1", draft_mlp=True)
    feats = synth.vision_features(wl.seeds["inputs"], wl.n_image, 1024)
    tw1, tw2 = synth.adapter_mlp(wl.seeds["weights"], "target", 1024, 4096, 4096)
    dw1, dw2 = synth.adapter_mlp(wl.seeds["weights"], "draft", 1024, 1024, 1024)
    dev = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)

    def image_from(gpu):
        v_t = torch.empty((wl.n_image, 4096), device="cuda", dtype=torch.float32)
        v_d = torch.empty((wl.n_image, 1024), device="cuda", dtype=torch.float32)
        gpu.image_adapter(feats, dev(tw1), dev(tw2), v_t)
        gpu.image_adapter(feats, dev(dw1), dev(dw2), v_d)
        o_t = OA.image_adapter(feats, synth.bf16_bits_to_f32(tw1), synth.bf16_bits_to_f32(tw2)).astype(F32)
        o_d = OA.image_adapter(feats, synth.bf16_bits_to_f32(dw1), synth.bf16_bits_to_f32(dw2)).astype(F32)
        return v_t, o_t, v_d, o_d

    rep = lockstep(wl, greedy=False, temperature=1.0, n_blocks=3, logit_tol=5e-2, image_from=image_from)
    assert rep["blocks"] == 3 and rep["max_logit_err"] < 1e-2 and rep["max_draft_logit_err"] < 1e-2


@pytest.mark.gpu
def test_table1_draft_text_only_lockstep():
    """Text-only draft of the Table-1 shape against the 2-layer LLaVA-7B-shaped target."""
    wl = synth.llava7b_workload(gamma=5, n_layers=2, draft_layers=4, draft="table1")
    rep = lockstep(wl, greedy=True, temperature=1.0, n_blocks=2, logit_tol=5e-2)
    assert rep["blocks"] == 2 and rep["max_draft_logit_err"] < 1e-2
