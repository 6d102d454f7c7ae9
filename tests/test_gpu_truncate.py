"""Top-k / top-p truncation on the device (spd_truncate_probs) against the CPU oracle: bit-exact
rows, and the rejection rule on truncated rows bit-exact end to end.  Integer masses and exact
fp32 comparisons define the kept set, one fp32 division per value the output, so there is no
tolerance."""
import numpy as np
import pytest

import synth
from oracle import sampling as S
from oracle import warp

from test_gpu_spd import _lib

F32 = np.float32
SETTINGS = [(50, 1.0), (0, 0.9), (40, 0.95), (1, 1.0), (0, 1.0), (0, 1e-4), (31999, 0.999)]


def _dev_truncate(spd, rows, top_k, top_p, in_place=False):
    import torch
    x = torch.from_numpy(np.ascontiguousarray(rows)).cuda()
    out = x if in_place else torch.full_like(x, float("nan"))
    spd.truncate_probs(x, out, top_k, top_p)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.gpu
@pytest.mark.parametrize("top_k,top_p", SETTINGS)
def test_truncated_rows_bit_exact_vocab_32000(top_k, top_p):
    spd = _lib()
    t_logits, d_logits = synth.microbench_logits(2, 5, 32000, 0.5)
    rows = np.concatenate([S.softmax_t(t_logits, 1.0).reshape(-1, 32000), S.softmax_t(d_logits, 1.0).reshape(-1, 32000)])
    want = warp.warp_rows(rows, top_k, top_p)
    got = _dev_truncate(spd, rows, top_k, top_p)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    kept = (want > 0).sum(axis=1)
    assert kept.min() >= 1 and (top_k < 1 or kept.max() <= top_k)
    assert np.array_equal(_dev_truncate(spd, rows, top_k, top_p, in_place=True).view(np.uint32), want.view(np.uint32))


@pytest.mark.gpu
@pytest.mark.parametrize("V", [1, 8, 33, 257, 1000, 50000])
def test_truncated_rows_with_many_ties_and_odd_sizes(V):
    """Probabilities quantised to a coarse grid (many equal values, zeros included): the cut
    falls inside a group of ties, which must be resolved by index."""
    spd = _lib()
    g = np.random.default_rng(V)
    raw = g.integers(0, 12, size=(6, V)).astype(F32)
    raw[:, 0] += 1
    rows = (raw / raw.sum(axis=1, keepdims=True)).astype(F32)
    rows[1] = F32(1.0) / F32(V)                     # every value equal
    rows[2, :] = 0
    rows[2, V // 2] = 1                             # one-hot
    for top_k, top_p in [(max(1, V // 3), 1.0), (0, 0.5), (max(1, V // 2), 0.7), (V + 5, 0.999), (3, 0.34)]:
        want = warp.warp_rows(rows, top_k, top_p)
        got = _dev_truncate(spd, rows, top_k, top_p)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (V, top_k, top_p)


@pytest.mark.gpu
@pytest.mark.parametrize("top_k,top_p", [(50, 1.0), (0, 0.9), (20, 0.8)])
def test_rule_on_truncated_rows_bit_exact(top_k, top_p):
    """Draft tokens drawn from the truncated q (oracle side, seeded uniforms), both rows truncated
    on the device, then the device's rejection rule: accepted counts and next tokens equal the
    oracle's on its own truncated rows."""
    import torch
    spd = _lib()
    B, gamma, V = 8, 5, 32000
    t_logits, d_logits = synth.microbench_logits(B, gamma, V, 0.5)
    p, q = S.softmax_t(t_logits, 1.0), S.softmax_t(d_logits, 1.0)
    pw, qw = warp.warp_rows(p, top_k, top_p), warp.warp_rows(q, top_k, top_p)
    u_draft = synth.uniforms(5, f"trunc.draft.{top_k}.{top_p}", (B, gamma))
    u = synth.uniforms(5, f"trunc.verify.{top_k}.{top_p}", (B, gamma + 1))
    ids = np.array([[S.sample_fixed_point(qw[b, j], u_draft[b, j]) for j in range(gamma)] for b in range(B)], np.int32)
    assert all(qw[b, j, ids[b, j]] > 0 for b in range(B) for j in range(gamma))
    want_acc, want_next = S.reject_sample_batch(pw, qw, ids, u)
    pd, qd = torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda()
    spd.truncate_probs(pd, pd, top_k, top_p)
    spd.truncate_probs(qd, qd, top_k, top_p)
    n_acc = torch.zeros(B, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(B, dtype=torch.int32, device="cuda")
    spd.reject_sample(pd, qd, torch.from_numpy(ids).cuda(), torch.from_numpy(u).cuda(), gamma, False, n_acc, nxt)
    torch.cuda.synchronize()
    assert np.array_equal(n_acc.cpu().numpy(), want_acc) and np.array_equal(nxt.cpu().numpy(), want_next)
    assert 0 < want_acc.sum() < B * gamma            # both branches of the rule ran


@pytest.mark.gpu
def test_truncate_argument_errors():
    import ctypes as C
    import torch
    spd = _lib()
    lib = spd.lib()
    x = torch.zeros((2, 64), device="cuda")
    host = np.zeros((2, 64), F32)
    p = C.c_void_p(x.data_ptr())
    f = C.c_float
    assert lib.spd_truncate_probs(p, p, 2, 64, 5, f(0.9), None) == spd.SPD_OK
    assert lib.spd_truncate_probs(None, p, 2, 64, 5, f(0.9), None) == spd.SPD_EINVAL
    assert lib.spd_truncate_probs(p, p, 0, 64, 5, f(0.9), None) == spd.SPD_EINVAL
    assert lib.spd_truncate_probs(p, p, 2, 64, 5, f(0.0), None) == spd.SPD_EINVAL
    assert lib.spd_truncate_probs(C.c_void_p(host.ctypes.data), p, 2, 64, 5, f(0.9), None) == spd.SPD_EINVAL
    assert lib.spd_truncate_probs(p, p, 2, 1 << 20, 5, f(0.9), None) == spd.SPD_EINVAL   # row larger than shared memory
    torch.cuda.synchronize()
