"""The allocation-free GEMM entry point against the regular one.

spd_skinny_gemm_noalloc is meant for hosts where this library may not call cudaMalloc or
cudaFree: programs whose device memory belongs to another allocator, latency-critical
loops that cannot afford the device-wide synchronisation an allocation implies, processes
with a memory budget fixed at start-up.  It keeps its scratch (barrier word, status block,
repacked weights) in a fixed array inside the library, shared by all calls.  This test calls
it several times in a row with different shapes and data -- each call sees whatever the one
before left in the scratch -- and compares each result with spd_skinny_gemm on the same inputs
and with an fp64 matrix product, checks that a warmed call leaves the amount of free device
memory exactly as it found it, that its status word reads clean afterwards, and that a matrix
too large for the fixed scratch is refused.

The file name sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest

import synth

F32 = np.float32


def _lib():
    from paper_2404_08856_b200 import build
    build.build()
    import paper_2404_08856_b200 as spd
    return spd


@pytest.mark.gpu
def test_noalloc_gemm_matches_regular_entry_point_twice_in_a_row():
    import torch
    spd = _lib()
    cases = [(6, 1000, 4096, 1), (3, 260, 688, 0), (8, 1536, 2048, 1)]   # the last reuses a dirty scratch
    for idx, (M, N, K, dtype) in enumerate(cases):
        g = np.random.default_rng(100 + idx)
        x = g.standard_normal((M, K)).astype(F32)
        w = (g.standard_normal((N, K)) * 0.05).astype(F32)
        if dtype == 1:
            wd = torch.from_numpy(synth.f32_to_bf16_bits(w).view(np.int16)).cuda()
        else:
            wd = torch.from_numpy(w).cuda()
        xd = torch.from_numpy(x).cuda()
        y_ref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        y_new = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        spd.skinny_gemm(xd, wd, y_ref, dtype)
        spd.skinny_gemm_noalloc(xd, wd, y_new, dtype)      # the first call per device does the set-up
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        y_new.fill_(float("nan"))
        spd.skinny_gemm_noalloc(xd, wd, y_new, dtype)      # warmed: must not allocate or free anything
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert spd.skinny_gemm_status(True) == spd.SPD_OK and spd.skinny_gemm_status(False) == spd.SPD_OK
        ref, new = y_ref.cpu().numpy(), y_new.cpu().numpy()
        assert np.isfinite(new).all()
        # same kernel, same arithmetic: the tolerance of the GEMM parity test is ample
        assert np.abs(new - ref).max() < 2e-4 * np.sqrt(K) * 0.05
        w_used = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(w)) if dtype == 1 else w
        want = x.astype(np.float64) @ w_used.astype(np.float64).T
        assert np.abs(new - want).max() < 2e-4 * np.sqrt(K) * 0.05


@pytest.mark.gpu
def test_noalloc_gemm_refuses_what_does_not_fit():
    import torch
    spd = _lib()
    M, N, K = 2, 4096, 4096                    # 32 MiB of bf16 weights > the 16 MiB scratch
    assert N * K * 2 > spd.NOALLOC_MAX_PACKED_BYTES
    x = torch.zeros(M, K, device="cuda")
    w = torch.zeros(N, K, dtype=torch.bfloat16, device="cuda")
    y = torch.full((M, N), 7.0, device="cuda")
    with pytest.raises(spd.SpdError) as e:
        spd.skinny_gemm_noalloc(x, w, y, 1)
    assert e.value.status == spd.SPD_EOVERFLOW
    torch.cuda.synchronize()
    assert float(y.min()) == 7.0               # nothing ran
