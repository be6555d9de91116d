"""rg_gemm_noalloc: the split-K GEMM for callers that cannot allocate device memory (a frozen
memory pool, a host framework that owns the allocator, a decode path that cannot take
cudaMalloc's synchronisation).  Its workspace is a fixed array inside the library, so the test
checks that it returns the same bits as rg_gemm with a caller-provided workspace, twice in a
row (the second call sees whatever the first left in the shared array), and that a shape whose
workspace exceeds the array is refused.  Collected last, so a failure here cannot hide others."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from paper_2609_11356_b200 import _cabi, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both(A, B, cuts, **epi):
    d = rg.rg_desc(cuts=cuts)
    M, N = A.shape[0], B.shape[0]
    At, Bt = synth.to_torch(A, DEV), synth.to_torch(B, DEV)
    kw = {k: synth.to_torch(v, DEV) if isinstance(v, np.ndarray) else v for k, v in epi.items()}
    ref = torch.empty((M, N), dtype=torch.bfloat16, device=DEV)
    ws = torch.empty(rg.rg_gemm_workspace_bytes(d, M, N), dtype=torch.uint8, device=DEV)
    rg.rg_gemm(d, At, Bt, ref, ws=ws, **kw)
    out = torch.empty((M, N), dtype=torch.bfloat16, device=DEV)
    out.view(torch.int16).fill_(-1)
    rg.rg_gemm_noalloc(d, At, Bt, out, **kw)
    torch.cuda.synchronize()
    return synth.from_torch(out), synth.from_torch(ref)


def test_noalloc_matches_rg_gemm_on_two_calls_in_a_row():
    # first call: the decode shape, 8 parts, fills 4 MiB of the shared array
    cuts = tuple(1792 * t for t in range(1, 8))
    A = synth.normal_bf16((32, 14336), 1.0, 4); B = synth.normal_bf16((4096, 14336), 0.02, 3)
    res = synth.normal_bf16((32, 4096), 1.0, 5)
    got, want = _both(A, B, cuts, residual=res)
    assert np.array_equal(got, want)
    # second call: a smaller, ragged problem that reuses the array with the first call's leftovers in it
    A2 = synth.spread_exponents_bf16(synth.normal_bf16((19, 1000), 1.0, 6), 7, -8, 8)
    B2 = synth.normal_bf16((301, 1000), 1.0, 8)
    bias = synth.uniform_bf16((301,), -0.1, 0.1, 9)
    got2, want2 = _both(A2, B2, (256, 512, 768), bias=bias, act=1)
    assert np.array_equal(got2, want2)
    # and the first problem again gives the first answer again
    got3, _ = _both(A, B, cuts, residual=res)
    assert np.array_equal(got3, want)
    assert rg.rg_device_status() == 0


def test_noalloc_refuses_what_does_not_fit_and_needs_no_scratch_without_cuts():
    d = rg.rg_desc(cuts=(1024,))
    M, N = 2048, 2048                     # 2 parts x 2048 x 2048 x 4 B = 32 MiB > the fixed 8 MiB
    assert rg.rg_gemm_workspace_bytes(d, M, N) > _cabi.RG_NOALLOC_WS_BYTES
    A = torch.zeros((M, 2048), dtype=torch.bfloat16, device=DEV); B = torch.zeros((N, 2048), dtype=torch.bfloat16, device=DEV)
    out = torch.full((M, N), 7.0, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(rg.RgError) as ei:
        rg.rg_gemm_noalloc(d, A, B, out)
    assert ei.value.status == 6           # RG_ERR_WORKSPACE, and nothing ran:
    torch.cuda.synchronize()
    assert torch.all(out == 7.0)
    # a descriptor without cuts has no parts to store: plain forwarding
    Ai = synth.int_valued_bf16((40, 128), -8, 8, 1); Bi = synth.int_valued_bf16((24, 128), -8, 8, 2)
    o2 = torch.empty((40, 24), dtype=torch.bfloat16, device=DEV)
    rg.rg_gemm_noalloc(rg.rg_desc(), synth.to_torch(Ai, DEV), synth.to_torch(Bi, DEV), o2)
    want = synth.bf16_bits_to_f32(Ai).astype(np.int64) @ synth.bf16_bits_to_f32(Bi).astype(np.int64).T
    assert np.array_equal(synth.from_torch(o2), synth.f32_to_bf16_bits(want.astype(np.float32)))   # one rounding to bf16
