"""Problems whose element counts and byte offsets pass 2^31 and 2^32: every index on the CUDA path is 64-bit.

Integer-valued inputs, so the expected values are exact integer sums whatever the order (Sec. 3.1: with
exact partial sums every tree gives the same value); they come from numpy on the host, never from the GPU.
"""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth
from _gpu_util import DEV, assert_bits_equal

pytestmark = pytest.mark.gpu


def _rows(total, g, n):
    return np.unique(np.concatenate([[0, 1, 127, 128, total - 129, total - 2, total - 1], g.integers(0, total, n)]))


@pytest.mark.parametrize("knobs", [dict(), dict(cta_group=1, BN=128), dict(cuts=(16,))])
def test_gemm_more_than_2_31_outputs(knobs):
    M, N, K = 66000, 32784, 48                                  # 2.16e9 outputs, 4.3 GB of bf16; N off the tile grid
    A = synth.int_valued_bf16((M, K), -3, 3, 5); B = synth.int_valued_bf16((N, K), -3, 3, 6)
    At, Bt = synth.to_torch(A, DEV), synth.to_torch(B, DEV)
    C = torch.empty((M, N), dtype=torch.bfloat16, device=DEV)
    C.view(torch.int16).fill_(-1)                                # NaN pattern: an unwritten element shows
    d = rg.rg_desc(**knobs)
    nb = rg.rg_gemm_workspace_bytes(d, M, N)                     # with a cut: two fp32 parts, 17 GB, offsets past 2^33
    ws = torch.empty(nb, dtype=torch.uint8, device=DEV) if nb else None
    rg.rg_gemm(d, At, Bt, C, ws=ws)
    torch.cuda.synchronize()
    g = np.random.default_rng(7)
    rows = _rows(M, g, 24)
    got = synth.from_torch(C[torch.as_tensor(rows, device=DEV)])
    Af = synth.bf16_bits_to_f32(A[rows]).astype(np.int64); Bf = synth.bf16_bits_to_f32(B).astype(np.int64)
    want = synth.f32_to_bf16_bits((Af @ Bf.T).astype(np.float32))   # |sum| <= 432: exact in fp32, rounded once to bf16
    assert_bits_equal(got, want, f"sampled rows of a 66000 x 32784 product {knobs}")
    # nothing unwritten anywhere: no element still holds the poison pattern
    assert int((C.view(torch.int16) == -1).sum().item()) == 0
    assert rg.rg_device_status() == 0


def test_row_reductions_more_than_2_31_elements():
    R, Cc = 70000, 32768                                        # 2.29e9 elements, 9.2 GB of fp32
    g = torch.Generator(device=DEV); g.manual_seed(11)
    x = torch.randint(-8, 9, (R, Cc), generator=g, device=DEV, dtype=torch.int32).to(torch.float32)
    out = torch.full((R,), float("nan"), dtype=torch.float32, device=DEV)
    rg.rg_reduce_rows(rg.rg_desc(), rg.RG_OP_SUM, x, out)
    torch.cuda.synchronize()
    r = np.random.default_rng(12)
    rows = _rows(R, r, 40)
    xs = x[torch.as_tensor(rows, device=DEV)].cpu().numpy()
    want = xs.astype(np.int64).sum(axis=1).astype(np.float32)   # |sum| < 2^24: every partial sum is exact
    assert_bits_equal(out.cpu().numpy()[rows], want, "row sums of a 70000 x 32768 matrix")
    assert not bool(torch.isnan(out).any().item())
    # the oracle agrees on a few of those rows (the tree itself, not only the exact value)
    few = rows[:6]
    wo, _ = rgo.reduce_rows(rgo.OP_SUM, xs[:6])
    assert_bits_equal(out.cpu().numpy()[few], wo, "oracle on sampled rows")
    # RMSNorm over the same rows of a bf16 matrix with as many elements (row offsets past 2^32 bytes)
    xb = x[:, :4096].to(torch.bfloat16)
    big = torch.empty((600000, 4096), dtype=torch.bfloat16, device=DEV)          # 2.46e9 elements
    big[:R] = xb; big[-R:] = xb
    y = torch.empty_like(big)
    w = synth.to_torch(synth.normal_bf16((4096,), 0.05, 3, mean=1.0), DEV)
    rg.rg_reduce_rows(rg.rg_desc(), rg.RG_OP_RMSNORM, big, y, weight=w, eps=1e-5)
    torch.cuda.synchronize()
    tail = np.array([600000 - R, 600000 - R + 1, 599999])
    src = synth.from_torch(big[torch.as_tensor(tail, device=DEV)])
    wy, _ = rgo.reduce_rows(rgo.OP_RMSNORM, src, weight=synth.from_torch(w), eps=1e-5)
    assert_bits_equal(synth.from_torch(y[torch.as_tensor(tail, device=DEV)]), wy, "RMSNorm rows past 2^32 bytes")
    assert rg.rg_device_status() == 0


def test_column_sum_more_than_2_31_elements():
    R, Cc = 300000, 8192                                        # 2.46e9 elements, 9.8 GB of fp32
    g = torch.Generator(device=DEV); g.manual_seed(13)
    x = torch.randint(-4, 5, (R, Cc), generator=g, device=DEV, dtype=torch.int32).to(torch.float32)
    out = torch.full((Cc,), float("nan"), dtype=torch.float32, device=DEV)
    nb = rg.rg_reduce_cols_workspace_bytes(R, Cc)
    ws = torch.empty(max(nb, 1), dtype=torch.uint8, device=DEV)
    rg.rg_reduce_cols(rg.rg_desc(), rg.RG_COLOP_SUM, x, out, ws=ws)
    torch.cuda.synchronize()
    cols = np.unique(np.concatenate([[0, 1, Cc - 1], np.random.default_rng(14).integers(0, Cc, 200)]))
    host = x[:, torch.as_tensor(cols, device=DEV)].cpu().numpy().astype(np.int64).sum(axis=0).astype(np.float32)   # integers below 2^24: exact
    assert_bits_equal(out.cpu().numpy()[cols], host, "column sums (host integers) of a 300000 x 8192 matrix")
    assert not bool(torch.isnan(out).any().item())
    assert rg.rg_device_status() == 0
