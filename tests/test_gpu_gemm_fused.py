"""Single-launch split-K (the merge inside the GEMM kernel): the same bits as the two-kernel path and as
the oracle, counters left at zero, whatever the shape, tree, part type, epilogue or operand type."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth
from tests._gpu_util import DEV, HW, HW8, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu


def fused_gemm(A, B, counters, *, out_dtype=rgo.BF16, bias=None, act=0, residual=None, **desc_kw):
    At = A if torch.is_tensor(A) else synth.to_torch(A, DEV)
    Bt = B if torch.is_tensor(B) else synth.to_torch(B, DEV)
    if At.dtype == torch.uint8:
        At, Bt = At.view(torch.float8_e4m3fn), Bt.view(torch.float8_e4m3fn)
        desc_kw.setdefault("in_dtype", rg.RG_F8E4M3)
    if At.dtype == torch.float16:
        desc_kw.setdefault("in_dtype", rg.RG_F16)
    M, N = At.shape[0], Bt.shape[0]
    d = rg.rg_desc(**desc_kw)
    tdt = {rgo.BF16: torch.bfloat16, rgo.F32: torch.float32, rgo.F16: torch.float16}[out_dtype]
    Ct = torch.empty((M, N), dtype=tdt, device=DEV)
    Ct.view(torch.int32 if out_dtype == rgo.F32 else torch.int16).fill_(-1)
    nb = rg.rg_gemm_workspace_bytes(d, M, N)
    ws = torch.full((max(nb, 16),), 0xFF, dtype=torch.uint8, device=DEV) if nb else None
    assert counters.numel() >= rg.rg_gemm_fused_merge_counters(d, M, N)
    bt = None if bias is None else synth.to_torch(bias, DEV)
    rt = None if residual is None else synth.to_torch(residual, DEV)
    rg.rg_gemm_fused_merge(d, At, Bt, Ct, counters, bias=bt, act=act, residual=rt, ws=ws)
    torch.cuda.synchronize()
    assert int(counters.abs().sum().item()) == 0, "counters must be left at zero"
    return synth.from_torch(Ct)


@pytest.fixture(scope="module")
def counters():
    return torch.zeros(8192, dtype=torch.int32, device=DEV)      # zeroed once; every call leaves it zero


@pytest.mark.parametrize("M,N,K,cuts", [(1, 64, 256, (128,)), (32, 4096, 14336, tuple(1792 * t for t in range(1, 8))),
                                        (7, 130, 1000, (16, 64, 144, 512)), (128, 520, 2048, (1024,)), (100, 96, 576, (192, 384)),
                                        (33, 70, 4096, tuple(64 * i for i in range(1, 64)))])
@pytest.mark.parametrize("tree", [rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED])
def test_same_bits_as_two_kernels_and_oracle(counters, M, N, K, cuts, tree):
    A = synth.normal_bf16((M, K), 1.0, 3 + M + K); B = synth.normal_bf16((N, K), 1.0, 4 + N)
    res = synth.normal_bf16((M, N), 1.0, 5)
    two = gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res)
    one = fused_gemm(A, B, counters, cuts=cuts, tree=tree, residual=res)
    assert_bits_equal(one, two, f"single launch vs two kernels {M}x{N}x{K} tree={tree}")
    if M * N <= 20000:
        want = rgo.gemm(A, B, cuts=cuts, tree=tree, atom_model=HW, residual=res)
        assert_bits_equal(one, want, "single launch vs oracle")


def test_part_types_epilogue_knobs_fp16_fp8_and_inner_span(counters):
    g = np.random.default_rng(2)
    A = synth.normal_bf16((70, 1024), 1.0, 1); B = synth.normal_bf16((200, 1024), 1.0, 2)
    bias = synth.uniform_bf16((200,), -0.1, 0.1, 3)
    cuts = (256, 512, 768)
    for pd, md in ((rgo.F32, rgo.F32), (rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16), (rgo.F16, rgo.F16)):
        for knobs in (dict(), dict(BN=64), dict(BN=112, BK=128), dict(BN=256, stages=2, raster=1)):
            for out in (rgo.BF16, rgo.F32):
                one = fused_gemm(A, B, counters, cuts=cuts, partial_dtype=pd, merge_dtype=md, bias=bias, act=1, out_dtype=out, **knobs)
                want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, partial_dtype=pd, merge_dtype=md, bias=bias, act=1, out_dtype=out)
                assert_bits_equal(one, want, f"partial={pd} merge={md} {knobs} out={out}")
    Ah = g.standard_normal((40, 512)).astype(np.float16); Bh = g.standard_normal((72, 512)).astype(np.float16)
    assert_bits_equal(fused_gemm(Ah, Bh, counters, cuts=(256,), out_dtype=rgo.F16), rgo.gemm(Ah, Bh, cuts=(256,), atom_model=HW, out_dtype=rgo.F16), "fp16")
    A8 = synth.normal_f8e4m3((33, 1024), 1.0, 7); B8 = synth.normal_f8e4m3((96, 1024), 1.0, 8)
    assert_bits_equal(fused_gemm(A8, B8, counters, cuts=(256, 640), out_dtype=rgo.F32), rgo.gemm(A8, B8, cuts=(256, 640), atom_model=HW8, out_dtype=rgo.F32), "fp8")
    assert_bits_equal(fused_gemm(A, B, counters, cuts=(512,), inner_span=128, out_dtype=rgo.F32),
                      rgo.gemm(A, B, cuts=(512,), inner_span=128, atom_model=HW, out_dtype=rgo.F32), "inner span")


def test_many_calls_share_counters_and_large_m_falls_back(counters):
    # decode loop: the same counters serve call after call, shapes alternating
    W1 = synth.normal_bf16((512, 2048), 0.05, 1); W2 = synth.normal_bf16((300, 1024), 0.05, 2)
    x1 = synth.normal_bf16((8, 2048), 1.0, 3); x2 = synth.normal_bf16((8, 1024), 1.0, 4)
    r1 = gpu_gemm(x1, W1, cuts=(512, 1024, 1536)); r2 = gpu_gemm(x2, W2, cuts=(512,))
    for _ in range(5):
        assert_bits_equal(fused_gemm(x1, W1, counters, cuts=(512, 1024, 1536)), r1, "repeat 1")
        assert_bits_equal(fused_gemm(x2, W2, counters, cuts=(512,)), r2, "repeat 2")
    # a shape that runs on the two-SM kernel ignores the counters and still gives the class's bits
    A = synth.normal_bf16((600, 512), 1.0, 5); B = synth.normal_bf16((1024, 512), 1.0, 6)
    assert_bits_equal(fused_gemm(A, B, counters, cuts=(256,), cta_group=2, BN=128), gpu_gemm(A, B, cuts=(256,)), "two-SM fallback")
    # many tiles and a multi-tile M on the one-CTA kernel
    assert_bits_equal(fused_gemm(A, B, counters, cuts=(128, 384), cta_group=1, BN=64), gpu_gemm(A, B, cuts=(128, 384)), "one-CTA, 5 x 16 tiles")
    assert rg.rg_device_status() == 0


def test_argument_errors(counters):
    A = torch.zeros((8, 256), dtype=torch.bfloat16, device=DEV); B = torch.zeros((64, 256), dtype=torch.bfloat16, device=DEV)
    C = torch.zeros((8, 64), dtype=torch.bfloat16, device=DEV)
    d = rg.rg_desc(cuts=(128,))
    ws = torch.empty(rg.rg_gemm_workspace_bytes(d, 8, 64), dtype=torch.uint8, device=DEV)
    with pytest.raises(rg.RgError):
        rg.rg_gemm_fused_merge(d, A, B, C, None, ws=ws)
    with pytest.raises(rg.RgError):
        rg.rg_gemm_fused_merge(d, A, B, C, counters[:1], ws=ws)
    with pytest.raises(rg.RgError):
        rg.rg_gemm_fused_merge(d, A, B, C, counters)                 # workspace missing
    rg.rg_gemm_fused_merge(rg.rg_desc(), A, B, C, None)              # no cuts: plain rg_gemm, no counters needed
