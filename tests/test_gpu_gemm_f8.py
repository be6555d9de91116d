"""GPU parity for e4m3 operands (32-wide tensor-core step): the CUDA path against the oracle, bit
for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth
from tests._gpu_util import DEV, HW8, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu


def _draws(M, N, K, seed):
    g = np.random.default_rng(seed)
    A = g.standard_normal((M, K)); B = g.standard_normal((N, K))
    yield "ordinary", synth.f32_to_f8e4m3_bits(A.astype(np.float32)), synth.f32_to_f8e4m3_bits(B.astype(np.float32))
    As = np.clip(A * np.exp2(g.integers(-7, 8, A.shape)), -448, 448); Bs = np.clip(B * np.exp2(g.integers(-7, 8, B.shape)), -448, 448)
    yield "spread", synth.f32_to_f8e4m3_bits(As.astype(np.float32)), synth.f32_to_f8e4m3_bits(Bs.astype(np.float32))


@pytest.mark.parametrize("M,N,K", [(1, 1, 32), (1, 8, 16), (3, 5, 48), (129, 65, 160), (300, 520, 1000), (513, 260, 2048)])
@pytest.mark.parametrize("knobs", [dict(), dict(BN=64), dict(cta_group=2, BN=128), dict(BN=48, cta_group=1), dict(BN=256, BK=128, stages=2),
                                   dict(cta_group=2, BN=64), dict(cta_group=2, BN=208, BK=128)])
def test_integer_inputs_exact(M, N, K, knobs):
    A = synth.int_valued_f8e4m3((M, K), -8, 8, 1 + K); B = synth.int_valued_f8e4m3((N, K), -8, 8, 2 + K)
    want = (synth.f8e4m3_bits_to_f32(A).astype(np.int64) @ synth.f8e4m3_bits_to_f32(B).astype(np.int64).T).astype(np.float32)
    assert_bits_equal(gpu_gemm(A, B, out_dtype=rgo.F32, **knobs), want, f"fp8 ints {M}x{N}x{K} {knobs}")


@pytest.mark.parametrize("M,N,K,cuts", [(100, 96, 64, ()), (64, 128, 4096, ()), (33, 70, 1006, ()), (40, 72, 2048, (512, 1024, 1536)),
                                        (300, 260, 1024, (256,)), (70, 130, 736, (32, 96, 704))])
def test_random_inputs_bit_exact_under_fitted_step_model(M, N, K, cuts):
    for name, A, B in _draws(M, N, K, 70 + K):
        want = rgo.gemm(A, B, cuts=cuts, atom_model=HW8, out_dtype=rgo.F32)
        for knobs in (dict(), dict(cta_group=2, BN=256), dict(BN=112, cta_group=1)):
            assert_bits_equal(gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32, **knobs), want, f"fp8 {M}x{N}x{K} {name} {knobs}")


def test_split_partials_epilogue_outputs_and_class():
    A, B = next(_draws(70, 200, 1024, 5))[1:]
    cuts = (256, 512, 768)
    bias = synth.uniform_bf16((200,), -0.1, 0.1, 2)
    res = synth.normal_bf16((70, 200), 1.0, 3)
    for pd, md in ((rgo.F32, rgo.F32), (rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16)):
        for tree in (rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED):
            for out in (rgo.BF16, rgo.F16, rgo.F32):
                got = gpu_gemm(A, B, cuts=cuts, tree=tree, partial_dtype=pd, merge_dtype=md, bias=bias, act=1, residual=res, out_dtype=out)
                want = rgo.gemm(A, B, cuts=cuts, tree=tree, atom_model=HW8, partial_dtype=pd, merge_dtype=md, bias=bias, act=1,
                                residual=res, out_dtype=out)
                assert_bits_equal(got, want, f"fp8 split partial={pd} merge={md} tree={tree} out={out}")
    d8 = rg.rg_desc(in_dtype=rg.RG_F8E4M3)
    assert d8.atom == rg.RG_ATOM_TC_F8_K32
    assert len({rg.rg_desc_class(d8), rg.rg_desc_class(rg.rg_desc()), rg.rg_desc_class(rg.rg_desc(in_dtype=rg.RG_F16))}) == 3
    # operands must be of the descriptor's input type
    with pytest.raises(rg.RgError):
        rg.rg_gemm(rg.rg_desc(), synth.to_torch(A, DEV).view(torch.float8_e4m3fn), synth.to_torch(B, DEV).view(torch.float8_e4m3fn),
                   torch.empty((70, 200), dtype=torch.bfloat16, device=DEV))


def test_inner_span_groups_bit_exact():
    A, B = list(_draws(50, 96, 1536, 9))[1][1:]
    for cuts, span in (((), 128), ((512, 1024), 256), ((768,), 384), ((), 32), ((512, 1024), 96), ((), 160)):   # 32 = one step per accumulator
        want = rgo.gemm(A, B, cuts=cuts, inner_span=span, atom_model=HW8, out_dtype=rgo.F32)
        assert_bits_equal(gpu_gemm(A, B, cuts=cuts, inner_span=span, out_dtype=rgo.F32), want, f"fp8 inner_span {span} cuts {cuts}")


def test_batch_and_tile_invariance_and_decode_shape():
    N, K = 512, 4096
    g = np.random.default_rng(4)
    B = synth.f32_to_f8e4m3_bits((g.standard_normal((N, K)) * 0.5).astype(np.float32))
    A = synth.f32_to_f8e4m3_bits(g.standard_normal((300, K)).astype(np.float32))
    cuts = (1024, 2048, 3072)
    full = gpu_gemm(A, B, cuts=cuts)
    for M in (1, 7, 32, 129):
        assert_bits_equal(gpu_gemm(A[:M], B, cuts=cuts), full[:M], f"fp8 batch invariance M={M}")
    ref = gpu_gemm(A, B)
    for knobs in (dict(BN=64), dict(BN=128, BK=128), dict(cta_group=2, BN=128), dict(cta_group=2, BN=256, BK=128), dict(BN=176, BK=256)):
        assert_bits_equal(gpu_gemm(A, B, **knobs), ref, f"fp8 tile config {knobs}")
    si, sj = g.integers(0, 300, 200), g.integers(0, N, 200)
    want = rgo.gemm_samples(A, B, si, sj, atom_model=HW8, out_dtype=rgo.BF16)
    assert_bits_equal(synth.bf16_bits_to_f32(ref[si, sj]), want, "fp8 sampled oracle")


def test_large_square_sampled_and_repeatable():
    n = 4096
    g = torch.Generator(device=DEV); g.manual_seed(5)
    A = torch.randn((n, n), generator=g, device=DEV).to(torch.float8_e4m3fn)
    B = torch.randn((n, n), generator=g, device=DEV).to(torch.float8_e4m3fn)
    c1 = gpu_gemm(A, B); c2 = gpu_gemm(A, B, cta_group=1, BN=128)
    assert_bits_equal(c1, c2, "fp8 4096^3 pair vs one-CTA")
    r = np.random.default_rng(6)
    si, sj = r.integers(0, n, 300), r.integers(0, n, 300)
    An = A.view(torch.uint8).cpu().numpy(); Bn = B.view(torch.uint8).cpu().numpy()
    want = rgo.gemm_samples(An, Bn, si, sj, atom_model=HW8, out_dtype=rgo.BF16)
    assert_bits_equal(synth.bf16_bits_to_f32(c1[si, sj]), want, "fp8 4096^3 sampled oracle")
    assert rg.rg_device_status() == 0


def test_host_buffer_form_matches_device_form():
    from paper_2609_11356_b200.api import rg_gemm_host, rg_gemm_host_scratch_bytes
    A, B = next(_draws(40, 72, 512, 8))[1:]
    want = gpu_gemm(A, B, cuts=(256,))
    d = rg.rg_desc(cuts=(256,), in_dtype=rg.RG_F8E4M3)
    At = torch.from_numpy(A).view(torch.float8_e4m3fn).pin_memory(); Bt = torch.from_numpy(B).view(torch.float8_e4m3fn).pin_memory()
    Ct = torch.empty((40, 72), dtype=torch.bfloat16).pin_memory()
    nb = rg_gemm_host_scratch_bytes(d, 40, 72, 512, rg.RG_BF16)
    scratch = torch.empty(nb, dtype=torch.uint8, device=DEV)
    rg_gemm_host(d, At, Bt, Ct, scratch)
    torch.cuda.synchronize()
    assert_bits_equal(synth.from_torch(Ct), want, "fp8 host-buffer form")
