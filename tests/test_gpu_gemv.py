"""GPU parity for the GEMV family (atom = RG_ATOM_SCALAR): bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth

from _gpu_util import DEV, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu
SC = rg.RG_ATOM_SCALAR


def _draw(M, N, K, seed, f16=False, spread=0):
    g = np.random.default_rng(seed)
    A = g.standard_normal((M, K)); B = g.standard_normal((N, K))
    if spread:
        A = A * np.exp2(g.integers(-spread, spread + 1, A.shape)); B = B * np.exp2(g.integers(-spread, spread + 1, B.shape))
    if f16:
        return A.astype(np.float16), B.astype(np.float16)
    return synth.f32_to_bf16_bits(A.astype(np.float32)), synth.f32_to_bf16_bits(B.astype(np.float32))


@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (1, 100, 1000), (3, 65, 4099), (8, 300, 14336), (13, 40, 520), (32, 64, 2048)])
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("fold", [0, 1])
def test_gemv_bit_exact(M, N, K, layout, fold):
    for f16 in (False, True):
        for spread in (0, 6):
            A, B = _draw(M, N, K, 7 + K, f16, spread)
            for fma in (0, 1):
                At, Bt = A, B
                if K % 8:      # rows must start on 16-byte boundaries: a view into a wider buffer
                    pad = 8 - K % 8
                    At = synth.to_torch(np.pad(A, ((0, 0), (0, pad))), DEV)[:, :K]
                    Bt = synth.to_torch(np.pad(B, ((0, 0), (0, pad))), DEV)[:, :K]
                got = gpu_gemm(At, Bt, atom=SC, gemv_layout=layout, gemv_fold=fold, fma=fma, out_dtype=rgo.F32)
                want = rgo.gemv(A, B, fma=fma, layout=layout, fold=fold, out_dtype=rgo.F32)
                assert_bits_equal(got, want, f"gemv {M}x{N}x{K} layout={layout} fold={fold} fma={fma} f16={f16} spread={spread}")


def test_gemv_closed_forms_epilogue_and_m_invariance():
    K, N = 14336, 512
    ones = synth.f32_to_bf16_bits(np.ones((4, K), np.float32))
    assert np.all(gpu_gemm(ones, ones[:1].repeat(N, 0), atom=SC, out_dtype=rgo.F32) == np.float32(K))
    A = synth.int_valued_bf16((9, 1000), -8, 8, 1); B = synth.int_valued_bf16((130, 1000), -8, 8, 2)
    want = (synth.bf16_bits_to_f32(A).astype(np.int64) @ synth.bf16_bits_to_f32(B).astype(np.int64).T).astype(np.float32)
    assert_bits_equal(gpu_gemm(A, B, atom=SC, out_dtype=rgo.F32), want, "integers")
    W = synth.normal_bf16((N, K), 0.02, 3); X = synth.normal_bf16((32, K), 1.0, 4)
    bias = synth.uniform_bf16((N,), -0.1, 0.1, 5); res = synth.normal_bf16((32, N), 1.0, 6)
    full = gpu_gemm(X, W, atom=SC, fma=1, bias=bias, act=1, residual=res)
    assert_bits_equal(full, rgo.gemv(X, W, fma=1, bias=bias, act=1, residual=res), "epilogue")
    for M in (1, 2, 5, 8, 9, 31):
        assert_bits_equal(gpu_gemm(X[:M], W, atom=SC, fma=1, bias=bias, act=1, residual=res[:M]), full[:M], f"rows at M={M}")
    # the family is its own class, and its two folds are two classes
    keys = {rg.rg_desc_class(rg.rg_desc()), rg.rg_desc_class(rg.rg_desc(atom=SC)), rg.rg_desc_class(rg.rg_desc(atom=SC, gemv_fold=1)),
            rg.rg_desc_class(rg.rg_desc(atom=SC, gemv_layout=1)), rg.rg_desc_class(rg.rg_desc(atom=SC, fma=1))}
    assert len(keys) == 5
    # and the folds really are different sums
    up = gpu_gemm(X, W, atom=SC, out_dtype=rgo.F32); down = gpu_gemm(X, W, atom=SC, gemv_fold=1, out_dtype=rgo.F32)
    assert (up.view(np.uint32) != down.view(np.uint32)).mean() > 0.05
