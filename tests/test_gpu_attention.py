"""GPU parity for attention with a fixed descriptor (App. F): the CUDA path against the oracle, bit
for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth
from tests._gpu_util import DEV, HW, assert_bits_equal

pytestmark = pytest.mark.gpu


def gpu_attention(Q, K, V, *, block_n, scale, heads=1, out_dtype=rgo.BF16, exp_base=0, causal=False):
    """Q [heads*Nq, d], K [heads*Nk, d], V [heads*Nk, d] as bf16 bit patterns."""
    d = Q.shape[1]; Nk = K.shape[0] // heads
    Vt = np.ascontiguousarray(V.reshape(heads, Nk, d).transpose(0, 2, 1)).reshape(heads * d, Nk)
    Nkp = (Nk + 7) // 8 * 8                                     # rows of Vt start on 16-byte boundaries
    vt = torch.zeros((heads * d, Nkp), dtype=torch.bfloat16, device=DEV)
    vt[:, :Nk] = synth.to_torch(Vt, DEV)
    tdt = {rgo.BF16: torch.bfloat16, rgo.F32: torch.float32, rgo.F16: torch.float16}[out_dtype]
    O = torch.empty((Q.shape[0], d), dtype=tdt, device=DEV)
    O.view(torch.int32 if out_dtype == rgo.F32 else torch.int16).fill_(-1)
    rg.rg_attention(rg.rg_attn_desc(block_n=block_n, scale=scale, heads=heads, exp_base=exp_base, mask=1 if causal else 0), synth.to_torch(Q, DEV), synth.to_torch(K, DEV), vt[:, :Nk], O)
    torch.cuda.synchronize()
    return synth.from_torch(O)


def _draw(Nq, Nk, d, seed, heads=1, spread=0):
    g = np.random.default_rng(seed)
    mk = lambda n: g.standard_normal((heads * n, d)) * (np.exp2(g.integers(-spread, spread + 1, (heads * n, d))) if spread else 1.0)
    return tuple(synth.f32_to_bf16_bits(mk(n).astype(np.float32)) for n in (Nq, Nk, Nk))


@pytest.mark.parametrize("Nq,Nk,d,w", [(128, 128, 128, 128), (128, 64, 64, 64), (1, 1, 64, 64), (5, 37, 128, 64), (130, 300, 128, 128),
                                       (257, 1000, 64, 128), (300, 520, 128, 64), (64, 2048, 128, 128)])
def test_single_head_bit_exact(Nq, Nk, d, w):
    Q, K, V = _draw(Nq, Nk, d, 7 + Nq + Nk)
    scale = float(np.float32(d ** -0.5))
    for out in (rgo.F32, rgo.BF16):
        got = gpu_attention(Q, K, V, block_n=w, scale=scale, out_dtype=out)
        want = rgo.attention(Q, K, V, block_n=w, scale=scale, atom_model=HW, out_dtype=out)
        assert_bits_equal(got, want, f"attention {Nq}x{Nk} d={d} w={w} out={out}")


@pytest.mark.parametrize("Nq,Nk,d,w", [(128, 128, 128, 128), (5, 37, 128, 64), (257, 1000, 64, 128), (300, 520, 128, 64)])
def test_base_two_variant_bit_exact(Nq, Nk, d, w):
    Q, K, V = _draw(Nq, Nk, d, 17 + Nq + Nk)
    scale = float(np.float32(d ** -0.5 * np.log2(np.e)))
    got = gpu_attention(Q, K, V, block_n=w, scale=scale, out_dtype=rgo.F32, exp_base=2)
    want = rgo.attention(Q, K, V, block_n=w, scale=scale, atom_model=HW, out_dtype=rgo.F32, exp_base=2)
    assert_bits_equal(got, want, f"attention base two {Nq}x{Nk} d={d} w={w}")


@pytest.mark.parametrize("base", [2, 0])
@pytest.mark.parametrize("Nq,Nk,d,w,scale", [(256, 512, 128, 128, 3.0), (130, 256, 64, 64, 6.0), (128, 384, 128, 128, 0.5)])
def test_wide_scores_underflow(Nq, Nk, d, w, scale, base):
    """Scores spread far past the underflow threshold below the row maximum: full key blocks in which some
    probabilities underflow to +0 and others do not (the chunk-level range test of the kernel must
    fall back to the per-element selects of the specified exponential)."""
    Q, K, V = _draw(Nq, Nk, d, 5 + Nq + Nk, spread=2)
    got = gpu_attention(Q, K, V, block_n=w, scale=scale, out_dtype=rgo.F32, exp_base=base)
    want = rgo.attention(Q, K, V, block_n=w, scale=scale, atom_model=HW, out_dtype=rgo.F32, exp_base=base)
    assert_bits_equal(got, want, f"wide scores {Nq}x{Nk} d={d} w={w} scale={scale} base={base}")


@pytest.mark.parametrize("N,d,w,base", [(128, 128, 128, 0), (300, 64, 64, 2), (1000, 128, 64, 0), (777, 128, 128, 2)])
def test_causal_bit_exact(N, d, w, base):
    H = 2
    Q, K, V = _draw(N, N, d, 31 + N, heads=H)
    scale = float(np.float32(d ** -0.5 * (np.log2(np.e) if base == 2 else 1.0)))
    got = gpu_attention(Q, K, V, block_n=w, scale=scale, heads=H, out_dtype=rgo.F32, exp_base=base, causal=True)
    for h in range(H):
        want = rgo.attention(Q[h * N:(h + 1) * N], K[h * N:(h + 1) * N], V[h * N:(h + 1) * N], block_n=w, scale=scale,
                             atom_model=HW, out_dtype=rgo.F32, exp_base=base, causal=True)
        assert_bits_equal(got[h * N:(h + 1) * N], want, f"causal N={N} d={d} w={w} base={base} head {h}")
    # the first query of every head sees one key
    assert_bits_equal(got[0], synth.bf16_bits_to_f32(V[0]), "first row")


def test_heads_block_width_and_spread_inputs():
    H, Nq, Nk, d = 3, 200, 333, 128
    Q, K, V = _draw(Nq, Nk, d, 11, heads=H, spread=3)
    scale = 0.11
    outs = {}
    for w in (64, 128):
        got = gpu_attention(Q, K, V, block_n=w, scale=scale, heads=H, out_dtype=rgo.F32)
        for h in range(H):
            want = rgo.attention(Q[h * Nq:(h + 1) * Nq], K[h * Nk:(h + 1) * Nk], V[h * Nk:(h + 1) * Nk], block_n=w, scale=scale,
                                 atom_model=HW, out_dtype=rgo.F32)
            assert_bits_equal(got[h * Nq:(h + 1) * Nq], want, f"head {h} w={w}")
        outs[w] = got
    # the key block width is part of the arithmetic: the two classes differ in bits and agree in value
    assert not np.array_equal(outs[64], outs[128]) and np.max(np.abs(outs[64] - outs[128])) < 0.05
    # close to double-precision softmax attention
    f = lambda b: synth.bf16_bits_to_f32(b).astype(np.float64)
    S = f(Q[:Nq]) @ f(K[:Nk]).T * scale
    P = np.exp(S - S.max(1, keepdims=True)); ref = (P / P.sum(1, keepdims=True)) @ f(V[:Nk])
    assert np.max(np.abs(outs[128][:Nq] - ref)) < 2.0 ** -7 * np.max(np.abs(f(V)))


def test_rows_are_independent_of_the_query_tile_and_runs_repeat():
    Nq, Nk, d = 300, 700, 128
    Q, K, V = _draw(Nq, Nk, d, 21)
    full = gpu_attention(Q, K, V, block_n=128, scale=0.09)
    assert_bits_equal(gpu_attention(Q, K, V, block_n=128, scale=0.09), full, "second run")
    for lo, hi in ((0, 1), (100, 229), (128, 300), (299, 300)):
        assert_bits_equal(gpu_attention(Q[lo:hi], K, V, block_n=128, scale=0.09), full[lo:hi], f"queries {lo}:{hi}")
    assert rg.rg_device_status() == 0


def test_strided_operands_and_fp16_output():
    H, Nq, Nk, d = 2, 150, 270, 64
    Q, K, V = _draw(Nq, Nk, d, 41, heads=H)
    scale = 0.125
    pad = lambda a, extra: torch.cat([synth.to_torch(a, DEV), torch.full((a.shape[0], extra), float("nan"), dtype=torch.bfloat16, device=DEV)], 1)
    Qp, Kp = pad(Q, 8), pad(K, 24)                          # leading dimensions 72 and 88: rows still 16-byte aligned
    Vt = np.ascontiguousarray(V.reshape(H, Nk, d).transpose(0, 2, 1)).reshape(H * d, Nk)
    vt = torch.full((H * d, 280), float("nan"), dtype=torch.bfloat16, device=DEV); vt[:, :Nk] = synth.to_torch(Vt, DEV)
    Op = torch.full((H * Nq, d + 8), float("nan"), dtype=torch.float16, device=DEV)
    rg.rg_attention(rg.rg_attn_desc(block_n=64, scale=scale, heads=H), Qp[:, :d], Kp[:, :d], vt[:, :Nk], Op[:, :d])
    torch.cuda.synchronize()
    got = Op[:, :d].cpu().numpy()
    assert torch.isnan(Op[:, d:]).all()                     # nothing written past the output's columns
    for h in range(H):
        want = rgo.attention(Q[h * Nq:(h + 1) * Nq], K[h * Nk:(h + 1) * Nk], V[h * Nk:(h + 1) * Nk], block_n=64, scale=scale,
                             atom_model=HW, out_dtype=rgo.F16)
        assert_bits_equal(got[h * Nq:(h + 1) * Nq], want, f"strided, fp16 out, head {h}")


def test_argument_errors():
    q = torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV); k = torch.zeros((256, 128), dtype=torch.bfloat16, device=DEV)
    vt = torch.zeros((128, 256), dtype=torch.bfloat16, device=DEV); o = torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(rg.RgError):
        rg.rg_attention(rg.rg_attn_desc(block_n=96, scale=1.0), q, k, vt, o)
    with pytest.raises(rg.RgError):
        rg.rg_attention(rg.rg_attn_desc(block_n=64, scale=1.0, mask=2), q, k, vt, o)
    with pytest.raises(rg.RgError):
        rg.rg_attention(rg.rg_attn_desc(block_n=64, scale=1.0, mask=1, block_m=256), q, k, vt, o)
    with pytest.raises(rg.RgError):
        rg.rg_attention(rg.rg_attn_desc(block_n=64, scale=1.0), q, k, vt[:, :200], o)
    with pytest.raises(rg.RgError):
        rg.rg_attention(rg.rg_attn_desc(block_n=64, scale=1.0, heads=3), q, k, vt, o)
