"""GPU parity: descriptor-fixed GEMM through the C ABI against the CPU oracle.

Bars: bit-exact for integer-valued inputs under every atom model; bit-exact on random inputs
under the probe-fitted tcgen05 model; against the paper's exact-sum model (Sec. 3.2.1) the
fp32 result stays within 1e-5*sqrt(K/4096) of sum|a*b| and a bf16 output within one ulp (plus
that fp32 allowance where the sum cancels);
GPU-vs-GPU bitwise identity across M, runs and every tile configuration of a class."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth

from _gpu_util import DEV, HW, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu


def _exact_int(A, B):
    return (synth.bf16_bits_to_f32(A).astype(np.int64) @ synth.bf16_bits_to_f32(B).astype(np.int64).T).astype(np.float32)


def _draws(M, N, K, seed, std_b=1.0):
    A = synth.normal_bf16((M, K), 1.0, seed); B = synth.normal_bf16((N, K), std_b, seed + 1)
    yield "ordinary", A, B
    yield "spread", synth.spread_exponents_bf16(A, seed + 2, -12, 12), synth.spread_exponents_bf16(B, seed + 3, -12, 12)


# ------------------------------------------------------------------ config 1
def test_tiny_descriptor_check_full_oracle_compare():
    """M=64 N=256 K=512, split at 256, pairwise merge, bf16 out: every element."""
    for name, A, B in _draws(64, 256, 512, 0):
        for out in (rgo.BF16, rgo.F32):
            got = gpu_gemm(A, B, cuts=(256,), out_dtype=out)
            want = rgo.gemm(A, B, cuts=(256,), atom_model=HW, out_dtype=out)
            assert_bits_equal(got, want, f"config 1 {name}")


# ------------------------------------------------------------------ exactness
@pytest.mark.parametrize("M,N,K", [(1, 1, 16), (1, 8, 8), (3, 5, 24), (128, 64, 64), (129, 65, 80), (300, 520, 1000),
                                   (7, 4096, 1024), (2000, 3000, 2048), (64, 100, 72)])
@pytest.mark.parametrize("knobs", [dict(), dict(BN=64), dict(BN=128, BK=128), dict(BN=256, stages=2, raster=1),
                                   dict(cta_group=1, BN=256), dict(cta_group=2, BN=256, BK=64), dict(BM=256, BN=128, BK=128, raster=4),
                                   dict(BN=112, BK=128), dict(BN=48, BK=256, cta_group=1), dict(BN=240, cta_group=1), dict(BN=16, cta_group=1),
                                   dict(cta_group=2, BN=32), dict(cta_group=2, BN=48, BK=128), dict(cta_group=2, BN=64, stages=2),
                                   dict(cta_group=2, BN=112, BK=128, raster=1), dict(cta_group=2, BN=240)])
def test_integer_inputs_exact(M, N, K, knobs):
    A = synth.int_valued_bf16((M, K), -8, 8, K + M); B = synth.int_valued_bf16((N, K), -8, 8, K + N + 1)
    assert_bits_equal(gpu_gemm(A, B, out_dtype=rgo.F32, **knobs), _exact_int(A, B), f"ints {M}x{N}x{K} {knobs}")


def test_closed_forms_and_dropped_tails():
    for K in (16, 1000, 4096, 14336):
        ones = synth.f32_to_bf16_bits(np.ones((130, K), np.float32))
        got = gpu_gemm(ones, ones[:70], out_dtype=rgo.F32)
        assert np.all(got == np.float32(K))         # the count of summed k: a lost tail would show
    alpha = np.array([1, 2, -3, 0.5], np.float32); beta = np.array([4, -1, 0.25], np.float32)
    A = synth.f32_to_bf16_bits(np.repeat(alpha[:, None], 2048, 1)); B = synth.f32_to_bf16_bits(np.repeat(beta[:, None], 2048, 1))
    got = gpu_gemm(A, B, cuts=(512, 1024), out_dtype=rgo.F32)
    assert np.array_equal(got, (2048 * np.outer(alpha, beta)).astype(np.float32))


@pytest.mark.parametrize("cuts", [(16,), (32, 48), (64,), (16, 64, 144), tuple(16 * i for i in range(1, 64))])
@pytest.mark.parametrize("tree", [rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED])
def test_integer_split_k_exact(cuts, tree):
    K = max(cuts) + 40
    A = synth.int_valued_bf16((70, K), -8, 8, 1); B = synth.int_valued_bf16((90, K), -8, 8, 2)
    assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, out_dtype=rgo.F32), _exact_int(A, B), f"cuts {cuts[:4]}")
    A = synth.int_valued_bf16((300, K), -8, 8, 3); B = synth.int_valued_bf16((260, K), -8, 8, 4)
    assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, out_dtype=rgo.F32, cta_group=2, BN=128), _exact_int(A, B),
                      f"two-SM tiles, cuts {cuts[:4]}")


# ------------------------------------------------------------------ atom model
@pytest.mark.parametrize("M,N,K,cuts", [(128, 64, 16, ()), (100, 96, 64, ()), (64, 128, 4096, ()), (32, 64, 1000, ()),
                                        (40, 72, 2048, (512, 1024, 1536)), (16, 64, 576, (192, 384))])
def test_random_inputs_bit_exact_under_fitted_atom_model(M, N, K, cuts):
    for name, A, B in _draws(M, N, K, 40 + K):
        want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, out_dtype=rgo.F32)
        for knobs in (dict(), dict(cta_group=2, BN=128), dict(cta_group=2, BN=256)):
            got = gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32, **knobs)
            assert_bits_equal(got, want, f"{M}x{N}x{K} {name} {knobs}")


@pytest.mark.parametrize("K", [512, 4096, 14336])
def test_error_bound_against_exact_sum_model(K):
    """Spec tolerance: |c_gpu - c_exact| <= 1e-5*sqrt(K/4096) * sum_k|a*b| in fp32, and a bf16
    output within one ulp of the exact-model bf16 output."""
    A = synth.normal_bf16((48, K), 1.0, 5); B = synth.normal_bf16((64, K), 0.02, 6)
    got = gpu_gemm(A, B, out_dtype=rgo.F32)
    ref = rgo.gemm(A, B, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)
    denom = np.abs(synth.bf16_bits_to_f32(A)).astype(np.float64) @ np.abs(synth.bf16_bits_to_f32(B)).astype(np.float64).T
    rel = np.abs(got.astype(np.float64) - ref.astype(np.float64)) / denom
    assert rel.max() <= 1e-5 * np.sqrt(K / 4096), rel.max()
    # bf16 output: both sides round once, so they differ by at most one output ulp plus the
    # allowed fp32 error (where the sum cancels, an ulp of the tiny result is far below that error)
    g16 = synth.bf16_bits_to_f32(gpu_gemm(A, B, out_dtype=rgo.BF16)).astype(np.float64)
    r16 = synth.bf16_bits_to_f32(rgo.gemm(A, B, atom_model=rgo.EXACT_RN, out_dtype=rgo.BF16)).astype(np.float64)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(r16), 2.0 ** -126))) - 7)
    assert np.all(np.abs(g16 - r16) <= ulp + 1e-5 * np.sqrt(K / 4096) * denom)
    big = np.abs(ref) > 0.05 * denom                      # no heavy cancellation: plain one-ulp statement
    assert np.all(np.abs(g16 - r16)[big] <= ulp[big])


def test_k576_walk_on_hardware_matches_the_models():
    """Sec. 4's walk: with 16-wide steps, r survives unless the pair straddles a step of r's part."""
    ms = list(range(1, 575))
    A = synth.f32_to_bf16_bits(np.stack([synth.lr_probe_row(576, 0, m, m + 1) for m in ms]))
    B = synth.f32_to_bf16_bits(np.ones((8, 576), np.float32))
    got = gpu_gemm(A, B, cuts=(192, 384), out_dtype=rgo.F32)[:, 0]
    assert_bits_equal(got, rgo.gemm(A, B, cuts=(192, 384), atom_model=HW, out_dtype=rgo.F32)[:, 0], "walk, fitted model")
    assert_bits_equal(got, rgo.gemm(A, B, cuts=(192, 384), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[:, 0], "walk, exact model")
    zeros = [m for m, v in zip(ms, got) if v == 0]
    assert zeros == [m for m in ms if (m % 16 == 15 and m < 192) or m == 383]


def test_position_independence_of_one_k_vector():
    """The same K-vector gives the same bits at any (row, column), tile shape and M (Sec. 3.2.2)."""
    K = 1024
    a = synth.spread_exponents_bf16(synth.normal_bf16((1, K), 1.0, 70), 71, -8, 8)
    b = synth.spread_exponents_bf16(synth.normal_bf16((1, K), 1.0, 72), 73, -8, 8)
    A = np.repeat(a, 300, 0); B = np.repeat(b, 600, 0)
    vals = set()
    for knobs in (dict(BN=64), dict(BN=128), dict(BN=256), dict(BN=256, BK=128), dict(cta_group=2, BN=256), dict(cta_group=2, BN=128),
                  dict(cta_group=1, BN=112, BK=256), dict(cta_group=1, BN=208), dict(cta_group=2, BN=48), dict(cta_group=2, BN=176, BK=128)):
        got = gpu_gemm(A, B, out_dtype=rgo.F32, **knobs)
        vals |= set(np.unique(got.view(np.uint32)).tolist())
    vals |= set(np.unique(gpu_gemm(A[:1], B[:5], out_dtype=rgo.F32).view(np.uint32)).tolist())
    assert len(vals) == 1


# ------------------------------------------------------------------ mutation power (App. E)
def test_oracle_mutations_are_caught():
    A = synth.spread_exponents_bf16(synth.normal_bf16((32, 2048), 1.0, 80), 81, -10, 10)
    B = synth.spread_exponents_bf16(synth.normal_bf16((64, 2048), 1.0, 82), 83, -10, 10)
    cuts = (256, 512, 768, 1024, 1280, 1536, 1792)
    got = gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32)
    assert_bits_equal(got, rgo.gemm(A, B, cuts=cuts, atom_model=HW, out_dtype=rgo.F32), "baseline")
    mutants = {
        "left merge": rgo.gemm(A, B, cuts=cuts, tree=rgo.TREE_LEFT, atom_model=HW, out_dtype=rgo.F32),
        "cut moved one step": rgo.gemm(A, B, cuts=(256, 512, 768, 1024, 1280, 1536, 1808), atom_model=HW, out_dtype=rgo.F32),
        "one cut fewer": rgo.gemm(A, B, cuts=cuts[:-1], atom_model=HW, out_dtype=rgo.F32),
        "backwards k": rgo.gemm(A[:, ::-1], B[:, ::-1], cuts=tuple(2048 - c for c in cuts[::-1]), atom_model=HW, out_dtype=rgo.F32),
        "exact-sum steps": rgo.gemm(A, B, cuts=cuts, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32),
        "8-wide steps": rgo.gemm(A, B, cuts=cuts, atom_model=rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, group=8, window_bits=25,
                                                                               exp_mode=1, final_round=0), out_dtype=rgo.F32),
    }
    for name, m in mutants.items():
        assert (m.view(np.uint32) != got.view(np.uint32)).mean() > 0.01, name


# ------------------------------------------------------------------ config 2: batch invariance
def test_batch_invariance_sweep():
    W = synth.device_normal((4096, 4096), 0.02, 1, torch.bfloat16, DEV)
    X = synth.device_normal((4096, 4096), 1.0, 2, torch.bfloat16, DEV)
    ref = gpu_gemm(X, W, BN=256, BK=64)                       # M = 4096, one descriptor
    for M in (1, 2, 7, 16, 64, 256, 1024, 4096):
        got = gpu_gemm(X[:M], W, BN=256, BK=64)
        assert_bits_equal(got, ref[:M], f"row bits at M={M}")
        got = gpu_gemm(X[:M], W)                               # tile chosen per M, same class
        assert_bits_equal(got, ref[:M], f"row bits at M={M}, tuned tiles")
        got = gpu_gemm(X[:M], W, cta_group=2, BN=256)          # a pair of SMs per 256-row tile, same class
        assert_bits_equal(got, ref[:M], f"row bits at M={M}, two-SM tiles")
    # a permutation of the rows permutes the output rows
    perm = torch.randperm(4096, generator=torch.Generator().manual_seed(0)).to(DEV)
    assert_bits_equal(gpu_gemm(X[perm], W), ref[perm.cpu().numpy()], "row permutation")
    # oracle on sampled elements
    g = np.random.default_rng(0)
    si, sj = g.integers(0, 4096, 400), g.integers(0, 4096, 400)
    want = rgo.gemm_samples(synth.from_torch(X), synth.from_torch(W), si, sj, atom_model=HW, out_dtype=rgo.BF16)
    assert_bits_equal(synth.bf16_bits_to_f32(ref[si, sj]), want, "config 2 sampled oracle")


def test_rows_up_to_64_take_the_narrow_step_and_keep_their_bits():
    """Problems of at most 64 rows run the 64-row tensor-core step, larger ones the 128-row step
    (another accumulator layout, the same products in the same order): a row's bits must not
    depend on which one computed it, for ragged shapes, K tails, cuts, accumulator groups, a
    narrowed partial type and the fused epilogue, and both must match the oracle."""
    N, K = 300, 1000
    W = synth.normal_bf16((N, K), 0.05, 71); X = synth.normal_bf16((200, K), 1.0, 72)
    bias = synth.uniform_bf16((N,), -0.1, 0.1, 73); res = synth.normal_bf16((200, N), 1.0, 74)
    variants = [dict(), dict(cuts=(256, 512)), dict(cuts=(320,), partial_dtype=rg.RG_BF16), dict(inner_span=256),
                dict(BN=48, BK=64), dict(BN=96, BK=256, stages=2)]
    for kw in variants:
        okw = {k: v for k, v in kw.items() if k in ("cuts", "partial_dtype", "inner_span")}
        big = gpu_gemm(X, W, out_dtype=rgo.F32, bias=bias, act=1, residual=res, **kw)          # 128-row step
        want = rgo.gemm(X, W, atom_model=HW, out_dtype=rgo.F32, bias=bias, act=1, residual=res, **okw)
        assert_bits_equal(big, want, f"200 rows {kw}")
        for M in (1, 7, 16, 33, 64):
            got = gpu_gemm(X[:M], W, out_dtype=rgo.F32, bias=bias, act=1, residual=res[:M], **kw)   # 64-row step
            assert_bits_equal(got, big[:M], f"{M} rows against 200 rows {kw}")
        got = gpu_gemm(X[:65], W, out_dtype=rgo.F32, bias=bias, act=1, residual=res[:65], **kw)     # back to 128
        assert_bits_equal(got, big[:65], f"65 rows against 200 rows {kw}")


# ------------------------------------------------------------------ config 3: decode split-K
@pytest.mark.parametrize("M", [1, 8, 32])
def test_decode_split_k_with_residual(M):
    K, N = 14336, 4096
    cuts = tuple(1792 * t for t in range(1, 8))
    W = synth.normal_bf16((N, K), 0.02, 3); X = synth.normal_bf16((32, K), 1.0, 4)[:M]
    res = synth.normal_bf16((32, N), 1.0, 5)[:M]
    got = gpu_gemm(X, W, cuts=cuts, residual=res)
    if M <= 8:
        want = rgo.gemm(X, W, cuts=cuts, atom_model=HW, residual=res, out_dtype=rgo.BF16)
        assert_bits_equal(got, want, f"config 3 M={M} every element")
    else:
        g = np.random.default_rng(1)
        si, sj = g.integers(0, M, 2000), g.integers(0, N, 2000)
        want = rgo.gemm_samples(X, W, si, sj, cuts=cuts, atom_model=HW, residual=res, out_dtype=rgo.BF16)
        assert_bits_equal(synth.bf16_bits_to_f32(got[si, sj]), want, "config 3 M=32 sampled")
    full = gpu_gemm(synth.normal_bf16((32, K), 1.0, 4), W, cuts=cuts, residual=synth.normal_bf16((32, N), 1.0, 5))
    assert_bits_equal(got, full[:M], "rows do not depend on M")
    for knobs in (dict(BN=128, BK=64), dict(BN=64, BK=256), dict(BN=32, BK=128), dict(BN=256, BK=128)):
        assert_bits_equal(gpu_gemm(X, W, cuts=cuts, residual=res, **knobs), got, f"tile knobs {knobs}")


# ------------------------------------------------------------------ config 4: fused epilogue
def test_fused_epilogue_small_every_element():
    A = synth.normal_bf16((70, 256), 1.0, 6); B = synth.normal_bf16((200, 256), 0.1, 7)
    bias = synth.uniform_bf16((200,), -0.1, 0.1, 8); res = synth.normal_bf16((70, 200), 1.0, 9)
    for kw in (dict(bias=bias), dict(act=1), dict(residual=res), dict(bias=bias, act=1), dict(bias=bias, act=1, residual=res)):
        for out in (rgo.BF16, rgo.F32):
            for cuts in ((), (128,)):
                got = gpu_gemm(A, B, cuts=cuts, out_dtype=out, **kw)
                want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, out_dtype=out, **kw)
                assert_bits_equal(got, want, f"epilogue {list(kw)} cuts={cuts}")
    b32 = synth.bf16_bits_to_f32(bias); r32 = synth.normal_f32((70, 200), 1.0, 10)
    got = gpu_gemm(A, B, bias=b32, act=1, residual=r32, out_dtype=rgo.F32)
    assert_bits_equal(got, rgo.gemm(A, B, atom_model=HW, bias=b32, act=1, residual=r32, out_dtype=rgo.F32), "fp32 bias/residual")


def test_silu_wide_range_every_element():
    """Pre-activations from far below the exponential's underflow to far above its overflow, mixed
    within rows: segments whose values all lie within +-87 take the select-free exponential, the
    others the full one, and both must match the specified exponential bit for bit."""
    for scale, seed in ((1.0, 40), (2.0, 41), (40.0, 42)):
        A = synth.normal_bf16((150, 256), scale, seed); B = synth.normal_bf16((330, 256), 1.0, seed + 10)
        bias = synth.uniform_bf16((330,), -0.1, 0.1, seed + 20)
        for kw in (dict(act=1), dict(bias=bias, act=1), dict(act=1, cta_group=2), dict(act=1, cuts=(128,))):
            got = gpu_gemm(A, B, out_dtype=rgo.F32, **kw)
            okw = {k: v for k, v in kw.items() if k != "cta_group"}
            want = rgo.gemm(A, B, atom_model=HW, out_dtype=rgo.F32, **okw)
            assert_bits_equal(got, want, f"silu scale={scale} {list(kw)}")
        if scale == 2.0:                                    # both kinds of 32-column segment occur
            v = np.abs(gpu_gemm(A, B, out_dtype=rgo.F32))[:, :320].reshape(150, 10, 32).max(axis=2)
            assert (v > 87).any() and (v <= 87).any()


def test_fused_epilogue_prefill_full_size_sampled():
    M, N, K = 8192, 14336, 4096
    X = synth.device_normal((M, K), 1.0, 6, torch.bfloat16, DEV)
    W = synth.device_normal((N, K), 0.02, 7, torch.bfloat16, DEV)
    bias = synth.device_uniform((N,), -0.1, 0.1, 8, torch.bfloat16, DEV)
    got = gpu_gemm(X, W, bias=bias, act=1)
    g = np.random.default_rng(2)
    si = np.concatenate([g.integers(0, M, 600), [0, M - 1, M - 1, 0]]); sj = np.concatenate([g.integers(0, N, 600), [0, N - 1, 0, N - 1]])
    want = rgo.gemm_samples(synth.from_torch(X), synth.from_torch(W), si, sj, atom_model=HW, bias=synth.from_torch(bias),
                            act=1, out_dtype=rgo.BF16)
    assert_bits_equal(synth.bf16_bits_to_f32(got[si, sj]), want, "config 4 sampled")
    assert not np.any((got & 0x7fff) > 0x7f80)          # no NaN pattern left: every element was written


# ------------------------------------------------------------------ config 5: one class, many tilings
def test_large_square_all_tile_configs_agree_bitwise():
    n = 8192
    A = synth.device_normal((n, n), 1.0, 11, torch.bfloat16, DEV)
    B = synth.device_normal((n, n), 1.0, 12, torch.bfloat16, DEV)
    configs = [dict(cta_group=1, BN=bn, BK=bk, stages=st, raster=ra) for bn in (64, 128, 256) for bk in (64, 128)
               for st in (0, 2) for ra in (0, 1)]
    configs += [dict(cta_group=2, BN=bn, BK=bk, stages=st, raster=ra) for bn in (128, 256) for bk in (64, 128)
                for st in (0, 2) for ra in (0, 1, 16)]
    configs += [dict(cta_group=1, BN=bn, BK=bk) for bn in (112, 176, 240) for bk in (64, 256)]
    configs += [dict(cta_group=2, BN=bn, BK=bk) for bn in (32, 64, 80, 160, 240) for bk in (64, 128)]
    keys = {rg.rg_desc_class(rg.rg_desc(**c)) for c in configs}
    assert len(keys) == 1
    ref = gpu_gemm(A, B, **configs[0])
    for c in configs[1:]:
        assert_bits_equal(gpu_gemm(A, B, **c), ref, f"tile config {c}")
    assert_bits_equal(gpu_gemm(A, B), ref, "default config, second run")
    g = np.random.default_rng(3)
    si, sj = g.integers(0, n, 500), g.integers(0, n, 500)
    want = rgo.gemm_samples(synth.from_torch(A), synth.from_torch(B), si, sj, atom_model=HW, out_dtype=rgo.BF16)
    assert_bits_equal(synth.bf16_bits_to_f32(ref[si, sj]), want, "config 5 sampled oracle")


# ------------------------------------------------------------------ edges
def test_edges_and_strided_operands():
    d = rg.rg_desc()
    A = torch.zeros((0, 64), dtype=torch.bfloat16, device=DEV); B = torch.zeros((8, 64), dtype=torch.bfloat16, device=DEV)
    rg.rg_gemm(d, A, B, torch.empty((0, 8), dtype=torch.bfloat16, device=DEV))          # M = 0: no-op
    # operands that are views with a leading dimension larger than K; odd N and fp32 / bf16 C views
    base_a = synth.int_valued_bf16((50, 96), -8, 8, 1); base_b = synth.int_valued_bf16((37, 96), -8, 8, 2)
    At = synth.to_torch(base_a, DEV)[:, 8:88]; Bt = synth.to_torch(base_b, DEV)[:, 8:88]
    want = _exact_int(np.ascontiguousarray(base_a[:, 8:88]), np.ascontiguousarray(base_b[:, 8:88]))
    assert_bits_equal(gpu_gemm(At, Bt, out_dtype=rgo.F32), want, "strided operands")
    Cbig = torch.zeros((50, 41), dtype=torch.bfloat16, device=DEV)
    rg.rg_gemm(d, At, Bt, Cbig[:, 2:39])
    torch.cuda.synchronize()
    assert_bits_equal(synth.from_torch(Cbig[:, 2:39].contiguous()), synth.f32_to_bf16_bits(want), "C view, odd offset")
    assert torch.all(Cbig[:, :2] == 0) and torch.all(Cbig[:, 39:] == 0)                 # neighbours untouched
    with pytest.raises(rg.RgError):
        rg.rg_gemm(d, synth.to_torch(base_a, DEV)[:, 1:65], Bt[:, :64], torch.empty((50, 37), dtype=torch.bfloat16, device=DEV))


def test_runs_are_bitwise_repeatable_and_device_healthy():
    A = synth.normal_bf16((512, 2048), 1.0, 90); B = synth.normal_bf16((768, 2048), 1.0, 91)
    ref = gpu_gemm(A, B, cuts=(1024,))
    for _ in range(5):
        assert_bits_equal(gpu_gemm(A, B, cuts=(1024,)), ref, "repeat")
    assert rg.rg_device_status() == 0


def test_host_buffer_form_matches_device_form():
    from paper_2609_11356_b200.api import rg_gemm_host, rg_gemm_host_scratch_bytes
    A = synth.normal_bf16((100, 520), 1.0, 30); B = synth.normal_bf16((260, 520), 1.0, 31)
    bias = synth.uniform_bf16((260,), -0.1, 0.1, 32)
    d = rg.rg_desc(cuts=(256,))
    Ah, Bh, bh = (synth.to_torch(t).pin_memory() for t in (A, B, bias))
    Ch = torch.empty((100, 260), dtype=torch.bfloat16).pin_memory()
    nb = rg_gemm_host_scratch_bytes(d, 100, 260, 520, rg.RG_BF16, bias=bh, act=1)
    scratch = torch.empty(nb, dtype=torch.uint8, device=DEV)
    rg_gemm_host(d, Ah, Bh, Ch, scratch, bias=bh, act=1)
    torch.cuda.synchronize()
    assert_bits_equal(synth.from_torch(Ch), gpu_gemm(A, B, cuts=(256,), bias=bias, act=1), "host-buffer GEMM")


# ------------------------------------------------------------------ parts at bf16 (Sec. 3.2.2)
@pytest.mark.parametrize("pd,md", [(rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16)])
@pytest.mark.parametrize("tree", [rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED])
def test_partial_and_merge_dtypes_bit_exact(pd, md, tree):
    for M, N, K, cuts in ((70, 200, 1024, (256, 512, 768)), (33, 130, 576, (192, 384)), (300, 260, 2048, tuple(256 * t for t in range(1, 8)))):
        for name, A, B in _draws(M, N, K, 60 + K):
            res = synth.normal_bf16((M, N), 1.0, 61)
            for knobs in (dict(), dict(cta_group=2, BN=128), dict(BN=48)):
                got = gpu_gemm(A, B, cuts=cuts, tree=tree, partial_dtype=pd, merge_dtype=md, residual=res, out_dtype=rgo.F32, **knobs)
                want = rgo.gemm(A, B, cuts=cuts, tree=tree, atom_model=HW, partial_dtype=pd, merge_dtype=md, residual=res, out_dtype=rgo.F32)
                assert_bits_equal(got, want, f"{M}x{N}x{K} {name} partial={pd} merge={md} {knobs}")
    # the three combinations are three classes
    keys = {rg.rg_desc_class(rg.rg_desc(cuts=(256,), partial_dtype=p_, merge_dtype=m_)) for p_, m_ in ((1, 1), (0, 1), (0, 0))}
    assert len(keys) == 3


# ------------------------------------------------------------------ fp16 operands
def _f16_draws(M, N, K, seed):
    g = np.random.default_rng(seed)
    A = g.standard_normal((M, K)); B = g.standard_normal((N, K))
    yield "ordinary", A.astype(np.float16), B.astype(np.float16)
    yield "spread", (A * np.exp2(g.integers(-6, 7, A.shape))).astype(np.float16), (B * np.exp2(g.integers(-6, 7, B.shape))).astype(np.float16)


def test_fp16_integer_inputs_exact_and_fp16_output():
    g = np.random.default_rng(1)
    for M, N, K in ((1, 8, 16), (129, 65, 80), (300, 520, 1000), (513, 260, 2048)):
        A = g.integers(-8, 9, (M, K)).astype(np.float16); B = g.integers(-8, 9, (N, K)).astype(np.float16)
        want = (A.astype(np.int64) @ B.astype(np.int64).T).astype(np.float32)
        for knobs in (dict(), dict(cta_group=2, BN=128), dict(BN=48, cta_group=1)):
            assert_bits_equal(gpu_gemm(A, B, out_dtype=rgo.F32, **knobs), want, f"fp16 ints {M}x{N}x{K} {knobs}")
        assert_bits_equal(gpu_gemm(A, B, out_dtype=rgo.F16), rgo.gemm(A, B, atom_model=HW, out_dtype=rgo.F16), "fp16 output")


@pytest.mark.parametrize("M,N,K,cuts", [(100, 96, 64, ()), (64, 128, 4096, ()), (40, 72, 2048, (512, 1024, 1536)), (300, 260, 1024, (256,))])
def test_fp16_random_inputs_bit_exact_under_fitted_atom_model(M, N, K, cuts):
    for name, A, B in _f16_draws(M, N, K, 70 + K):
        want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, out_dtype=rgo.F32)
        for knobs in (dict(), dict(cta_group=2, BN=256), dict(BN=112, cta_group=1)):
            assert_bits_equal(gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32, **knobs), want, f"fp16 {M}x{N}x{K} {name} {knobs}")


def test_fp16_split_partials_epilogue_and_class():
    A, B = next(_f16_draws(70, 200, 1024, 5))[1:]
    cuts = (256, 512, 768)
    bias = np.random.default_rng(2).uniform(-0.1, 0.1, 200).astype(np.float16)
    res = np.random.default_rng(3).standard_normal((70, 200)).astype(np.float16)
    for pd, md in ((rgo.F32, rgo.F32), (rgo.F16, rgo.F32), (rgo.F16, rgo.F16), (rgo.BF16, rgo.BF16)):
        for out in (rgo.F16, rgo.F32):
            got = gpu_gemm(A, B, cuts=cuts, partial_dtype=pd, merge_dtype=md, bias=bias, act=1, residual=res, out_dtype=out)
            want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, partial_dtype=pd, merge_dtype=md, bias=bias, act=1, residual=res, out_dtype=out)
            assert_bits_equal(got, want, f"fp16 split partial={pd} merge={md} out={out}")
    assert rg.rg_desc_class(rg.rg_desc(in_dtype=rg.RG_F16)) != rg.rg_desc_class(rg.rg_desc())
    # operands must be of the descriptor's input type
    with pytest.raises(rg.RgError):
        rg.rg_gemm(rg.rg_desc(), synth.to_torch(A, DEV), synth.to_torch(B, DEV), torch.empty((70, 200), dtype=torch.float16, device=DEV))


# ------------------------------------------------------------------ second level of the cut nest
def test_inner_span_groups_bit_exact():
    """Sec. 3.2.2 / App. E: an accumulator closed every inner_span k, groups chained at fp32."""
    a = np.zeros((1, 192), np.float32); a[0, 0] = 1.0; a[0, 64] = 2.0 ** -24; a[0, 80] = 2.0 ** -24
    ones = synth.f32_to_bf16_bits(np.ones((8, 192), np.float32)); ab = synth.f32_to_bf16_bits(a)
    assert gpu_gemm(ab, ones, out_dtype=rgo.F32)[0, 0] == np.float32(1.0)                       # one chain: both ties lost
    assert gpu_gemm(ab, ones, out_dtype=rgo.F32, inner_span=64)[0, 0] == np.float32(1 + 2.0 ** -23)   # second group sums to 2^-23 first
    for M, N, K, cuts in ((70, 200, 1024, ()), (300, 130, 1000, ()), (33, 260, 2048, (512, 1024, 1536)), (129, 64, 4096, (2048,))):
        for name, A, B in _draws(M, N, K, 90 + K):
            for span in (16, 48, 64, 80, 128, 448):         # 16 = an accumulator per instruction (the two-rounding plan)
                for knobs in (dict(), dict(BN=64), dict(BN=112, stages=2), dict(BN=256), dict(BN=208, raster=1),
                              dict(cta_group=2, BN=256), dict(cta_group=2, BN=128, stages=3)):
                    got = gpu_gemm(A, B, cuts=cuts, inner_span=span, out_dtype=rgo.F32, **knobs)
                    want = rgo.gemm(A, B, cuts=cuts, inner_span=span, atom_model=HW, out_dtype=rgo.F32)
                    assert_bits_equal(got, want, f"{M}x{N}x{K} {name} span={span} {knobs}")
    A = synth.int_valued_bf16((200, 1000), -8, 8, 1); B = synth.int_valued_bf16((300, 1000), -8, 8, 2)
    assert_bits_equal(gpu_gemm(A, B, inner_span=128, out_dtype=rgo.F32), _exact_int(A, B), "ints under a nest")
    bias = synth.uniform_bf16((300,), -0.1, 0.1, 3)
    assert_bits_equal(gpu_gemm(A, B, inner_span=192, bias=bias, act=1), rgo.gemm(A, B, inner_span=192, atom_model=HW, bias=bias, act=1),
                      "nest with fused epilogue")
    # a problem large enough for the default plan to take the two-SM kernel, on sampled outputs
    Ab = synth.normal_bf16((2304, 1024), 1.0, 5); Bb = synth.normal_bf16((2560, 1024), 1.0, 6)
    gsi = np.random.default_rng(7)
    si, sj = gsi.integers(0, 2304, 600), gsi.integers(0, 2560, 600)
    for span in (16, 64, 192):
        got = gpu_gemm(Ab, Bb, inner_span=span, out_dtype=rgo.F32)
        assert_bits_equal(got[si, sj], rgo.gemm_samples(Ab, Bb, si, sj, inner_span=span, atom_model=HW, out_dtype=rgo.F32), f"large, span {span}")
        assert_bits_equal(gpu_gemm(Ab, Bb, inner_span=span, out_dtype=rgo.F32, cta_group=1, BN=128), got, f"large, span {span}: one-CTA kernel agrees")
    k0 = rg.rg_desc_class(rg.rg_desc()); k1 = rg.rg_desc_class(rg.rg_desc(inner_span=64)); k2 = rg.rg_desc_class(rg.rg_desc(inner_span=128))
    assert len({k0, k1, k2}) == 3
    for bad in (dict(inner_span=40), dict(inner_span=8), dict(inner_span=64, BK=128), dict(inner_span=64, cta_group=2, BK=128)):
        assert rg.rg_desc_validate(rg.rg_desc(**bad), 64, 256, 512) == 3
    assert rg.rg_device_status() == 0


# ------------------------------------------------------------------ the planner's choices are speed knobs
@pytest.mark.parametrize("seed", range(48))
def test_library_chosen_tiles_on_random_shapes_equal_a_fixed_tile(seed):
    """Whatever kernel, tile width and stage width the planner picks for a shape (one-CTA tiles of any multiple of
    16 columns, two-SM tiles of any width from 32, 64- to 256-wide K stages), the bits are those of one fixed
    configuration of the same class, and sampled elements are the oracle's."""
    g = np.random.default_rng(7000 + seed)
    M = int(g.choice([g.integers(1, 130), g.integers(129, 600), g.integers(600, 2600)]))
    N = int(g.choice([g.integers(8, 300), g.integers(300, 2100), g.integers(2100, 6200)]))
    K = int(g.choice([64, 80, 256, 520, 1000, 1024, 2048, 4096]))
    A = synth.device_normal((M, K), 1.0, 100 + seed, torch.bfloat16, DEV)
    B = synth.device_normal((N, K), 1.0, 200 + seed, torch.bfloat16, DEV)
    ref = gpu_gemm(A, B, out_dtype=rgo.F32, cta_group=1, BN=128, BK=64)
    assert_bits_equal(gpu_gemm(A, B, out_dtype=rgo.F32), ref, f"library's choice for {M}x{N}x{K}")
    if M > 128:
        bn = int(g.choice(np.arange(32, 257, 16)))
        assert_bits_equal(gpu_gemm(A, B, out_dtype=rgo.F32, cta_group=2, BN=bn, BK=int(g.choice([64, 128]))), ref, f"two-SM tiles of {bn} columns, {M}x{N}x{K}")
    si, sj = g.integers(0, M, 24), g.integers(0, N, 24)
    want = rgo.gemm_samples(synth.from_torch(A), synth.from_torch(B), si, sj, atom_model=HW, out_dtype=rgo.F32)
    assert_bits_equal(ref[si, sj], want, f"sampled oracle {M}x{N}x{K}")
    assert rg.rg_device_status() == 0
