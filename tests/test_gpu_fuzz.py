"""Descriptor-space fuzz (App. E: "a sweep of the plan-parameter space rather than of shapes"): random
descriptors -- cuts, merge tree, part and merge types, inner span, operand type, tile knobs, epilogue --
on small random shapes, every element against the oracle, ordinary and exponent-spread draws."""
import numpy as np
import pytest

import paper_2609_11356_b200 as rg
from oracle import rgo

from _gpu_util import HW, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu


def _case(g):
    M = int(g.choice([1, 7, 33, 64, 65, 128, 129, 200, 300]))      # up to 64 rows: the 64-row tensor-core step
    N = int(g.choice([8, 40, 64, 130, 256, 328]))
    K = int(g.choice([64, 192, 576, 1000, 1024, 2048]))
    f16 = bool(g.integers(0, 2))
    nest = bool(g.integers(0, 3) == 0)
    step = 16
    ncut = int(g.integers(0, 5))
    pts = sorted(set(int(x) * step for x in g.integers(1, max(2, K // step), ncut) if 0 < int(x) * step < K))
    desc = dict(cuts=tuple(pts), tree=int(g.integers(0, 2)))
    pd, md = [(rgo.F32, rgo.F32), (rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16), (rgo.F16, rgo.F32), (rgo.F16, rgo.F16)][int(g.integers(0, 5))]
    desc.update(partial_dtype=pd, merge_dtype=md)
    knobs = {}
    if nest:
        desc["inner_span"] = int(g.choice([16, 48, 64, 128, 320]))
        knobs = [dict(), dict(BN=64), dict(BN=96, stages=2), dict(BN=256), dict(cta_group=2, BN=128), dict(cta_group=2, BN=256)][int(g.integers(0, 6))]
    else:
        knobs = [dict(), dict(BN=64, BK=128), dict(cta_group=2, BN=128), dict(cta_group=2, BN=256, BK=64), dict(BN=48, cta_group=1),
                 dict(BN=208, cta_group=1, raster=1), dict(BN=128, BK=256, cta_group=1, stages=1), dict(cta_group=2, BN=80),
                 dict(cta_group=2, BN=192, BK=128)][int(g.integers(0, 9))]
    epi = {}
    out = [rgo.BF16, rgo.F32, rgo.F16][int(g.integers(0, 3))]
    knobs = dict(knobs, b_static=int(g.integers(0, 3)))       # a promise about in-flight work: never moves a bit (with cuts and few rows it also changes the grid)
    return M, N, K, f16, desc, knobs, out


@pytest.mark.parametrize("seed", range(150))
def test_random_descriptor_matches_oracle(seed):
    g = np.random.default_rng(1000 + seed)
    M, N, K, f16, desc, knobs, out = _case(g)
    spread = 6 if f16 else 10
    A = g.standard_normal((M, K)); B = g.standard_normal((N, K))
    if seed % 2:
        A = A * np.exp2(g.integers(-spread, spread + 1, A.shape)); B = B * np.exp2(g.integers(-spread, spread + 1, B.shape))
    if f16:
        A, B = A.astype(np.float16), B.astype(np.float16)
        conv = lambda x: np.asarray(x, np.float32).astype(np.float16)
    else:
        from paper_2609_11356_b200 import synth
        A, B = synth.f32_to_bf16_bits(A.astype(np.float32)), synth.f32_to_bf16_bits(B.astype(np.float32))
        conv = lambda x: synth.f32_to_bf16_bits(np.asarray(x, np.float32))
    epi = {}
    if g.integers(0, 2): epi["bias"] = conv(g.uniform(-0.5, 0.5, N))
    if g.integers(0, 2): epi["act"] = 1
    if g.integers(0, 2): epi["residual"] = g.standard_normal((M, N)).astype(np.float32)
    got = gpu_gemm(A, B, out_dtype=out, **desc, **knobs, **epi)
    want = rgo.gemm(A, B, atom_model=HW, out_dtype=out, **desc, **epi)
    assert_bits_equal(got, want, f"seed {seed}: {M}x{N}x{K} f16={f16} {desc} {knobs} {list(epi)} out={out}")
    assert rg.rg_device_status() == 0


@pytest.mark.parametrize("seed", range(100))
def test_random_reduction_matches_oracle(seed):
    """Row reductions over random widths, types, alignments and launch shapes, bit for bit."""
    import torch
    from _gpu_util import DEV, gpu_reduce
    from paper_2609_11356_b200 import synth
    g = np.random.default_rng(5000 + seed)
    op = int(g.integers(0, 3))
    bf = bool(g.integers(0, 2))
    R = int(g.choice([1, 3, 37, 150, 400]))
    Cc = int(g.choice([1, 5, 31, 128, 1000, 4096, 4100, 8192, 20000, 33001, 70000])) if R <= 37 else int(g.choice([7, 256, 1000, 4096, 9000]))
    pad_l, pad_r = (int(g.integers(0, 9)), int(g.integers(0, 9))) if g.integers(0, 2) else (0, 0)
    scale = float(g.choice([1.0, 100.0]))
    full = synth.normal_f32((R, Cc + pad_l + pad_r), scale, 5000 + seed)
    if seed % 3 == 0:
        full = synth.spread_exponents_f32(full, seed, -8, 8)
    if bf:
        full = synth.f32_to_bf16_bits(full)
    x = np.ascontiguousarray(full[:, pad_l:pad_l + Cc])
    xt = synth.to_torch(full, DEV)[:, pad_l:pad_l + Cc]
    knobs = {}
    if g.integers(0, 2):
        knobs = dict(BN=int(g.choice([32, 64, 128, 256, 512, 1024])), stages=int(g.choice([1, 2, 4, 8])))
    kw = {}
    if op == rg.RG_OP_RMSNORM:
        kw = dict(eps=1e-5, fma=int(g.integers(0, 2)))
        if g.integers(0, 2):
            w = synth.normal_f32((Cc,), 0.05, seed, mean=1.0)
            kw["weight"] = synth.f32_to_bf16_bits(w) if (bf and g.integers(0, 2)) else w
    fma = kw.pop("fma", 0)
    got, gaux = gpu_reduce(op, xt, **kw, fma=fma, **knobs)
    want, waux = rgo.reduce_rows(op, x, fma=fma, **kw)
    assert_bits_equal(got, want, f"seed {seed}: op={op} bf16={bf} {R}x{Cc} pad=({pad_l},{pad_r}) {knobs}")
    if waux is not None:
        assert_bits_equal(gaux, waux, f"seed {seed}: aux")


@pytest.mark.parametrize("seed", range(60))
def test_random_fp8_descriptor_matches_oracle(seed):
    """The same sweep on e4m3 operands (32-wide step): cuts, trees, part types, spans, knobs, epilogue."""
    from _gpu_util import HW8
    from paper_2609_11356_b200 import synth
    g = np.random.default_rng(9000 + seed)
    M = int(g.choice([1, 7, 33, 64, 65, 129, 200, 300])); N = int(g.choice([8, 40, 130, 256, 328]))
    K = int(g.choice([64, 190, 576, 1000, 1024, 2048]))
    nest = bool(g.integers(0, 3) == 0)
    step = 32
    pts = sorted(set(int(x) * step for x in g.integers(1, max(2, K // step), int(g.integers(0, 5))) if 0 < int(x) * step < K))
    desc = dict(cuts=tuple(pts), tree=int(g.integers(0, 2)))
    pd, md = [(rgo.F32, rgo.F32), (rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16), (rgo.F16, rgo.F16)][int(g.integers(0, 4))]
    desc.update(partial_dtype=pd, merge_dtype=md)
    if nest:
        desc["inner_span"] = int(g.choice([32, 96, 128, 256, 640]))
        knobs = [dict(), dict(BN=64), dict(BN=96, stages=2), dict(BN=256), dict(cta_group=2, BN=128), dict(cta_group=2, BN=256)][int(g.integers(0, 6))]
    else:
        knobs = [dict(), dict(BN=64, BK=128), dict(cta_group=2, BN=128), dict(cta_group=2, BN=256, BK=64), dict(BN=48, cta_group=1),
                 dict(BN=208, cta_group=1, raster=1)][int(g.integers(0, 6))]
    out = [rgo.BF16, rgo.F32, rgo.F16][int(g.integers(0, 3))]
    A = g.standard_normal((M, K)); B = g.standard_normal((N, K))
    if seed % 2:
        A = A * np.exp2(g.integers(-7, 8, A.shape)); B = B * np.exp2(g.integers(-7, 8, B.shape))
    A = synth.f32_to_f8e4m3_bits(np.clip(A, -448, 448).astype(np.float32)); B = synth.f32_to_f8e4m3_bits(np.clip(B, -448, 448).astype(np.float32))
    epi = {}
    if g.integers(0, 2): epi["bias"] = synth.f32_to_bf16_bits(g.uniform(-0.5, 0.5, N).astype(np.float32))
    if g.integers(0, 2): epi["act"] = 1
    if g.integers(0, 2): epi["residual"] = g.standard_normal((M, N)).astype(np.float32)
    got = gpu_gemm(A, B, out_dtype=out, **desc, **knobs, **epi)
    want = rgo.gemm(A, B, atom_model=HW8, out_dtype=out, **desc, **epi)
    assert_bits_equal(got, want, f"seed {seed}: fp8 {M}x{N}x{K} {desc} {knobs} {list(epi)} out={out}")
    assert rg.rg_device_status() == 0


@pytest.mark.parametrize("seed", range(60))
def test_random_gemv_and_column_reduction_match_oracle(seed):
    """GEMV family (layouts, folds, fma, both operand types, ragged K) and column reductions (sum, dot,
    fma, both leaf types, unaligned views), bit for bit."""
    import torch
    from _gpu_util import DEV
    from paper_2609_11356_b200 import synth
    g = np.random.default_rng(12000 + seed)
    # ---- GEMV
    M = int(g.choice([1, 2, 3, 4, 5, 9])); N = int(g.choice([1, 7, 64, 300])); K = int(g.choice([8, 24, 250, 256, 1000, 4099, 8192]))
    f16 = bool(g.integers(0, 2)); fma = int(g.integers(0, 2)); layout = int(g.integers(0, 2)); fold = int(g.integers(0, 2))
    A = g.standard_normal((M, K)) * np.exp2(g.integers(-6, 7, (M, K))); B = g.standard_normal((N, K)) * np.exp2(g.integers(-6, 7, (N, K)))
    if f16:
        A, B = A.astype(np.float16), B.astype(np.float16)
    else:
        A, B = synth.f32_to_bf16_bits(A.astype(np.float32)), synth.f32_to_bf16_bits(B.astype(np.float32))
    Kp = (K + 7) // 8 * 8                                      # rows start on 16-byte boundaries
    def padded(a):
        t = torch.zeros((a.shape[0], Kp), dtype=torch.float16 if f16 else torch.bfloat16, device=DEV)
        t[:, :K] = synth.to_torch(a, DEV)
        return t[:, :K]
    out = [rgo.BF16, rgo.F32][int(g.integers(0, 2))]
    got = gpu_gemm(padded(A), padded(B), out_dtype=out, atom=rg.RG_ATOM_SCALAR, fma=fma, gemv_layout=layout, gemv_fold=fold)
    want = rgo.gemv(A, B, fma=fma, layout=layout, fold=fold, out_dtype=out)
    assert_bits_equal(got, want, f"seed {seed}: gemv {M}x{N}x{K} f16={f16} fma={fma} layout={layout} fold={fold}")
    # ---- column reduction
    R = int(g.choice([1, 5, 33, 256, 257, 700, 3000])); Cc = int(g.choice([1, 3, 100, 128, 131, 520]))
    op = int(g.integers(0, 2)); cfma = int(g.integers(0, 2)); bf = bool(g.integers(0, 2))
    off = int(g.integers(0, 4)) if g.integers(0, 2) else 0
    x = synth.normal_f32((R, Cc + off + 3), 100.0, 12000 + seed); y = synth.normal_f32((R, Cc + off + 3), 1.0, 13000 + seed)
    if bf:
        x, y = synth.f32_to_bf16_bits(x), synth.f32_to_bf16_bits(y)
    xt, yt = synth.to_torch(x, DEV)[:, off:off + Cc], synth.to_torch(y, DEV)[:, off:off + Cc]
    o = torch.full((Cc,), float("nan"), dtype=torch.float32, device=DEV)
    nb = rg.rg_reduce_cols_workspace_bytes(R, Cc)
    ws = torch.full((max(nb, 16),), 0xFF, dtype=torch.uint8, device=DEV)
    rg.rg_reduce_cols(rg.rg_desc(fma=cfma), op, xt, o, y=yt if op else None, ws=ws if nb else None)
    torch.cuda.synchronize()
    want = rgo.reduce_cols(op, x[:, off:off + Cc], y[:, off:off + Cc] if op else None, fma=cfma)
    assert_bits_equal(o.cpu().numpy(), want, f"seed {seed}: cols op={op} {R}x{Cc} bf16={bf} fma={cfma} off={off}")
    assert rg.rg_device_status() == 0


@pytest.mark.parametrize("seed", range(24))
def test_random_attention_matches_oracle(seed):
    """Attention descriptors (block width, base, head size, heads) on random ragged shapes, bit for bit."""
    from test_gpu_attention import gpu_attention
    from paper_2609_11356_b200 import synth
    g = np.random.default_rng(20000 + seed)
    H = int(g.choice([1, 2, 3])); Nq = int(g.choice([1, 17, 128, 130, 300])); Nk = int(g.choice([1, 40, 64, 129, 500, 1100]))
    d = int(g.choice([64, 128])); w = int(g.choice([64, 128])); base = int(g.choice([0, 2]))
    spread = int(g.choice([0, 2]))
    causal = bool(g.integers(0, 2))
    if causal:
        Nk = Nq
    mk = lambda n: synth.f32_to_bf16_bits((g.standard_normal((H * n, d)) * np.exp2(g.integers(-spread, spread + 1, (H * n, d)))).astype(np.float32))
    Q, K, V = mk(Nq), mk(Nk), mk(Nk)
    scale = float(np.float32(d ** -0.5 * (np.log2(np.e) if base == 2 else 1.0)))
    out = [rgo.F32, rgo.BF16][int(g.integers(0, 2))]
    got = gpu_attention(Q, K, V, block_n=w, scale=scale, heads=H, out_dtype=out, exp_base=base, causal=causal)
    for h in range(H):
        want = rgo.attention(Q[h * Nq:(h + 1) * Nq], K[h * Nk:(h + 1) * Nk], V[h * Nk:(h + 1) * Nk], block_n=w, scale=scale,
                             atom_model=HW, out_dtype=out, exp_base=base, causal=causal)
        assert_bits_equal(got[h * Nq:(h + 1) * Nq], want, f"seed {seed}: attention causal={causal} H={H} {Nq}x{Nk} d={d} w={w} base={base} head {h}")
    assert rg.rg_device_status() == 0
