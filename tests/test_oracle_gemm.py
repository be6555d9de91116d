"""Pins for the GEMM oracle (Sec. 3.2): the printed K = 576 walk, exact integer products under
every atom model, closed forms, an independent exact-rational atom, mutation power checks."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import rgo
from paper_2609_11356_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
Lf, rf = np.float32(1024.0), np.float32(2.0 ** -15)

MODELS = {
    "exact_rn": rgo.EXACT_RN,
    "seq_fma": rgo.SEQ_FMA,
    "seq_nofma": rgo.SEQ_NOFMA,
    "align_rz_24": rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=24, final_round=0),
    "align_rn_30_g8": rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=30, group=8, final_round=1),
    "align_floor_26_eop": rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=26, exp_mode=1,
                                        addend_round=1, final_round=0),
    "align_noacc": rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=25, acc_in_window=0, final_round=1),
}


def _bf(x):
    return synth.f32_to_bf16_bits(np.asarray(x, np.float32))


def _gold(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        rows.append((int(k), rf if v == "r" else np.float32(0.0)))
    return rows


def test_printed_k576_walk_sequential_parts():
    """Sec. 4: three parts of 192, merged left to right; every m of the walk in one GEMM."""
    gold = _gold("splitk_walk_k576.txt")
    A = np.zeros((len(gold), 576), np.float32)
    for row, (m, _) in enumerate(gold):
        A[row] = synth.lr_probe_row(576, 0, m, m + 1)
    B = np.ones((1, 576), np.float32)
    for tree in (rgo.TREE_LEFT, rgo.TREE_BALANCED):  # identical shapes for three parts
        Cm = rgo.gemm(_bf(A), _bf(B), cuts=(192, 384), tree=tree, atom_model=rgo.SEQ_FMA, out_dtype=rgo.F32)
        want = np.array([w for _, w in gold], np.float32)
        assert np.array_equal(Cm[:, 0], want)


def test_k576_walk_under_exact_atoms_differs_as_predicted():
    """With exact 16-wide atoms a pair inside one atom cancels before the accumulator sees it,
    so r survives unless the pair straddles an atom boundary of r's own part."""
    ms = list(range(1, 575))
    A = np.stack([synth.lr_probe_row(576, 0, m, m + 1) for m in ms])
    Cm = rgo.gemm(_bf(A), _bf(np.ones((1, 576), np.float32)), cuts=(192, 384), atom_model=rgo.EXACT_RN,
                  out_dtype=rgo.F32)[:, 0]
    for m, got in zip(ms, Cm):
        straddle_atom = (m % 16 == 15)
        zero = (straddle_atom and m < 192) or m == 383
        assert got == (np.float32(0) if zero else rf), m


def test_printed_contiguous_grouping_as_split():
    rows = []
    for line in open(os.path.join(GOLD, "contiguous_grouping_8.txt")):
        if not line.startswith("#") and line.strip():
            p, v = line.split()
            rows.append((int(p), rf if v == "r" else np.float32(0)))
    A = np.stack([synth.lr_probe_row(8, 0, p, p + 1) for p, _ in rows])
    Cm = rgo.gemm(_bf(A), _bf(np.ones((1, 8), np.float32)), cuts=(4,), atom_model=rgo.SEQ_NOFMA, out_dtype=rgo.F32)
    assert np.array_equal(Cm[:, 0], np.array([w for _, w in rows], np.float32))


@pytest.mark.parametrize("name", list(MODELS))
@pytest.mark.parametrize("K,cuts", [(512, (256,)), (1000, ()), (14336, tuple(1792 * t for t in range(1, 8))),
                                    (72, (16, 48))])
def test_integer_inputs_give_exact_products(name, K, cuts):
    """|a|,|b| <= 8: every partial sum is an integer below 2^24, so any order and any atom
    model with a window of at least 21 bits returns the exact dot product."""
    M, N = 5, 7
    A = synth.int_valued_bf16((M, K), -8, 8, seed=K)
    B = synth.int_valued_bf16((N, K), -8, 8, seed=K + 1)
    want = synth.bf16_bits_to_f32(A).astype(np.int64) @ synth.bf16_bits_to_f32(B).astype(np.int64).T
    for tree in (rgo.TREE_LEFT, rgo.TREE_BALANCED):
        got = rgo.gemm(A, B, cuts=cuts, tree=tree, atom_model=MODELS[name], out_dtype=rgo.F32)
        assert np.array_equal(got.astype(np.int64), want) and np.all(got == want.astype(np.float32))


@pytest.mark.parametrize("name", list(MODELS))
def test_closed_forms(name):
    K = 4096
    ones = _bf(np.ones((3, K), np.float32))
    got = rgo.gemm(ones, ones, atom_model=MODELS[name], out_dtype=rgo.F32)
    assert np.all(got == np.float32(K))          # all-ones: the count of summed k (App. D)
    alpha = np.array([1, 2, -3, 0.5], np.float32)
    beta = np.array([4, -1, 0.25], np.float32)
    A = _bf(np.repeat(alpha[:, None], K, 1)); B = _bf(np.repeat(beta[:, None], K, 1))
    got = rgo.gemm(A, B, cuts=(1024, 2048), atom_model=MODELS[name], out_dtype=rgo.F32)
    assert np.array_equal(got, (K * np.outer(alpha, beta)).astype(np.float32))
    # a dropped tail would show: K not a multiple of the atom
    got = rgo.gemm(ones[:, :1000], ones[:, :1000], atom_model=MODELS[name], out_dtype=rgo.F32)
    assert np.all(got == np.float32(1000))


# ---- EXACT_RN against exact rational arithmetic (Python integers), an independent route
def _frac_bf16(h):
    s = -1 if h >> 15 else 1
    e, m = (h >> 7) & 0xff, h & 0x7f
    return s * (Fraction(m, 128) * Fraction(2) ** -126 if e == 0 else (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127))


def _rn_f32(q: Fraction) -> np.float32:
    if q == 0:
        return np.float32(0.0)
    s, a = (-1 if q < 0 else 1), abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    lsb = max(e - 23, -149)
    scaled = a / Fraction(2) ** lsb
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n & 1):
        n += 1
    return np.float32(s * float(n) * 2.0 ** lsb) if n * 2.0 ** lsb < 2.0 ** 128 else np.float32(s * np.inf)


@pytest.mark.parametrize("spread", [2, 12, 40, 110])
def test_exact_atom_against_rationals(spread):
    g = np.random.default_rng(spread)
    for trial in range(300):
        n = int(g.integers(1, 17))
        a = synth.f32_to_bf16_bits((g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n))).astype(np.float32))
        b = synth.f32_to_bf16_bits((g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n))).astype(np.float32))
        acc = np.float32(g.standard_normal() * 2.0 ** int(g.integers(-spread, spread + 1)))
        exact = Fraction(float(acc)) + sum(_frac_bf16(int(x)) * _frac_bf16(int(y)) for x, y in zip(a, b))
        assert rgo.atom(rgo.EXACT_RN, acc, a, b) == _rn_f32(exact)
        if n == 1:  # a one-product atom is a fused multiply-add
            assert rgo.atom(rgo.EXACT_RN, acc, a, b) == rgo.atom(rgo.SEQ_FMA, acc, a, b)


def test_exact_atom_ties_and_cancellation():
    one = _bf([1.0])[0]
    # {1, 2^-24}: exact tie, RN-even keeps 1;  {1+2^-23 (acc), 2^-24} rounds up to even
    assert rgo.atom(rgo.EXACT_RN, 0.0, [one, _bf([2.0 ** -24])[0]], [one, one]) == np.float32(1.0)
    assert rgo.atom(rgo.EXACT_RN, np.float32(1 + 2.0 ** -23), [_bf([2.0 ** -24])[0]], [one]) == np.float32(1 + 2.0 ** -22)
    # {1, 2^-24, 2^-25}: above the tie, rounds up; a sequential chain would lose both
    a = _bf([1.0, 2.0 ** -24, 2.0 ** -25])
    assert rgo.atom(rgo.EXACT_RN, 0.0, a, [one] * 3) == np.float32(1 + 2.0 ** -23)
    assert rgo.atom(rgo.SEQ_FMA, 0.0, a, [one] * 3) == np.float32(1.0)
    # +L, -L, r inside one exact atom: r survives; sequentially it is absorbed
    a = _bf([2.0 ** -15, 1024.0, -1024.0])
    assert rgo.atom(rgo.EXACT_RN, 0.0, a, [one] * 3) == rf
    assert rgo.atom(rgo.SEQ_FMA, 0.0, a, [one] * 3) == np.float32(0.0)


def test_bf16_products_exact_so_fma_flag_is_inert():
    g = np.random.default_rng(5)
    A = synth.normal_bf16((4, 256), 1.0, 11); B = synth.normal_bf16((6, 256), 1.0, 12)
    c1 = rgo.gemm(A, B, atom_model=rgo.SEQ_FMA, out_dtype=rgo.F32)
    c2 = rgo.gemm(A, B, atom_model=rgo.SEQ_NOFMA, out_dtype=rgo.F32)
    assert np.array_equal(c1, c2)


def test_align_trunc_wide_window_equals_exact_on_narrow_spread():
    wide = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=90, final_round=1)
    A = synth.normal_bf16((8, 512), 1.0, 21); B = synth.normal_bf16((8, 512), 1.0, 22)
    assert np.array_equal(rgo.gemm(A, B, atom_model=wide, out_dtype=rgo.F32),
                          rgo.gemm(A, B, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32))


def test_align_trunc_window_drops_small_addends():
    one = _bf([1.0])[0]
    m = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=24, final_round=0)
    a = _bf([1.0, 2.0 ** -25, -1.0])
    assert rgo.atom(m, 0.0, a, [one] * 3) == np.float32(0.0)           # 2^-25 is below the window
    a = _bf([1.0, 2.0 ** -20, -1.0])
    assert rgo.atom(m, 0.0, a, [one] * 3) == np.float32(2.0 ** -20)    # inside it
    # floor vs truncate on a negative addend below the window
    mf = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=24, addend_round=1, final_round=0)
    a = _bf([1.0, -2.0 ** -30])
    assert rgo.atom(m, 0.0, a, [one] * 2) == np.float32(1.0)
    assert rgo.atom(mf, 0.0, a, [one] * 2) == np.float32(1.0 - 2.0 ** -24)


# ---- mutation power: descriptors that differ must be told apart (App. E)
def _parts_gemm(vals, cuts, tree):
    """one row, one column; part s holds vals[s] at its first k"""
    K = 16 * len(vals) if not cuts else None
    bounds = [0] + list(cuts)
    Kt = bounds[-1] + 16
    a = np.zeros((1, Kt), np.float32)
    for s, v in enumerate(vals):
        a[0, bounds[s]] = v
    return rgo.gemm(_bf(a), _bf(np.ones((1, Kt), np.float32)), cuts=cuts, tree=tree,
                    atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[0, 0]


def test_merge_tree_left_vs_balanced_and_reversed():
    cuts = tuple(16 * t for t in range(1, 8))
    vals = [0, Lf, -Lf, rf, 0, 0, 0, 0]              # L in p1, -L in p2, r in p3
    assert _parts_gemm(vals, cuts, rgo.TREE_LEFT) == rf
    assert _parts_gemm(vals, cuts, rgo.TREE_BALANCED) == np.float32(0.0)
    vals = [rf, 0, 0, 0, 0, 0, Lf, -Lf]              # forwards: r + (L-L) = r ; reversed merge absorbs r
    assert _parts_gemm(vals, cuts, rgo.TREE_LEFT) == np.float32(0.0)   # ((r+..)+L)-L
    assert _parts_gemm(vals, cuts, rgo.TREE_BALANCED) == rf
    assert _parts_gemm(vals[::-1], cuts, rgo.TREE_LEFT) == rf          # backwards partials differ


def test_cut_moved_by_one_atom_is_detected():
    a = np.zeros((1, 64), np.float32)
    a[0, 0], a[0, 16], a[0, 32] = rf, Lf, -Lf
    ones = _bf(np.ones((1, 64), np.float32))
    at32 = rgo.gemm(_bf(a), ones, cuts=(32,), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[0, 0]
    at16 = rgo.gemm(_bf(a), ones, cuts=(16,), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[0, 0]
    assert at32 == np.float32(0.0) and at16 == rf


def test_partials_and_merge_consistent():
    A = synth.normal_bf16((4, 512), 1.0, 0); B = synth.normal_bf16((5, 512), 1.0, 1)
    P = rgo.gemm_partials(A, B, cuts=(256,), atom_model=rgo.EXACT_RN)
    full = rgo.gemm(A, B, cuts=(256,), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)
    assert np.array_equal(full, P[0] + P[1])
    # each partial is the unsplit GEMM of its own K range
    assert np.array_equal(P[1], rgo.gemm(A[:, 256:], B[:, 256:], atom_model=rgo.EXACT_RN, out_dtype=rgo.F32))


def test_row_permutation_and_m_invariance():
    A = synth.normal_bf16((16, 256), 1.0, 2); B = synth.normal_bf16((8, 256), 0.02, 3)
    full = rgo.gemm(A, B, cuts=(128,), out_dtype=rgo.BF16)
    perm = np.random.default_rng(0).permutation(16)
    assert np.array_equal(rgo.gemm(A[perm], B, cuts=(128,), out_dtype=rgo.BF16), full[perm])
    assert np.array_equal(rgo.gemm(A[:3], B, cuts=(128,), out_dtype=rgo.BF16), full[:3])


def test_epilogue_indexing_and_order():
    M, N, K = 6, 5, 64
    A = synth.int_valued_bf16((M, K), -4, 4, 1); B = synth.int_valued_bf16((N, K), -4, 4, 2)
    bias = _bf(np.arange(N, dtype=np.float32) * 3 - 5)                 # distinct per column
    res = _bf((np.arange(M * N, dtype=np.float32).reshape(M, N) % 17) * 2 - 9)   # distinct per (i, j)
    dot = synth.bf16_bits_to_f32(A).astype(np.int64) @ synth.bf16_bits_to_f32(B).astype(np.int64).T
    want = dot + synth.bf16_bits_to_f32(bias).astype(np.int64)[None, :] + synth.bf16_bits_to_f32(res).astype(np.int64)
    got = rgo.gemm(A, B, bias=bias, residual=res, out_dtype=rgo.F32)
    assert np.array_equal(got, want.astype(np.float32))
    # fp32 bias / residual take the same path
    got = rgo.gemm(A, B, bias=synth.bf16_bits_to_f32(bias), residual=synth.bf16_bits_to_f32(res), out_dtype=rgo.F32)
    assert np.array_equal(got, want.astype(np.float32))
    # order bias -> SiLU -> residual, one rounding at the end: zero product isolates the epilogue
    Z = np.zeros((M, K), np.uint16)
    got = rgo.gemm(Z, B, bias=bias, act=1, residual=res, out_dtype=rgo.F32)
    b64 = synth.bf16_bits_to_f32(bias).astype(np.float64)[None, :]
    r64 = synth.bf16_bits_to_f32(res).astype(np.float64)
    want64 = b64 / (1 + np.exp(-b64)) + r64
    assert np.allclose(got, want64, rtol=3e-7, atol=1e-6)
    wrong = (b64 + r64) / (1 + np.exp(-(b64 + r64)))
    assert not np.allclose(got, wrong, rtol=1e-3, atol=1e-3)
    # bf16 output: exactly one rounding of the fp32 value
    got16 = rgo.gemm(Z, B, bias=bias, act=1, residual=res, out_dtype=rgo.BF16)
    assert np.array_equal(got16, synth.f32_to_bf16_bits(got))


# ---- parts written at bf16, sum kept at fp32 or bf16 (Sec. 3.2.2: partial_dtype / merge_dtype)
def test_partial_and_merge_dtypes():
    A = synth.normal_bf16((6, 512), 1.0, 50); B = synth.normal_bf16((7, 512), 1.0, 51)
    cuts = (128, 256, 384)
    P32 = rgo.gemm_partials(A, B, cuts=cuts, atom_model=rgo.EXACT_RN)
    P16 = rgo.gemm_partials(A, B, cuts=cuts, atom_model=rgo.EXACT_RN, partial_dtype=rgo.BF16)
    # a bf16 part is the fp32 part rounded once (library conversion as the independent route)
    import torch
    want = torch.from_numpy(P32).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(P16, want)
    # parts at bf16, sum at fp32: the fp32 tree over the rounded parts
    c_16_32 = rgo.gemm(A, B, cuts=cuts, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32, partial_dtype=rgo.BF16)
    assert np.array_equal(c_16_32, (P16[0] + P16[1]) + (P16[2] + P16[3]))
    # both at bf16: every add rounded to bf16, checked with torch's bf16 adds (correctly rounded)
    t = torch.from_numpy(P16).to(torch.bfloat16)
    want = ((t[0] + t[1]) + (t[2] + t[3])).to(torch.float32).numpy()
    c_16_16 = rgo.gemm(A, B, cuts=cuts, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32, partial_dtype=rgo.BF16, merge_dtype=rgo.BF16)
    assert np.array_equal(c_16_16, want)
    want_left = (((t[0] + t[1]) + t[2]) + t[3]).to(torch.float32).numpy()
    c_left = rgo.gemm(A, B, cuts=cuts, tree=rgo.TREE_LEFT, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32,
                      partial_dtype=rgo.BF16, merge_dtype=rgo.BF16)
    assert np.array_equal(c_left, want_left)
    # the three recorded combinations are three different classes of bits on ordinary inputs
    c_32_32 = rgo.gemm(A, B, cuts=cuts, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)
    assert not np.array_equal(c_32_32, c_16_32) and not np.array_equal(c_16_32, c_16_16)
    # small integers are exact at every type, so all combinations agree with the integer product
    Ai = synth.int_valued_bf16((5, 64), -2, 2, 1); Bi = synth.int_valued_bf16((4, 64), -2, 2, 2)
    exact = (synth.bf16_bits_to_f32(Ai).astype(np.int64) @ synth.bf16_bits_to_f32(Bi).astype(np.int64).T).astype(np.float32)
    for pd, md in ((rgo.F32, rgo.F32), (rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16)):
        got = rgo.gemm(Ai, Bi, cuts=(16, 32, 48), out_dtype=rgo.F32, partial_dtype=pd, merge_dtype=md)
        assert np.array_equal(got, exact)


# ---- fp16 operands (the paper's headline input type): same pins, another operand decode
def _f16(x):
    return np.asarray(x, np.float32).astype(np.float16)


def test_fp16_integer_products_and_closed_forms():
    g = np.random.default_rng(0)
    for K, cuts in ((512, (256,)), (1000, ()), (72, (16, 48))):
        A = _f16(g.integers(-8, 9, (5, K))); B = _f16(g.integers(-8, 9, (7, K)))
        want = (A.astype(np.int64) @ B.astype(np.int64).T).astype(np.float32)
        for name, m in MODELS.items():
            got = rgo.gemm(A, B, cuts=cuts, atom_model=m, out_dtype=rgo.F32)
            assert np.array_equal(got, want), (name, K)
    ones = _f16(np.ones((3, 4096)))
    assert np.all(rgo.gemm(ones, ones, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32) == np.float32(4096))
    # fp16 output: one rounding to binary16 (2049 is not representable: ties to even 2048)
    assert np.all(rgo.gemm(_f16(np.ones((2, 2049))), _f16(np.ones((2, 2049))), out_dtype=rgo.F16) == np.float16(2048))


@pytest.mark.parametrize("spread", [2, 8, 14])
def test_fp16_exact_atom_against_rationals(spread):
    g = np.random.default_rng(100 + spread)
    for trial in range(300):
        n = int(g.integers(1, 17))
        a = _f16(g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n)))
        b = _f16(g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n)))
        acc = np.float32(g.standard_normal() * 2.0 ** int(g.integers(-spread, spread + 1)))
        exact = Fraction(float(acc)) + sum(Fraction(float(x)) * Fraction(float(y)) for x, y in zip(a, b))
        assert rgo.atom(rgo.EXACT_RN, acc, a, b) == _rn_f32(exact)
        if n == 1:
            assert rgo.atom(rgo.EXACT_RN, acc, a, b) == rgo.atom(rgo.SEQ_FMA, acc, a, b)
    # fp16 subnormal operands take part exactly
    a = np.array([2.0 ** -24, 2.0 ** -20], np.float16); b = np.array([1.0, 2.0 ** -4], np.float16)
    assert rgo.atom(rgo.EXACT_RN, 0.0, a, b) == np.float32(2.0 ** -24 + 2.0 ** -24)


# ---- fp8 e4m3 operands (Sec. 2: the fp8 GEMMs; a 32-wide step)
def _with_k32(m):
    import dataclasses
    return dataclasses.replace(m, atom_k=32, group=(32 if m.group == 16 else m.group))


def test_fp8_integer_products_and_closed_forms():
    for K, cuts in ((512, (256,)), (1000, ()), (96, (32, 64))):
        A = synth.int_valued_f8e4m3((5, K), -8, 8, 40 + K); B = synth.int_valued_f8e4m3((7, K), -8, 8, 41 + K)
        Ai = synth.f8e4m3_bits_to_f32(A).astype(np.int64); Bi = synth.f8e4m3_bits_to_f32(B).astype(np.int64)
        want = (Ai @ Bi.T).astype(np.float32)
        for name, m in MODELS.items():
            got = rgo.gemm(A, B, cuts=cuts, atom_model=_with_k32(m), out_dtype=rgo.F32)
            assert np.array_equal(got, want), (name, K)
    ones = synth.f32_to_f8e4m3_bits(np.ones((3, 4096), np.float32))
    assert np.all(rgo.gemm(ones, ones, atom_model=_with_k32(rgo.EXACT_RN), out_dtype=rgo.F32) == np.float32(4096))
    # rank one: every product alpha*beta, K of them
    a = synth.f32_to_f8e4m3_bits(np.full((2, 640), 1.5, np.float32)); b = synth.f32_to_f8e4m3_bits(np.full((3, 640), -0.375, np.float32))
    assert np.all(rgo.gemm(a, b, atom_model=_with_k32(rgo.EXACT_RN), out_dtype=rgo.F32) == np.float32(640 * 1.5 * -0.375))


@pytest.mark.parametrize("spread", [1, 4, 7])
def test_fp8_exact_atom_against_rationals(spread):
    g = np.random.default_rng(300 + spread)
    for trial in range(300):
        n = int(g.integers(1, 33))
        a = synth.f32_to_f8e4m3_bits((g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n))).astype(np.float32))
        b = synth.f32_to_f8e4m3_bits((g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n))).astype(np.float32))
        acc = np.float32(g.standard_normal() * 2.0 ** int(g.integers(-spread, spread + 1)))
        af = synth.f8e4m3_bits_to_f32(a); bf = synth.f8e4m3_bits_to_f32(b)
        exact = Fraction(float(acc)) + sum(Fraction(float(x)) * Fraction(float(y)) for x, y in zip(af, bf))
        assert rgo.atom(_with_k32(rgo.EXACT_RN), acc, a, b) == _rn_f32(exact)
    # subnormal operands take part exactly: 2^-9 * 1 + 2^-6 * 2^-3
    a = np.array([0x01, 0x08], np.uint8); b = np.array([0x38, 0x20], np.uint8)
    assert rgo.f8e4m3_to_f32(0x20) == 2.0 ** -3
    assert rgo.atom(_with_k32(rgo.EXACT_RN), 0.0, a, b) == np.float32(2.0 ** -9 + 2.0 ** -9)


# ---- second level of the cut nest (Sec. 3.2.2 k_cuts; App. E per-group accumulation)
def test_inner_span_worked_example_and_closed_forms():
    """k=0: 1; k=32 and k=48: 2^-24 each (different 16-wide steps).  One chain: 1 + 2^-24 ties back to 1,
    twice.  Closed every 32: the second group holds 2^-24 + 2^-24 = 2^-23 and 1 + 2^-23 is exact.
    Closed every 16: each 2^-24 meets the running sum alone and is lost again."""
    a = np.zeros((1, 96), np.float32); a[0, 0] = 1.0; a[0, 32] = 2.0 ** -24; a[0, 48] = 2.0 ** -24
    ones = _bf(np.ones((1, 96), np.float32))
    for m in (rgo.EXACT_RN, rgo.TCGEN05_BF16_B200):
        assert rgo.gemm(_bf(a), ones, atom_model=m, out_dtype=rgo.F32)[0, 0] == np.float32(1.0)
        assert rgo.gemm(_bf(a), ones, atom_model=m, out_dtype=rgo.F32, inner_span=32)[0, 0] == np.float32(1 + 2.0 ** -23)
        assert rgo.gemm(_bf(a), ones, atom_model=m, out_dtype=rgo.F32, inner_span=16)[0, 0] == np.float32(1.0)
        assert rgo.gemm(_bf(a), ones, atom_model=m, out_dtype=rgo.F32, inner_span=96)[0, 0] == np.float32(1.0)   # one group = no cut
    # integers are exact under any nest; a span that does not divide the part leaves a short last group
    A = synth.int_valued_bf16((4, 1000), -8, 8, 1); B = synth.int_valued_bf16((5, 1000), -8, 8, 2)
    want = (synth.bf16_bits_to_f32(A).astype(np.int64) @ synth.bf16_bits_to_f32(B).astype(np.int64).T).astype(np.float32)
    for span in (16, 64, 128, 448):
        for cuts in ((), (512,)):
            assert np.array_equal(rgo.gemm(A, B, cuts=cuts, inner_span=span, out_dtype=rgo.F32), want)
    # the groups restart inside every part: a part equals the unsplit GEMM of its own K range under the same nest
    A = synth.normal_bf16((3, 512), 1.0, 3); B = synth.normal_bf16((4, 512), 1.0, 4)
    P = rgo.gemm_partials(A, B, cuts=(192,), inner_span=128)
    assert np.array_equal(P[1], rgo.gemm(A[:, 192:], B[:, 192:], inner_span=128, out_dtype=rgo.F32))
    # and the nest is visible on ordinary inputs
    assert not np.array_equal(rgo.gemm(A, B, out_dtype=rgo.F32), rgo.gemm(A, B, inner_span=64, out_dtype=rgo.F32))
    # group sums against the definition: chain of group results, each an unsplit GEMM of its own range
    g = [rgo.gemm(A[:, k:k + 128], B[:, k:k + 128], out_dtype=rgo.F32) for k in range(0, 512, 128)]
    assert np.array_equal(rgo.gemm(A, B, inner_span=128, out_dtype=rgo.F32), ((g[0] + g[1]) + g[2]) + g[3])


def test_one_step_groups_are_separately_rounded_steps_chained_at_fp32():
    """inner_span = one step (Sec. 3.2.2, `use_fast_accum` off; App. E, per-instruction accumulation): every
    instruction's result is formed from a zero accumulator and reaches the running sum in a rounding of its
    own.  Spelled out from the pinned pieces: one step from zero (`rgo.atom`), then one fp32 add."""
    g = np.random.default_rng(16)
    for model, width, draw in ((rgo.TCGEN05_BF16_B200, 16, "bf16"), (rgo.EXACT_RN, 16, "bf16"), (_with_k32(rgo.TCGEN05_F8E4M3_B200), 32, "e4m3")):
        K = 7 * width + width // 2                                     # a short last step
        x = (g.standard_normal((3, K)) * np.exp2(g.integers(-5, 6, (3, K)))).astype(np.float32)
        y = (g.standard_normal((2, K)) * np.exp2(g.integers(-5, 6, (2, K)))).astype(np.float32)
        A, B = (_bf(x), _bf(y)) if draw == "bf16" else (synth.f32_to_f8e4m3_bits(np.clip(x, -448, 448)), synth.f32_to_f8e4m3_bits(np.clip(y, -448, 448)))
        for span_steps in (1, 2, 3):
            got = rgo.gemm(A, B, atom_model=model, out_dtype=rgo.F32, inner_span=span_steps * width)
            for i in range(3):
                for j in range(2):
                    run = None
                    for k0 in range(0, K, span_steps * width):
                        acc = np.float32(0.0)
                        for s0 in range(k0, min(K, k0 + span_steps * width), width):   # the steps of one group, chained in the accumulator
                            acc = rgo.atom(model, acc, A[i, s0:s0 + width], B[j, s0:s0 + width])
                        run = acc if run is None else rgo.add_f32(run, acc)           # the group reaches the running sum rounded
                    assert got[i, j] == run, (draw, span_steps, i, j)
        # and it is a different sum from the single chain
        assert not np.array_equal(rgo.gemm(A, B, atom_model=model, out_dtype=rgo.F32, inner_span=width),
                                  rgo.gemm(A, B, atom_model=model, out_dtype=rgo.F32))
