"""The finite-window step family of the oracle (Sec. 3.2.1: what one matrix instruction does to its
products and the incoming accumulator) against an independent restatement in exact rational
arithmetic.

The oracle evaluates the family with shifts on 128-bit integers and a long accumulator; here every
quantity is a `fractions.Fraction`, exponents come from comparisons with powers of two, truncation is
`int()` / `math.floor` of an exact quotient and the final rounding is written from the definition of
binary32.  The two share nothing, so a wrong shift, a window off by one bit, a mishandled sign under
floor, or an accumulator aligned at the wrong weight in the oracle fails here for some parameter set.
What stays taken from hardware after this file are only the parameter *values* of the member that
reproduces a B200 (window 25, exponent Ea + Eb, truncation, RZ), not the machinery that evaluates it.
"""
import dataclasses
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import rgo
from paper_2609_11356_b200 import synth

TWO = Fraction(2)

# (exponent field width, fraction field width, bias) of the operand formats
FORMATS = {rgo.BF16: (8, 7, 127), rgo.F16: (5, 10, 15), rgo.F8E4M3: (4, 3, 7)}


def _decode(bits: int, fmt: int):
    """(value as a Fraction, exponent the format assigns to the operand).  A subnormal operand carries
    the format's smallest normal exponent, whatever its leading bit is."""
    ew, fw, bias = FORMATS[fmt]
    sign = -1 if (bits >> (ew + fw)) & 1 else 1
    e = (bits >> fw) & ((1 << ew) - 1)
    f = bits & ((1 << fw) - 1)
    if e == 0:
        return sign * Fraction(f, 1 << fw) * TWO ** (1 - bias), 1 - bias
    return sign * (1 + Fraction(f, 1 << fw)) * TWO ** (e - bias), e - bias


def _floor_log2(q: Fraction) -> int:
    """The e with 2^e <= |q| < 2^(e+1), found by comparison."""
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    while TWO ** e > a:
        e -= 1
    while TWO ** (e + 1) <= a:
        e += 1
    return e


def _to_f32(q: Fraction, nearest: bool) -> np.float32:
    """Round an exact value to binary32: toward zero, or to nearest with ties to even."""
    if q == 0:
        return np.float32(0.0)
    s, a = (-1 if q < 0 else 1), abs(q)
    lsb = max(_floor_log2(a) - 23, -149)
    scaled = a / TWO ** lsb
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if nearest and (rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1)):
        n += 1
    return np.float32(s * math.ldexp(n, lsb))


def _window_step(acc: np.float32, a_bits, b_bits, fmt: int, m: rgo.AtomModel) -> np.float32:
    """One internal step, from the definition: every addend is aligned to the largest exponent present,
    kept to `window_bits` bits below it, the kept parts are added exactly and the sum is rounded once."""
    prods, exps = [], []
    for x, y in zip(a_bits, b_bits):
        vx, ex = _decode(int(x), fmt)
        vy, ey = _decode(int(y), fmt)
        v = vx * vy
        prods.append(v)
        if v != 0:
            exps.append(ex + ey if m.exp_mode else _floor_log2(v))
    accq = Fraction(float(acc))
    if m.acc_in_window and accq != 0:
        exps.append(_floor_log2(accq))
    if not exps:
        return np.float32(acc)                                  # nothing but zeros: the accumulator passes
    quantum = TWO ** (max(exps) - min(m.window_bits, 90))       # weight of the window's last bit

    def keep(v: Fraction) -> Fraction:
        units = v / quantum
        kept = math.floor(units) if m.addend_round == 1 else int(units)   # floor, or truncation toward zero
        return kept * quantum

    total = sum(keep(v) for v in prods)
    total += keep(accq) if m.acc_in_window else accq
    return _to_f32(total, nearest=bool(m.final_round))


def _window_atom(acc, a_bits, b_bits, fmt, m):
    g = m.group if m.group > 0 else len(a_bits)
    for u0 in range(0, len(a_bits), g):
        acc = _window_step(acc, a_bits[u0:u0 + g], b_bits[u0:u0 + g], fmt, m)
    return acc


def _draw_operands(g, n, spread, fmt):
    x = (g.standard_normal(n) * np.exp2(g.integers(-spread, spread + 1, n))).astype(np.float32)
    if g.random() < 0.3:                                        # near-cancelling neighbours stress the window's edge
        x[1::2] = -x[: n // 2 * 2: 2] * np.float32(1 + 2.0 ** -int(g.integers(1, 7)))
    if g.random() < 0.2:
        x[int(g.integers(0, n))] = 0.0
    if fmt == rgo.BF16:
        return synth.f32_to_bf16_bits(x)
    if fmt == rgo.F16:
        return x.astype(np.float16).view(np.uint16)
    return synth.f32_to_f8e4m3_bits(x)


def _call_oracle(m, acc, a, b, fmt):
    if fmt == rgo.F8E4M3:
        return rgo.atom(m, acc, a.astype(np.uint8), b.astype(np.uint8))
    if fmt == rgo.F16:
        return rgo.atom(m, acc, a.view(np.float16), b.view(np.float16))
    return rgo.atom(m, acc, a, b)


def _same(x: np.float32, y: np.float32) -> bool:
    return np.float32(x).view(np.uint32) == np.float32(y).view(np.uint32) or (x == 0 and y == 0)


CASES = [(rgo.BF16, 2), (rgo.BF16, 12), (rgo.BF16, 40), (rgo.F16, 2), (rgo.F16, 6), (rgo.F16, 12),
         (rgo.F8E4M3, 1), (rgo.F8E4M3, 4), (rgo.F8E4M3, 7)]


@pytest.mark.parametrize("fmt,spread", CASES)
def test_window_family_against_rationals_over_random_parameter_sets(fmt, spread):
    g = np.random.default_rng(1000 * fmt + spread)
    width = 32 if fmt == rgo.F8E4M3 else 16
    for trial in range(320):
        m = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, atom_k=width,
                          group=int(g.choice([4, 8, 16, 32][: 4 if width == 32 else 3])),
                          window_bits=int(g.integers(6, 41)), exp_mode=int(g.integers(0, 2)),
                          acc_in_window=int(g.integers(0, 2)), addend_round=int(g.integers(0, 2)),
                          final_round=int(g.integers(0, 2)))
        n = int(g.integers(1, width + 1))
        a = _draw_operands(g, n, spread, fmt); b = _draw_operands(g, n, spread, fmt)
        acc = np.float32(0.0) if g.random() < 0.15 else np.float32(g.standard_normal() * 2.0 ** int(g.integers(-2 * spread, 2 * spread + 1)))
        want = _window_atom(acc, a, b, fmt, m)
        got = _call_oracle(m, acc, a, b, fmt)
        assert _same(got, want), (trial, m, acc, a.tolist(), b.tolist(), got, want)


@pytest.mark.parametrize("base,fmt", [(rgo.TCGEN05_BF16_B200, rgo.BF16), (rgo.TCGEN05_BF16_B200, rgo.F16),
                                      (rgo.TCGEN05_F8E4M3_B200, rgo.F8E4M3)])
def test_selected_members_against_rationals(base, fmt):
    """The two members the library's GPU tests compare against, full-width steps, chained like a K walk."""
    g = np.random.default_rng(77 + fmt)
    width = base.atom_k
    spreads = (1, 3, 7) if fmt == rgo.F8E4M3 else (2, 6, 12) if fmt == rgo.F16 else (2, 12, 40)
    for spread in spreads:
        for trial in range(120):
            acc_o = acc_r = np.float32(0.0)
            for step in range(4):                               # four chained steps: the accumulator re-enters the window
                a = _draw_operands(g, width, spread, fmt); b = _draw_operands(g, width, spread, fmt)
                acc_o = _call_oracle(base, acc_o, a, b, fmt)
                acc_r = _window_atom(acc_r, a, b, fmt, base)
                assert _same(acc_o, acc_r), (spread, trial, step)


def test_subnormal_operands_and_accumulator():
    """A subnormal operand keeps its true value but carries the smallest normal exponent (exp_mode 1);
    a subnormal accumulator is aligned at its true leading bit."""
    m1 = dataclasses.replace(rgo.TCGEN05_BF16_B200)
    m0 = dataclasses.replace(m1, exp_mode=0)
    g = np.random.default_rng(9)
    for trial in range(200):
        a = g.integers(0, 0x80, 16).astype(np.uint16) | (g.integers(0, 2, 16).astype(np.uint16) << 15)   # bf16 subnormals and zeros
        b = synth.f32_to_bf16_bits((g.standard_normal(16) * np.exp2(g.integers(100, 126, 16))).astype(np.float32))
        acc = np.float32(g.standard_normal() * 2.0 ** -140) if trial % 2 else np.float32(g.standard_normal() * 2.0 ** -20)
        for m in (m0, m1):
            assert _same(rgo.atom(m, acc, a, b), _window_atom(acc, a, b, rgo.BF16, m)), (trial, m.exp_mode)


def test_restatement_itself_on_hand_cases():
    """The rational restatement checked by hand, so that the comparison above is not two wrong answers
    agreeing: values worked out on paper from the definition."""
    one = int(synth.f32_to_bf16_bits(np.array([1.0], np.float32))[0])

    def bf(v):
        return [int(t) for t in synth.f32_to_bf16_bits(np.asarray(v, np.float32))]

    m = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=24, final_round=0)
    # {1, 2^-25, -1}: 2^-25 lies below the 24-bit window under 2^0 and is dropped
    assert _window_atom(np.float32(0), bf([1.0, 2.0 ** -25, -1.0]), [one] * 3, rgo.BF16, m) == 0.0
    # {1, 2^-24, -1}: the window's last bit has weight 2^-24, so it is kept
    assert _window_atom(np.float32(0), bf([1.0, 2.0 ** -24, -1.0]), [one] * 3, rgo.BF16, m) == np.float32(2.0 ** -24)
    # floor of a small negative addend is minus one unit of the window; truncation drops it
    mf = dataclasses.replace(m, addend_round=1)
    assert _window_atom(np.float32(0), bf([1.0, -2.0 ** -30]), [one] * 2, rgo.BF16, mf) == np.float32(1 - 2.0 ** -24)
    assert _window_atom(np.float32(0), bf([1.0, -2.0 ** -30]), [one] * 2, rgo.BF16, m) == np.float32(1.0)
    # 1.5 * 1.5 = 2.25: normalised exponent 1, operand exponents 0 + 0.  With a 4-bit window the unit is
    # 2^-3 (normalised) or 2^-4 (Ea + Eb), and 2^-4 survives only in the second
    m4n = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=4, exp_mode=0, final_round=0)
    m4o = dataclasses.replace(m4n, exp_mode=1)
    a, b = bf([1.5, 2.0 ** -4]), bf([1.5, 1.0])
    assert _window_atom(np.float32(0), a, b, rgo.BF16, m4n) == np.float32(2.25)
    assert _window_atom(np.float32(0), a, b, rgo.BF16, m4o) == np.float32(2.25 + 2.0 ** -4)
    # an accumulator outside the window keeps all its bits; inside, it is cut like a product
    mo = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=8, acc_in_window=0, final_round=1)
    mi = dataclasses.replace(mo, acc_in_window=1)
    acc = np.float32(2.0 ** -12)
    assert _window_atom(acc, bf([1.0, -1.0]), [one] * 2, rgo.BF16, mo) == acc
    assert _window_atom(acc, bf([1.0, -1.0]), [one] * 2, rgo.BF16, mi) == 0.0
    # final rounding: 1 + 2^-24 + 2^-25 is above the tie (RN rounds up, RZ cuts); 1 + 2^-24 is the tie (even: 1)
    wide_rn = rgo.AtomModel(model=rgo.ATOM_ALIGN_TRUNC, window_bits=40, final_round=1)
    wide_rz = dataclasses.replace(wide_rn, final_round=0)
    a = bf([1.0, 2.0 ** -24, 2.0 ** -25])
    assert _window_atom(np.float32(0), a, [one] * 3, rgo.BF16, wide_rn) == np.float32(1 + 2.0 ** -23)
    assert _window_atom(np.float32(0), a, [one] * 3, rgo.BF16, wide_rz) == np.float32(1.0)
    assert _window_atom(np.float32(0), a[:2], [one] * 2, rgo.BF16, wide_rn) == np.float32(1.0)
    # and the oracle gives the same on each of these
    for mm, aa, bb, ac in ((m, bf([1.0, 2.0 ** -25, -1.0]), [one] * 3, 0.0), (mf, bf([1.0, -2.0 ** -30]), [one] * 2, 0.0),
                           (m4o, bf([1.5, 2.0 ** -4]), bf([1.5, 1.0]), 0.0), (m4n, bf([1.5, 2.0 ** -4]), bf([1.5, 1.0]), 0.0),
                           (mi, bf([1.0, -1.0]), [one] * 2, acc), (mo, bf([1.0, -1.0]), [one] * 2, acc),
                           (wide_rn, a, [one] * 3, 0.0), (wide_rz, a, [one] * 3, 0.0)):
        assert _same(rgo.atom(mm, ac, aa, bb), _window_atom(np.float32(ac), aa, bb, rgo.BF16, mm))
