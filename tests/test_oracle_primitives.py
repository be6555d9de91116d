"""Pins for the oracle's primitives: conversions, single fp32 operations, the specified exp."""
import math

import numpy as np
import pytest
import torch

from oracle import rgo
from paper_2609_11356_b200 import synth


def test_bf16_widening_exhaustive():
    # every one of the 65,536 patterns: bf16 is the top half of binary32
    for h in range(0, 65536, 1):
        f = np.float32(rgo.lib().rgo_bf16_to_f32(h))
        assert f.view(np.uint32) == np.uint32(h << 16) or (math.isnan(f) and (h & 0x7fff) > 0x7f80)


def test_bf16_round_trip_exhaustive():
    for h in range(65536):
        if (h & 0x7fff) > 0x7f80:
            continue
        f = np.uint32(h << 16).view(np.float32)
        assert rgo.f32_to_bf16(f) == h


def test_bf16_narrowing_matches_library_rne():
    # independent route: torch's CPU conversion is round-to-nearest-even
    g = np.random.default_rng(0)
    x = g.standard_normal(200000).astype(np.float32) * np.exp2(g.integers(-60, 60, 200000)).astype(np.float32)
    # exact ties and their neighbours
    base = (g.integers(0, 0x7f7f, 20000).astype(np.uint32) << 16)
    ties = np.concatenate([base | 0x8000, (base | 0x8000) + 1, (base | 0x8000) - 1]).astype(np.uint32).view(np.float32)
    x = np.concatenate([x, ties, -ties])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([rgo.f32_to_bf16(v) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_tie_goes_to_even():
    # 1 + 2^-8 is exactly between bf16(1) and bf16(1 + 2^-7): even mantissa wins
    assert rgo.f32_to_bf16(np.float32(1 + 2.0 ** -8)) == 0x3F80
    assert rgo.f32_to_bf16(np.float32(1 + 2.0 ** -7 + 2.0 ** -8)) == 0x3F82


def test_add_mul_single_rounding():
    # double arithmetic then one rounding equals a correctly rounded fp32 add / mul
    g = np.random.default_rng(1)
    a = (g.standard_normal(50000) * np.exp2(g.integers(-30, 30, 50000))).astype(np.float32)
    b = (g.standard_normal(50000) * np.exp2(g.integers(-30, 30, 50000))).astype(np.float32)
    for x, y in zip(a[:20000], b[:20000]):
        assert rgo.add_f32(x, y) == np.float32(np.float64(x) + np.float64(y))
        assert rgo.mul_f32(x, y) == np.float32(np.float64(x) * np.float64(y))
    assert (np.float32(1.0) + np.float32(2.0 ** -24)) == np.float32(1.0)  # tie to even
    assert rgo.add_f32(1.0, 2.0 ** -24) == np.float32(1.0)
    assert rgo.add_f32(1.0 + 2.0 ** -23, 2.0 ** -24) == np.float32(1.0 + 2.0 ** -22)
    # -0 is the additive identity, +0 is not
    assert np.signbit(rgo.add_f32(-0.0, -0.0)) and not np.signbit(rgo.add_f32(-0.0, 0.0))


def _ulp_err(got: float, exact: float) -> float:
    if exact == 0:
        return abs(got)
    e = math.floor(math.log2(abs(exact)))
    ulp = 2.0 ** (max(e, -126) - 23)
    return abs(float(got) - exact) / ulp


def test_expf_accuracy_monotone_and_clamps():
    xs = np.linspace(-87.3, 88.7, 200001).astype(np.float32)
    prev = -1.0
    worst = 0.0
    for x in xs:
        y = float(rgo.expf(x))
        worst = max(worst, _ulp_err(y, math.exp(float(x))))
        assert y >= prev
        prev = y
    assert worst <= 2.0, worst
    assert rgo.expf(0.0) == np.float32(1.0)
    assert rgo.expf(-0.0) == np.float32(1.0)
    assert rgo.expf(89.0) == np.float32(np.inf)
    assert rgo.expf(-88.0) == np.float32(0.0)
    assert rgo.expf(-1e30) == np.float32(0.0)
    assert math.isnan(float(rgo.expf(np.float32(np.nan))))
    # dense around zero and around the reduction boundaries n*ln2/2
    for k in range(-60, 61):
        for d in (-3e-7, 0.0, 3e-7):
            x = np.float32(k * 0.34657359 + d)
            assert _ulp_err(float(rgo.expf(x)), math.exp(float(x))) <= 2.0


def test_silu():
    assert rgo.silu(0.0) == np.float32(0.0)
    xs = np.linspace(-30, 30, 20001).astype(np.float32)
    for x in xs:
        want = float(x) / (1.0 + math.exp(-float(x)))
        assert _ulp_err(float(rgo.silu(x)), want) <= 4.0
    assert rgo.silu(-200.0) == np.float32(-0.0)  # x / inf
    assert rgo.silu(200.0) == np.float32(200.0)


def test_f16_widening_exhaustive():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = allbits.view(np.float16).astype(np.float32)
    got = np.array([rgo.lib().rgo_f16_to_f32(int(h)) for h in allbits], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32)) and np.all(np.isnan(got[nan]))


def test_f16_narrowing_matches_library_rne():
    g = np.random.default_rng(2)
    x = (g.standard_normal(200000) * np.exp2(g.integers(-30, 18, 200000))).astype(np.float32)
    h = g.integers(0, 0x7bff, 30000).astype(np.uint16)                       # exact ties between neighbours
    lo = h.view(np.float16).astype(np.float64); hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    ties = ((lo + hi) / 2).astype(np.float32)
    near = np.concatenate([np.nextafter(ties, np.float32(np.inf)), np.nextafter(ties, np.float32(-np.inf))])
    edge = np.array([65504, 65519.99, 65520, 65536, 1e9, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0001, 2.0 ** -26, 0.0, -0.0,
                     6.1e-5, 6.097e-5, np.inf], dtype=np.float32)
    x = np.concatenate([x, ties, -ties, near, edge, -edge])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    got = np.array([rgo.f32_to_f16(v) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
    for h16 in range(0, 0x7c00):                                            # round trip of every finite pattern
        assert rgo.f32_to_f16(np.uint16(h16).view(np.float16).astype(np.float32)) == h16


def test_f8e4m3_widening_exhaustive_and_landmarks():
    allbits = np.arange(256, dtype=np.uint8)
    want = synth.f8e4m3_bits_to_f32(allbits)                       # torch's conversion, an independent routine
    got = np.array([rgo.f8e4m3_to_f32(int(h)) for h in allbits], dtype=np.float32)
    nan = np.isnan(want)
    assert list(np.nonzero(nan)[0]) == [0x7f, 0xff]                # the only NaN patterns; no infinities
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32)) and np.all(np.isnan(got[nan]))
    # landmarks of the 1-4-3 format with bias 7
    assert rgo.f8e4m3_to_f32(0x7e) == 448.0 and rgo.f8e4m3_to_f32(0xfe) == -448.0
    assert rgo.f8e4m3_to_f32(0x01) == 2.0 ** -9 and rgo.f8e4m3_to_f32(0x07) == 7 * 2.0 ** -9
    assert rgo.f8e4m3_to_f32(0x08) == 2.0 ** -6 and rgo.f8e4m3_to_f32(0x38) == 1.0 and rgo.f8e4m3_to_f32(0x3c) == 1.5
    assert np.float32(rgo.f8e4m3_to_f32(0x80)).view(np.uint32) == 0x80000000


def test_exp2f_accuracy_exact_powers_monotone_and_clamps():
    g = np.random.default_rng(4)
    x = np.concatenate([g.uniform(-126, 128, 200000), g.uniform(-2, 2, 100000), g.uniform(-40, 0, 100000)]).astype(np.float32)
    got = np.array([rgo.exp2f(v) for v in x], dtype=np.float32)
    ref = np.exp2(x.astype(np.float64))
    ulp = np.spacing(ref.astype(np.float32)).astype(np.float64)
    assert np.max(np.abs(got.astype(np.float64) - ref) / ulp) <= 2.0
    for n in range(-126, 128):                                   # integers: exact powers of two
        assert rgo.exp2f(n) == np.float32(2.0) ** n
    assert rgo.exp2f(0.5) == np.float32(np.sqrt(2.0)) or abs(float(rgo.exp2f(0.5)) - 2 ** 0.5) < 2e-7
    grid = np.linspace(-30, 30, 200001).astype(np.float32)
    vals = np.array([rgo.exp2f(v) for v in grid], dtype=np.float32)
    assert np.all(np.diff(vals) >= 0)
    assert rgo.exp2f(-126.0) == np.float32(2.0 ** -126) and rgo.exp2f(np.float32(-126.00001)) == 0 and rgo.exp2f(-1e30) == 0
    assert rgo.exp2f(-np.inf) == 0 and np.isinf(rgo.exp2f(128.0)) and np.isinf(rgo.exp2f(np.inf)) and np.isnan(rgo.exp2f(np.nan))
    assert rgo.exp2f(np.float32(127.99999)) < np.inf


def test_exp_array_is_the_scalar_functions_in_a_loop():
    g = np.random.default_rng(9)
    x = np.concatenate([g.uniform(-100, 100, 500), [0.0, -0.0, np.inf, -np.inf, np.nan, 88.8, -87.4, 128.0, -126.5]]).astype(np.float32)
    for base2 in (False, True):
        y = rgo.exp_array(x, base2)
        for xi, yi in zip(x, y):
            want = rgo.exp2f(xi) if base2 else rgo.expf(xi)
            assert (np.isnan(yi) and np.isnan(want)) or np.float32(yi).view(np.uint32) == np.float32(want).view(np.uint32)
    for xi, yi in zip(x, rgo.silu_array(x)):
        want = rgo.silu(xi)
        assert (np.isnan(yi) and np.isnan(want)) or np.float32(yi).view(np.uint32) == np.float32(want).view(np.uint32)
