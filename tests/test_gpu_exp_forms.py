"""The exponentials as the kernels compute them, against the oracle's, value by value.

The paper's attention kernel calls the hardware's base-two exponential (App. F); this library fixes exp and exp2
as sequences of IEEE operations, and the kernels use forms of them with range selects removed where the argument's
range is known, one of them with packed fp32x2 instructions.  Each form is run on the device over its domain
(random bit patterns, the domain's ends, zeros, subnormals, and the twelve arguments on which a packed multiply in
front of the packed rounding add once changed the result) and compared bit for bit with `rgo.exp_array`.
"""
import numpy as np
import pytest
import torch

from oracle import rgo
from paper_2609_11356_b200.api import RgError, rg_selftest_exp
from _gpu_util import DEV, assert_bits_equal

pytestmark = pytest.mark.gpu

# arguments in [-87.33655, 0] whose product with log2(e), rounded once, and whose exact product round to different integers
HAZARDS = np.array([0xc0d2b77c, 0xc2a180d8, 0xc2a2e3bc, 0xc14214ca, 0xc158430d, 0xc2490340, 0xc283013c, 0xc2a70c69, 0xc16e7150,
                    0xc0ff1402, 0xc28cb579, 0xc25f3183], dtype=np.uint32)
LO_E = np.float32(-87.33655)                     # below it the base-e form's result is +0
N = 1 << 21


def _bits_between(lo_bits, hi_bits, seed):
    g = np.random.default_rng(seed)
    return g.integers(lo_bits, hi_bits + 1, N, dtype=np.uint64).astype(np.uint32)


def _run(form, x):
    xt = torch.from_numpy(x.view(np.float32).copy()).to(DEV)
    y = torch.full_like(xt, float("nan"))
    rg_selftest_exp(form, xt, y)
    torch.cuda.synchronize()
    return y.cpu().numpy()


def _special(lo, hi):
    """ends of [lo, hi], their neighbours inside, zeros, subnormals, small and integer arguments"""
    v = [lo, np.nextafter(lo, np.float32(0)), hi, -0.0, 0.0, -1e-45, -1e-40, -1.1754944e-38, -1e-20, -0.5, -1.0, -1.5, -2.0, -2.5,
         -0.6931472, -0.34657359, -10.0, -64.0, -80.0, -86.99, -87.0]
    v = np.array(v, dtype=np.float32)
    return v[(v >= lo) & (v <= hi)].view(np.uint32)


@pytest.mark.parametrize("form,base2", [(0, False), (1, True)])
def test_full_range_forms_on_random_bit_patterns(form, base2):
    x = np.concatenate([_bits_between(0, 0xffffffff, 1 + form), HAZARDS,
                        np.array([np.inf, -np.inf, np.nan, 88.72284, 88.722847, 128.0, 127.99999, -126.0, -126.00001, -149.0, -150.0, 0.0, -0.0],
                                 dtype=np.float32).view(np.uint32)])
    assert_bits_equal(_run(form, x), rgo.exp_array(x.view(np.float32), base2), f"form {form}")


def test_epilogue_form_for_magnitudes_up_to_87():
    hi = np.array([87.0], np.float32).view(np.uint32)[0]
    mag = np.concatenate([_bits_between(0, int(hi), 3), _special(np.float32(-87.0), np.float32(0.0)) & 0x7fffffff, HAZARDS & 0x7fffffff])
    mag = mag[mag <= hi]
    for sign in (0, 0x80000000):
        x = (mag | np.uint32(sign)).astype(np.uint32)
        assert_bits_equal(_run(2, x), rgo.exp_array(x.view(np.float32)), f"epilogue form, sign bit {sign:#x}")


def test_attention_packed_base_e_form():
    lo = LO_E.view(np.uint32)
    x = np.concatenate([HAZARDS, _bits_between(0x80000000, int(lo), 4), _special(LO_E, np.float32(0.0)) | np.uint32(0x80000000)])
    x = x[(x >= 0x80000000) & (x <= lo)]
    for shift in (0, 1):                          # every argument in both halves of a packed pair
        xs = np.roll(x, shift)
        assert_bits_equal(_run(3, xs), rgo.exp_array(xs.view(np.float32)), f"packed base-e form, pairing {shift}")
    # an odd count: the last element has no partner
    assert_bits_equal(_run(3, x[:1001]), rgo.exp_array(x[:1001].view(np.float32)), "odd count")


def test_attention_base_two_forms():
    lo = np.array([-126.0], np.float32).view(np.uint32)[0]
    x = np.concatenate([_bits_between(0x80000000, int(lo), 5), _special(np.float32(-126.0), np.float32(0.0)) | np.uint32(0x80000000)])
    x = x[(x >= 0x80000000) & (x <= lo)]
    assert_bits_equal(_run(4, x), rgo.exp_array(x.view(np.float32), True), "range-free base-two form on [-126, 0]")
    # the form with the underflow and NaN selects: every non-positive value, -inf and negative NaNs included, and +0
    neg = np.concatenate([_bits_between(0x80000000, 0xffffffff, 6), x[:4096], np.array([0], np.uint32),
                          np.array([-np.inf, -126.00001, -127.0, -149.5, -1e30], np.float32).view(np.uint32)])
    assert_bits_equal(_run(5, neg), rgo.exp_array(neg.view(np.float32), True), "base-two form for x <= 0 or NaN")


def test_softmax_normaliser_form():
    neg = np.concatenate([_bits_between(0x80000000, 0xffffffff, 7), HAZARDS, np.array([0], np.uint32),
                          _special(LO_E, np.float32(0.0)) | np.uint32(0x80000000),
                          np.array([-np.inf, -87.33656, -88.0, -100.0, -1e30], np.float32).view(np.uint32)])
    assert_bits_equal(_run(6, neg), rgo.exp_array(neg.view(np.float32)), "base-e form for x <= 0 or NaN")


def test_epilogue_silu_on_segments_of_32():
    g = np.random.default_rng(8)
    seg = []
    seg.append(g.standard_normal((20000, 32)).astype(np.float32) * 3)                  # every magnitude small: range-free form
    big = g.standard_normal((20000, 32)).astype(np.float32) * 3
    big[np.arange(20000), g.integers(0, 32, 20000)] = (g.uniform(87.0, 200.0, 20000) * g.choice([-1, 1], 20000)).astype(np.float32)
    seg.append(big)                                                                    # one magnitude above 87: general form
    seg.append(_bits_between(0, 0xffffffff, 9)[: 32 * 20000].view(np.float32).reshape(-1, 32))   # anything, NaN and inf included
    edge = np.zeros((8, 32), np.float32)
    edge[0, :8] = [87.0, -87.0, 87.00001, -87.00001, 88.72284, -88.72284, 0.0, -0.0]
    edge[1, :6] = [np.inf, -np.inf, np.nan, 1e-45, -1e-45, 3.4e38]
    edge[2, :] = np.linspace(-20, 20, 32, dtype=np.float32)
    seg.append(edge)
    x = np.concatenate(seg).reshape(-1)
    assert_bits_equal(_run(7, x.view(np.uint32)), rgo.silu_array(x), "epilogue SiLU")


def test_arguments():
    x = torch.zeros(4, device=DEV)
    with pytest.raises(RgError):
        rg_selftest_exp(8, x, x)
    with pytest.raises(RgError):
        rg_selftest_exp(7, x, x)                  # SiLU segments are 32 wide
    rg_selftest_exp(0, x[:0], x[:0])              # nothing to do
    y = torch.empty_like(x)
    rg_selftest_exp(0, x, y); torch.cuda.synchronize()
    assert y.tolist() == [1.0] * 4
