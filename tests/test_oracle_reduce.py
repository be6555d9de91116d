"""Pins for the row-reduction oracles: sum, RMSNorm, softmax normaliser."""
import math

import numpy as np
import pytest

from oracle import rgo
from paper_2609_11356_b200 import synth


def _topdown(v):
    n = len(v)
    if n == 1:
        return v[0]
    p = 1 << ((n - 1).bit_length() - 1)
    return np.float32(_topdown(v[:p]) + _topdown(v[p:]))


def test_row_sum_is_the_tree_per_row():
    x = synth.normal_f32((5, 777), 1.0, 0)
    out, _ = rgo.reduce_rows(rgo.OP_SUM, x)
    for r in range(5):
        assert out[r] == _topdown(list(x[r]))
    out_l, _ = rgo.reduce_rows(rgo.OP_SUM, x, tree=rgo.TREE_LEFT)
    acc = x[2, 0]
    for c in range(1, 777):
        acc = np.float32(acc + x[2, c])
    assert out_l[2] == acc


def test_row_sum_bf16_leaves_and_integers():
    xi = synth.int_valued_bf16((3, 4096), -100, 100, 4)
    out, _ = rgo.reduce_rows(rgo.OP_SUM, xi)
    assert np.array_equal(out, synth.bf16_bits_to_f32(xi).astype(np.int64).sum(1).astype(np.float32))


def test_row_sum_cancellation_pairs_close_to_double():
    x = synth.add_cancellation_pairs(synth.normal_f32((4, 32768), 100.0, 13), 14)
    out, _ = rgo.reduce_rows(rgo.OP_SUM, x)
    ref = x.astype(np.float64).sum(1)
    # error bound of pairwise summation: depth * eps * sum|x|
    bound = 15 * 2.0 ** -24 * np.abs(x.astype(np.float64)).sum(1)
    assert np.all(np.abs(out - ref) <= bound)


def test_rmsnorm_against_double_and_closed_forms():
    C = 4096
    x = synth.normal_bf16((6, C), 1.0, 9)
    w = synth.normal_bf16((C,), 0.05, 10, mean=1.0)
    y, rinv = rgo.reduce_rows(rgo.OP_RMSNORM, x, weight=w, eps=1e-5)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64); wf = synth.bf16_bits_to_f32(w).astype(np.float64)
    ref = xf / np.sqrt((xf ** 2).mean(1, keepdims=True) + np.float64(np.float32(1e-5))) * wf
    got = synth.bf16_bits_to_f32(y).astype(np.float64)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7)
    assert np.all(np.abs(got - ref) <= 1.01 * ulp)          # within one bf16 ulp of the exact value
    assert np.mean(got == synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(ref.astype(np.float32)))) > 0.99
    # all-equal row, unit weight: c / sqrt(c^2 + eps)
    for cval in (0.5, 2.0, -3.0):
        xr = synth.f32_to_bf16_bits(np.full((1, 1024), cval, np.float32))
        yr, _ = rgo.reduce_rows(rgo.OP_RMSNORM, xr, eps=1e-5, out_dtype=rgo.F32)
        want = cval / math.sqrt(cval * cval + float(np.float32(1e-5)))
        assert np.all(np.abs(yr - want) <= 2 * 2.0 ** -24 * abs(want) * 2)
    # powers of two with eps = 0: exact
    xr = np.full((1, 256), 4.0, np.float32)
    yr, ri = rgo.reduce_rows(rgo.OP_RMSNORM, xr, eps=0.0)
    assert ri[0] == np.float32(0.25) and np.all(yr == np.float32(1.0))
    # weight indexes the column
    wcol = np.arange(256, dtype=np.float32)
    yr, _ = rgo.reduce_rows(rgo.OP_RMSNORM, xr, weight=wcol, eps=0.0)
    assert np.array_equal(yr[0], wcol)


def test_rmsnorm_fma_flag():
    # bf16 leaves: squares are exact, so the flag cannot move a bit
    x = synth.normal_bf16((4, 512), 1.0, 3)
    y0, r0 = rgo.reduce_rows(rgo.OP_RMSNORM, x, fma=0, eps=1e-5)
    y1, r1 = rgo.reduce_rows(rgo.OP_RMSNORM, x, fma=1, eps=1e-5)
    assert np.array_equal(y0, y1) and np.array_equal(r0, r1)
    # fp32 leaves: the fused level-0 node keeps the second square unrounded
    x = np.array([[1.0, 1.0 + 2.0 ** -12]], np.float32)
    _, r0 = rgo.reduce_rows(rgo.OP_RMSNORM, x, fma=0, eps=0.0)
    _, r1 = rgo.reduce_rows(rgo.OP_RMSNORM, x, fma=1, eps=0.0)
    ss0 = np.float32(np.float32(1.0) + np.float32(np.float32(1 + 2.0 ** -12) ** 2))
    ss1 = np.float32(1.0 + (1 + 2.0 ** -12) ** 2)
    assert r0[0] == np.float32(1.0) / np.sqrt(np.float32(ss0 / np.float32(2)))
    assert r1[0] == np.float32(1.0) / np.sqrt(np.float32(ss1 / np.float32(2)))


def test_softmax_normaliser():
    # identical values: every leaf is exp(0) = 1, the sum is exactly C
    x = np.full((2, 4096), 3.25, np.float32)
    Z, m = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, x)
    assert np.all(Z == np.float32(4096)) and np.all(m == np.float32(3.25))
    # cancellation rows: only the +1e8 entries survive the shift by the row max
    x = synth.add_cancellation_pairs(synth.normal_f32((4, 32768), 100.0, 13), 14, pairs=64)
    Z, m = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, x)
    assert Z[0] == np.float32(64) and Z[2] == np.float32(64) and m[0] == np.float32(1e8)
    # ordinary rows against double
    for rr in (1, 3):
        xd = x[rr].astype(np.float64)
        ref = np.exp(xd - xd.max()).sum()
        assert abs(float(Z[rr]) - ref) <= 4e-6 * ref
        assert m[rr] == x[rr].max()
    # a single column
    Z, m = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, np.array([[5.0], [-2.0]], np.float32))
    assert np.all(Z == np.float32(1.0))


# ---- reductions along the other axis (column sums; the LayerNorm weight-gradient shape)
def test_col_sum_is_the_tree_per_column_over_rows_in_order():
    x = synth.normal_f32((777, 6), 1.0, 5)
    out = rgo.reduce_cols(0, x)
    for c in range(6):
        assert out[c] == _topdown(list(x[:, c]))                 # independent top-down restatement of the tree
    # left fold spelled out
    out_l = rgo.reduce_cols(0, x, tree=rgo.TREE_LEFT)
    acc = x[0, 3]
    for r in range(1, 777):
        acc = np.float32(acc + x[r, 3])
    assert out_l[3] == acc
    # integer leaves: exact under any tree; all ones: R
    xi = np.random.default_rng(1).integers(-100, 101, (1000, 9)).astype(np.float32)
    assert np.array_equal(rgo.reduce_cols(0, xi), xi.astype(np.int64).sum(0).astype(np.float32))
    assert np.all(rgo.reduce_cols(0, np.ones((4097, 3), np.float32)) == 4097)
    # bf16 leaves widen exactly
    xb = synth.int_valued_bf16((300, 4), -50, 50, 2)
    assert np.array_equal(rgo.reduce_cols(0, xb), synth.bf16_bits_to_f32(xb).astype(np.int64).sum(0).astype(np.float32))


def test_col_sum_probe_tells_the_tree_from_its_neighbours():
    # +L, -L, r placed along the rows of one column: r survives exactly when +L and -L meet before r joins them
    L, r = np.float32(1024.0), np.float32(2.0 ** -15)
    def col(n, pos_r, pos_p, pos_m):
        v = np.zeros((n, 1), np.float32); v[pos_r] = r; v[pos_p] = L; v[pos_m] = -L
        return v
    # rows 2,3 pair at level 0 in the balanced tree: +L and -L cancel before r (row 0) arrives
    assert rgo.reduce_cols(0, col(8, 0, 2, 3))[0] == r
    # rows 1,2 do not pair at level 0 (pairs are (0,1), (2,3)): r at row 0 is absorbed by +L
    assert rgo.reduce_cols(0, col(8, 0, 1, 2))[0] == 0
    # the left fold absorbs r at row 0 in both placements, and keeps it when it comes last
    assert rgo.reduce_cols(0, col(8, 0, 2, 3), tree=rgo.TREE_LEFT)[0] == 0
    assert rgo.reduce_cols(0, col(8, 7, 2, 3), tree=rgo.TREE_LEFT)[0] == r
    # unpaired last row moves up unchanged: n = 5, rows (0,1), (2,3) pair, row 4 joins at the top
    v = np.zeros((5, 1), np.float32); v[0] = L; v[1] = r; v[2] = -L; v[4] = r
    assert rgo.reduce_cols(0, v)[0] == r                           # (L+r -> L) + (-L) = 0, then + r


def test_col_dot_products_round_once_and_fma_flag():
    g = np.random.default_rng(3)
    x = g.standard_normal((513, 5)).astype(np.float32); y = g.standard_normal((513, 5)).astype(np.float32)
    out = rgo.reduce_cols(1, x, y)
    for c in range(5):
        assert out[c] == _topdown([np.float32(a * b) for a, b in zip(x[:, c], y[:, c])])
    # against double: 513 terms, a few ulp of the sum of magnitudes
    ref = (x.astype(np.float64) * y.astype(np.float64)).sum(0)
    assert np.all(np.abs(out - ref) <= 16 * 2.0 ** -24 * np.abs(x.astype(np.float64) * y).sum(0))
    # integer-valued: exact; equals the sum path on the elementwise product
    xi = g.integers(-30, 31, (400, 4)).astype(np.float32); yi = g.integers(-30, 31, (400, 4)).astype(np.float32)
    assert np.array_equal(rgo.reduce_cols(1, xi, yi), (xi * yi).astype(np.int64).sum(0).astype(np.float32))
    assert np.array_equal(rgo.reduce_cols(1, x, y), rgo.reduce_cols(0, (x * y).astype(np.float32)))
    # fma: the second product of each level-0 pair is not rounded before the add.  a^2 = 1 + 2^-11 + 2^-24
    # rounds to 1 + 2^-11; -RN(a^2) + a^2 is 0 with two roundings and the residual 2^-24 fused
    a = np.float32(1 + 2.0 ** -12)
    xx = np.array([[a], [a]], np.float32); yy = np.array([[-a], [a]], np.float32)
    assert rgo.reduce_cols(1, xx, yy)[0] == 0
    assert rgo.reduce_cols(1, xx, yy, fma=1)[0] == np.float32(2.0 ** -24)
    assert rgo.reduce_cols(1, xx, yy, fma=1, tree=rgo.TREE_LEFT)[0] == np.float32(2.0 ** -24)
    # the transpose relation: a column reduction is the row reduction of the transposed matrix
    xt = np.ascontiguousarray(x.T)
    rows, _ = rgo.reduce_rows(rgo.OP_SUM, xt)
    assert np.array_equal(rgo.reduce_cols(0, x), rows)
