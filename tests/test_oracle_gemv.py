"""Pins for the GEMV family oracle (Sec. 3.2.2 "GEMV"; Sec. 4 "Strided grouping")."""
import os

import numpy as np
import pytest

from oracle import rgo
from paper_2609_11356_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
L, r = np.float32(1024.0), np.float32(2.0 ** -15)


def _bf(x):
    return synth.f32_to_bf16_bits(np.asarray(x, np.float32))


def test_printed_strided_grouping_is_two_lanes_of_tile_one():
    """(a0+a2+a4+a6)+(a1+a3+a5+a7): two lanes, tiles of one element dealt alternately, one fold."""
    rows = [(int(k), r if v == "r" else np.float32(0)) for k, v in
            (ln.split() for ln in open(os.path.join(GOLD, "strided_grouping_8.txt")) if not ln.startswith("#") and ln.strip())]
    A = np.zeros((len(rows), 8), np.float32)
    for n, (ridx, _) in enumerate(rows):
        A[n, 0], A[n, 6], A[n, ridx] = L, -L, r
    got = rgo.gemv(_bf(A), _bf(np.ones((1, 8))), lanes=2, tile=1, layout=0, out_dtype=rgo.F32)[:, 0]
    assert np.array_equal(got, np.array([w for _, w in rows], np.float32))
    # the contiguous deal of the same eight terms is the other printed grouping: (a0..a3)+(a4..a7)
    rows = [(int(k), r if v == "r" else np.float32(0)) for k, v in
            (ln.split() for ln in open(os.path.join(GOLD, "contiguous_grouping_8.txt")) if not ln.startswith("#") and ln.strip())]
    A = np.zeros((len(rows), 8), np.float32)
    for n, (p, _) in enumerate(rows):
        A[n, 0], A[n, p], A[n, p + 1] = r, L, -L
    got = rgo.gemv(_bf(A), _bf(np.ones((1, 8))), lanes=2, tile=1, layout=1, out_dtype=rgo.F32)[:, 0]
    assert np.array_equal(got, np.array([w for _, w in rows], np.float32))


def test_count_up_and_count_down_folds_are_different_trees():
    """Four lanes, one element each: count-up pairs (0,1),(2,3); count-down pairs (0,2),(1,3)."""
    ones = _bf(np.ones((1, 4)))
    a = np.array([[r, L, -L, 0]], np.float32)          # L and -L in lanes 1 and 2
    assert rgo.gemv(_bf(a), ones, lanes=4, tile=1, fold=0, out_dtype=rgo.F32)[0, 0] == np.float32(0)   # (r+L)+(-L+0)
    a = np.array([[r, L, 0, -L]], np.float32)          # L and -L in lanes 1 and 3: a pair only when counting down
    assert rgo.gemv(_bf(a), ones, lanes=4, tile=1, fold=0, out_dtype=rgo.F32)[0, 0] == np.float32(0)   # (r+L)+(0-L)
    assert rgo.gemv(_bf(a), ones, lanes=4, tile=1, fold=1, out_dtype=rgo.F32)[0, 0] == r               # (r+0)+(L-L)
    # brute force: every placement of r, L, -L over 8 lanes against explicit trees
    for i in range(8):
        for j in range(8):
            for k in range(8):
                if len({i, j, k}) < 3:
                    continue
                v = np.zeros(8, np.float32); v[i], v[j], v[k] = r, L, -L
                up = rgo.tree_sum(v, rgo.TREE_BALANCED)
                rev = [int(format(t, "03b")[::-1], 2) for t in range(8)]
                down = rgo.tree_sum(v[rev], rgo.TREE_BALANCED)
                a8 = _bf(v[None, :]); o8 = _bf(np.ones((1, 8)))
                assert rgo.gemv(a8, o8, lanes=8, tile=1, fold=0, out_dtype=rgo.F32)[0, 0] == up
                assert rgo.gemv(a8, o8, lanes=8, tile=1, fold=1, out_dtype=rgo.F32)[0, 0] == down


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("fold", [0, 1])
def test_integers_exact_and_tails(layout, fold):
    for K in (1, 7, 8, 100, 1000, 14336):
        A = synth.int_valued_bf16((3, K), -8, 8, K); B = synth.int_valued_bf16((5, K), -8, 8, K + 1)
        want = (synth.bf16_bits_to_f32(A).astype(np.int64) @ synth.bf16_bits_to_f32(B).astype(np.int64).T).astype(np.float32)
        for fma in (0, 1):
            assert np.array_equal(rgo.gemv(A, B, fma=fma, layout=layout, fold=fold, out_dtype=rgo.F32), want)
    ones = _bf(np.ones((2, 4099)))
    assert np.all(rgo.gemv(ones, ones, layout=layout, fold=fold, out_dtype=rgo.F32) == np.float32(4099))


def test_lane_chain_is_sequential_and_fma_matters_only_for_inexact_products():
    # one lane, tile = K: a plain fma chain, equal to the SEQ GEMM oracle
    A = synth.normal_bf16((4, 300), 1.0, 1); B = synth.normal_bf16((6, 300), 1.0, 2)
    assert np.array_equal(rgo.gemv(A, B, lanes=1, tile=300, out_dtype=rgo.F32), rgo.gemm(A, B, atom_model=rgo.SEQ_FMA, out_dtype=rgo.F32))
    assert np.array_equal(rgo.gemv(A, B, fma=0, out_dtype=rgo.F32), rgo.gemv(A, B, fma=1, out_dtype=rgo.F32))   # bf16 products are exact
    # against double: |error| <= depth * eps * sum|ab|
    got = rgo.gemv(A, B, out_dtype=rgo.F32).astype(np.float64)
    a64, b64 = synth.bf16_bits_to_f32(A).astype(np.float64), synth.bf16_bits_to_f32(B).astype(np.float64)
    assert np.all(np.abs(got - a64 @ b64.T) <= 20 * 2.0 ** -24 * (np.abs(a64) @ np.abs(b64).T))
    # epilogue indexing as in the GEMM
    bias = _bf(np.arange(6) - 2.0); res = _bf(np.arange(24).reshape(4, 6) % 5 - 2.0)
    Ai = synth.int_valued_bf16((4, 64), -4, 4, 3); Bi = synth.int_valued_bf16((6, 64), -4, 4, 4)
    want = synth.bf16_bits_to_f32(Ai).astype(np.int64) @ synth.bf16_bits_to_f32(Bi).astype(np.int64).T + \
        synth.bf16_bits_to_f32(bias).astype(np.int64)[None, :] + synth.bf16_bits_to_f32(res).astype(np.int64)
    assert np.array_equal(rgo.gemv(Ai, Bi, bias=bias, residual=res, out_dtype=rgo.F32), want.astype(np.float32))
