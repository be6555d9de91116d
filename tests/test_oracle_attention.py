"""Pins for the attention oracle (App. F): the online-softmax recurrence over key blocks."""
import numpy as np
import pytest

from oracle import rgo
from paper_2609_11356_b200 import synth


def _bf(x):
    return synth.f32_to_bf16_bits(np.asarray(x, np.float32))


def _f(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def _ref64(Q, K, V, scale):
    S = (_f(Q) @ _f(K).T) * scale
    P = np.exp(S - S.max(1, keepdims=True))
    return (P / P.sum(1, keepdims=True)) @ _f(V)


@pytest.mark.parametrize("Nq,Nk,d,w", [(5, 64, 32, 64), (7, 300, 64, 128), (3, 1000, 128, 128), (4, 257, 128, 64), (2, 16, 16, 16)])
@pytest.mark.parametrize("model", ["exact", "hw"])
def test_close_to_double_softmax_attention(Nq, Nk, d, w, model):
    g = np.random.default_rng(Nk + d)
    Q, K, V = _bf(g.standard_normal((Nq, d))), _bf(g.standard_normal((Nk, d))), _bf(g.standard_normal((Nk, d)))
    m = rgo.EXACT_RN if model == "exact" else rgo.TCGEN05_BF16_B200
    out = rgo.attention(Q, K, V, block_n=w, scale=d ** -0.5, atom_model=m, out_dtype=rgo.F32)
    ref = _ref64(Q, K, V, d ** -0.5)
    # the probabilities are narrowed to bf16 before the second product: 2^-9 relative per term
    assert np.max(np.abs(out - ref)) <= 2.0 ** -8 * np.max(np.abs(_f(V))) + 1e-6


def test_uniform_keys_and_single_key_closed_forms():
    d = 32
    q = _bf(np.ones((3, d)))
    # every key identical: all probabilities are exp(0) = 1, the row sum of a block is its width
    # (exact), l = Nk, and O = (sum of Nk copies of v) / Nk = v when Nk * v is exact
    K = _bf(np.tile(np.linspace(-1, 1, d, dtype=np.float32), (256, 1)))
    v = np.arange(d, dtype=np.float32) / 4
    V = _bf(np.tile(v, (256, 1)))
    for w in (16, 64, 128, 256):
        out = rgo.attention(q, K, V, block_n=w, scale=0.25, atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32)
        assert np.array_equal(out, np.tile(v, (3, 1))), w
    # a single key: the output is that key's value row, whatever the score
    out = rgo.attention(q, K[:1], V[:1], block_n=64, scale=3.0, out_dtype=rgo.F32)
    assert np.array_equal(out, np.tile(v, (3, 1)))
    # one key dominates by more than the underflow threshold: its value row exactly
    K2 = _bf(np.zeros((100, d))); K2[37] = _bf(np.full(d, 8.0))
    V2 = _bf(np.random.default_rng(0).standard_normal((100, d)))
    out = rgo.attention(q, K2, V2, block_n=32, scale=1.0, out_dtype=rgo.F32)
    assert np.array_equal(out, np.tile(synth.bf16_bits_to_f32(V2[37]), (3, 1)))


def test_one_block_is_the_plain_definition_and_block_width_is_part_of_the_arithmetic():
    g = np.random.default_rng(5)
    d, Nk = 64, 128
    Q, K, V = _bf(g.standard_normal((6, d))), _bf(g.standard_normal((Nk, d))), _bf(g.standard_normal((Nk, d)))
    scale = np.float32(d ** -0.5)
    one = rgo.attention(Q, K, V, block_n=128, scale=scale, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)
    # spelled out with the pinned pieces: scores by the GEMM oracle, exp, tree sum, narrowing, second GEMM, one division
    S = rgo.gemm(Q, K, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32) * scale
    want = np.empty_like(one)
    for i in range(6):
        mrow = S[i].max()
        p = np.array([rgo.expf(np.float32(x - mrow)) for x in S[i]], np.float32)
        l = rgo.tree_sum(p)
        pv = rgo.gemm(_bf(p)[None, :], np.ascontiguousarray(V.T), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[0]
        want[i] = pv / l
    assert np.array_equal(one, want)
    # two blocks: a rounding at the boundary, so (some) bits move; the values stay close
    two = rgo.attention(Q, K, V, block_n=64, scale=scale, atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)
    assert not np.array_equal(one, two) and np.max(np.abs(one - two)) < 4e-3    # the narrowing to bf16 happens at another scale
    # the recurrence spelled out for two blocks on one row
    i = 2
    m1 = S[i, :64].max(); p1 = np.array([rgo.expf(np.float32(x - m1)) for x in S[i, :64]], np.float32)
    l1 = rgo.tree_sum(p1); o1 = rgo.gemm(_bf(p1)[None, :], np.ascontiguousarray(V[:64].T), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[0]
    m2 = max(m1, S[i, 64:].max()); a = rgo.expf(np.float32(m1 - m2))
    p2 = np.array([rgo.expf(np.float32(x - m2)) for x in S[i, 64:]], np.float32)
    l2 = np.float32(np.float32(a * l1) + rgo.tree_sum(p2))
    o2 = (np.float32(a) * o1).astype(np.float32) + rgo.gemm(_bf(p2)[None, :], np.ascontiguousarray(V[64:].T), atom_model=rgo.EXACT_RN, out_dtype=rgo.F32)[0]
    assert np.array_equal(two[i], (o2.astype(np.float32) / l2).astype(np.float32))


def test_ragged_last_block_and_row_independence():
    g = np.random.default_rng(9)
    d = 32
    Q, K, V = _bf(g.standard_normal((9, d))), _bf(g.standard_normal((150, d))), _bf(g.standard_normal((150, d)))
    full = rgo.attention(Q, K, V, block_n=64, scale=0.2, atom_model=rgo.TCGEN05_BF16_B200)
    # rows are independent: any subset of queries gives the same bits
    assert np.array_equal(rgo.attention(Q[3:5], K, V, block_n=64, scale=0.2, atom_model=rgo.TCGEN05_BF16_B200), full[3:5])
    # absent keys contribute exactly nothing: appending keys whose probabilities underflow changes no bit
    Kx = np.concatenate([K, _bf(np.full((42, d), -100.0) * np.sign(synth.bf16_bits_to_f32(Q[0]))[None, :])])
    far = rgo.attention(Q[:1], Kx, np.concatenate([V, V[:42]]), block_n=64, scale=0.2, atom_model=rgo.TCGEN05_BF16_B200)
    assert np.array_equal(far, full[:1])


def test_base_two_exponential_variant():
    g = np.random.default_rng(12)
    d, Nk = 64, 300
    Q, K, V = _bf(g.standard_normal((5, d))), _bf(g.standard_normal((Nk, d))), _bf(g.standard_normal((Nk, d)))
    scale = d ** -0.5
    e = rgo.attention(Q, K, V, block_n=128, scale=scale, atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32)
    b2 = rgo.attention(Q, K, V, block_n=128, scale=np.float32(scale * np.log2(np.e)), atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32, exp_base=2)
    ref = _ref64(Q, K, V, scale)
    assert not np.array_equal(e, b2)                      # another class of bits
    assert np.max(np.abs(b2 - ref)) <= 2.0 ** -8 * np.max(np.abs(_f(V))) + 1e-6
    # uniform keys: probabilities 2^0 = 1 exactly, so the closed form holds in base two as well
    Ku = _bf(np.tile(np.linspace(-1, 1, d, dtype=np.float32), (256, 1))); v = np.arange(d, dtype=np.float32) / 4
    out = rgo.attention(_bf(np.ones((2, d))), Ku, _bf(np.tile(v, (256, 1))), block_n=64, scale=0.3, out_dtype=rgo.F32, exp_base=2)
    assert np.array_equal(out, np.tile(v, (2, 1)))


def test_causal_masking():
    g = np.random.default_rng(21)
    d, N = 32, 300
    Q, K, V = _bf(g.standard_normal((N, d))), _bf(g.standard_normal((N, d))), _bf(g.standard_normal((N, d)))
    scale = d ** -0.5
    out = rgo.attention(Q, K, V, block_n=64, scale=scale, atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32, causal=True)
    # against double-precision causal softmax attention
    S = (_f(Q) @ _f(K).T) * scale
    S[np.triu_indices(N, 1)] = -np.inf
    P = np.exp(S - S.max(1, keepdims=True)); ref = (P / P.sum(1, keepdims=True)) @ _f(V)
    assert np.max(np.abs(out - ref)) <= 2.0 ** -8 * np.max(np.abs(_f(V))) + 1e-6
    # the first query sees one key: its value row exactly; a row never depends on later keys or values
    assert np.array_equal(out[0], synth.bf16_bits_to_f32(V[0]))
    K2, V2 = K.copy(), V.copy(); K2[200:] = _bf(g.standard_normal((100, d))); V2[200:] = _bf(g.standard_normal((100, d)))
    out2 = rgo.attention(Q, K2, V2, block_n=64, scale=scale, atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32, causal=True)
    assert np.array_equal(out[:200], out2[:200]) and not np.array_equal(out[200:], out2[200:])
    # rows of the first tile equal unmasked attention over their own prefix only when the prefix is a whole
    # number of blocks and nothing above the diagonal is live: row 63 with 64-wide blocks
    pref = rgo.attention(Q[63:64], K[:64], V[:64], block_n=64, scale=scale, atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32)
    assert np.allclose(out[63], pref[0], atol=1e-6)
    # with block_n dividing block_m and exp(0) = 1 exact, a fully masked block is an exact no-op
    # (alpha = 1, every probability 0), so the query tile height moves no bit here
    out256 = rgo.attention(Q, K, V, block_n=64, scale=scale, atom_model=rgo.TCGEN05_BF16_B200, out_dtype=rgo.F32, causal=True, block_m=256)
    assert np.array_equal(out, out256)
