"""Pins for the dependence trees (Sec. 3.1, Sec. 5.1): printed examples, brute force over every
tree shape on small n, a top-down restatement on large n, exact integer sums."""
import os

import numpy as np
import pytest

from oracle import rgo

GOLD = os.path.join(os.path.dirname(__file__), "golden")
L = np.float32(1024.0)
r = np.float32(2.0 ** -15)


def _gold(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        rows.append((int(k), r if v == "r" else np.float32(0.0)))
    return rows


def test_printed_strided_grouping():
    # (a0+a2+a4+a6)+(a1+a3+a5+a7): each group a chain, then one add
    for ridx, want in _gold("strided_grouping_8.txt"):
        v = np.zeros(8, np.float32)
        v[0], v[6], v[ridx] = L, -L, r
        g0 = rgo.tree_sum(v[0::2], rgo.TREE_LEFT)
        g1 = rgo.tree_sum(v[1::2], rgo.TREE_LEFT)
        assert rgo.add_f32(g0, g1) == want


def test_printed_contiguous_grouping_as_left_chains():
    for p, want in _gold("contiguous_grouping_8.txt"):
        v = np.zeros(8, np.float32)
        v[0], v[p], v[p + 1] = r, L, -L
        got = rgo.add_f32(rgo.tree_sum(v[:4], rgo.TREE_LEFT), rgo.tree_sum(v[4:], rgo.TREE_LEFT))
        assert got == want


# ---- brute force: every binary tree over n labelled leaves, up to swapping an add's inputs
def _all_trees(leaves):
    leaves = tuple(leaves)
    if len(leaves) == 1:
        yield leaves[0]
        return
    first, rest = leaves[0], leaves[1:]
    n = len(rest)
    for mask in range(1 << n):
        left = (first,) + tuple(rest[i] for i in range(n) if mask >> i & 1)
        right = tuple(rest[i] for i in range(n) if not mask >> i & 1)
        if not right:
            continue
        for a in _all_trees(left):
            for b in _all_trees(right):
                yield (a, b)


def _eval(t, v):
    if isinstance(t, tuple):
        return np.float32(_eval(t[0], v) + _eval(t[1], v))
    return v[t]


def _probes(n):
    out = []
    for i in range(n):
        for j in range(n):
            for k in range(n):
                if len({i, j, k}) == 3:
                    v = [np.float32(0.0)] * n
                    v[i], v[j], v[k] = r, L, -L
                    out.append(v)
    return out


def _intended(n, tree):
    if tree == rgo.TREE_LEFT:
        t = 0
        for i in range(1, n):
            t = (t, i)
        return t
    nodes = list(range(n))
    while len(nodes) > 1:
        nxt = [(nodes[2 * t], nodes[2 * t + 1]) for t in range(len(nodes) // 2)]
        if len(nodes) & 1:
            nxt.append(nodes[-1])
        nodes = nxt
    return nodes[0]


@pytest.mark.parametrize("n", [2, 3, 4, 5, 6])
@pytest.mark.parametrize("tree", [rgo.TREE_LEFT, rgo.TREE_BALANCED])
def test_tree_is_the_intended_one_among_all_shapes(n, tree):
    probes = _probes(n) if n >= 3 else [[r, L], [L, r]]
    oracle_sig = tuple(float(rgo.tree_sum(np.array(v, np.float32), tree)) for v in probes)
    trees = list(_all_trees(range(n)))
    dfact = 1
    for k in range(2 * n - 3, 0, -2):
        dfact *= k
    assert len(trees) == dfact  # (2n-3)!! classes
    sigs = {}
    for t in trees:
        sigs.setdefault(tuple(float(_eval(t, v)) for v in probes), []).append(t)
    if n >= 3:
        assert len(sigs) == len(trees)  # the probes separate every class
    assert sigs[oracle_sig] == [_canon(_intended(n, tree), trees)]


def _leafset(t):
    return frozenset([t]) if not isinstance(t, tuple) else _leafset(t[0]) | _leafset(t[1])


def _key(t):
    if not isinstance(t, tuple):
        return t
    return frozenset([_key(t[0]), _key(t[1])])


def _canon(t, trees):
    k = _key(t)
    m = [u for u in trees if _key(u) == k]
    assert len(m) == 1
    return m[0]


# ---- large n: top-down restatement (split at the largest power of two below n)
def _topdown(v):
    n = len(v)
    if n == 1:
        return v[0]
    p = 1 << ((n - 1).bit_length() - 1)
    return np.float32(_topdown(v[:p]) + _topdown(v[p:]))


@pytest.mark.parametrize("n", [1, 2, 3, 5, 6, 7, 11, 100, 1000, 4096, 4097, 5000, 32768])
def test_balanced_tree_against_topdown(n):
    g = np.random.default_rng(n)
    v = (g.standard_normal(n) * np.exp2(g.integers(-12, 12, n))).astype(np.float32)
    assert rgo.tree_sum(v, rgo.TREE_BALANCED) == _topdown(list(v))


@pytest.mark.parametrize("n", [4096, 32768, 3000])
def test_random_probe_triples_on_large_trees(n):
    g = np.random.default_rng(7)
    for _ in range(200):
        i, j, k = g.choice(n, 3, replace=False)
        v = np.zeros(n, np.float32)
        v[i], v[j], v[k] = r, L, -L
        # r survives iff it is outside the smallest aligned block holding both L's
        blk = 1
        while j // blk != k // blk:
            blk *= 2
        want = np.float32(0.0) if i // blk == j // blk else r
        assert rgo.tree_sum(v, rgo.TREE_BALANCED) == want
        # chain: r survives iff it comes after both
        assert rgo.tree_sum(v, rgo.TREE_LEFT) == (r if i > max(j, k) else np.float32(0.0))


def test_integer_sums_exact():
    g = np.random.default_rng(3)
    for n in (1, 17, 4096, 32768, 33333):
        v = g.integers(-64, 65, n)
        for tree in (rgo.TREE_LEFT, rgo.TREE_BALANCED):
            assert rgo.tree_sum(v.astype(np.float32), tree) == np.float32(v.sum())
            assert rgo.tree_sum(np.ones(n, np.float32), tree) == np.float32(n)


def test_balanced_differs_from_chain_on_cancellation():
    v = np.zeros(8, np.float32)
    v[0], v[2], v[3] = r, L, -L
    assert rgo.tree_sum(v, rgo.TREE_BALANCED) == r      # (r+0) + (L-L)
    assert rgo.tree_sum(v, rgo.TREE_LEFT) == np.float32(0.0)
