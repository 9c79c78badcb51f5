"""Pins of the oracle's prefix side: longest common prefix, trie metric d_T = -log2 P(s ^ s'),
parents, and the enumeration checks on a 4-symbol vocabulary (all strings of length <= 6)."""
import itertools
import math
import os

import numpy as np


def _chain(rng, V=4):
    P = rng.dirichlet(np.ones(V), size=V)          # P[prev][next], previous token of position 0 is 0
    return P


def _all_strings(V, maxlen):
    out = [()]
    for m in range(1, maxlen + 1):
        out += list(itertools.product(range(V), repeat=m))
    return out


def _prob(P, s):
    p, prev = 1.0, 0
    for t in s:
        p *= P[prev][t]; prev = t
    return p


def test_enumeration_on_four_symbols(orc):
    rng = np.random.default_rng(21)
    P = _chain(rng)
    strings = _all_strings(4, 6)
    assert len(strings) == 5461
    for m in range(7):                                            # the trie's level-m nodes carry total mass 1
        assert abs(sum(_prob(P, s) for s in strings if len(s) == m) - 1) < 1e-12
    S, n = len(strings), 6
    tokens = np.full((S, n), -1, np.int32)
    lens = np.zeros(S, np.int32)
    logp2 = np.zeros((S, n), np.float32)
    for i, s in enumerate(strings):
        lens[i] = len(s); prev = 0
        for j, t in enumerate(s):
            tokens[i, j] = t; logp2[i, j] = math.log2(P[prev][t]); prev = t
    lcp, dT, parent, shared = orc.prefix_dedup(tokens, lens, logp2)
    # literal definition on a sample of pairs (all pairs for the 341 strings of length <= 4)
    idx = [i for i, s in enumerate(strings) if len(s) <= 4]
    pick = rng.integers(0, S, (20000, 2)).tolist() + [(a, b) for a in idx[::3] for b in idx]
    for a, b in pick:
        common = os.path.commonprefix([strings[a], strings[b]])
        assert lcp[a, b] == len(common)
        assert abs(dT[a, b] + math.log2(_prob(P, common))) < 1e-4
    # d_T(s,s) = -log2 P(s); empty common prefix -> 0 (Remark after Def. 2)
    for a in rng.integers(0, S, 300):
        assert abs(dT[a, a] + math.log2(_prob(P, strings[a]))) < 1e-4
    assert np.all(dT[0] == 0) and np.all(lcp[0] == 0)
    assert np.array_equal(lcp, lcp.T)
    # what the definition yields for three sequences: lcp(a,c) >= min(lcp(a,b), lcp(b,c)), so
    # d_T(a,c) >= min(d_T(a,b), d_T(b,c)) when measured along a
    tri = rng.integers(0, S, (50000, 3))
    a, b, c = tri[:, 0], tri[:, 1], tri[:, 2]
    assert np.all(lcp[a, c] >= np.minimum(lcp[a, b], lcp[b, c]))
    # parent = earliest among the earlier sessions with the longest common prefix
    for a in rng.integers(1, S, 300):
        row = lcp[a, :a]
        if row.max() == 0:
            assert parent[a] == -1 and shared[a] == 0
        else:
            assert parent[a] == int(np.argmax(row)) and shared[a] == row.max()
    assert parent[0] == -1 and shared[0] == 0


def test_dedup_parents_handcrafted(orc):
    tok = np.array([[1, 2, 3, 4, 5, 6],
                    [1, 2, 3, 9, 9, 9],
                    [7, 7, 7, 7, 7, 7],
                    [1, 2, 3, 9, 9, 1],
                    [1, 2, 3, 4, 5, 6]], np.int32)
    lens = np.array([6, 6, 6, 6, 4], np.int32)
    lp = -np.ones((5, 6), np.float32)
    lcp, dT, parent, shared = orc.prefix_dedup(tok, lens, lp)
    assert parent.tolist() == [-1, 0, -1, 1, 0] and shared.tolist() == [0, 3, 0, 5, 4]
    assert lcp[4, 0] == 4 and dT[4, 0] == 4.0 and dT[1, 3] == 5.0 and dT[2, 0] == 0.0


def test_token_entropy_bounds_symbol_entropy_by_enumeration(orc):
    """Thm. 1 on the 4-symbol vocabulary: the coded symbols of position i are a function of the
    token prefix, so H(symbols_i | t_<i) <= H(t_i | t_<i), with equality when the map token ->
    symbol vector is one-to-one (distinct table rows)."""
    rng = np.random.default_rng(22)
    P = _chain(rng)
    d = 32
    T = rng.standard_normal((4, d)).astype(np.float16)
    T[3] = T[2]                                                    # two tokens with the same KV vector
    for prev in range(4):
        lg = np.log(P[prev]).astype(np.float16)[None, :]
        idx, w, *_ = orc.topk_softmax(lg, None, 4)
        mu, s2 = orc.mixture(T, idx[0], w[0])
        syms = [tuple(orc.quantise(T[t], mu, 0.02).tolist()) for t in range(4)]
        Ht = -(P[prev] * np.log2(P[prev])).sum()
        mass = {}
        for t in range(4):
            mass[syms[t]] = mass.get(syms[t], 0.0) + P[prev][t]
        Hs = -sum(m * math.log2(m) for m in mass.values())
        assert len(mass) == 3 and Hs < Ht                          # merged rows lose exactly their split
        merged = P[prev][2] + P[prev][3]
        split = -(P[prev][2] * math.log2(P[prev][2] / merged) + P[prev][3] * math.log2(P[prev][3] / merged))
        assert abs((Ht - Hs) - split) < 1e-12
