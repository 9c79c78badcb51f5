"""Trie-based prefix index (Sec. 7.3): pins of the brute-force oracle, then the library's host-side
trie against it on random insert / lookup / evict traffic.  No GPU is involved."""
import math
import os

import numpy as np
import pytest

import paper_2604_15356_b200 as plc
from oracle.trie import TrieOracle


def _seqs(rng, count, V=5, lo=0, hi=12):
    out = []
    for _ in range(count):
        n = int(rng.integers(lo, hi + 1))
        tok = rng.integers(0, V, n).astype(np.int32)
        # log2 P(x_j | x_<j) is a property of the prefix (Def. 1): derive it from the prefix itself
        lp = np.array([-(0.2 + (hash(tuple(tok[:j + 1].tolist())) % 2801) / 1000.0) for j in range(n)], np.float32)
        out.append((tok, lp))
    return out


def test_oracle_on_a_hand_made_trie():
    o = TrieOracle()
    lp = [-1.0] * 6
    assert o.insert(10, [1, 2, 3, 4], lp) == 4
    assert o.insert(11, [1, 2, 5], lp) == 3
    assert o.insert(12, [7], lp) == 1
    assert o.best_match([1, 2, 3, 9]) == (10, 3, 3.0)            # deepest stored ancestor: [1,2,3]
    assert o.best_match([1, 2, 9]) == (10, 2, 2.0)               # two candidates: [1,2,3,4] < [1,2,5]
    assert o.best_match([1, 2, 5, 5, 5]) == (11, 3, 3.0)
    assert o.best_match([9, 9]) == (10, 0, 0.0)                   # empty common prefix: d_T = 0
    assert o.best_match([]) == (10, 0, 0.0)
    assert o.n_nodes() == 4 + 1 + 1
    o.evict(10)
    assert o.best_match([1, 2, 3, 9]) == (11, 2, 2.0) and o.n_nodes() == 3 + 1
    o.evict(11); o.evict(12)
    assert o.best_match([1]) == (-1, 0, 0.0) and o.n_nodes() == 0


def test_oracle_pruning_at_epsilon():
    """A node is kept only while P(prefix) >= epsilon (cumulative surprisal <= -log2 epsilon)."""
    o = TrieOracle(epsilon=2.0 ** -5)
    assert o.insert(1, [3, 3, 3, 3, 3, 3, 3], [-2.0] * 7) == 2    # 2, 4 bits kept; 6 > 5 pruned
    assert o.insert(2, [3, 3, 4], [-2.0, -2.0, -1.0]) == 3        # 5 bits: exactly epsilon stays
    assert o.best_match([3, 3, 3, 3]) == (1, 2, 4.0)              # cannot match deeper than what is kept
    assert o.best_match([3, 3, 4, 0]) == (2, 3, 5.0)
    # d_T(s, s) = -log2 P(s) for a stored, unpruned s (Remark after Def. 2)
    p = TrieOracle()
    lp = [-0.5, -1.25, -2.0]
    p.insert(7, [4, 5, 6], lp)
    assert p.best_match([4, 5, 6]) == (7, 3, 3.75)


def test_oracle_lcp_is_the_maximum_over_stored(orc):
    rng = np.random.default_rng(3)
    o = TrieOracle()
    data = _seqs(rng, 40)
    for i, (tok, lp) in enumerate(data):
        o.insert(i, tok, lp)
    for q, _ in _seqs(rng, 200):
        ident, lcp, dT = o.best_match(q)
        ref = max(len(os.path.commonprefix([list(q), list(t)])) for t, _ in data)
        assert lcp == ref and ident >= 0
        assert len(os.path.commonprefix([list(q), list(data[ident][0])])) == ref
        assert abs(dT + float(data[ident][1][:lcp].astype(np.float64).sum())) < 1e-9


@pytest.mark.parametrize("eps", [0.0, 2.0 ** -9])
def test_library_trie_matches_oracle_under_random_traffic(eps):
    plc.build()
    rng = np.random.default_rng(11)
    lib, o = plc.TrieIndex(eps), TrieOracle(eps)
    live, next_id = [], 0
    for step in range(1500):
        r = rng.random()
        if r < 0.45 or not live:
            tok, lp = _seqs(rng, 1, V=4, hi=14)[0]
            assert lib.insert(next_id, tok, lp) == o.insert(next_id, tok, lp)
            live.append(next_id); next_id += 1
        elif r < 0.65:
            ident = live.pop(int(rng.integers(len(live))))
            lib.evict(ident); o.evict(ident)
        q = _seqs(rng, 1, V=4, hi=16)[0][0]
        gi, gl, gd = lib.best_match(q)
        oi, ol, od = o.best_match(q)
        assert (gi, gl) == (oi, ol) and abs(gd - od) <= 1e-5 * max(1.0, od)
        nodes, prefixes = lib.stats()
        assert prefixes == len(live) and nodes == o.n_nodes()
    with pytest.raises(plc.PlcError):
        lib.insert(live[0], [1], [-1.0])                         # id already stored
    with pytest.raises(plc.PlcError):
        lib.evict(10 ** 6)                                        # unknown id
    for ident in live:
        lib.evict(ident)
    assert lib.stats() == (0, 0) and lib.best_match([1, 2])[0] == -1


def test_index_agrees_with_batched_dedup_oracle(orc):
    """Inserting sessions in arrival order and asking for the best match before each insert gives
    the shared_len of the batched prefix dedup (same longest common prefix, Prop. 2)."""
    rng = np.random.default_rng(5)
    S, n = 20, 30
    tokens = rng.integers(0, 3, (S, n)).astype(np.int32)
    tokens[5, :12] = tokens[2, :12]; tokens[9, :20] = tokens[5, :20]
    lens = np.full(S, n, np.int32)
    lp = np.array([[-(0.5 + (hash(tuple(tokens[s, :j + 1].tolist())) % 1501) / 1000.0) for j in range(n)]
                   for s in range(S)], np.float32)
    lcp, dT, parent, shared = orc.prefix_dedup(tokens, lens, lp)
    plc.build()
    t = plc.TrieIndex()
    for s in range(S):
        ident, m, d = t.best_match(tokens[s])
        assert m == shared[s]
        if m > 0:
            assert lcp[s, ident] == m and abs(d - dT[s, ident]) < 1e-4 * max(1.0, d)
        t.insert(s, tokens[s], lp[s])
