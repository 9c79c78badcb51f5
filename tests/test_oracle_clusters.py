"""Pins of the oracle's semantic prefix clusters (Def. 3: clusters of sessions at a trie-metric
threshold, centroid = most probable member) and of the storage they give (Cor. 3)."""
import numpy as np
import torch

from paper_2604_15356_b200 import synth


def _sessions(S=24, n=120, seed=5, V=64):
    table = synth.markov_table(V, 6.0, seed, max_states=32)
    tokens, keys, leaf, plen = synth.trie_sessions(table, S, n, seed + 1, 8, 30)
    # log-probabilities that are a function of the token prefix, as a model's are
    u = synth.hashed_normal(keys, 0, 1, seed + 2)[..., 0]
    logp2 = -(0.2 + 2.5 * torch.sigmoid(u)).to(torch.float32)
    g = torch.Generator().manual_seed(seed + 3)
    lens = torch.randint(n // 2, n + 1, (S,), generator=g, dtype=torch.int32)
    return tokens.numpy(), lens.numpy(), logp2.numpy()


def _cut_partition(tokens, lens, logp2, delta):
    """Independent construction: cut every session's path at the first prefix whose cost reaches
    delta; two sessions share a cluster iff they share that prefix (the cut of the trie at cost delta)."""
    keys = []
    for s in range(tokens.shape[0]):
        cost = np.cumsum(-logp2[s, :lens[s]].astype(np.float64))
        hit = np.nonzero(cost >= delta)[0]
        keys.append(("cut",) + tuple(tokens[s, :hit[0] + 1].tolist()) if len(hit) else ("alone", s))
    first = {}
    return np.array([first.setdefault(k, s) for s, k in enumerate(keys)], np.int32)


def test_clusters_are_the_cut_of_the_trie(orc):
    tokens, lens, logp2 = _sessions()
    lcp, dT, _, _ = orc.prefix_dedup(tokens, lens, logp2)
    seen = set()
    for delta in (0.0, 3.3, 17.7, 41.3, 77.7, 130.1, 1e9):
        cl, ce, be = orc.prefix_clusters(lcp, dT, delta)
        assert np.array_equal(cl, _cut_partition(tokens, lens, logp2, delta)), delta
        seen.add(len(set(cl.tolist())))
        # an equivalence: members of one cluster are pairwise within the threshold, others are not
        for a in range(len(cl)):
            for b in range(len(cl)):
                if a != b:
                    assert (cl[a] == cl[b]) == (dT[a, b] >= delta)
        # centroid: the most probable member (Def. 3), the same for the whole cluster
        for a in range(len(cl)):
            members = np.nonzero(cl == cl[a])[0]
            total = np.array([-logp2[m, :lens[m]].astype(np.float64).sum() for m in members])
            assert ce[a] == members[np.argmin(total)]
            assert be[a] == (0 if ce[a] == a else lcp[a, ce[a]])
    assert 1 in seen and len(cl) in seen and len(seen) >= 4       # one cluster ... all singletons
    # refinement: a larger threshold only splits clusters
    prev = None
    for delta in (0.0, 10.0, 40.0, 90.0, 200.0):
        cl, _, _ = orc.prefix_clusters(lcp, dT, delta)
        if prev is not None:
            for a in range(len(cl)):
                for b in range(len(cl)):
                    assert not (cl[a] == cl[b]) or prev[a] == prev[b]
        prev = cl


def test_literal_inequality_is_not_transitive(orc):
    """Why the threshold is read as d_T >= delta: with '<=' sessions a, b that share a long prefix and
    c that shares a short one give a ~ c, c ~ b but not a ~ b."""
    tokens = np.array([[1, 2, 3, 4, 5, 6], [1, 2, 3, 4, 5, 7], [1, 9, 9, 9, 9, 9]], np.int32)
    lens = np.array([6, 6, 6], np.int32)
    logp2 = np.full((3, 6), -2.0, np.float32)
    lcp, dT, _, _ = orc.prefix_dedup(tokens, lens, logp2)
    assert dT[0, 2] <= 3 and dT[2, 1] <= 3 and not dT[0, 1] <= 3              # literal reading: no partition
    cl, ce, be = orc.prefix_clusters(lcp, dT, 3.0)
    assert cl.tolist() == [0, 0, 2] and ce.tolist() == [0, 0, 2] and be.tolist() == [0, 5, 0]


def test_storage_of_a_clustering_is_cor3(orc):
    """Cor. 3: relative cost = 1 - f (1 - tail/n) when a fraction f of equal-length sessions sits in a
    cluster (beside its centroid) with mean tail length `tail`."""
    tokens, lens, logp2 = _sessions(S=32, n=100, seed=9)
    lens[:] = 100
    lcp, dT, _, _ = orc.prefix_dedup(tokens, lens, logp2)
    cl, ce, be = orc.prefix_clusters(lcp, dT, 60.0)
    stored = (lens - be).sum()
    dependants = ce != np.arange(len(ce))
    f = dependants.mean()
    assert 0.2 < f < 0.95 and 1 < len(set(cl.tolist())) < len(cl)
    tail = (lens - be)[dependants].mean()
    assert abs(stored / lens.sum() - (1 - f * (1 - tail / 100))) < 1e-12
    # the coder charges exactly those positions (Prop. 2)
    V, d, K = 64, 64, 8
    table = synth.markov_table(V, 6.0, 9, max_states=32)
    T = synth.make_tables(1, 1, V, d, 11)
    tk = torch.from_numpy(tokens)
    kv = synth.make_kv(T, tk, 0.05, 12, keys=synth.prefix_keys(tk))
    logits = synth.position_logits(table, tk)
    cfg = orc.Config(1, 1, d, V, K, 0.02, 0.0, 32, 0)
    enc = orc.encode(cfg, T.numpy(), kv.numpy(), logits.numpy(), None, pos_begin=be.tolist(), pos_end=lens.tolist())
    assert enc["stats"].coded_positions == stored
    # and a dependant's prefix is the centroid's KV (Lemma 1 / Prop. 1(a)): nothing is lost
    for s in np.nonzero(dependants)[0][:6]:
        assert torch.equal(kv[:, :, s, :, :be[s]], kv[:, :, ce[s], :, :be[s]])
