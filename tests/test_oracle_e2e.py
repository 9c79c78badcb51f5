"""Whole-path pins of the oracle on the Tiny configuration, and calibration of the synthetic source."""
import math
import os

import numpy as np
import torch

from paper_2604_15356_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_numbers.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def tiny(seed=20260416, S=1, n=512, L=1, H=1, d=64, V=256, K=16, pp=12.0, sigma=0.05):
    table = synth.markov_table(V, pp, seed)
    tokens = synth.sample_tokens(table, S, n, seed + 1)
    logits = synth.position_logits(table, tokens)
    T = synth.make_tables(L, H, V, d, seed + 2)
    kv = synth.make_kv(T, tokens, sigma, seed + 3)
    return table, tokens.numpy(), logits.numpy(), T.numpy(), kv.numpy()


def test_source_perplexity_matches_the_papers_bits_per_token(orc):
    """Cor. 1: the per-token bound is log2(perplexity): 3.3 bits at 10, 4.3 bits at 20."""
    g = _gold()
    assert abs(math.log2(10) - g["bits_per_token_pp10"]) < 0.05
    assert abs(math.log2(20) - g["bits_per_token_pp20"]) < 0.05
    assert abs(2 * 80 * 64 * 128 * 3 - g["turboquant_bits_token"]) < 0.005e6
    assert abs(2 * 80 * 64 * 128 * 16 - g["fp16_bits_token"]) < 0.005e7
    assert abs(g["turboquant_bits_token"] / g["bits_per_token_pp20"] / g["ratio_vs_turboquant"] - 1) < 0.01
    for pp in (10.0, 20.0):
        table = synth.markov_table(512, pp, 5)
        tokens = synth.sample_tokens(table, 4, 3000, 6)
        logits = synth.position_logits(table, tokens)
        _, _, _, _, lp = orc.topk_softmax(logits.numpy().reshape(-1, 512), tokens.numpy().reshape(-1), 8)
        assert abs(-lp.mean() / math.log2(pp) - 1) < 0.05


def test_tiny_roundtrip_bounds_and_rate(orc):
    table, tokens, logits, T, kv = tiny()
    cfg = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 256, 0)
    enc = orc.encode(cfg, T, kv, logits, tokens, export=True)
    st = enc["stats"]
    assert st.n_chunks == 4 and st.coded_positions == 512
    rc, out, sym = orc.decode(cfg, T, logits, enc, kv.shape, export=True)
    assert rc == 0 and np.array_equal(sym, enc["sym"])
    assert np.abs(out.astype(np.float64) - kv.astype(np.float64)).max() <= 0.02 / 2 + 1e-3   # Prop. 3
    # the stream is within the per-chunk state flush of the model's code length
    bits = 8 * st.payload_bytes
    assert st.ideal_bits + 512 * st.n_chunks - 4 <= bits <= st.ideal_bits * 1.001 + 1024 * st.n_chunks + 64
    assert st.payload_bytes == int(enc["chunk_bytes"].sum())
    # token-level bound for context: mean surprisal ~ log2(12)
    assert abs(st.token_bits / 512 / math.log2(12) - 1) < 0.15
    # chunks start on 16-byte boundaries and do not overlap
    off = enc["chunk_offset"].reshape(-1).astype(np.int64); nb = enc["chunk_bytes"].reshape(-1).astype(np.int64)
    assert np.all(off % 16 == 0) and np.all(off[1:] >= off[:-1] + nb[:-1])


def test_shared_prefix_costs_zero_bits_and_tail_is_coded(orc):
    """Prop. 2: positions up to the divergence are stored by pointer, the tail is delta coded."""
    table, tokens, logits, T, kv = tiny(S=2, n=96)
    cfg = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 32, 0)
    full = orc.encode(cfg, T, kv, logits, tokens)
    part = orc.encode(cfg, T, kv, logits, tokens, pos_begin=[0, 96], pos_end=[96, 96])
    assert part["chunk_bytes"][1].sum() == 0 and np.array_equal(part["chunk_bytes"][0], full["chunk_bytes"][0])
    tail = orc.encode(cfg, T, kv, logits, tokens, pos_begin=[0, 40], pos_end=[96, 96], export=True)
    assert tail["stats"].coded_positions == 96 + 56
    rc, out, _ = orc.decode(cfg, T, logits, tail, kv.shape, pos_begin=[0, 40], pos_end=[96, 96])
    assert rc == 0
    assert not out[:, :, 1, :, :40].any()                                             # prefix not written
    assert np.abs(out[:, :, 1, :, 40:] - kv[:, :, 1, :, 40:].astype(np.float32)).max() <= 0.011
    # relative storage of Cor. 3 with f = 1/2 of the sessions in the cluster and tail 56 of 96
    rel = tail["stats"].coded_positions / (2 * 96)
    assert abs(rel - (1 - 0.5 * (1 - 56 / 96))) < 1e-12


def test_noise_free_point_mass_codes_to_nothing(orc):
    """Def. 6 with a point-mass prediction: every residual is zero and the chunk is its flush."""
    table, tokens, logits, T, kv = tiny(n=64, sigma=0.0)
    lg = np.full(logits.shape, -40.0, np.float16)
    np.put_along_axis(lg[0], tokens[0][:, None].astype(np.int64), np.float16(40.0), axis=1)
    cfg = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 64, 0)
    enc = orc.encode(cfg, T, kv, lg, tokens, export=True)
    assert not enc["sym"].any() and np.all(enc["q"] == orc.Q_MIN)
    assert enc["stats"].payload_bytes <= 2 * (128 + 8) and enc["stats"].token_bits < 1e-9


def test_dense_variant_roundtrip(orc):
    table, tokens, logits, T, kv = tiny(n=48, V=96, K=96)
    cfg = orc.Config(1, 1, 64, 96, 96, 0.02, 0.0, 16, 1)
    enc = orc.encode(cfg, T, kv, logits, tokens, export=True)
    rc, out, sym = orc.decode(cfg, T, logits, enc, kv.shape, export=True)
    assert rc == 0 and np.array_equal(sym, enc["sym"])
    assert np.abs(out - kv.astype(np.float32)).max() <= 0.011
    # the bf16 contraction stays close to the exact K = V mixture
    cfg2 = orc.Config(1, 1, 64, 96, 96, 0.02, 0.0, 16, 0)
    enc2 = orc.encode(cfg2, T, kv, logits, tokens, export=True)
    assert np.abs(enc["mu"] - enc2["mu"]).max() < 0.05


def test_synth_is_deterministic_and_prefix_keyed():
    table = synth.markov_table(128, 12.0, 3, max_states=32)
    tok, keys, leaf, plen = synth.trie_sessions(table, 6, 200, 9, 10, 40)
    tok2, keys2, _, _ = synth.trie_sessions(table, 6, 200, 9, 10, 40)
    assert torch.equal(tok, tok2) and torch.equal(keys, keys2)
    T = synth.make_tables(1, 2, 128, 32, 4)
    kv = synth.make_kv(T, tok, 0.05, 5, keys=keys)
    for a in range(6):
        for b in range(a):
            m = int((tok[a] == tok[b]).to(torch.int8).cumprod(0).sum())
            same_leaf = int(leaf[a]) == int(leaf[b])
            assert m >= min(int(plen[a]), int(plen[b])) if same_leaf else True
            k = int((keys[a] == keys[b]).to(torch.int8).cumprod(0).sum())
            assert torch.equal(kv[:, :, a, :, :k], kv[:, :, b, :, :k])          # Lemma 1 on the shared prefix
    z = synth.hashed_normal(torch.arange(200000), 3, 8, 1).double()
    assert abs(float(z.mean())) < 0.01 and abs(float(z.std()) - 1) < 0.01
