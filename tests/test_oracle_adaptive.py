"""Pins of the oracle's surprisal-adaptive quantiser (Def. 7): b_i = max(1, floor(b0 h_i / hbar))
bits per component, realised as the step delta * 2^(b0 - b_i)."""
import math

import numpy as np

from paper_2604_15356_b200 import synth


def test_bits_formula(orc):
    b0, hbar = 8, 3.5
    assert orc.adaptive_bits(hbar, b0, hbar, 16) == b0                       # average surprisal -> target depth
    assert orc.adaptive_bits(0.0, b0, hbar, 16) == 1                         # max(1, .)
    assert orc.adaptive_bits(0.1, b0, hbar, 16) == 1
    assert orc.adaptive_bits(2 * hbar, b0, hbar, 16) == 2 * b0
    assert orc.adaptive_bits(2 * hbar, b0, hbar, 4) == b0 + 4                # cap
    assert orc.adaptive_bits(0.99 * hbar, b0, hbar, 16) == 7                 # floor, not round
    assert orc.adaptive_bits(1.126 * hbar, b0, hbar, 16) == 9
    hs = np.linspace(0, 30, 500)
    bs = [orc.adaptive_bits(float(h), b0, hbar, 6) for h in hs]
    assert all(b2 >= b1 for b1, b2 in zip(bs, bs[1:])) and min(bs) == 1 and max(bs) == b0 + 6
    ref = [min(b0 + 6, max(1, math.floor(b0 * float(np.float32(h)) / hbar))) for h in hs]
    assert sum(a != b for a, b in zip(bs, ref)) <= 2                         # only exact-boundary cases may move


def _workload(V=256, n=200, pp=12.0, seed=77):
    table = synth.markov_table(V, pp, seed, max_states=64)
    tokens = synth.sample_tokens(table, 1, n, seed + 1)
    logits = synth.position_logits(table, tokens)
    T = synth.make_tables(1, 1, V, 64, seed + 2)
    kv = synth.make_kv(T, tokens, 0.05, seed + 3)
    return tokens.numpy(), logits.numpy(), T.numpy(), kv.numpy()


def test_average_depth_and_per_position_error_bound(orc):
    tokens, logits, T, kv = _workload()
    _, _, _, _, lp = orc.topk_softmax(logits[0], tokens[0], 16)
    hbar = float(-lp.mean())
    b0, delta = 6, 0.02
    cfg = orc.Config(1, 1, 64, 256, 16, delta, 0.0, 64, 0, b0, 10, hbar)
    enc = orc.encode(cfg, T, kv, logits, tokens, export=True)
    bits = enc["bits"][0]
    ref = np.clip(np.floor(b0 * (-lp).astype(np.float32) / np.float32(hbar)), 1, b0 + 10)
    assert (bits != ref).sum() <= 1
    # floor loses less than one bit, max(1,.) can only add: the mean depth stays just below b0
    assert b0 - 1 < bits.mean() < b0 + 0.5
    assert bits.min() >= 1 and bits.max() > b0 and len(set(bits.tolist())) > 4
    rc, out, _ = orc.decode(cfg, T, logits, enc, kv.shape, tokens=tokens)
    assert rc == 0
    err = np.abs(out[0, 0, 0, 0].astype(np.float64) - kv[0, 0, 0, 0].astype(np.float64)).max(-1)   # per position
    step = delta * 2.0 ** (b0 - bits)
    assert np.all(err <= step / 2 + 1e-3)                                   # Prop. 3 with the position's own step
    # surprising positions are kept more precisely than predictable ones
    assert err[bits >= b0 + 2].max() < err[bits <= b0 - 2].max()
    # decoding without the tokens is refused (the step cannot be recomputed)
    assert orc.decode(cfg, T, logits, enc, kv.shape)[0] == orc.E_INVALID


def test_constant_surprisal_reproduces_the_fixed_step_coder(orc):
    """If every token has the average surprisal, b_i = b0 everywhere and nothing changes."""
    tokens, logits, T, kv = _workload(n=96)
    flat = np.zeros_like(logits)                                            # uniform distribution: h_i = log2 V
    hbar = math.log2(256)
    fixed = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 32, 0)
    adapt = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 32, 0, 7, 4, hbar)
    a = orc.encode(fixed, T, kv, flat, tokens)
    b = orc.encode(adapt, T, kv, flat, tokens)
    assert np.all(b["bits"] == 7)
    assert a["stats"].payload_bytes == b["stats"].payload_bytes
    assert np.array_equal(a["payload"][:int(a["stats"].payload_bytes) + 64], b["payload"][:int(a["stats"].payload_bytes) + 64])


def test_more_bits_cost_more_bytes(orc):
    tokens, logits, T, kv = _workload(n=128)
    hbar = 3.6
    cfg_lo = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 64, 0, 4, 8, hbar)
    cfg_hi = orc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 64, 0, 4, 8, hbar / 2)      # same tokens look twice as surprising
    lo = orc.encode(cfg_lo, T, kv, logits, tokens)["stats"].payload_bytes
    hi = orc.encode(cfg_hi, T, kv, logits, tokens)["stats"].payload_bytes
    assert hi > lo * 1.2
