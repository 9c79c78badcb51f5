"""The oracle's integer decisions against the plain definitions written out in double.

The oracle decides three integers in binary32 (symbol, scale class, adaptive depth), because an
integer decided by floating point has to be decided in one stated precision on both sides of a
codec.  These pins tie each of them back to the plain formula: the two may differ only where the
real-valued argument sits on a rounding boundary to within the binary32 error, by one unit, and on
a bounded fraction of realistic inputs.

  * Def. 6 + uniform quantiser:  sym = rint((KV - KV^) / delta), ties to even;
  * scale class:                 q = clamp(rint(4 log2(sigma_tot^2 / delta^2)), -24, 135)
                                   = clamp(rint(8 log2(sigma_tot / delta)), ...);
  * Def. 7:                      b = min(b0 + extra, max(1, floor(b0 h / hbar))).
"""
import math

import numpy as np
import pytest

from paper_2604_15356_b200 import synth


def _slice(S, n, L, H, d, V, K, pp, alpha, seed, max_states=64):
    table = synth.markov_table(V, pp, seed, alpha=alpha, max_states=max_states)
    tokens = synth.sample_tokens(table, S, n, seed + 1)
    logits = synth.position_logits(table, tokens)
    T = synth.make_tables(L, H, V, d, seed + 2)
    kv = synth.make_kv(T, tokens, 0.05, seed + 3)
    return tokens.numpy(), logits.numpy(), T.numpy(), kv.numpy()


CASES = [
    # the Tiny configuration in full
    dict(S=1, n=512, L=1, H=1, d=64, V=256, K=16, pp=12.0, alpha=0.0, delta=0.02, seed=20260416),
    # a slice with the shapes and logit statistics of the Llama-2-7B configuration
    dict(S=1, n=96, L=1, H=2, d=128, V=32000, K=64, pp=15.0, alpha=1.1, delta=0.02, seed=20260417),
    # fine and coarse steps
    dict(S=1, n=128, L=1, H=1, d=128, V=1024, K=32, pp=4.0, alpha=0.0, delta=0.005, seed=5),
    dict(S=1, n=128, L=1, H=1, d=128, V=1024, K=32, pp=50.0, alpha=0.0, delta=0.08, seed=6),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "V%d_d%d_delta%g" % (c["V"], c["d"], c["delta"]))
def test_symbols_and_classes_follow_the_plain_definitions(orc, case):
    c = case
    tokens, logits, T, kv = _slice(c["S"], c["n"], c["L"], c["H"], c["d"], c["V"], c["K"], c["pp"], c["alpha"], c["seed"])
    delta = float(np.float32(c["delta"]))                      # the step the codec is given (a binary32 number)
    cfg = orc.Config(c["L"], c["H"], c["d"], c["V"], c["K"], c["delta"], 0.0, 64, 0)
    enc = orc.encode(cfg, T, kv, logits, None, export=True)
    S, n, L, H, d, V, K = (c[k] for k in ("S", "n", "L", "H", "d", "V", "K"))
    idx, w, *_ = orc.topk_softmax(logits.reshape(S * n, V), None, K)
    n_sym = n_sym_diff = n_q = n_q_diff = 0
    for s in range(S):
        for i in range(n):
            for l in range(L):
                for a in range(2):
                    for h in range(H):
                        mu, s2 = orc.mixture(T[l, a, h], idx[s * n + i], w[s * n + i])
                        x = kv[l, a, s, h, i].astype(np.float64)
                        # Def. 6 and the uniform quantiser, in double
                        t = (x - mu) / delta
                        ref = np.rint(t)
                        got = enc["sym"][s, i, l, a, h]
                        diff = got != ref
                        n_sym += d
                        n_sym_diff += int(diff.sum())
                        if diff.any():
                            assert np.abs(got - ref)[diff].max() == 1
                            assert np.abs(t - np.floor(t) - 0.5)[diff].max() < 1e-3
                        # scale class, in double
                        qref = -24 if s2 <= 0 else int(min(135, max(-24, np.rint(4 * math.log2(s2 / delta ** 2)))))
                        qgot = int(enc["q"][s, i, l, a, h])
                        n_q += 1
                        if qgot != qref:
                            n_q_diff += 1
                            tq = 4 * math.log2(s2 / delta ** 2)
                            assert abs(qgot - qref) == 1 and abs(tq - math.floor(tq) - 0.5) < 1e-5
                        # the same class said with sigma: round(8 log2(sigma / delta))
                        if s2 > 0:
                            tq8 = 8 * math.log2(math.sqrt(s2) / delta)
                            if abs(tq8 - math.floor(tq8) - 0.5) > 1e-5:
                                assert qgot == int(min(135, max(-24, np.rint(tq8))))
    assert n_sym_diff <= max(1, 1e-4 * n_sym), (n_sym_diff, n_sym)
    assert n_q_diff <= max(1, 1e-4 * n_q), (n_q_diff, n_q)


def test_quantiser_boundary_rate_on_dense_grid(orc):
    """Residuals spread evenly over many steps: the binary32 decision differs from rint((kv - mu) / delta)
    on fewer than 1e-4 of them, always by one and always within 1e-3 of a half-integer."""
    rng = np.random.default_rng(12)
    d = 256
    for delta in (0.005, 0.02, 0.08):
        de = float(np.float32(delta))
        n_diff = n = 0
        for _ in range(400):
            x = (rng.standard_normal(d) * 1.2).astype(np.float16)
            mu = rng.standard_normal(d) * 0.6
            got = orc.quantise(x, mu, delta)
            t = (x.astype(np.float64) - mu) / de
            ref = np.rint(t)
            diff = got != ref
            n += d
            n_diff += int(diff.sum())
            if diff.any():
                assert np.abs(got - ref)[diff].max() == 1
                assert np.abs(t - np.floor(t) - 0.5)[diff].max() < 1e-3
        assert n_diff < 1e-4 * n, (delta, n_diff, n)


def test_class_boundary_rate(orc):
    """round(4 log2 v) decided on exponent + four binary32 thresholds against the double formula, for v
    over the whole range the workloads produce (sigma / delta from 1/8 to 2^16): the two differ only
    within 1e-5 of a rounding boundary, i.e. on a few inputs in a million."""
    rng = np.random.default_rng(13)
    v = np.exp2(rng.uniform(-6.0, 33.0, 400000))
    got = np.array([orc.class_from_v(float(np.float32(x))) for x in v])
    t = 4 * np.log2(np.float32(v).astype(np.float64))
    ref = np.clip(np.rint(t), orc.Q_MIN, orc.Q_MAX).astype(int)
    diff = got != ref
    assert diff.mean() < 1e-4
    if diff.any():
        assert np.abs(got - ref)[diff].max() == 1
        assert np.abs(t - np.floor(t) - 0.5)[diff].max() < 1e-5


def test_adaptive_depth_boundary_rate(orc):
    """Def. 7's floor decided in binary32 against floor(b0 h / hbar) in double, on surprisals drawn from
    a Markov source: equal except within 1e-5 of an integer."""
    tokens, logits, T, kv = _slice(1, 4000, 1, 1, 64, 512, 16, 12.0, 0.0, 91)
    _, _, _, _, lp = orc.topk_softmax(logits[0], tokens[0], 16)
    h = -lp
    hbar = float(np.float32(h.mean()))
    for b0, extra in ((6, 4), (8, 12), (3, 0)):
        got = np.array([orc.adaptive_bits(float(x), b0, hbar, extra) for x in h])
        r = b0 * h.astype(np.float32).astype(np.float64) / hbar
        ref = np.minimum(b0 + extra, np.maximum(1, np.floor(r))).astype(int)
        diff = got != ref
        assert diff.mean() < 1e-3
        if diff.any():
            assert np.abs(got - ref)[diff].max() == 1 and np.abs(r - np.rint(r))[diff].max() < 1e-5
