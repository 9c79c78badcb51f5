"""Pins of the oracle's zero-rate rule (Thm. 3 / Cor. 6: a position whose residual variance does not
exceed the target distortion D needs no bits; the decoder takes KV' = KV^)."""
import math

import numpy as np
import torch

from paper_2604_15356_b200 import synth


def test_threshold_class(orc):
    # Cor. 6's operating point: D = step^2 / 12 (the noise of a uniform quantiser) -> 4 log2(1/12) - 1/2 = -14.84
    for step in (0.01, 0.02, 0.5, 3.0):
        assert orc.zero_class(step * step / 12.0, step) == -15
    assert orc.zero_class(0.02 ** 2, 0.02) == -1                  # D = step^2: floor(0 - 1/2)
    assert orc.zero_class(0.0, 0.02) < -1000 and orc.zero_class(-1.0, 0.02) < -1000     # off
    # the class comparison is conservative: skipped => sigma^2 <= D; and nothing clearly below D is kept
    rng = np.random.default_rng(5)
    step, D = 0.02, 3.1e-5
    zc = orc.zero_class(D, step)
    for s2 in np.exp(rng.uniform(math.log(D) - 3, math.log(D) + 3, 4000)):
        q = orc.scale_class(float(s2), 0.0, step)
        if q <= zc:
            assert s2 <= D * (1 + 1e-6)
        if s2 <= D * 2.0 ** -0.25 * (1 - 1e-6) and q > -24:
            assert q <= zc
    # halving the step moves the threshold by 8 classes (used by the adaptive step)
    assert orc.zero_class(D, step / 2) == zc + 8 and orc.zero_class(D, step * 4) == zc - 16


def test_skipped_positions_cost_nothing_in_the_chunk_coder(orc):
    rng = np.random.default_rng(6)
    P, d = 40, 64
    sym = rng.integers(-20, 21, (P, d)).astype(np.int32)
    q = rng.integers(-10, 40, P).astype(np.int32)
    skip = rng.random(P) < 0.4
    qs = q.copy(); qs[skip] = orc.q_skip()
    full, _, _ = orc.rans_encode_chunk(sym[~skip], q[~skip])
    part, ideal, _ = orc.rans_encode_chunk(sym, qs)
    assert np.array_equal(full, part)                            # exactly the stream of the kept positions
    rc, back = orc.rans_decode_chunk(part, qs, d)
    assert rc == 0 and np.array_equal(back[~skip], sym[~skip]) and not back[skip].any()
    allskip, ideal0, _ = orc.rans_encode_chunk(sym, np.full(P, orc.q_skip(), np.int32))
    assert len(allskip) == 128 and ideal0 == 0.0                 # the 32 untouched states only
    assert np.array_equal(np.frombuffer(allskip.tobytes(), np.uint32), np.full(32, 1 << 16, np.uint32))


def _peaked_workload(V=128, n=400, d=64, K=16, seed=91):
    """Positions of very different entropy (near-uniform rows up to point masses)."""
    logits = synth.peaked_logits(1, n, V, seed)
    T = synth.make_tables(1, 1, V, d, seed + 1)
    return logits, T, K


def test_distortion_stays_below_D_and_rate_drops(orc):
    """Noise-free KV whose token is drawn from the same (top-K, renormalised) distribution the
    predictor uses: E||KV - KV^||^2 / d = sigma_mix^2 (Thm. 2), so over the skipped positions the mean
    squared error per component stays below D; kept positions keep the step/2 bound."""
    logits, T, K = _peaked_workload()
    n, V, d = logits.shape[1], logits.shape[2], T.shape[-1]
    idx, w, _, _, _ = orc.topk_softmax(logits[0].numpy(), None, K)
    rng = np.random.default_rng(92)
    delta = 0.02
    D = 0.3
    reps, se, cnt, kept_max = 24, 0.0, 0, 0.0
    skipped_any = None
    for r in range(reps):
        u = rng.random(n)
        pick = (np.cumsum(w, 1) < u[:, None]).sum(1).clip(0, K - 1)
        tok = idx[np.arange(n), pick]
        kv = T[:, :, :, torch.from_numpy(tok).long(), :].reshape(1, 2, 1, 1, n, d).contiguous()   # [L][2][S][H][n][d]
        cfg = orc.Config(1, 1, d, V, K, delta, 0.0, 64, 0)
        cfg.zero_D = D
        enc = orc.encode(cfg, T.numpy(), kv.numpy(), logits.numpy(), None, export=True)
        rc, out, _ = orc.decode(cfg, T.numpy(), logits.numpy(), enc, kv.shape)
        assert rc == 0
        q = enc["q"].reshape(n, 2)
        sk = q <= orc.zero_class(D, delta)                        # [n][kv]
        if skipped_any is None:
            skipped_any = sk
            assert 0.1 < sk.mean() < 0.9                          # the workload exercises both branches
            assert enc["stats"].skipped_vectors == sk.sum()
            assert not enc["sym"].reshape(n, 2, d)[sk].any()
        err = out.astype(np.float64)[0, :, 0, 0] - kv.numpy().astype(np.float64)[0, :, 0, 0]      # [kv][n][d]
        err = np.transpose(err, (1, 0, 2))
        assert np.array_equal(out[0, :, 0, 0].transpose(1, 0, 2)[sk], enc["mu"].reshape(n, 2, d)[sk])   # KV' = KV^ exactly
        se += (err[sk] ** 2).sum(); cnt += err[sk].size
        kept_max = max(kept_max, np.abs(err[~sk]).max())
    # what Thm. 2 predicts for exactly these positions: the mean of their mixture variances
    Tn = T.numpy()
    s2 = np.array([[orc.mixture(Tn[0, a, 0], idx[i], w[i])[1] for a in range(2)] for i in range(n)])
    expect = s2[skipped_any].mean()
    assert s2[skipped_any].max() <= D and expect > 0.02 * D      # a real distortion, and below the target
    assert abs(se / cnt - expect) <= 0.1 * expect, (se / cnt, expect)
    assert se / cnt <= D
    assert kept_max <= delta / 2 + 1e-3


def test_rule_off_is_the_plain_coder_and_rule_on_is_smaller(orc):
    logits, T, K = _peaked_workload(seed=95)
    n, V, d = logits.shape[1], logits.shape[2], T.shape[-1]
    g = torch.Generator().manual_seed(96)
    tok = torch.randint(0, V, (1, n), generator=g, dtype=torch.int32)
    kv = synth.make_kv(T, tok, 0.0, 97)
    a = orc.Config(1, 1, d, V, K, 0.02, 0.0, 64, 0)
    b = orc.Config(1, 1, d, V, K, 0.02, 0.0, 64, 0); b.zero_D = 0.0
    c = orc.Config(1, 1, d, V, K, 0.02, 0.0, 64, 0); c.zero_D = 0.02 ** 2 / 12
    ea, eb, ec = (orc.encode(x, T.numpy(), kv.numpy(), logits.numpy(), None) for x in (a, b, c))
    assert np.array_equal(ea["payload"][:ea["stats"].payload_bytes + 64], eb["payload"][:eb["stats"].payload_bytes + 64])
    assert eb["stats"].skipped_vectors == 0 and ec["stats"].skipped_vectors > 0
    assert ec["stats"].payload_bytes < ea["stats"].payload_bytes
    # more tolerated distortion, more skipped positions (monotone)
    last = 0
    for D in (1e-6, 1e-4, 1e-2, 1.0, 100.0):
        x = orc.Config(1, 1, d, V, K, 0.02, 0.0, 64, 0); x.zero_D = D
        sk = orc.encode(x, T.numpy(), kv.numpy(), logits.numpy(), None)["stats"].skipped_vectors
        assert sk >= last
        last = sk
    assert last == 2 * n                                          # D above every variance: nothing is coded
