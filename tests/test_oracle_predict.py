"""Pins of the oracle's prediction side: number formats, top-K softmax, mixture, variance, class,
quantiser.  Every expected value here comes from numpy/torch/scipy library routines, closed forms or
the paper's statements, never from the oracle itself."""
import math

import numpy as np
import pytest
import torch


def test_half_to_double_all_patterns(orc):
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([orc.lib().plo_half_to_double(int(b)) for b in bits])
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin], ref[fin])
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isinf(got), np.isinf(ref))


def test_round_bf16_matches_torch(orc):
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(4000), np.exp(rng.uniform(-40, 10, 4000)),
                        [1.0, 1.00390625, 1.01171875, 0.0, -3.0, 257.0, 258.0]])
    x32 = x.astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([orc.lib().plo_round_bf16(float(v)) for v in x32])
    assert np.array_equal(got, ref)
    # exact ties go to the even 8-bit significand
    assert orc.lib().plo_round_bf16(1.00390625) == 1.0          # 1 + 2^-8  -> 1
    assert orc.lib().plo_round_bf16(1.01171875) == 1.015625     # 1 + 3*2^-8 -> 1 + 2^-6


def _np_topk(lg, K):
    V = lg.shape[0]
    order = np.lexsort((np.arange(V), -lg.astype(np.float64)))
    return order[:K]


@pytest.mark.parametrize("V,K", [(256, 16), (1000, 64), (37, 37), (64, 1)])
def test_topk_softmax_against_library_softmax(orc, V, K):
    rng = np.random.default_rng(V + K)
    N = 12
    lg = (rng.standard_normal((N, V)) * 2.5).astype(np.float16)
    lg[3, :] = np.float16(0.5)                       # all equal: ties resolved by index
    lg[4, ::3] = lg[4, 0]                            # many ties at one value
    tok = rng.integers(0, V, N).astype(np.int32)
    idx, w, lse, zk, lp = orc.topk_softmax(lg, tok, K)
    p = torch.softmax(torch.from_numpy(lg.astype(np.float64)), dim=1).numpy()
    for n in range(N):
        ref = _np_topk(lg[n], K)
        assert np.array_equal(idx[n], ref)
        np.testing.assert_allclose(w[n], p[n, ref] / p[n, ref].sum(), rtol=1e-12)
        assert abs(w[n].sum() - 1) < 1e-12
        assert abs(zk[n] - p[n, ref].sum()) < 1e-12                  # Thm. 4(a): acceptance = top-k mass
        assert abs(lp[n] - math.log2(p[n, tok[n]])) < 1e-9
        assert abs(lse[n] - float(torch.logsumexp(torch.from_numpy(lg[n].astype(np.float64)), 0))) < 1e-12
    if K == V:
        assert np.allclose(zk, 1.0, atol=1e-12)                      # Z_V = 1
        for n in range(N):
            np.testing.assert_allclose(w[n], p[n, idx[n]], rtol=1e-12)   # K = V is the full softmax


def test_topk_tie_order_is_value_then_index(orc):
    lg = np.array([[1.0, 3.0, 3.0, -1.0, 3.0, 2.0, 2.0, 0.0]], np.float16)
    idx, w, *_ = orc.topk_softmax(lg, None, 5)
    assert idx[0].tolist() == [1, 2, 4, 5, 6]
    lg[0, 0] = np.float16(-0.0); lg[0, 7] = np.float16(0.0)          # -0 and +0 are equal logits
    idx, *_ = orc.topk_softmax(lg, None, 8)
    assert idx[0].tolist() == [1, 2, 4, 5, 6, 0, 7, 3]


def test_mixture_point_mass_gives_zero_residual(orc):
    """Def. 5/6: a point mass on the true token predicts its vector exactly; R = 0, variance 0
    (Thm. 4(b): zero at k = 1)."""
    rng = np.random.default_rng(3)
    T = rng.standard_normal((50, 64)).astype(np.float16)
    mu, s2 = orc.mixture(T, [17], [1.0])
    assert np.array_equal(mu, T[17].astype(np.float64)) and s2 == 0.0
    sym = orc.quantise(T[17], mu, 0.02)
    assert not sym.any()
    # sharply peaked logits: top-1 weight -> 1 and the prediction tends to the true row
    lg = np.full((1, 50), -30.0, np.float16); lg[0, 17] = 30.0
    idx, w, lse, zk, lp = orc.topk_softmax(lg, np.array([17], np.int32), 8)
    mu, s2 = orc.mixture(T, idx[0], w[0])
    assert idx[0, 0] == 17 and np.abs(mu - T[17]).max() < 1e-20 and s2 < 1e-20 and abs(lp[0]) < 1e-12


def test_mixture_equals_matmul_and_variance_definition(orc):
    rng = np.random.default_rng(4)
    V, d = 300, 128
    T = rng.standard_normal((V, d)).astype(np.float16)
    lg = (rng.standard_normal((1, V)) * 3).astype(np.float16)
    idx, w, *_ = orc.topk_softmax(lg, None, V)
    mu, s2 = orc.mixture(T, idx[0], w[0])
    p = torch.softmax(torch.from_numpy(lg[0].astype(np.float64)), 0).numpy()
    T64 = T.astype(np.float64)
    np.testing.assert_allclose(mu, p @ T64, rtol=0, atol=1e-13)           # Def. 5 as a matrix product
    var = (p @ (T64 ** 2) - (p @ T64) ** 2).sum() / d                     # Var = E[F^2] - E[F]^2
    assert abs(s2 - var) < 1e-12
    # two equally likely rows: mu is the midpoint, sigma2 = ||a-b||^2 / (4 d)
    mu2, s22 = orc.mixture(T, [5, 9], [0.5, 0.5])
    np.testing.assert_allclose(mu2, (T64[5] + T64[9]) / 2, atol=1e-15)
    assert abs(s22 - ((T64[5] - T64[9]) ** 2).sum() / (4 * d)) < 1e-13
    # linearity in the weights
    a, _ = orc.mixture(T, [1, 2, 3], [0.2, 0.3, 0.5])
    b, _ = orc.mixture(T, [1, 2, 3], [0.6, 0.1, 0.3])
    c, _ = orc.mixture(T, [1, 2, 3], [0.4, 0.2, 0.4])
    np.testing.assert_allclose(c, (a + b) / 2, atol=1e-15)


def test_residual_second_moment_is_mixture_variance(orc):
    """Thm. 2: E||R||^2 = Var_t[F(t)] when t is drawn from the predicting distribution."""
    rng = np.random.default_rng(5)
    V, d, K = 400, 64, 16
    T = rng.standard_normal((V, d)).astype(np.float16)
    lg = (rng.standard_normal((1, V)) * 2).astype(np.float16)
    idx, w, *_ = orc.topk_softmax(lg, None, K)
    mu, s2 = orc.mixture(T, idx[0], w[0])
    draws = rng.choice(idx[0], size=200000, p=w[0])
    R = T[draws].astype(np.float64) - mu
    emp = (R ** 2).sum(1).mean() / d
    assert abs(emp / s2 - 1) < 0.01


def test_dense_mixture_against_torch_bf16(orc):
    rng = np.random.default_rng(6)
    V, d = 500, 64
    T = rng.standard_normal((V, d)).astype(np.float16)
    lg = (rng.standard_normal(V) * 2).astype(np.float16)
    lse = float(torch.logsumexp(torch.from_numpy(lg.astype(np.float64)), 0))
    mu, s2 = orc.dense_mixture(T, lg, lse)
    p = torch.exp(torch.from_numpy(lg.astype(np.float64)) - lse)
    # exp in double, then one rounding to bf16: go through float64 -> bf16 with torch
    pb = p.to(torch.bfloat16).to(torch.float64)
    # torch rounds float64->bf16 directly (single rounding), as the oracle does
    Tb = torch.from_numpy(T.astype(np.float32)).to(torch.bfloat16).to(torch.float64)
    ref = (pb[None, :] @ Tb)[0].numpy()
    np.testing.assert_allclose(mu, ref, atol=1e-13)
    n2 = ((Tb ** 2).sum(1) / d).to(torch.bfloat16).to(torch.float64)
    var = max(0.0, float(pb @ n2) - float((ref ** 2).sum()) / d)
    assert abs(s2 - var) < 1e-12
    # without the bf16 roundings it is Def. 5; the roundings move it by < 2^-8 relative per term
    full = (p[None, :] @ torch.from_numpy(T.astype(np.float64)))[0].numpy()
    assert np.abs(mu - full).max() < 2 ** -7 * np.abs(T.astype(np.float64)).max()


def test_class_is_round_8log2_sigma(orc):
    rng = np.random.default_rng(7)
    v = np.exp(rng.uniform(math.log(1e-3), math.log(1e9), 20000)).astype(np.float32)
    t = 4 * np.log2(v.astype(np.float64))
    safe = np.abs(t - np.floor(t) - 0.5) > 1e-5        # away from the rounding boundary
    got = np.array([orc.class_from_v(float(x)) for x in v])
    ref = np.clip(np.rint(t), orc.Q_MIN, orc.Q_MAX).astype(int)
    assert np.array_equal(got[safe], ref[safe])
    assert np.all(np.diff(got[np.argsort(v)]) >= 0)     # monotone in v
    assert orc.class_from_v(0.0) == orc.Q_MIN and orc.class_from_v(1e-30) == orc.Q_MIN
    assert orc.class_from_v(1.0) == 0 and orc.class_from_v(4.0) == 8 and orc.class_from_v(1e30) == orc.Q_MAX
    # sigma_tot / delta = 40  ->  8 log2 40 = 42.58 -> 43
    assert orc.scale_class(0.8 ** 2, 0.0, 0.02) == 43
    assert orc.scale_class(0.0, 0.05, 0.02) == round(8 * math.log2(2.5))


def test_class_params_keep_the_scale(orc):
    for q in range(orc.Q_MIN, orc.Q_MAX + 1):
        s, qp = orc.class_params(q)
        assert abs(2 ** (qp / 8) * 2 ** s - 2 ** (q / 8)) < 1e-9 * 2 ** (q / 8)
        assert -24 <= qp <= 15 and 0 <= s <= 15
        if s > 0:
            assert 2.0 <= 2 ** (qp / 8) < 4.0
        else:
            assert q < 16


def test_quantise_reconstruct_error_bound_and_idempotence(orc):
    """Prop. 3, 'Correctness': the error of the recovered KV is the quantisation error of R."""
    rng = np.random.default_rng(8)
    d = 128
    for delta in (0.005, 0.02, 0.08):
        kv = (rng.standard_normal(d) * 1.5).astype(np.float16)
        mu = rng.standard_normal(d) * 0.7
        sym = orc.quantise(kv, mu, delta)
        t = (kv.astype(np.float64) - mu) / float(np.float32(delta))
        ref = np.rint(t)                                                       # Def. 6 + uniform quantiser, in double
        moved = sym != ref                                                     # only exact-boundary cases may move
        assert moved.sum() <= 1 and np.abs(sym - ref).max() <= 1
        assert not moved.any() or np.abs(t - np.floor(t) - 0.5)[moved].max() < 1e-3
        out = orc.reconstruct(mu, sym, delta)
        assert np.abs(out.astype(np.float64) - kv.astype(np.float64)).max() <= delta / 2 + 1e-6
        # re-quantising the reconstruction (kept in float64 here) returns the same symbols
        ref2 = np.rint((out.astype(np.float64) - mu.astype(np.float32).astype(np.float64)) / delta)
        assert np.array_equal(ref2, sym)
    # ties to even, decided in binary32
    mu0 = np.zeros(4)
    assert orc.quantise(np.array([0.5, 1.5, 2.5, -0.5], np.float16), mu0, 1.0).tolist() == [0, 2, 2, 0]
