"""Pins of the oracle's linear-embedding predictor (Sec. 7.1): KV^ ~ c + A Ebar with
Ebar = E_{t~P}[E(t)], in the arithmetic of two chained bf16 contractions."""
import numpy as np
import torch

from paper_2604_15356_b200 import synth


def _bf(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).to(torch.float64).numpy()


def _model(V=300, d=64, dm=48, seed=5):
    E, A, c = synth.make_linear_model(1, 1, V, d, dm, seed)
    return E.numpy(), A.numpy(), c.numpy()


def test_expected_embedding_and_apply_against_library_ops(orc):
    E, A, c = _model()
    rng = np.random.default_rng(1)
    lg = (rng.standard_normal(300) * 2).astype(np.float16)
    lse = float(torch.logsumexp(torch.from_numpy(lg.astype(np.float64)), 0))
    ebar = orc.expected_embedding(E, lg, lse)
    p = torch.exp(torch.from_numpy(lg.astype(np.float64)) - lse).to(torch.bfloat16).to(torch.float64).numpy()
    ref = torch.from_numpy(p @ _bf(E)).to(torch.bfloat16).to(torch.float64).numpy()      # exact sum, one rounding
    assert np.array_equal(ebar, ref)
    mu = orc.linear_apply(A[0, 0, 0], c[0, 0, 0], ebar)
    np.testing.assert_allclose(mu, c[0, 0, 0].astype(np.float64) + _bf(A[0, 0, 0]) @ ebar, atol=1e-13)
    # linear in its argument
    x, y = rng.standard_normal(48), rng.standard_normal(48)
    z = np.zeros(48)
    f = lambda v: orc.linear_apply(A[0, 0, 0], c[0, 0, 0], v)
    np.testing.assert_allclose(f(x) + f(y) - f(z), f(x + y), atol=1e-12)


def test_linear_predictor_is_def5_applied_to_a_linear_kv_function(orc):
    """If F(t) = c + A E(t), then sum_t P(t) F(t) = c + A sum_t P(t) E(t) (Def. 5 and Sec. 7.1):
    the two-stage prediction equals the full-vocabulary mixture of the candidate vectors c + A E(v)
    up to the roundings of the chained contraction."""
    E, A, c = _model()
    rng = np.random.default_rng(2)
    lg = (rng.standard_normal(300) * 2.5).astype(np.float16)
    lse = float(torch.logsumexp(torch.from_numpy(lg.astype(np.float64)), 0))
    mu = orc.linear_apply(A[0, 0, 0], c[0, 0, 0], orc.expected_embedding(E, lg, lse))
    p = torch.softmax(torch.from_numpy(lg.astype(np.float64)), 0).numpy()
    Tlin = c[0, 0, 0].astype(np.float64) + _bf(E) @ _bf(A[0, 0, 0]).T                 # [V][d]
    ref = p @ Tlin
    assert np.abs(mu - ref).max() < 2 ** -7 * np.abs(Tlin).max()
    # variance: Var_t[F] = E||F||^2 - ||E F||^2 per component (Thm. 2)
    n2b = orc.linear_rownorms(E, A[0, 0, 0], c[0, 0, 0])
    np.testing.assert_array_equal(n2b, _bf((Tlin ** 2).sum(1) / 64))


def test_point_mass_predicts_the_candidate_vector(orc):
    """Def. 5/6: a point mass on token x predicts F(x) = c + A E(x): zero residual."""
    E, A, c = _model()
    lg = np.full(300, -40.0, np.float16); lg[123] = 40.0
    lse = float(torch.logsumexp(torch.from_numpy(lg.astype(np.float64)), 0))
    ebar = orc.expected_embedding(E, lg, lse)
    assert np.array_equal(ebar, _bf(E[123]))
    mu = orc.linear_apply(A[0, 0, 0], c[0, 0, 0], ebar)
    target = c[0, 0, 0].astype(np.float64) + _bf(A[0, 0, 0]) @ _bf(E[123])
    assert np.array_equal(mu, target)


def test_whole_path_roundtrip_with_the_linear_predictor(orc):
    S, n, L, H, d, V, dm, K, CP, delta = 1, 80, 1, 2, 64, 200, 32, 8, 32, 0.02
    table = synth.markov_table(V, 12.0, 9, max_states=32)
    tokens = synth.sample_tokens(table, S, n, 10)
    logits = synth.position_logits(table, tokens).numpy()
    E, A, c = synth.make_linear_model(L, H, V, d, dm, 11)
    kv = synth.make_kv_linear(E, A, c, tokens, 0.05, 12).numpy()
    cfg = orc.linear_config(L, H, d, V, K, delta, CP, E.numpy(), A.numpy(), c.numpy())
    enc = orc.encode(cfg, None, kv, logits, None, export=True)
    rc, out, sym = orc.decode(cfg, None, logits, enc, kv.shape, export=True)
    assert rc == 0 and np.array_equal(sym, enc["sym"])
    assert np.abs(out - kv.astype(np.float32)).max() <= delta / 2 + 1e-3
    # the prediction carries information: residuals are much smaller than the vectors themselves
    res = enc["sym"].astype(np.float64) * delta
    assert res.std() < 0.9 * kv.astype(np.float64).std()
