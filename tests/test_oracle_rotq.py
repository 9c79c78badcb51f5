"""Pins of the oracle's rotated fixed-rate quantiser (Prop. 3 step 3: a per-vector quantiser applied to
the residual; here sign flips, an orthonormal Hadamard transform and a b-bit scalar quantiser)."""
import numpy as np
import pytest
from scipy.linalg import hadamard


def _vec(d, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal(d) * scale, rng.integers(0, 2, d).astype(np.uint8)


@pytest.mark.parametrize("d", [2, 32, 128, 256])
def test_rotation_is_the_library_hadamard_matrix(orc, d):
    r, neg = _vec(d, d)
    eps = 1.0 - 2.0 * neg
    want = hadamard(d).astype(np.float64) @ (eps * r) / np.sqrt(d)
    np.testing.assert_allclose(orc.rotq_rotate(r, neg), want, rtol=0, atol=1e-12)


def test_rotation_textbook_case_and_invariants(orc):
    y = orc.rotq_rotate(np.array([3.0, 1.0]), np.zeros(2, np.uint8))
    np.testing.assert_allclose(y, [4 / np.sqrt(2), 2 / np.sqrt(2)], atol=1e-15)
    y = orc.rotq_rotate(np.array([3.0, 1.0]), np.array([0, 1], np.uint8))          # second component negated first
    np.testing.assert_allclose(y, [2 / np.sqrt(2), 4 / np.sqrt(2)], atol=1e-15)
    r, neg = _vec(128, 7)
    y = orc.rotq_rotate(r, neg)
    assert abs(np.linalg.norm(y) - np.linalg.norm(r)) < 1e-12                      # orthonormal
    np.testing.assert_allclose(orc.rotq_unrotate(y, neg), r, atol=1e-12)           # inverse
    e = np.zeros(64); e[5] = 1.0                                                   # a spike spreads evenly
    assert np.allclose(np.abs(orc.rotq_rotate(e, np.zeros(64, np.uint8))), 1 / 8)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_quantiser_levels_and_error_bound(orc, bits):
    d, L = 128, 1 << bits
    for seed in range(5):
        r, neg = _vec(d, 100 + seed, scale=0.3)
        mu = np.random.default_rng(seed).standard_normal(d)
        kv = (mu + r).astype(np.float16)
        scale, code = orc.rotq_quantise(kv, mu, neg, bits)
        res = kv.astype(np.float32).astype(np.float64) - mu.astype(np.float32).astype(np.float64)
        y = orc.rotq_rotate(res, neg)
        assert scale == np.float32(np.abs(y.astype(np.float32)).max())
        assert code.min() >= 0 and code.max() <= L - 1
        k = int(np.argmax(np.abs(y)))                                               # the extreme component sits in an end level
        assert code[k] == (L - 1 if y[k] > 0 else 0)
        yq = float(scale) * ((code + 0.5) * 2.0 / L - 1.0)
        assert np.abs(yq - y).max() <= float(scale) / L * (1 + 1e-5)
        # levels are the literal mid-rise cells of [-s, s]
        cell = np.clip(np.floor((y / float(scale) + 1.0) * L / 2), 0, L - 1)
        inner = np.abs((y / float(scale) + 1.0) * L / 2 - np.round((y / float(scale) + 1.0) * L / 2)) > 1e-4
        assert np.array_equal(code[inner], cell[inner].astype(np.int32))
        out = orc.rotq_reconstruct(mu, neg, bits, scale, code)
        err = out.astype(np.float64) - kv.astype(np.float64)
        assert np.linalg.norm(err) <= np.sqrt(d) * float(scale) / L * (1 + 1e-4) + 1e-5    # Prop. 3: error on KV = error on R
        assert np.abs(orc.rotq_rotate(err, neg)).max() <= float(scale) / L * (1 + 1e-4) + 1e-5


def test_zero_residual_and_bad_arguments(orc):
    mu = np.linspace(-1, 1, 64)
    kv = mu.astype(np.float16)
    scale, code = orc.rotq_quantise(kv, kv.astype(np.float64), np.zeros(64, np.uint8), 3)
    assert scale == 0 and np.all(code == 4)
    out = orc.rotq_reconstruct(kv.astype(np.float64), np.zeros(64, np.uint8), 3, scale, code)
    assert np.array_equal(out, kv.astype(np.float32))
    with pytest.raises(ValueError):
        orc.rotq_quantise(kv[:48], mu[:48], np.zeros(48, np.uint8), 3)                 # not a power of two
    with pytest.raises(ValueError):
        orc.rotq_quantise(kv, mu, np.zeros(64, np.uint8), 9)


@pytest.mark.parametrize("d,bits", [(32, 3), (64, 1), (128, 4), (256, 8)])
def test_record_layout(orc, d, bits):
    rng = np.random.default_rng(d + bits)
    code = rng.integers(0, 1 << bits, d).astype(np.int32)
    rec = orc.rotq_pack(code, 1.25, bits)
    assert len(rec) == 4 + d * bits // 8
    assert rec[:4].view(np.float32)[0] == np.float32(1.25)
    scale, back = orc.rotq_unpack(rec, d, bits)
    assert scale == np.float32(1.25) and np.array_equal(back, code)
    # literal reading of the layout: word g*b+p, bit l = bit p of the code of lane l's g-th component
    R, G = d // 8, d // 32
    words = rec[4:].view(np.uint32)
    for g in range(G):
        for p in range(bits):
            for l in (0, 1, 7, 16, 31):
                j = 8 * (l % R) + G * (l // R) + g
                assert (int(words[g * bits + p]) >> l) & 1 == (int(code[j]) >> p) & 1
    one = np.zeros(d, np.int32); one[0] = 1                                          # a single set bit lands in word 0, bit 0
    w = orc.rotq_pack(one, 0.0, bits)[4:].view(np.uint32)
    assert w[0] == 1 and not w[1:].any()
