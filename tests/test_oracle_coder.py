"""Pins of the oracle's entropy-coding side: frequency tables, the interleaved rANS chunk coder and
its code length.  Expected values are closed forms of the discretised Laplace law, code-length
identities, and an independent decoder written here from the format's definition."""
import math

import numpy as np
import pytest

M = 1 << 15


def _laplace_mass(qp):
    """Closed-form P(hi) of the discretised Laplace of std 2^(qp/8): index by zigzag symbol."""
    x = math.sqrt(2.0) / 2 ** (qp / 8)
    p = np.zeros(64)
    p[0] = 1 - math.exp(-x / 2)
    for k in range(1, 32):
        m = 0.5 * (math.exp(-(k - 0.5) * x) - math.exp(-(k + 0.5) * x))
        p[2 * k - 1] = p[2 * k] = m
    p[63] = math.exp(-31.5 * x)
    return p


def test_tables_are_valid_and_close_to_laplace(orc):
    for qp in range(-24, 16):
        f, c = orc.build_table(qp)
        assert f.sum() == M and f.min() >= 1
        assert c[0] == 0 and c[64] == M and np.array_equal(np.diff(c.astype(np.int64)), f)
        mag = f[1:63:2]
        assert np.array_equal(mag, f[2:63:2])                      # symmetric in the sign
        assert np.all(np.diff(mag.astype(np.int64)) <= 0)
        p = _laplace_mass(qp)
        assert abs(p.sum() - 1) < 1e-12
        err = np.abs(f / M - p)
        assert err[1:].max() <= 2 ** -14 + 1e-9                    # floor to >= 1 and truncation
        assert err[0] <= 70 / M                                    # symbol 0 absorbs the normalisation
    with pytest.raises(ValueError):
        orc.build_table(16)


def test_table_constants_closed_form(orc):
    for qp in (-24, -3, 0, 8, 15):
        th, rh = orc.table_constants(qp)
        x = math.sqrt(2.0) / 2 ** (qp / 8)
        assert abs(th - 2 ** 32 * math.exp(-x)) <= 0.5 + 1e-3
        assert abs(rh - 2 ** 32 * math.exp(-x / 2)) <= 0.5 + 1e-3


def _py_decode(data, q, d, orc):
    """Independent decoder written from the format's definition (forward word order)."""
    G, R = d // 32, d // 8
    x = [int.from_bytes(data[4 * l:4 * l + 4].tobytes(), "little") for l in range(32)]
    words = data[128:].view("<u2").astype(np.int64).tolist()
    rp = 0
    out = np.zeros((len(q), d), np.int64)
    for p, qq in enumerate(q):
        s, qp = orc.class_params(int(qq))
        f, c = orc.build_table(qp)
        f = f.astype(np.int64).tolist(); c = c.astype(np.int64).tolist()
        for g in range(G):
            lo = [0] * 32
            for b in range(s):
                plane = words[rp] | (words[rp + 1] << 16); rp += 2
                for l in range(32):
                    lo[l] |= ((plane >> l) & 1) << b
            zzs = []
            for l in range(32):
                slot = x[l] & (M - 1)
                zz = max(i for i in range(64) if c[i] <= slot)
                x[l] = f[zz] * (x[l] >> 15) + slot - c[zz]
                if x[l] < (1 << 16):
                    x[l] = (x[l] << 16) | words[rp]; rp += 1
                zzs.append(zz)
            for l in range(32):
                if zzs[l] == 63:
                    raw = words[rp] | (words[rp + 1] << 16); rp += 2
                    hi = raw - (1 << 32) if raw >= (1 << 31) else raw
                else:
                    hi = (zzs[l] + 1) // 2 if zzs[l] & 1 else -(zzs[l] // 2)
                out[p, 8 * (l % R) + G * (l // R) + g] = hi if s == 0 else (hi << s) + lo[l] - (1 << (s - 1))
    assert rp == len(words) and all(v == 1 << 16 for v in x)
    return out


def _laplace_symbols(rng, P, d, q):
    sc = 2.0 ** (np.asarray(q) / 8.0) / math.sqrt(2.0)
    return np.rint(rng.laplace(0.0, 1.0, (P, d)) * sc[:, None]).astype(np.int32)


def test_rans_roundtrip_and_python_decoder(orc):
    rng = np.random.default_rng(11)
    P, d = 6, 64
    q = np.array([-24, 0, 15, 16, 43, 70], np.int32)
    sym = _laplace_symbols(rng, P, d, q)
    sym[2, 5] = 100000; sym[3, 7] = -77777; sym[0, 0] = -(1 << 30); sym[5, 63] = 1 << 30   # escapes
    data, ideal, nesc = orc.rans_encode_chunk(sym, q)
    assert nesc >= 4
    rc, back = orc.rans_decode_chunk(data, q, d)
    assert rc == 0 and np.array_equal(back, sym)
    assert np.array_equal(_py_decode(data, q, d, orc), sym)


@pytest.mark.parametrize("d,P", [(32, 1), (64, 37), (128, 256), (256, 5)])
def test_rans_roundtrip_random_classes(orc, d, P):
    rng = np.random.default_rng(d + P)
    q = rng.integers(-24, 136, P).astype(np.int32)
    sym = _laplace_symbols(rng, P, d, np.minimum(q, 120))
    data, ideal, nesc = orc.rans_encode_chunk(sym, q)
    rc, back = orc.rans_decode_chunk(data, q, d)
    assert rc == 0 and np.array_equal(back, sym)


def test_rans_degenerate_streams(orc):
    d = 128
    for sym, q in [(np.zeros((40, d), np.int32), np.full(40, -24, np.int32)),                   # all zero
                   (np.full((3, d), 12345678, np.int32), np.full(3, 0, np.int32)),             # all escapes
                   (np.full((3, d), -(1 << 30), np.int32), np.full(3, 135, np.int32)),         # most planes
                   (np.zeros((0, d), np.int32), np.zeros(0, np.int32))]:                       # empty chunk
        data, ideal, nesc = orc.rans_encode_chunk(sym, q)
        rc, back = orc.rans_decode_chunk(data, q, d)
        assert rc == 0 and np.array_equal(back, sym)
    data, _, _ = orc.rans_encode_chunk(np.zeros((0, d), np.int32), np.zeros(0, np.int32))
    assert len(data) == 128                                                                     # states only
    # all-zero symbols in the sharpest class cost almost nothing beyond the flush
    data, ideal, _ = orc.rans_encode_chunk(np.zeros((256, d), np.int32), np.full(256, -24, np.int32))
    assert ideal < 0.01 * 256 * d and len(data) <= 128 + ideal / 8 + 4


def test_code_length_is_sum_of_minus_log2_p(orc):
    """The ideal length is sum -log2 P(symbol) under the tables plus raw bits, and the stream is
    within the state flush of it (32 lanes x 32-bit states, 16 of them information-free)."""
    rng = np.random.default_rng(12)
    P, d = 256, 128
    for qv in (3, 20, 43):
        q = np.full(P, qv, np.int32)
        sym = _laplace_symbols(rng, P, d, q)
        data, ideal, nesc = orc.rans_encode_chunk(sym, q)
        s, qp = orc.class_params(qv)
        f, _ = orc.build_table(qp)
        u = sym.astype(np.int64) + ((1 << (s - 1)) if s else 0)
        hi = u >> s
        zz = np.where(np.abs(hi) > 31, 63, np.where(hi > 0, 2 * hi - 1, -2 * hi))
        ref = np.log2(M / f[zz]).sum() + 32.0 * (zz == 63).sum() + s * P * d
        assert abs(ideal - ref) < 1e-6 * ref
        bits = 8 * len(data)
        assert ideal + 16 * 32 - 1 <= bits <= ideal + 32 * 32 + 0.001 * ideal + 16
        # and the model is a good one for Laplace data: within 3 % of the empirical entropy
        vals, cnt = np.unique(sym, return_counts=True)
        H = -(cnt / cnt.sum() * np.log2(cnt / cnt.sum())).sum() * P * d
        assert ideal < 1.05 * H + 2000


def test_decoder_rejects_damaged_chunks(orc):
    rng = np.random.default_rng(13)
    P, d = 32, 128
    q = np.full(P, 43, np.int32)
    sym = _laplace_symbols(rng, P, d, q)
    data, _, _ = orc.rans_encode_chunk(sym, q)
    for cut in (0, 64, 128, len(data) // 2, len(data) - 2):
        rc, _ = orc.rans_decode_chunk(data[:cut], q, d)
        assert rc == orc.E_CORRUPT
    rc, _ = orc.rans_decode_chunk(np.concatenate([data, np.zeros(2, np.uint8)]), q, d)
    assert rc == orc.E_CORRUPT
    bad = data.copy(); bad[3] = 0; bad[2] = 0                    # a start state below 2^16
    assert orc.rans_decode_chunk(bad, q, d)[0] == orc.E_CORRUPT
    hits = 0
    for i in range(40):
        bad = data.copy(); bad[128 + 7 * i] ^= 0x5A
        rc, back = orc.rans_decode_chunk(bad, q, d)
        hits += (rc == orc.E_CORRUPT) or not np.array_equal(back, sym)
    assert hits == 40
