"""ctypes front end of the CPU oracle (oracle/plc_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg call this;
the CUDA library and its Python binding never do, and nothing here imports them.  The C file is
compiled with gcc on first use (or by ``build()``) into ``oracle/libplc_oracle.so``.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "plc_oracle.c")
_SO = os.path.join(_HERE, "libplc_oracle.so")

OK, E_INVALID, E_CAPACITY, E_CORRUPT = 0, 1, 4, 5
Q_MIN, Q_MAX = -24, 135
PROB_M = 1 << 15
ESC = 63


def build(force=False):
    """Compile the oracle with gcc -O2 (no intrinsics, no threads)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


class Config(C.Structure):
    _fields_ = [("L", C.c_int32), ("H", C.c_int32), ("d", C.c_int32), ("V", C.c_int32), ("K", C.c_int32),
                ("delta", C.c_float), ("sigma_floor", C.c_float), ("chunk_pos", C.c_int32), ("dense", C.c_int32),
                ("adaptive_b0", C.c_int32), ("adaptive_extra", C.c_int32), ("adaptive_hbar", C.c_float),
                ("lin_dm", C.c_int32), ("lin_E", C.c_void_p), ("lin_A", C.c_void_p), ("lin_c", C.c_void_p),
                ("zero_D", C.c_float)]


class KVStrides(C.Structure):
    _fields_ = [("layer", C.c_int64), ("kv", C.c_int64), ("session", C.c_int64), ("head", C.c_int64),
                ("pos", C.c_int64)]


class Stats(C.Structure):
    _fields_ = [("ideal_bits", C.c_double), ("token_bits", C.c_double), ("payload_bytes", C.c_uint64),
                ("n_chunks", C.c_uint64), ("n_escapes", C.c_uint64), ("coded_positions", C.c_uint64),
                ("skipped_vectors", C.c_uint64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.plo_half_to_double.restype = C.c_double
        _lib.plo_half_to_double.argtypes = [C.c_uint16]
        _lib.plo_round_bf16.restype = C.c_double
        _lib.plo_round_bf16.argtypes = [C.c_double]
        _lib.plo_class_from_v.argtypes = [C.c_float]
        _lib.plo_class.argtypes = [C.c_double, C.c_float, C.c_float]
    return _lib


def _p(a, t=C.c_void_p):
    return None if a is None else a.ctypes.data_as(t)


def _h(a):
    """fp16 array -> contiguous uint16 view."""
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    return a.view(np.uint16)


def topk_softmax(logits, tokens, K):
    """logits [N,V] float16, tokens [N] int32 or None -> idx [N,K] i32, w [N,K] f64, lse, zk, logp2 [N] f64."""
    lg = _h(logits)
    N, V = lg.shape
    idx = np.zeros((N, K), np.int32)
    w = np.zeros((N, K), np.float64)
    lse = np.zeros(N, np.float64)
    zk = np.zeros(N, np.float64)
    lp = np.zeros(N, np.float64)
    tk = None if tokens is None else np.ascontiguousarray(tokens, dtype=np.int32)
    rc = lib().plo_topk_softmax(_p(lg), _p(tk), C.c_int64(N), V, K, _p(idx), _p(w), _p(lse), _p(zk), _p(lp))
    if rc:
        raise ValueError(f"plo_topk_softmax rc={rc}")
    return idx, w, lse, zk, lp


def mixture(table, idx, w):
    """table [V,d] float16, idx [K], w [K] -> mu [d] f64, sigma2."""
    tb = _h(table)
    d = tb.shape[1]
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    w = np.ascontiguousarray(w, dtype=np.float64)
    mu = np.zeros(d, np.float64)
    s2 = C.c_double()
    lib().plo_mixture(_p(tb), d, _p(idx), _p(w), len(idx), _p(mu), C.byref(s2))
    return mu, s2.value


def dense_mixture(table, logits_row, lse):
    tb = _h(table)
    V, d = tb.shape
    lg = _h(logits_row)
    mu = np.zeros(d, np.float64)
    s2 = C.c_double()
    lib().plo_dense_mixture(_p(tb), V, d, _p(lg), C.c_double(lse), _p(mu), C.byref(s2))
    return mu, s2.value


def scale_class(sigma2, sigma_floor, delta):
    return lib().plo_class(C.c_double(sigma2), C.c_float(sigma_floor), C.c_float(delta))


def class_from_v(v):
    return lib().plo_class_from_v(C.c_float(v))


def class_params(q):
    s, qp = C.c_int(), C.c_int()
    lib().plo_class_params(int(q), C.byref(s), C.byref(qp))
    return s.value, qp.value


def adaptive_bits(h, b0, hbar, extra):
    """Def. 7: bits per component at surprisal h (bits), capped at b0 + extra."""
    lib().plo_adaptive_bits.argtypes = [C.c_float, C.c_int, C.c_float, C.c_int]
    return lib().plo_adaptive_bits(C.c_float(h), int(b0), C.c_float(hbar), int(extra))


def linear_config(L, H, d, V, K, delta, chunk_pos, E, A, c):
    """Config of the linear-embedding predictor (Sec. 7.1): E [V,dm], A [L,2,H,d,dm], c [L,2,H,d], all float16.
    The arrays are kept alive on the returned object."""
    Eb, Ab, cb = _h(E), _h(A), _h(c)
    cfg = Config(L, H, d, V, K, delta, 0.0, chunk_pos, 2, 0, 0, 0.0, Eb.shape[1], Eb.ctypes.data, Ab.ctypes.data, cb.ctypes.data)
    cfg._keep = (Eb, Ab, cb)
    return cfg


def zero_class(D, step):
    """Largest scale class the zero-rate rule (Thm. 3) skips at target distortion D and this step."""
    lib().plo_zero_class.restype = C.c_int
    return int(lib().plo_zero_class(C.c_double(D), C.c_double(step)))


def q_skip():
    """Class value that marks a position without symbols in rans_encode_chunk / rans_decode_chunk."""
    return int(lib().plo_q_skip())


def expected_embedding(E, logits_row, lse):
    Eb = _h(E); lg = _h(logits_row)
    V, dm = Eb.shape
    out = np.zeros(dm, np.float64)
    lib().plo_expected_embedding(_p(Eb), V, dm, _p(lg), C.c_double(lse), _p(out))
    return out


def linear_apply(A, c, x):
    Ab, cb = _h(A), _h(c)
    d, dm = Ab.shape
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.zeros(d, np.float64)
    lib().plo_linear_apply(_p(Ab), _p(cb), d, dm, _p(x), _p(out))
    return out


def linear_rownorms(E, A, c):
    Eb, Ab, cb = _h(E), _h(A), _h(c)
    V, dm = Eb.shape
    out = np.zeros(V, np.float64)
    lib().plo_linear_rownorms(_p(Eb), _p(Ab), _p(cb), V, Ab.shape[0], dm, _p(out))
    return out


def quantise(kv, mu, delta):
    x = _h(kv)
    mu = np.ascontiguousarray(mu, dtype=np.float64)
    sym = np.zeros(x.shape[0], np.int32)
    lib().plo_quantise(_p(x), _p(mu), x.shape[0], C.c_float(delta), _p(sym))
    return sym


def reconstruct(mu, sym, delta):
    mu = np.ascontiguousarray(mu, dtype=np.float64)
    sym = np.ascontiguousarray(sym, dtype=np.int32)
    out = np.zeros(len(sym), np.float32)
    lib().plo_reconstruct(_p(mu), _p(sym), len(sym), C.c_float(delta), _p(out))
    return out


def table_constants(qp):
    th, rh = C.c_uint32(), C.c_uint32()
    rc = lib().plo_table_constants(int(qp), C.byref(th), C.byref(rh))
    if rc:
        raise ValueError("bad table id")
    return th.value, rh.value


def build_table(qp):
    f = np.zeros(64, np.uint32)
    c = np.zeros(65, np.uint32)
    rc = lib().plo_build_table(int(qp), _p(f), _p(c))
    if rc:
        raise ValueError("bad table id")
    return f, c


def rans_encode_chunk(sym, q, cap=None):
    """sym [P,d] int32, q [P] int32 -> (bytes ndarray u8, ideal_bits, n_escapes)."""
    sym = np.ascontiguousarray(sym, dtype=np.int32)
    q = np.ascontiguousarray(q, dtype=np.int32)
    P, d = sym.shape
    if cap is None:
        cap = 128 + 8 * P * d + 64
    out = np.zeros(cap, np.uint8)
    nb, ideal, nesc = C.c_uint64(), C.c_double(), C.c_uint64()
    rc = lib().plo_rans_encode_chunk(_p(sym), _p(q), P, d, _p(out), C.c_uint64(cap), C.byref(nb), C.byref(ideal),
                                     C.byref(nesc))
    if rc == E_CAPACITY:
        raise OverflowError(nb.value)
    if rc:
        raise ValueError(f"plo_rans_encode_chunk rc={rc}")
    return out[:nb.value].copy(), ideal.value, nesc.value


def rans_decode_chunk(data, q, d):
    """Returns (rc, sym [P,d])."""
    data = np.ascontiguousarray(data, dtype=np.uint8)
    q = np.ascontiguousarray(q, dtype=np.int32)
    P = len(q)
    sym = np.zeros((P, d), np.int32)
    rc = lib().plo_rans_decode_chunk(_p(data), C.c_uint64(len(data)), _p(q), P, d, _p(sym))
    return rc, sym


def prefix_dedup(tokens, lens, logp2):
    """tokens [S,n] i32, lens [S] i32, logp2 [S,n] f32 -> lcp [S,S] i32, dT [S,S] f64, parent, shared_len."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    logp2 = np.ascontiguousarray(logp2, dtype=np.float32)
    S, n = tokens.shape
    lcp = np.zeros((S, S), np.int32)
    dT = np.zeros((S, S), np.float64)
    parent = np.zeros(S, np.int32)
    shared = np.zeros(S, np.int32)
    lib().plo_prefix_dedup(_p(tokens), _p(lens), _p(logp2), S, C.c_int64(n), _p(lcp), _p(dT), _p(parent), _p(shared))
    return lcp, dT, parent, shared


def prefix_clusters(lcp, dT, delta):
    """Def. 3 on the matrices of prefix_dedup -> cluster [S] (smallest member), centroid [S], begin [S]."""
    lcp = np.ascontiguousarray(lcp, dtype=np.int32)
    dT = np.ascontiguousarray(dT, dtype=np.float64)
    S = lcp.shape[0]
    cl, ce, be = (np.zeros(S, np.int32) for _ in range(3))
    lib().plo_prefix_clusters(_p(lcp), _p(dT), S, C.c_double(delta), _p(cl), _p(ce), _p(be))
    return cl, ce, be


def rotq_rotate(r, neg):
    """Sign flips and orthonormal Hadamard transform of one vector (Prop. 3 step 3, rotated quantiser)."""
    r = np.ascontiguousarray(r, dtype=np.float64)
    neg = np.ascontiguousarray(neg, dtype=np.uint8)
    y = np.zeros_like(r)
    lib().plo_rotq_rotate(_p(r), _p(neg), len(r), _p(y))
    return y


def rotq_unrotate(y, neg):
    y = np.ascontiguousarray(y, dtype=np.float64)
    neg = np.ascontiguousarray(neg, dtype=np.uint8)
    r = np.zeros_like(y)
    lib().plo_rotq_unrotate(_p(y), _p(neg), len(y), _p(r))
    return r


def rotq_quantise(kv_vec, mu, neg, bits):
    """kv_vec [d] float16, mu [d] f64 -> (scale float32, codes [d] int32)."""
    kvv = _h(kv_vec)
    mu = np.ascontiguousarray(mu, dtype=np.float64)
    neg = np.ascontiguousarray(neg, dtype=np.uint8)
    d = len(mu)
    code = np.zeros(d, np.int32)
    sc = C.c_float()
    rc = lib().plo_rotq_quantise(_p(kvv), _p(mu), _p(neg), d, int(bits), C.byref(sc), _p(code))
    if rc:
        raise ValueError("rotq_quantise: bad arguments")
    return np.float32(sc.value), code


def rotq_reconstruct(mu, neg, bits, scale, code):
    mu = np.ascontiguousarray(mu, dtype=np.float64)
    neg = np.ascontiguousarray(neg, dtype=np.uint8)
    code = np.ascontiguousarray(code, dtype=np.int32)
    out = np.zeros(len(mu), np.float32)
    rc = lib().plo_rotq_reconstruct(_p(mu), _p(neg), len(mu), int(bits), C.c_float(float(scale)), _p(code), _p(out))
    if rc:
        raise ValueError("rotq_reconstruct: bad arguments")
    return out


def rotq_pack(code, scale, bits):
    code = np.ascontiguousarray(code, dtype=np.int32)
    d = len(code)
    rec = np.zeros(4 + d * bits // 8, np.uint8)
    rc = lib().plo_rotq_pack(_p(code), C.c_float(float(scale)), d, int(bits), _p(rec))
    if rc:
        raise ValueError("rotq_pack: bad arguments")
    return rec


def rotq_unpack(rec, d, bits):
    rec = np.ascontiguousarray(rec, dtype=np.uint8)
    code = np.zeros(d, np.int32)
    sc = C.c_float()
    rc = lib().plo_rotq_unpack(_p(rec), d, int(bits), C.byref(sc), _p(code))
    if rc:
        raise ValueError("rotq_unpack: bad arguments")
    return np.float32(sc.value), code


def _strides(kv):
    """kv laid out [L,2,S,H,n,d] (any permutation of a contiguous array works): element strides."""
    es = kv.itemsize
    st = [s // es for s in kv.strides]
    return KVStrides(st[0], st[1], st[2], st[3], st[4])


def max_chunks_for(n, chunk_pos):
    return (n + chunk_pos - 1) // chunk_pos


def encode(cfg, T, kv, logits, tokens, pos_begin=None, pos_end=None, export=False):
    """Whole-path encode.

    T [L,2,H,V,d] f16; kv a float16 array indexed [L,2,S,H,n,d] (strides free, d contiguous);
    logits [S,n,V] f16; tokens [S,n] i32 or None.  Returns a dict with payload, chunk_offset,
    chunk_bytes ([S,L,2,H,max_chunks]), stats and, with export=True, sym/q/mu ([S,n,L,2,H(,d)]).
    """
    if T is None:                                   # linear-embedding predictor: shapes come from the config
        Tb = None
        L, H, V, d = cfg.L, cfg.H, cfg.V, cfg.d
    else:
        Tb = _h(T)
        L, _, H, V, d = Tb.shape
    assert kv.dtype == np.float16 and kv.strides[-1] == 2
    kvv = kv.view(np.uint16)
    lg = _h(logits)
    S, n, _ = lg.shape
    tk = None if tokens is None else np.ascontiguousarray(tokens, dtype=np.int32)
    pb = None if pos_begin is None else np.ascontiguousarray(pos_begin, dtype=np.int32)
    pe = None if pos_end is None else np.ascontiguousarray(pos_end, dtype=np.int32)
    mc = max_chunks_for(n, cfg.chunk_pos)
    nslots = S * L * 2 * H * mc
    cap = nslots * (128 + 16) + 8 * S * n * L * 2 * H * d + 64   # worst case of the format
    payload = np.zeros(cap, np.uint8)
    off = np.zeros(nslots, np.uint64)
    nby = np.zeros(nslots, np.uint32)
    stats = Stats()
    sym = q = mu = None
    bits = np.zeros((S, n), np.int32) if cfg.adaptive_b0 > 0 else None
    if export:
        sym = np.zeros((S, n, L, 2, H, d), np.int32)
        q = np.zeros((S, n, L, 2, H), np.int32)
        mu = np.zeros((S, n, L, 2, H, d), np.float32)
    st = _strides(kv)
    rc = lib().plo_encode(C.byref(cfg), _p(Tb), C.c_void_p(kvv.ctypes.data), C.byref(st), _p(lg), _p(tk), S, n,
                          _p(pb), _p(pe), mc, _p(payload), C.c_uint64(cap), _p(off), _p(nby), C.byref(stats),
                          _p(sym), _p(q), _p(mu), _p(bits))
    if rc:
        raise ValueError(f"plo_encode rc={rc}")
    shape = (S, L, 2, H, mc)
    return dict(payload=payload, chunk_offset=off.reshape(shape), chunk_bytes=nby.reshape(shape), stats=stats,
                sym=sym, q=q, mu=mu, bits=bits, max_chunks=mc)


def decode(cfg, T, logits, enc, kv_shape, pos_begin=None, pos_end=None, export=False, tokens=None):
    """Whole-path decode of the dict ``encode`` returned.  kv_shape = (L,2,S,H,n,d); returns float32 KV'."""
    Tb = None if T is None else _h(T)
    lg = _h(logits)
    S, n, _ = lg.shape
    pb = None if pos_begin is None else np.ascontiguousarray(pos_begin, dtype=np.int32)
    pe = None if pos_end is None else np.ascontiguousarray(pos_end, dtype=np.int32)
    out = np.zeros(kv_shape, np.float32)
    st = _strides(out)
    L, _, _, H, _, d = kv_shape
    sym = np.zeros((S, n, L, 2, H, d), np.int32) if export else None
    off = np.ascontiguousarray(enc["chunk_offset"]).reshape(-1)
    nby = np.ascontiguousarray(enc["chunk_bytes"]).reshape(-1)
    tk = None if tokens is None else np.ascontiguousarray(tokens, dtype=np.int32)
    rc = lib().plo_decode(C.byref(cfg), _p(Tb), _p(lg), _p(tk), S, n, _p(pb), _p(pe), enc["max_chunks"], _p(enc["payload"]),
                          _p(off), _p(nby), _p(out), C.byref(st), _p(sym))
    return rc, out, sym


# ---------------------------------------------------------------------------------------------
# The same oracle on several host cores.  Streams are independent across heads (nothing couples
# them in the codec), so the whole-path encode is cut along the head axis, every slice is coded by
# the unchanged single-threaded `encode` in a process of its own, and the exports are put back
# together.  Processes are started with "spawn": a fork after the parent has touched CUDA hangs.

def host_cores():
    """Cores this process may run on."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _config_fields(cfg):
    return [getattr(cfg, name) for name, _ in Config._fields_]


def _encode_slice(job):
    fields, T, kv, logits, tokens, pos_begin, pos_end, export, linear = job
    if linear is not None:
        E, A, c = linear
        L, _, H, d, dm = A.shape
        cfg = linear_config(L, H, d, fields[3], fields[4], fields[5], fields[7], E, A, c)
        cfg.zero_D = fields[16]
    else:
        cfg = Config(*fields[:12], 0, None, None, None, fields[16])
        cfg.H = T.shape[2]
    enc = encode(cfg, T, kv, logits, tokens, pos_begin, pos_end, export=export)
    st = enc["stats"]
    stats = {name: getattr(st, name) for name, _ in Stats._fields_}
    return dict(sym=enc["sym"], q=enc["q"], mu=enc["mu"], bits=enc["bits"], stats=stats,
                chunk_bytes=enc["chunk_bytes"])


def encode_parallel(cfg, T, kv, logits, tokens=None, pos_begin=None, pos_end=None, export=False, workers=None, linear=None):
    """`encode` cut along the head axis over `workers` processes (default: the host's cores).
    linear = (E, A, c) for the linear-embedding predictor (then T is None).  Returns the merged
    exports (sym / q / mu as [S,n,L,2,H(,d)]), chunk_bytes [S,L,2,H,max_chunks], a dict of summed
    statistics, and the number of processes used; payload bytes are not kept."""
    import multiprocessing as mp
    H = cfg.H
    workers = max(1, min(H, workers or host_cores()))
    bounds = [(H * k // workers, H * (k + 1) // workers) for k in range(workers)]
    fields = _config_fields(cfg)
    jobs = []
    for lo, hi in bounds:
        Ts = None if T is None else np.ascontiguousarray(T[:, :, lo:hi])
        kvs = np.ascontiguousarray(kv[:, :, :, lo:hi])
        lin = None if linear is None else (linear[0], np.ascontiguousarray(linear[1][:, :, lo:hi]),
                                           np.ascontiguousarray(linear[2][:, :, lo:hi]))
        jobs.append((fields, Ts, kvs, logits, tokens, pos_begin, pos_end, export, lin))
    if workers == 1:
        parts = [_encode_slice(jobs[0])]
    else:
        with mp.get_context("spawn").Pool(workers) as pool:
            parts = pool.map(_encode_slice, jobs)
    out = dict(workers=workers, bits=parts[0]["bits"])
    out["chunk_bytes"] = np.concatenate([p["chunk_bytes"] for p in parts], axis=3)
    if export:
        out["sym"] = np.concatenate([p["sym"] for p in parts], axis=4)
        out["q"] = np.concatenate([p["q"] for p in parts], axis=4)
        out["mu"] = np.concatenate([p["mu"] for p in parts], axis=4)
    stats = {k: sum(p["stats"][k] for p in parts) for k in parts[0]["stats"]}
    stats["token_bits"] = parts[0]["stats"]["token_bits"]          # a property of the positions, not of the heads
    stats["coded_positions"] = parts[0]["stats"]["coded_positions"]
    out["stats"] = stats
    return out


def _roundtrip_slice(job):
    import time
    fields, T, kv, logits, tokens = job
    cfg = Config(*fields[:12], 0, None, None, None, fields[16])
    cfg.H = T.shape[2]
    t0 = time.perf_counter()
    enc = encode(cfg, T, kv, logits, tokens)
    t1 = time.perf_counter()
    rc, out, _ = decode(cfg, T, logits, enc, kv.shape, tokens=tokens if cfg.adaptive_b0 > 0 else None)
    t2 = time.perf_counter()
    st = enc["stats"]
    return dict(rc=rc, encode_s=t1 - t0, decode_s=t2 - t1, payload_bytes=int(st.payload_bytes), ideal_bits=float(st.ideal_bits),
                token_bits=float(st.token_bits), max_err=float(np.abs(out - kv.astype(np.float32)).max()))


def roundtrip_parallel(cfg, T, kv, logits, tokens=None, workers=None):
    """Encode then decode, cut along the head axis over `workers` processes; every process times
    its own two calls.  Returns the slowest process's times (the job's time with one process per
    slice), the summed statistics and the number of processes."""
    import multiprocessing as mp
    H = cfg.H
    workers = max(1, min(H, workers or host_cores()))
    fields = _config_fields(cfg)
    jobs = []
    for k in range(workers):
        lo, hi = H * k // workers, H * (k + 1) // workers
        jobs.append((fields, np.ascontiguousarray(T[:, :, lo:hi]), np.ascontiguousarray(kv[:, :, :, lo:hi]), logits, tokens))
    if workers == 1:
        parts = [_roundtrip_slice(jobs[0])]
    else:
        with mp.get_context("spawn").Pool(workers) as pool:
            parts = pool.map(_roundtrip_slice, jobs)
    return dict(workers=workers, rc=max(p["rc"] for p in parts),
                encode_s=max(p["encode_s"] for p in parts), decode_s=max(p["decode_s"] for p in parts),
                seconds=max(p["encode_s"] + p["decode_s"] for p in parts),
                payload_bytes=sum(p["payload_bytes"] for p in parts), ideal_bits=sum(p["ideal_bits"] for p in parts),
                token_bits=parts[0]["token_bits"], max_err=max(p["max_err"] for p in parts))
