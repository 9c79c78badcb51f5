"""Predictive delta coding of the KV cache for B200 (sm_100a): thin Python binding of libplc.so.

The binding only marshals arguments (torch device tensors -> raw pointers, the current torch stream
-> cudaStream_t).  Every step of the path runs in the library's CUDA kernels; there is no CPU or
PyTorch fallback: if the shared library is missing, ``lib()`` raises.
"""
import ctypes as C
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INC = os.path.join(os.path.dirname(_HERE), "include")
_SO = os.path.join(_HERE, "libplc.so")
_SOURCES = ["plc_api.cu", "plc_topk.cu", "plc_prefix.cu", "plc_codec.cu", "plc_dense.cu", "plc_static.cu", "plc_trie.cu"]

OK, E_INVALID, E_SHAPE, E_ALIGN, E_CAPACITY, E_CORRUPT, E_STATE, E_CUDA = range(8)
PRED_TOPK, PRED_DENSE, PRED_LINEAR = 0, 1, 2
OUT_F32, OUT_F16 = 0, 1

EXPORTS = ["plc_create", "plc_destroy", "plc_reserve", "plc_topk_softmax", "plc_prefix_dedup", "plc_encode",
           "plc_decode", "plc_append_step", "plc_append_flush", "plc_append_sizes", "plc_sync_status",
           "plc_get_stats", "plc_table_constants", "plc_build_table", "plc_set_profiling", "plc_last_kernel_ms",
           "plc_launch_count", "plc_rans_encode_static", "plc_encode_adaptive", "plc_decode_adaptive",
           "plc_trie_create", "plc_trie_destroy", "plc_trie_insert", "plc_trie_best_match", "plc_trie_evict",
           "plc_trie_stats", "plc_create_linear", "plc_prefix_clusters", "plc_rotq_record_bytes", "plc_encode_rotq",
           "plc_decode_rotq", "plc_poll_status", "plc_last_schedule", "plc_kernel_ms"]


def sources():
    return [os.path.join(_CSRC, s) for s in _SOURCES if os.path.exists(os.path.join(_CSRC, s))]


def build(force=False, verbose=False):
    """Compile libplc.so for sm_100a with nvcc (in-tree)."""
    srcs = sources()
    deps = srcs + [os.path.join(_CSRC, "plc_common.cuh"), os.path.join(_INC, "plc.h")]
    if not force and os.path.exists(_SO) and all(os.path.getmtime(_SO) >= os.path.getmtime(d) for d in deps):
        return _SO
    cmd = ["nvcc", "-t", "0", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-shared", "-I" + _INC, "-o", _SO] + srcs
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return _SO


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("vocab", C.c_int32),
                ("top_k", C.c_int32), ("delta", C.c_float), ("sigma_floor", C.c_float), ("chunk_pos", C.c_int32),
                ("variant", C.c_int32), ("out_dtype", C.c_int32), ("adaptive_b0", C.c_int32),
                ("adaptive_extra", C.c_int32), ("adaptive_hbar", C.c_float), ("zero_rate_D", C.c_float)]


class KVView(C.Structure):
    _fields_ = [("base_dev", C.c_void_p), ("stride_layer", C.c_int64), ("stride_kv", C.c_int64),
                ("stride_session", C.c_int64), ("stride_head", C.c_int64), ("stride_pos", C.c_int64)]


class Streams(C.Structure):
    _fields_ = [("payload_dev", C.c_void_p), ("payload_capacity", C.c_uint64), ("chunk_offset_dev", C.c_void_p),
                ("chunk_bytes_dev", C.c_void_p), ("total_bytes_dev", C.c_void_p), ("max_chunks", C.c_int32)]


class DebugBuffers(C.Structure):
    _fields_ = [("sym_dev", C.c_void_p), ("q_dev", C.c_void_p), ("mu_dev", C.c_void_p), ("bits_dev", C.c_void_p),
                ("count_ideal_bits", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("payload_bytes", C.c_uint64), ("n_chunks", C.c_uint64), ("n_escapes", C.c_uint64),
                ("coded_vectors", C.c_uint64), ("skipped_vectors", C.c_uint64), ("ideal_bits", C.c_double)]


class RotqParams(C.Structure):
    _fields_ = [("bits", C.c_int32), ("sign_bits", C.c_uint32 * 8)]


class LinearModel(C.Structure):
    _fields_ = [("E_dev", C.c_void_p), ("A_dev", C.c_void_p), ("c_dev", C.c_void_p), ("d_model", C.c_int32)]


class SessionBatch(C.Structure):
    _fields_ = [("B", C.c_int32), ("steps", C.c_int32), ("open_sym_dev", C.c_void_p), ("open_q_dev", C.c_void_p),
                ("streams", Streams)]


_lib = None


def lib():
    """Loads libplc.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise RuntimeError(f"{_SO} not found: run paper_2604_15356_b200.build() (nvcc, sm_100a) first")
        _lib = C.CDLL(_SO)
        _lib.plc_launch_count.restype = C.c_uint64
    return _lib


class PlcError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: plc_status {code}")
        self.code = code


def _check(rc, where):
    if rc != OK:
        raise PlcError(rc, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def kv_view(kv):
    """torch tensor indexed [L][2][S][H][n][d] (any strides with d contiguous) -> KVView."""
    assert kv.dim() == 6 and kv.stride(5) == 1
    s = kv.stride()
    return KVView(kv.data_ptr(), s[0], s[1], s[2], s[3], s[4])


class StreamSet:
    """Device buffers of a coded output: payload, per-chunk index, byte cursor."""

    def __init__(self, n_streams, max_chunks, capacity, device="cuda", guard=0):
        """guard > 0 allocates that many extra bytes behind the stated capacity, filled with 0xA5, so
        that a test can show nothing was written past the capacity (``guard_intact``)."""
        import torch
        self.capacity = int(capacity)
        self.payload = torch.empty(self.capacity + int(guard), dtype=torch.uint8, device=device)
        if guard:
            self.payload[self.capacity:] = 0xA5
        self.chunk_offset = torch.zeros(n_streams * max_chunks, dtype=torch.int64, device=device)
        self.chunk_bytes = torch.zeros(n_streams * max_chunks, dtype=torch.int32, device=device)
        self.total_bytes = torch.zeros(1, dtype=torch.int64, device=device)
        self.max_chunks = max_chunks
        self.n_streams = n_streams

    def c(self):
        return Streams(self.payload.data_ptr(), self.capacity, self.chunk_offset.data_ptr(),
                       self.chunk_bytes.data_ptr(), self.total_bytes.data_ptr(), self.max_chunks)

    def guard_intact(self):
        return bool((self.payload[self.capacity:] == 0xA5).all())

    def chunk(self, slot):
        """Bytes of one chunk as a CPU numpy array."""
        off = int(self.chunk_offset[slot]); nb = int(self.chunk_bytes[slot]) & 0xFFFFFFFF
        return self.payload[off:off + nb].cpu().numpy()


class Context:
    """One parameter set + candidate table T ([L][2][H][V][d] float16 on the device)."""

    def __init__(self, T, top_k, delta, chunk_pos=256, sigma_floor=0.0, variant=PRED_TOPK, out_dtype=OUT_F32,
                 adaptive=None, zero_rate_D=0.0):
        """adaptive = (b0, extra, hbar) turns on the surprisal-adaptive step (Def. 7); encode / decode
        then need the tokens.  zero_rate_D > 0 turns on the zero-rate rule (Thm. 3)."""
        L, two, H, V, d = T.shape
        assert two == 2 and T.is_cuda and T.is_contiguous()
        self.T = T
        b0, extra, hbar = adaptive if adaptive else (0, 0, 0.0)
        self.cfg = Config(L, H, d, V, top_k, delta, sigma_floor, chunk_pos, variant, out_dtype, b0, extra, hbar, zero_rate_D)
        self.W = 2 * L * H
        self._h = C.c_void_p()
        _check(lib().plc_create(C.byref(self._h), C.byref(self.cfg), _ptr(T)), "plc_create")

    @classmethod
    def linear(cls, E, A, c, delta, chunk_pos=256, sigma_floor=0.0, out_dtype=OUT_F32, zero_rate_D=0.0):
        """Context of the linear-embedding predictor (Sec. 7.1): E [V][dm], A [L][2][H][d][dm],
        c [L][2][H][d], float16 on the device."""
        V, dm = E.shape
        L, two, H, d, dm2 = A.shape
        assert two == 2 and dm2 == dm and tuple(c.shape) == (L, 2, H, d)
        assert all(t.is_cuda and t.is_contiguous() for t in (E, A, c))
        self = cls.__new__(cls)
        self.T = None
        self._model = (E, A, c)
        self.cfg = Config(L, H, d, V, 1, delta, sigma_floor, chunk_pos, PRED_LINEAR, out_dtype, 0, 0, 0.0, zero_rate_D)
        self.W = 2 * L * H
        self._h = C.c_void_p()
        m = LinearModel(E.data_ptr(), A.data_ptr(), c.data_ptr(), dm)
        _check(lib().plc_create_linear(C.byref(self._h), C.byref(self.cfg), C.byref(m)), "plc_create_linear")
        return self

    def close(self):
        if getattr(self, "_h", None):
            lib().plc_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def max_chunks(self, n):
        return (n + self.cfg.chunk_pos - 1) // self.cfg.chunk_pos

    def reserve(self, positions):
        _check(lib().plc_reserve(self._h, C.c_int64(positions)), "plc_reserve")

    def topk_softmax(self, logits, tokens=None, want=("idx", "w", "lse", "zk", "logp2")):
        import torch
        N = logits.numel() // self.cfg.vocab
        K = self.cfg.top_k
        dev = logits.device
        out = {}
        if "idx" in want:
            out["idx"] = torch.empty(N, K, dtype=torch.int32, device=dev)
        if "w" in want:
            out["w"] = torch.empty(N, K, dtype=torch.float32, device=dev)
        for k in ("lse", "zk"):
            if k in want:
                out[k] = torch.empty(N, dtype=torch.float32, device=dev)
        if "logp2" in want and tokens is not None:
            out["logp2"] = torch.empty(N, dtype=torch.float32, device=dev)
        _check(lib().plc_topk_softmax(self._h, _ptr(logits), _ptr(tokens), C.c_int64(N), _ptr(out.get("idx")),
                                      _ptr(out.get("w")), _ptr(out.get("lse")), _ptr(out.get("zk")),
                                      _ptr(out.get("logp2")), _stream()), "plc_topk_softmax")
        return out

    def prefix_dedup(self, tokens, lens, logp2):
        import torch
        S, stride = tokens.shape
        dev = tokens.device
        lcp = torch.empty(S, S, dtype=torch.int32, device=dev)
        dT = torch.empty(S, S, dtype=torch.float32, device=dev)
        parent = torch.empty(S, dtype=torch.int32, device=dev)
        shared = torch.empty(S, dtype=torch.int32, device=dev)
        _check(lib().plc_prefix_dedup(self._h, _ptr(tokens), _ptr(lens), _ptr(logp2), S, C.c_int64(stride), _ptr(lcp),
                                      _ptr(dT), _ptr(parent), _ptr(shared), _stream()), "plc_prefix_dedup")
        return lcp, dT, parent, shared

    def rotq_params(self, bits, neg):
        """neg: d booleans (component j negated before the transform)."""
        p = RotqParams()
        p.bits = int(bits)
        for j, v in enumerate(neg):
            if v:
                p.sign_bits[j >> 5] |= 1 << (j & 31)
        return p

    def rotq_record_bytes(self, bits):
        b = C.c_uint64()
        _check(lib().plc_rotq_record_bytes(self._h, int(bits), C.byref(b)), "plc_rotq_record_bytes")
        return b.value

    def encode_rotq(self, kv, logits, params, records, pos_begin=None, pos_end=None):
        """Rotated fixed-rate quantiser (Prop. 3 step 3): records uint8 [S*W*n*record_bytes] on the device."""
        S, n = logits.shape[0], logits.shape[1]
        view = kv if isinstance(kv, KVView) else kv_view(kv)
        _check(lib().plc_encode_rotq(self._h, C.byref(view), _ptr(logits), S, n, _ptr(pos_begin), _ptr(pos_end),
                                     C.byref(params), _ptr(records), C.c_uint64(records.numel() * records.element_size()),
                                     _stream()), "plc_encode_rotq")

    def decode_rotq(self, records, logits, params, kv_out, pos_begin=None, pos_end=None):
        S, n = logits.shape[0], logits.shape[1]
        view = kv_out if isinstance(kv_out, KVView) else kv_view(kv_out)
        _check(lib().plc_decode_rotq(self._h, _ptr(records), C.c_uint64(records.numel() * records.element_size()),
                                     _ptr(logits), S, n, _ptr(pos_begin), _ptr(pos_end), C.byref(params), C.byref(view),
                                     _stream()), "plc_decode_rotq")

    def prefix_clusters(self, lcp, dT, delta):
        """Def. 3 on the outputs of prefix_dedup -> (cluster, centroid, begin), each [S] int32."""
        import torch
        S = lcp.shape[0]
        out = [torch.empty(S, dtype=torch.int32, device=lcp.device) for _ in range(3)]
        _check(lib().plc_prefix_clusters(self._h, _ptr(lcp), _ptr(dT), S, C.c_float(delta), _ptr(out[0]), _ptr(out[1]),
                                         _ptr(out[2]), _stream()), "plc_prefix_clusters")
        return tuple(out)

    def encode(self, kv, logits, streams, pos_begin=None, pos_end=None, debug=None, tokens=None):
        S, n = logits.shape[0], logits.shape[1]
        view = kv if isinstance(kv, KVView) else kv_view(kv)
        st = streams.c()
        if tokens is not None:
            _check(lib().plc_encode_adaptive(self._h, C.byref(view), _ptr(logits), _ptr(tokens), S, n, _ptr(pos_begin),
                                             _ptr(pos_end), C.byref(st), None if debug is None else C.byref(debug),
                                             _stream()), "plc_encode_adaptive")
            return
        _check(lib().plc_encode(self._h, C.byref(view), _ptr(logits), S, n, _ptr(pos_begin), _ptr(pos_end),
                                C.byref(st), None if debug is None else C.byref(debug), _stream()), "plc_encode")

    def decode(self, streams, logits, kv_out, pos_begin=None, pos_end=None, debug=None, tokens=None):
        S, n = logits.shape[0], logits.shape[1]
        view = kv_out if isinstance(kv_out, KVView) else kv_view(kv_out)
        st = streams.c()
        if tokens is not None:
            _check(lib().plc_decode_adaptive(self._h, C.byref(st), _ptr(logits), _ptr(tokens), S, n, _ptr(pos_begin),
                                             _ptr(pos_end), C.byref(view), None if debug is None else C.byref(debug),
                                             _stream()), "plc_decode_adaptive")
            return
        _check(lib().plc_decode(self._h, C.byref(st), _ptr(logits), S, n, _ptr(pos_begin), _ptr(pos_end),
                                C.byref(view), None if debug is None else C.byref(debug), _stream()), "plc_decode")

    def sync_status(self):
        return lib().plc_sync_status(self._h, _stream())

    def poll_status(self):
        """(status code, raw bits) of the device status word, without waiting for enqueued work."""
        bits = C.c_uint32()
        rc = lib().plc_poll_status(self._h, C.byref(bits))
        return rc, bits.value

    def last_schedule(self):
        """(queues, SMs per queue) of the most recent top-K encode / decode launch."""
        nq, g = C.c_int32(), C.c_int32()
        _check(lib().plc_last_schedule(self._h, C.byref(nq), C.byref(g)), "plc_last_schedule")
        return nq.value, g.value

    def set_profiling(self, on=True):
        _check(lib().plc_set_profiling(self._h, int(on)), "plc_set_profiling")

    def last_kernel_ms(self, which):
        """Duration of the most recent fused kernel: which = 0 encode, 1 decode."""
        ms = C.c_float()
        _check(lib().plc_last_kernel_ms(self._h, int(which), C.byref(ms)), "plc_last_kernel_ms")
        return ms.value

    def kernel_ms(self, which, reset=False):
        """(mean duration in ms, launches) of the profiled launches of one kind since the last reset."""
        ms, cnt = C.c_float(), C.c_int32()
        _check(lib().plc_kernel_ms(self._h, int(which), C.byref(ms), C.byref(cnt), int(reset)), "plc_kernel_ms")
        return ms.value, cnt.value

    def stats(self, reset=False):
        s = Stats()
        _check(lib().plc_get_stats(self._h, C.byref(s), int(reset), _stream()), "plc_get_stats")
        return s

    def new_session_batch(self, B, max_chunks, capacity):
        import torch
        a, b = C.c_uint64(), C.c_uint64()
        _check(lib().plc_append_sizes(self._h, B, C.byref(a), C.byref(b)), "plc_append_sizes")
        sb = AppendBatch()
        sb.open_sym = torch.zeros(a.value // 4, dtype=torch.int32, device=self.T.device)
        sb.open_q = torch.zeros(b.value // 4, dtype=torch.int32, device=self.T.device)
        sb.streams = StreamSet(B * self.W, max_chunks, capacity, self.T.device)
        sb.c = SessionBatch(B, 0, sb.open_sym.data_ptr(), sb.open_q.data_ptr(), sb.streams.c())
        return sb

    def append_step(self, sb, kv_step, logits_step):
        _check(lib().plc_append_step(self._h, C.byref(sb.c), _ptr(kv_step), _ptr(logits_step), _stream()),
               "plc_append_step")

    def append_flush(self, sb):
        _check(lib().plc_append_flush(self._h, C.byref(sb.c), _stream()), "plc_append_flush")


class AppendBatch:
    """Python-side holder of a plc_session_batch and the tensors it points to."""


def rans_encode_static(sym, q, n_pos, chunk_index, streams, status):
    """Codes chunk ``chunk_index`` of every stream from symbols / classes on the device, using only
    the library's static working memory (no allocation inside the call).

    sym [n_streams][chunk_capacity][d] int32, q [n_streams][chunk_capacity] int32, status: one int32
    device word that receives 0 or the error bits.  Returns the plc_status of the host-side checks."""
    n_streams, cap, d = sym.shape
    st = streams.c()
    return lib().plc_rans_encode_static(_ptr(sym), _ptr(q), n_streams, int(n_pos), d, cap, int(chunk_index),
                                        C.byref(st), _ptr(status), _stream())


class TrieIndex:
    """Host-side prefix index (Sec. 7.3): insert / best_match / evict over numpy int32 token arrays."""

    def __init__(self, epsilon=0.0):
        self._h = C.c_void_p()
        _check(lib().plc_trie_create(C.byref(self._h), C.c_float(epsilon)), "plc_trie_create")

    def __del__(self):
        try:
            if self._h:
                lib().plc_trie_destroy(self._h)
                self._h = C.c_void_p()
        except Exception:
            pass

    def insert(self, ident, tokens, logp2):
        import numpy as np
        tk = np.ascontiguousarray(tokens, dtype=np.int32); lp = np.ascontiguousarray(logp2, dtype=np.float32)
        kept = C.c_int32()
        _check(lib().plc_trie_insert(self._h, int(ident), tk.ctypes.data_as(C.c_void_p), lp.ctypes.data_as(C.c_void_p),
                                     len(tk), C.byref(kept)), "plc_trie_insert")
        return kept.value

    def best_match(self, tokens):
        import numpy as np
        tk = np.ascontiguousarray(tokens, dtype=np.int32)
        ident, lcp, dT = C.c_int32(), C.c_int32(), C.c_float()
        _check(lib().plc_trie_best_match(self._h, tk.ctypes.data_as(C.c_void_p), len(tk), C.byref(ident), C.byref(lcp),
                                         C.byref(dT)), "plc_trie_best_match")
        return ident.value, lcp.value, dT.value

    def evict(self, ident):
        _check(lib().plc_trie_evict(self._h, int(ident)), "plc_trie_evict")

    def stats(self):
        a, b = C.c_int64(), C.c_int64()
        _check(lib().plc_trie_stats(self._h, C.byref(a), C.byref(b)), "plc_trie_stats")
        return a.value, b.value


def table_constants(qp):
    th, rh = C.c_uint32(), C.c_uint32()
    _check(lib().plc_table_constants(int(qp), C.byref(th), C.byref(rh)), "plc_table_constants")
    return th.value, rh.value


def build_table(qp):
    import numpy as np
    f = np.zeros(64, np.uint32)
    c = np.zeros(65, np.uint32)
    _check(lib().plc_build_table(int(qp), f.ctypes.data_as(C.c_void_p), c.ctypes.data_as(C.c_void_p)),
           "plc_build_table")
    return f, c


def launch_count():
    return int(lib().plc_launch_count())
