"""Parity at the benchmark configurations' full sizes, in the launch configurations bench.py times:
`llama2-7b` in full; `70b-longctx` (131 072 positions, one global work queue) and the dedup
configuration (V = 128 256, per-SM work queues with stealing) on a subset of the layers that leaves
the work-queue decision unchanged; prefix dedup at 64 sessions x 8192 tokens; the append path at
256 sessions x 512 streams.

The oracle cannot run 10^7 .. 10^8 vectors, so it recomputes sampled chunks one by one; everything
else is checked through properties that hold at any size (decode inverts encode within delta/2, the
index is consistent, the byte count adds up)."""
import math

import numpy as np
import pytest
import torch

import paper_2604_15356_b200 as plc
from paper_2604_15356_b200 import workloads

pytestmark = pytest.mark.gpu


def oracle_chunk(orc, logits_rows, table, kv_rows, K, delta):
    """Symbols [P][d] and classes [P] of one chunk of one stream, by the oracle, from the inputs."""
    P, d = kv_rows.shape
    idx, wt, *_ = orc.topk_softmax(logits_rows, None, K)
    sym_o = np.zeros((P, d), np.int32); q_o = np.zeros(P, np.int32)
    for p in range(P):
        mu, s2 = orc.mixture(table, idx[p], wt[p])
        q_o[p] = orc.scale_class(s2, 0.0, delta)
        sym_o[p] = orc.quantise(kv_rows[p], mu, delta)
    return sym_o, q_o


class Tally:
    """Counts symbol / class disagreements over sampled chunks; each must be by one unit."""

    def __init__(self):
        self.n_sym = self.n_diff = self.n_q = self.n_qdiff = 0

    def add(self, sym_g, sym_o, q_g, q_o):
        self.n_sym += sym_o.size; self.n_diff += int((sym_g != sym_o).sum())
        self.n_q += q_o.size; self.n_qdiff += int((q_g != q_o).sum())
        assert np.abs(sym_g - sym_o).max() <= 1 and np.abs(q_g - q_o).max() <= 1

    def check(self):
        assert self.n_sym > 0
        assert self.n_diff <= max(1, 1e-4 * self.n_sym), (self.n_diff, self.n_sym)
        assert self.n_qdiff <= max(1, 1e-2 * self.n_q), (self.n_qdiff, self.n_q)


def check_sampled_chunk(orc, st, slot, q_g, logits_rows, table, kv_rows, K, delta, tally):
    """The GPU's bytes of one chunk: the oracle's decoder reads them (with the GPU's classes), its
    coder reproduces them bit for bit, and the symbols are the oracle's own up to rounding boundaries."""
    d = kv_rows.shape[1]
    got = st.chunk(slot)
    rc, sym_g = orc.rans_decode_chunk(got, q_g, d)
    assert rc == 0, slot
    ref, _, _ = orc.rans_encode_chunk(sym_g, q_g)
    assert np.array_equal(ref, got), slot
    sym_o, q_o = oracle_chunk(orc, logits_rows, table, kv_rows, K, delta)
    tally.add(sym_g, sym_o, q_g, q_o)


def need_memory(gb):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip(f"needs about {gb} GB of device memory")
    plc.build()
    return torch.device("cuda:0")


def test_full_size_sampled_chunks_and_properties(orc):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    free, _ = torch.cuda.mem_get_info()
    if free < 70e9:
        pytest.skip("needs about 60 GB of device memory")
    plc.build()
    dev = torch.device("cuda:0")
    w = workloads.build("llama2-7b", dev, seed=20260415)
    cfg = w["cfg"]
    S, n, L, H, d, V, K, CP, delta = (cfg[k] for k in ("S", "n", "L", "H", "d", "V", "K", "chunk_pos", "delta"))
    W = 2 * L * H
    ctx = plc.Context(w["T"], K, delta, chunk_pos=CP)
    mc = ctx.max_chunks(n)
    st = plc.StreamSet(S * W, mc, int(0.70 * w["kv"].numel() * 2), dev)
    q = torch.empty(S, n, W, dtype=torch.int32, device=dev)
    ctx.encode(w["kv"], w["logits"], st, debug=plc.DebugBuffers(None, q.data_ptr(), None))
    assert ctx.sync_status() == plc.OK
    stats = ctx.stats()
    assert stats.n_chunks == S * W * mc and stats.coded_vectors == S * n * W

    # index properties: aligned, disjoint, sizes add up
    off = st.chunk_offset.cpu().numpy().astype(np.int64)
    nby = st.chunk_bytes.cpu().numpy().astype(np.int64)
    assert np.all(off % 16 == 0) and np.all(nby > 128)
    order = np.argsort(off)
    assert np.all(off[order][1:] >= off[order][:-1] + nby[order][:-1])
    assert int(nby.sum()) == stats.payload_bytes
    assert int(st.total_bytes) == int(((nby + 15) // 16 * 16).sum())
    bits_per_comp = 8 * stats.payload_bytes / (S * n * W * d)
    assert 6.5 < bits_per_comp < 8.5

    # sampled chunks, recomputed by the oracle from the same inputs
    rng = np.random.default_rng(5)
    picks = [(int(rng.integers(S)), int(rng.integers(W)), int(rng.integers(mc))) for _ in range(10)]
    picks += [(0, 0, 0), (S - 1, W - 1, mc - 1)]
    n_sym = n_diff = n_qdiff = 0
    for s, t, c in picks:
        l, a, h = t // (2 * H), (t // H) % 2, t % H
        p0 = c * CP
        lg = w["logits"][s, p0:p0 + CP].cpu().numpy()
        tab = w["T"][l, a, h].cpu().numpy()
        kv = w["kv"][l, a, s, h, p0:p0 + CP].cpu().numpy()
        idx, wt, *_ = orc.topk_softmax(lg, None, K)
        sym_o = np.zeros((CP, d), np.int32); q_o = np.zeros(CP, np.int32)
        for p in range(CP):
            mu, s2 = orc.mixture(tab, idx[p], wt[p])
            q_o[p] = orc.scale_class(s2, 0.0, delta)
            sym_o[p] = orc.quantise(kv[p], mu, delta)
        q_g = q[s, p0:p0 + CP, t].cpu().numpy()
        got = st.chunk((s * W + t) * mc + c)
        rc, sym_g = orc.rans_decode_chunk(got, q_g, d)
        assert rc == 0, (s, t, c)                                   # the oracle's decoder reads the GPU's bytes
        ref, _, _ = orc.rans_encode_chunk(sym_g, q_g)
        assert np.array_equal(ref, got)                             # and its coder reproduces them bit for bit
        n_sym += sym_o.size; n_diff += int((sym_g != sym_o).sum()); n_qdiff += int((q_g != q_o).sum())
        assert np.abs(sym_g - sym_o).max() <= 1 and np.abs(q_g - q_o).max() <= 1
    assert n_diff <= max(1, 1e-4 * n_sym), (n_diff, n_sym)
    assert n_qdiff <= 0.01 * len(picks) * CP

    # decode inverts encode everywhere (Prop. 3): |KV' - KV| <= delta/2 + 1e-3 over the whole tensor
    del q
    out = torch.empty(w["kv"].shape, dtype=torch.float32, device=dev)
    ctx.decode(st, w["logits"], out)
    assert ctx.sync_status() == plc.OK
    worst = 0.0
    for l in range(L):
        worst = max(worst, float((out[l] - w["kv"][l].float()).abs().max()))
    assert worst <= delta / 2 + 1e-3, worst


def test_longctx_global_queue_sampled_chunks(orc):
    """`70b-longctx`, top-K: one session of 131 072 positions, chunk_pos 256 (512 chunks per table), so
    the resident warps span 13 consecutive tables = 107 MB <= L2 and the kernels take their work from
    ONE global queue.  4 of the 80 layers (64 tables >= the 13 spanned, so the queue decision is the
    full configuration's); sampled chunks recomputed by the oracle."""
    dev = need_memory(40)
    w = workloads.build("70b-longctx", dev, seed=20260418, L=4)
    cfg = w["cfg"]
    S, n, L, H, d, V, K, CP, delta = (cfg[k] for k in ("S", "n", "L", "H", "d", "V", "K", "chunk_pos", "delta"))
    assert (S, n, V, K, CP) == (1, 131072, 32000, 64, 256)
    W = 2 * L * H
    ctx = plc.Context(w["T"], K, delta, chunk_pos=CP)
    mc = ctx.max_chunks(n)
    st = plc.StreamSet(S * W, mc, int(0.70 * w["kv"].numel() * 2), dev)
    q = torch.empty(S, n, W, dtype=torch.int32, device=dev)
    ctx.encode(w["kv"], w["logits"], st, debug=plc.DebugBuffers(None, q.data_ptr(), None, None, 1))
    assert ctx.sync_status() == plc.OK
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    assert ctx.last_schedule() == (1, sms)                         # one queue for the whole GPU
    stats = ctx.stats()
    assert stats.n_chunks == S * W * mc and stats.coded_vectors == S * n * W
    nby = st.chunk_bytes.cpu().numpy().astype(np.int64)
    assert int(nby.sum()) == stats.payload_bytes and np.all(nby > 128)
    assert stats.ideal_bits <= 8 * stats.payload_bytes <= stats.ideal_bits * 1.001 + 1040 * stats.n_chunks
    rng = np.random.default_rng(6)
    picks = [(int(rng.integers(W)), int(rng.integers(mc))) for _ in range(6)] + [(0, 0), (W - 1, mc - 1)]
    tally = Tally()
    for t, c in picks:
        l, a, h = t // (2 * H), (t // H) % 2, t % H
        p0 = c * CP
        check_sampled_chunk(orc, st, t * mc + c, q[0, p0:p0 + CP, t].cpu().numpy(), w["logits"][0, p0:p0 + CP].cpu().numpy(),
                            w["T"][l, a, h].cpu().numpy(), w["kv"][l, a, 0, h, p0:p0 + CP].cpu().numpy(), K, delta, tally)
    tally.check()
    del q
    out = torch.empty(w["kv"].shape, dtype=torch.float32, device=dev)
    ctx.decode(st, w["logits"], out)
    assert ctx.sync_status() == plc.OK
    assert ctx.last_schedule() == (1, sms)
    assert float((out - w["kv"].float()).abs().max()) <= delta / 2 + 1e-3


def test_dedup_shape_prefix_and_per_sm_queues(orc):
    """The dedup configuration at its own shapes: 64 sessions x 8192 tokens from the seeded 8-leaf prefix
    trie, V = 128 256.  (1) log2 P of every token by the top-K kernel against the oracle's
    log-sum-exp of the 4096 distinct rows of the Markov source; (2) LCP, d_T, parents, shared lengths
    at 64 x 8192 against the oracle fed its own log-probabilities: exact / 1e-4; (3) the tails of the
    first 8 sessions coded with 2 of the 32 layers (32 tables of 32.8 MB: the 25 tables the resident
    warps would span are far beyond L2 whatever the layer count, so the kernels use the same 25 work
    queues of 6 SMs, with stealing, as the full configuration), sampled chunks by the oracle."""
    dev = need_memory(60)
    from paper_2604_15356_b200 import synth
    cfg = dict(workloads.CONFIGS["llama3-8b-dedup"])
    S, n, H, d, V, K, CP, delta = (cfg[k] for k in ("S", "n", "H", "d", "V", "K", "chunk_pos", "delta"))
    L, Sb, seed = 2, 8, 20260417
    table = synth.markov_table(V, cfg["pp"], seed, alpha=cfg["alpha"], max_states=4096, device=dev)
    tokens, keys, leaf, plen = synth.trie_sessions(table, S, n, seed + 1, 128, 1024)
    torch.cuda.empty_cache()
    T = synth.make_tables(L, H, V, d, seed + 2, device=dev)
    ctx = plc.Context(T, K, delta, chunk_pos=CP)
    ctx.reserve(Sb * n)
    W, mc = ctx.W, ctx.max_chunks(n)
    # (1) edge weights of the trie
    logp2 = torch.empty(S, n, dtype=torch.float32, device=dev)
    for b0 in range(0, S, Sb):
        lg = synth.position_logits(table, tokens[b0:b0 + Sb])
        logp2[b0:b0 + Sb] = ctx.topk_softmax(lg, tokens[b0:b0 + Sb].reshape(-1), want=("logp2",))["logp2"].view(Sb, n)
        del lg
    tab = table.cpu().numpy()
    _, _, lse_o, _, _ = orc.topk_softmax(tab, None, 1)                       # natural log-sum-exp of each distinct row
    tk = tokens.cpu().numpy().astype(np.int64)
    prev = np.concatenate([np.zeros((S, 1), np.int64), tk[:, :-1]], axis=1) % tab.shape[0]
    lp_o = (tab[prev, tk].astype(np.float64) - lse_o[prev]) / math.log(2.0)
    np.testing.assert_allclose(logp2.cpu().numpy(), lp_o, rtol=1e-4, atol=1e-4)
    # (2) prefix dedup at full size
    lens = torch.full((S,), n, dtype=torch.int32, device=dev)
    lens[5] = n - 1000; lens[17] = 3000
    lcp, dT, parent, shared = ctx.prefix_dedup(tokens, lens, logp2)
    lcp_o, dT_o, par_o, sh_o = orc.prefix_dedup(tk.astype(np.int32), lens.cpu().numpy(), lp_o.astype(np.float32))
    assert np.array_equal(lcp.cpu().numpy(), lcp_o)
    np.testing.assert_allclose(dT.cpu().numpy(), dT_o, rtol=1e-4, atol=1e-3)
    assert np.array_equal(parent.cpu().numpy(), par_o) and np.array_equal(shared.cpu().numpy(), sh_o)
    assert (par_o >= 0).sum() == S - 1 and sh_o[1:].min() >= 128              # at least the trie's root segment is shared
    # (3) tails of the first batch of sessions
    tb = tokens[:Sb]
    lg = synth.position_logits(table, tb)
    kv = synth.make_kv(T, tb, cfg["sigma"], seed + 3, keys=keys[:Sb])
    pb, pe = shared[:Sb].contiguous(), lens[:Sb].contiguous()
    st = plc.StreamSet(Sb * W, mc, int(0.70 * kv.numel() * 2) + (1 << 20), dev)
    q = torch.empty(Sb, n, W, dtype=torch.int32, device=dev)
    ctx.encode(kv, lg, st, pb, pe, debug=plc.DebugBuffers(None, q.data_ptr(), None))
    assert ctx.sync_status() == plc.OK
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    nq, g = ctx.last_schedule()
    assert g == (Sb * mc) // 40 and nq == min(-(-sms // g), W) and nq > 1     # per-SM-group queues, as at L = 32
    pbh, peh = pb.cpu().numpy(), pe.cpu().numpy()
    coded = int(np.maximum(peh - pbh, 0).sum())
    assert ctx.stats().coded_vectors == coded * W                             # Prop. 2: shared prefixes cost nothing
    rng = np.random.default_rng(7)
    tally = Tally()
    picks = 0
    while picks < 8:
        s_, t, c = int(rng.integers(Sb)), int(rng.integers(W)), int(rng.integers(mc))
        p0 = int(pbh[s_]) + c * CP
        if p0 >= peh[s_]:
            assert int(st.chunk_bytes[(s_ * W + t) * mc + c]) == 0
            continue
        P = min(CP, int(peh[s_]) - p0)
        l, a, h = t // (2 * H), (t // H) % 2, t % H
        check_sampled_chunk(orc, st, (s_ * W + t) * mc + c, q[s_, p0:p0 + P, t].cpu().numpy(), lg[s_, p0:p0 + P].cpu().numpy(),
                            T[l, a, h].cpu().numpy(), kv[l, a, s_, h, p0:p0 + P].cpu().numpy(), K, delta, tally)
        picks += 1
    tally.check()
    del q
    out = torch.zeros(kv.shape, dtype=torch.float32, device=dev)
    ctx.decode(st, lg, out, pb, pe)
    assert ctx.sync_status() == plc.OK
    for s_ in range(Sb):
        b, e = int(pbh[s_]), int(peh[s_])
        if e > b:
            assert float((out[:, :, s_, :, b:e] - kv[:, :, s_, :, b:e].float()).abs().max()) <= delta / 2 + 1e-3
        assert not out[:, :, s_, :, :b].any()


def test_append_full_batch_sampled_chunks(orc):
    """The streaming configuration at full width: 256 sessions x 512 streams (32 layers, 8 KV heads),
    V = 32000, 32-position chunks; 70 append steps = two sealed chunks and a flushed remainder of 6.
    After each seal the open chunk still holds the sealed positions' symbols and classes: sampled
    (session, table) pairs are compared with the oracle's symbols and re-coded by the oracle's coder."""
    dev = need_memory(30)
    from paper_2604_15356_b200 import synth
    cfg = dict(workloads.CONFIGS["append"])
    B, L, H, d, V, K, CP, delta = (cfg[k] for k in ("S", "L", "H", "d", "V", "K", "chunk_pos", "delta"))
    steps, seed = 70, 20260419
    W = 2 * L * H
    table = synth.markov_table(V, cfg["pp"], seed, device=dev)
    tokens = synth.sample_tokens(table, B, steps, seed + 1)
    logits = synth.position_logits(table, tokens)                             # [B][steps][V]
    T = synth.make_tables(L, H, V, d, seed + 2, device=dev)
    ctx = plc.Context(T, K, delta, chunk_pos=CP)
    sb = ctx.new_session_batch(B, 3, int(steps * B * W * d * 1.4) + (1 << 20))
    rng = np.random.default_rng(8)
    picks = [(int(rng.integers(B)), int(rng.integers(W))) for _ in range(10)] + [(0, 0), (B - 1, W - 1)]
    pb = torch.tensor([p[0] for p in picks], device=dev); pt = torch.tensor([p[1] for p in picks], device=dev)
    kv_keep = np.zeros((len(picks), steps, d), np.float16)
    g = torch.Generator(device=dev); g.manual_seed(seed + 3)
    open_sym = sb.open_sym.view(2, B, W, CP, d); open_q = sb.open_q.view(2, B, W, CP)   # chunk c fills buffer c mod 2
    sealed = {}
    lat = []
    for i in range(steps):
        tok = tokens[:, i].to(torch.int64)
        kv_step = (T[:, :, :, tok, :].permute(0, 1, 3, 2, 4).float() +
                   cfg["sigma"] * torch.randn(L, 2, B, H, d, device=dev, generator=g)).to(torch.float16).contiguous()
        flat = kv_step.permute(2, 0, 1, 3, 4).reshape(B, W, d)                # [B][table][d], table = (l*2 + kv)*H + h
        kv_keep[:, i] = flat[pb, pt].cpu().numpy()
        lg = logits[:, i, :].contiguous()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.append_step(sb, kv_step, lg)
        e1.record()
        lat.append((e0, e1))
        if (i + 1) % CP == 0:
            c = (i + 1) // CP - 1
            sealed[c] = (open_sym[c & 1][pb, pt].cpu().numpy(), open_q[c & 1][pb, pt].cpu().numpy(), CP)
    # a completed chunk is coded a slice of the streams per step: after 70 steps chunk 0 is in the container
    # in full (coded by steps 32 .. 63), chunk 1 only for the slices of steps 64 .. 69
    torch.cuda.synchronize()
    nby = sb.streams.chunk_bytes.view(B * W, 3).cpu().numpy()
    item = np.arange(B * W)                                               # item = table * B + session
    slot_of_item = (item % B) * W + item // B
    assert np.all(nby[:, 0] > 128)
    assert np.all((nby[slot_of_item, 1] > 0) == (item * CP // (B * W) <= steps % CP)) and not nby[:, 2].any()
    ctx.append_flush(sb)
    c = steps // CP
    sealed[c] = (open_sym[c & 1][pb, pt].cpu().numpy(), open_q[c & 1][pb, pt].cpu().numpy(), steps % CP)
    # every step costs about the same: no step carries the coding of all streams at once
    ms = sorted(a.elapsed_time(b) for a, b in lat[CP:])
    assert ms[-1] <= 2.0 * ms[len(ms) // 2], (ms[len(ms) // 2], ms[-1])
    assert ctx.sync_status() == plc.OK
    stats = ctx.stats()
    assert stats.n_chunks == B * W * 3 and stats.coded_vectors == B * W * steps
    tally = Tally()
    lgn = logits.cpu().numpy()
    for j, (b, t) in enumerate(picks):
        l, a, h = t // (2 * H), (t // H) % 2, t % H
        tab = T[l, a, h].cpu().numpy()
        for c, (sym_all, q_all, P) in sealed.items():
            sym_g, q_g = sym_all[j, :P], q_all[j, :P]
            ref, _, _ = orc.rans_encode_chunk(sym_g, q_g)
            assert np.array_equal(sb.streams.chunk((b * W + t) * 3 + c), ref), (b, t, c)
            sym_o, q_o = oracle_chunk(orc, lgn[b, c * CP:c * CP + P], tab, kv_keep[j, c * CP:c * CP + P], K, delta)
            tally.add(sym_g, sym_o, q_g, q_o)
    tally.check()
    # and the streams decode as a bulk encode's would
    out = torch.empty(L, 2, B, H, steps, d, dtype=torch.float16, device=dev)
    ctx2 = plc.Context(T, K, delta, chunk_pos=CP, out_dtype=plc.OUT_F16)
    ctx2.decode(sb.streams, logits, out)
    assert ctx2.sync_status() == plc.OK
    got = out.permute(2, 0, 1, 3, 4, 5).reshape(B, W, steps, d)[pb, pt].float().cpu().numpy()
    assert np.abs(got - kv_keep.astype(np.float32)).max() <= delta / 2 + 1e-3 + 8 * 2 ** -11
