"""Parity at the benchmark's full size (workload `llama2-7b`: 4 x 4096 tokens, 32 layers, 32 KV
heads, d = 128, V = 32000, K = 64, chunk_pos = 256), in the launch configuration bench.py times.

The oracle cannot run 33.5 M vectors, so it recomputes sampled chunks one by one; everything else is
checked through properties that hold at any size (decode inverts encode within delta/2, the index is
consistent, the byte count adds up)."""
import numpy as np
import pytest
import torch

import paper_2604_15356_b200 as plc
from paper_2604_15356_b200 import workloads

pytestmark = pytest.mark.gpu


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
