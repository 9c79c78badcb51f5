"""The allocation-free chunk coder (plc_rans_encode_static) against the append path's own sealing.

Some callers may not allocate device memory where they seal a chunk (a serving loop on a frozen
memory pool, a plugin with a fixed budget), so they cannot hold a context.  This entry point codes
chunks from symbols and classes with nothing but the library's static device array.  It must write
byte for byte what plc_append_flush writes for the same symbols -- on a first call and again on a
second call that finds the previous call's leftovers in the shared array.
"""
import numpy as np
import pytest
import torch

import paper_2604_15356_b200 as plc
from paper_2604_15356_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_coder_matches_append_sealing_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    plc.build()
    dev = torch.device("cuda:0")
    B, L, H, d, V, K, CP = 3, 1, 2, 128, 512, 32, 32
    for steps, seed in ((20, 61), (32, 62)):          # a partly filled chunk, then a full one (32*128 = the limit)
        table = synth.markov_table(V, 12.0, seed, max_states=64)
        tokens = synth.sample_tokens(table, B, steps, seed + 1)
        logits = synth.position_logits(table, tokens).to(dev)
        T = synth.make_tables(L, H, V, d, seed + 2)
        kv = synth.make_kv(T, tokens, 0.05, seed + 3).to(dev)
        ctx = plc.Context(T.to(dev), K, 0.02, chunk_pos=CP)
        W = ctx.W
        cap = 3 * B * CP * W * d + 4096
        sb = ctx.new_session_batch(B, 1, cap)
        for i in range(steps):
            ctx.append_step(sb, kv[:, :, :, :, i, :].contiguous(), logits[:, i, :].contiguous())
        ctx.append_flush(sb)                            # codes whatever the steps have not coded yet
        assert ctx.sync_status() == plc.OK
        ref = [sb.streams.chunk(s) for s in range(B * W)]
        assert all(len(r) > 128 for r in ref)
        sym = sb.open_sym.view(2, B * W, CP, d)[0]      # chunk 0 sits in the first of the two open buffers
        q = sb.open_q.view(2, B * W, CP)[0]
        status = torch.full((1,), 77, dtype=torch.int32, device=dev)
        for call in range(2):                           # two calls in a row share the static array
            out = plc.StreamSet(B * W, 1, cap, dev)
            assert plc.rans_encode_static(sym, q, steps, 0, out, status) == plc.OK
            torch.cuda.synchronize()
            assert int(status) == 0
            for s in range(B * W):
                assert np.array_equal(out.chunk(s), ref[s]), (steps, call, s)
            assert int(out.total_bytes) == int(sb.streams.total_bytes)
        # a payload buffer that is too small is reported through the status word, nothing is overrun
        small = plc.StreamSet(B * W, 1, 1024, dev, guard=1 << 16)
        assert plc.rans_encode_static(sym, q, steps, 0, small, status) == plc.OK
        torch.cuda.synchronize()
        assert int(status) == 1 and int(small.total_bytes) == int(sb.streams.total_bytes)
        assert small.guard_intact()
        # a byte cursor that is not a multiple of 16 is reported (bit 16) and nothing is written
        odd = plc.StreamSet(B * W, 1, cap, dev)
        odd.payload.fill_(0x5A)
        odd.total_bytes.fill_(4)
        assert plc.rans_encode_static(sym, q, steps, 0, odd, status) == plc.OK
        torch.cuda.synchronize()
        assert int(status) == 16 and bool((odd.payload == 0x5A).all())
    # sizes beyond the static working memory are refused on the host
    big_sym = torch.zeros(2, 64, 128, dtype=torch.int32, device=dev)
    big_q = torch.zeros(2, 64, dtype=torch.int32, device=dev)
    out = plc.StreamSet(2, 1, 1 << 16, dev)
    assert plc.rans_encode_static(big_sym, big_q, 33, 0, out, status) == plc.E_SHAPE
    assert plc.rans_encode_static(big_sym, big_q, 32, 1, out, status) == plc.E_SHAPE      # chunk index out of range
    # an out-of-range class is clamped and flagged, not used as a table index
    big_q[1, 3] = 9999
    assert plc.rans_encode_static(big_sym, big_q, 8, 0, out, status) == plc.OK
    torch.cuda.synchronize()
    assert int(status) == 4
