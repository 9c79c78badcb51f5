"""The oracle run on several host cores (oracle.encode_parallel: one unchanged single-threaded
encode per slice of heads, in processes of their own) gives exactly what the serial oracle gives."""
import numpy as np

from paper_2604_15356_b200 import synth


def _inputs(S=1, n=40, L=2, H=4, d=64, V=300):
    table = synth.markov_table(V, 12.0, 1, max_states=64)
    tokens = synth.sample_tokens(table, S, n, 2)
    logits = synth.position_logits(table, tokens)
    T = synth.make_tables(L, H, V, d, 3)
    kv = synth.make_kv(T, tokens, 0.05, 4)
    return tokens, logits, T, kv


def test_parallel_equals_serial_topk_and_dense(orc):
    tokens, logits, T, kv = _inputs()
    L, _, H, V, d = T.shape
    for dense in (0, 1):
        cfg = orc.Config(L, H, d, V, 8, 0.02, 0.0, 16, dense)
        a = orc.encode(cfg, T.numpy(), kv.numpy(), logits.numpy(), tokens.numpy(), export=True)
        b = orc.encode_parallel(cfg, T.numpy(), kv.numpy(), logits.numpy(), tokens.numpy(), export=True, workers=3)
        assert b["workers"] == 3
        for k in ("sym", "q", "mu", "chunk_bytes"):
            assert np.array_equal(a[k], b[k]), k
        assert a["stats"].payload_bytes == b["stats"]["payload_bytes"] and a["stats"].n_chunks == b["stats"]["n_chunks"]
        assert abs(a["stats"].ideal_bits - b["stats"]["ideal_bits"]) < 1e-6
        assert abs(a["stats"].token_bits - b["stats"]["token_bits"]) < 1e-9
        assert a["stats"].coded_positions == b["stats"]["coded_positions"]


def test_parallel_equals_serial_linear_predictor(orc):
    tokens, logits, T, kv = _inputs()
    L, _, H, V, d = T.shape
    E, A, c = synth.make_linear_model(L, H, V, d, 64, 5)
    kv = synth.make_kv_linear(E, A, c, tokens, 0.05, 6)
    cfg = orc.linear_config(L, H, d, V, 1, 0.02, 16, E.numpy(), A.numpy(), c.numpy())
    a = orc.encode(cfg, None, kv.numpy(), logits.numpy(), None, export=True)
    b = orc.encode_parallel(cfg, None, kv.numpy(), logits.numpy(), None, export=True, workers=2,
                            linear=(E.numpy(), A.numpy(), c.numpy()))
    for k in ("sym", "q", "mu", "chunk_bytes"):
        assert np.array_equal(a[k], b[k]), k
    assert a["stats"].payload_bytes == b["stats"]["payload_bytes"]
