"""Named synthetic workloads (shapes of the benchmark configurations) built with ``synth``.

Input construction only: nothing here belongs to the codec.  Keyword overrides let tests build the
same recipe at a reduced size.
"""
import torch

from . import synth

# S sessions x n tokens, L layers, H KV heads, d head dim, V vocab, K top-K, pp perplexity,
# alpha Zipf skew of the Markov logits, delta step, chunk_pos positions per coded chunk.
CONFIGS = {
    "tiny": dict(S=1, n=512, L=1, H=1, d=64, V=256, K=16, pp=12.0, alpha=0.0, delta=0.02, chunk_pos=256, sigma=0.05),
    "llama2-7b": dict(S=4, n=4096, L=32, H=32, d=128, V=32000, K=64, pp=15.0, alpha=1.1, delta=0.02, chunk_pos=256,
                      sigma=0.05),
    "llama3-8b-dedup": dict(S=64, n=8192, L=32, H=8, d=128, V=128256, K=64, pp=12.0, alpha=0.0, delta=0.02,
                            chunk_pos=256, sigma=0.05),
    "70b-longctx": dict(S=1, n=131072, L=80, H=8, d=128, V=32000, K=64, pp=20.0, alpha=0.0, delta=0.02,
                        chunk_pos=256, sigma=0.05),
    "append": dict(S=256, n=512, L=32, H=8, d=128, V=32000, K=64, pp=12.0, alpha=0.0, delta=0.02, chunk_pos=32,
                   sigma=0.05),
}


def build(name, device, seed=20260415, **override):
    """Returns dict(cfg, tokens [S][n] i32, logits [S][n][V] f16, T [L][2][H][V][d] f16,
    kv [L][2][S][H][n][d] f16), all on ``device``.  With the override ``dm`` the candidate table is
    replaced by a linear model (E [V][dm], A [L][2][H][d][dm], c [L][2][H][d]) and T is None."""
    cfg = dict(CONFIGS[name])
    cfg.update(override)
    S, n, L, H, d, V = cfg["S"], cfg["n"], cfg["L"], cfg["H"], cfg["d"], cfg["V"]
    table = synth.markov_table(V, cfg["pp"], seed, alpha=cfg["alpha"], max_states=cfg.get("max_states", 4096),
                               device=device)
    tokens = synth.sample_tokens(table, S, n, seed + 1)
    logits = synth.position_logits(table, tokens)
    del table
    if cfg.get("dm"):          # KV function linear in the token embedding (Sec. 7.1) instead of a candidate table
        E, A, c = synth.make_linear_model(L, H, V, d, int(cfg["dm"]), seed + 2, device=device)
        kv = synth.make_kv_linear(E, A, c, tokens, cfg["sigma"], seed + 3)
        if torch.device(device).type == "cuda":
            torch.cuda.empty_cache()
        return dict(cfg=cfg, tokens=tokens, logits=logits, T=None, kv=kv, E=E, A=A, c=c)
    T = synth.make_tables(L, H, V, d, seed + 2, device=device)
    kv = synth.make_kv(T, tokens, cfg["sigma"], seed + 3)
    if torch.device(device).type == "cuda":
        torch.cuda.empty_cache()
    return dict(cfg=cfg, tokens=tokens, logits=logits, T=T, kv=kv)
