"""Seeded synthetic inputs: Markov token source, per-position logits, candidate tables T, KV tensors.

This module only produces input arrays.  It contains none of the codec's arithmetic and is the one
module that both the CUDA library's callers and the CPU oracle's callers import: both sides receive
the same arrays unchanged.  Everything is torch, runs on CPU or on a CUDA device, and is a pure
function of its seeds.

Recipe (shapes follow the configurations of the benchmark definition; the model names there only
lend shapes):
  * R = min(V, max_states) context states, state(x) = x mod R (first-order Markov source).
  * base[r][v] = -alpha * ln(1 + rank(v)) + g[r][v], g ~ N(0,1), rank a fixed permutation;
    logits = tau * base, tau found by bisection so that the mean row entropy is ln(target
    perplexity); stored as float16.
  * tokens: x_{-1} = 0, x_i drawn from softmax(logits[state(x_{i-1})]) by inverse CDF.
  * per-position logits handed to the codec: logits[s][i] = table[state(x_{i-1})].
  * T [L][2][H][V][d] float16 ~ N(0,1).
  * KV[l][kv][s][h][i][:] = float16(T[l][kv][h][x_i] + sigma * z), z ~ N(0,1) from a counter-based
    hash of (seed, key[s][i], l, kv, h, j); equal keys give equal noise, so sessions that share a
    token prefix (and are given equal keys there) share their KV exactly on that prefix.
"""
import math

import torch


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def markov_table(V, target_pp, seed, alpha=0.0, max_states=4096, device="cpu"):
    """Returns float16 logits table [R][V] whose mean row perplexity is target_pp."""
    R = min(V, max_states)
    g = _gen(seed, device)
    noise = torch.randn(R, V, generator=g, device=device, dtype=torch.float32)
    if alpha:
        rank = torch.randperm(V, generator=g, device=device).to(torch.float32)
        noise = noise - alpha * torch.log1p(rank)[None, :]
    target = math.log(target_pp)

    def mean_entropy(tau):
        lp = torch.log_softmax(noise * tau, dim=1)
        return float(-(lp.exp() * lp).sum(1).mean())

    lo, hi = 0.0, 64.0
    for _ in range(40):
        mid = 0.5 * (lo + hi)
        if mean_entropy(mid) > target:
            lo = mid
        else:
            hi = mid
    tau = 0.5 * (lo + hi)
    return (noise * tau).to(torch.float16)


def sample_tokens(table, S, n, seed, first_state=0, start=None):
    """Markov sampling by inverse CDF.  Returns int32 tokens [S][n].

    ``start`` (int64 [S]) gives the token that precedes position 0 of each session (default 0).
    """
    device = table.device
    R, V = table.shape
    g = _gen(seed, device)
    u = torch.rand(S, n, generator=g, device=device, dtype=torch.float64)
    cdf = torch.softmax(table.to(torch.float64), dim=1).cumsum(1)
    cdf = cdf / cdf[:, -1:]
    prev = torch.full((S,), first_state, dtype=torch.int64, device=device) if start is None else start.to(torch.int64)
    out = torch.empty(S, n, dtype=torch.int32, device=device)
    for i in range(n):
        rows = cdf[prev % R]
        x = torch.searchsorted(rows, u[:, i:i + 1].contiguous()).squeeze(1).clamp_(max=V - 1)
        out[:, i] = x.to(torch.int32)
        prev = x
    return out


def position_logits(table, tokens, start=None):
    """logits[s][i] = table[state(x_{i-1})] with x_{-1} = start[s] (default 0).  float16 [S][n][V]."""
    R = table.shape[0]
    S, n = tokens.shape
    first = torch.zeros(S, 1, dtype=torch.int64, device=tokens.device) if start is None else start.view(S, 1).to(torch.int64)
    prev = torch.cat([first, tokens[:, :-1].to(torch.int64)], dim=1)
    return table[prev % R]


def make_tables(L, H, V, d, seed, device="cpu"):
    """T [L][2][H][V][d] float16 ~ N(0,1)."""
    g = _gen(seed, device)
    T = torch.empty(L, 2, H, V, d, dtype=torch.float16, device=device)
    for l in range(L):
        T[l] = torch.randn(2, H, V, d, generator=g, device=device, dtype=torch.float32).to(torch.float16)
    return T


_M64 = (1 << 64) - 1


def _wrap(c):
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def _mix64(x):
    """splitmix64 finaliser on int64 tensors (arithmetic modulo 2^64)."""
    x = (x ^ ((x >> 30) & 0x3FFFFFFFF)) * _wrap(0xBF58476D1CE4E5B9)
    x = (x ^ ((x >> 27) & 0x1FFFFFFFFF)) * _wrap(0x94D049BB133111EB)
    return x ^ ((x >> 31) & 0x1FFFFFFFF)


def hashed_normal(keys, stream, d, seed):
    """Standard normals [..., d] that are a pure function of (seed, key, stream, component)."""
    dev = keys.device
    j = torch.arange(d, device=dev, dtype=torch.int64)
    base = _mix64(keys.to(torch.int64) * _wrap(0x9E3779B97F4A7C15) + _wrap(int(seed)))[..., None]
    h = _mix64(base + (j + 1) * _wrap(0xD1B54A32D192ED03) + _wrap(int(stream) * 0x8CB92BA72F3D8DD7))
    h2 = _mix64(h + _wrap(0x2545F4914F6CDD1D))
    u1 = (((h >> 11) & ((1 << 53) - 1)).to(torch.float64) + 0.5) / float(1 << 53)
    u2 = (((h2 >> 11) & ((1 << 53) - 1)).to(torch.float64) + 0.5) / float(1 << 53)
    return (torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)).to(torch.float32)


def prefix_keys(tokens):
    """int64 [S][n] rolling hash of the token prefix x_0..x_i: equal prefixes give equal keys, so KV
    built from these keys is a function of the token prefix alone."""
    S, n = tokens.shape
    keys = torch.empty(S, n, dtype=torch.int64, device=tokens.device)
    k = torch.zeros(S, dtype=torch.int64, device=tokens.device)
    tok = tokens.to(torch.int64)
    for i in range(n):
        k = _mix64(k * _wrap(0x9E3779B97F4A7C15) + tok[:, i] + 1)
        keys[:, i] = k
    return keys


def make_kv(T, tokens, sigma, seed, keys=None, out=None):
    """KV [L][2][S][H][n][d] float16 = T[l][kv][h][x_i] + sigma * noise(key[s][i])."""
    L, _, H, V, d = T.shape
    S, n = tokens.shape
    dev = T.device
    if keys is None:
        keys = torch.arange(S * n, device=dev, dtype=torch.int64).view(S, n)
    if out is None:
        out = torch.empty(L, 2, S, H, n, d, dtype=torch.float16, device=dev)
    tok = tokens.to(torch.int64)
    for l in range(L):
        for a in range(2):
            for h in range(H):
                rows = T[l, a, h][tok].to(torch.float32)              # [S][n][d]
                if sigma:
                    rows = rows + sigma * hashed_normal(keys, (l * 2 + a) * H + h, d, seed)
                out[l, a, :, h] = rows.to(torch.float16)
    return out


def trie_sessions(table, S, n, seed, seg_lo, seg_hi, depth=3):
    """Sessions that share system prefixes drawn from a seeded binary prefix trie.

    The trie has depth+1 levels (1+2+...+2^depth segments); each segment is Markov-sampled,
    length U[seg_lo, seg_hi]; a session picks one of the 2^depth leaves uniformly, takes that
    root-to-leaf path as its prefix and continues sampling.  Returns tokens int32 [S][n], keys
    int64 [S][n] (a hash of the token prefix, so equal exactly where prefixes are equal), leaf [S],
    prefix_len [S].
    """
    dev = table.device
    g = _gen(seed, "cpu")
    nseg = (1 << (depth + 1)) - 1
    seg_len = torch.randint(seg_lo, seg_hi + 1, (nseg,), generator=g)
    segs = [None] * nseg
    for node in range(nseg):
        parent = (node - 1) // 2 if node else -1
        start = None if parent < 0 else segs[parent][:, -1].to(torch.int64)
        segs[node] = sample_tokens(table, 1, int(seg_len[node]), seed * 1000 + 17 + node, start=start)
    leaf = torch.randint(0, 1 << depth, (S,), generator=g)
    tokens = torch.zeros(S, n, dtype=torch.int32, device=dev)
    plen = torch.zeros(S, dtype=torch.int32)
    for s in range(S):
        node = (1 << depth) - 1 + int(leaf[s])
        path = []
        while node >= 0:
            path.append(node)
            node = (node - 1) // 2 if node else -1
        path.reverse()
        pos = 0
        for nd in path:
            m = min(int(seg_len[nd]), n - pos)
            tokens[s, pos:pos + m] = segs[nd][0, :m]
            pos += m
        plen[s] = pos
    # every session continues from its prefix's last token; the continuations are drawn for all
    # sessions at once (one uniform stream per session) and cut to the length each one needs
    last = tokens[torch.arange(S, device=dev), (plen.to(dev).to(torch.int64) - 1).clamp_(min=0)].to(torch.int64)
    cont = sample_tokens(table, S, n, seed * 1000 + 500, start=last)
    for s in range(S):
        pos = int(plen[s])
        if pos < n:
            tokens[s, pos:] = cont[s, :n - pos]
    return tokens, prefix_keys(tokens), leaf, plen


def peaked_logits(S, n, V, seed, lo=0.5, hi=40.0, device="cpu"):
    """Logits [S][n][V] float16 whose entropy differs widely from position to position:
    row = scale * N(0,1)^V with scale log-uniform in [lo, hi] (near-uniform rows up to point masses)."""
    g = _gen(seed, device)
    base = torch.randn(S, n, V, generator=g, device=device, dtype=torch.float32)
    u = torch.rand(S, n, generator=g, device=device, dtype=torch.float32)
    scale = torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo)))
    return (base * scale[..., None]).to(torch.float16)


def make_linear_model(L, H, V, d, dm, seed, device="cpu"):
    """Parameters of a KV function that is linear in the token embedding, F(t) = c + A E(t):
    E [V][dm] ~ N(0,1), A [L][2][H][d][dm] ~ N(0, 1/dm), c [L][2][H][d] ~ N(0, 0.01), all float16."""
    g = _gen(seed, device)
    E = torch.randn(V, dm, generator=g, device=device, dtype=torch.float32).to(torch.float16)
    A = (torch.randn(L, 2, H, d, dm, generator=g, device=device, dtype=torch.float32) / dm ** 0.5).to(torch.float16)
    c = (0.1 * torch.randn(L, 2, H, d, generator=g, device=device, dtype=torch.float32)).to(torch.float16)
    return E, A, c


def make_kv_linear(E, A, c, tokens, sigma, seed, keys=None):
    """KV [L][2][S][H][n][d] float16 = c + A E[x_i] + sigma * noise(key[s][i]) (computed in float32)."""
    L, _, H, d, dm = A.shape
    S, n = tokens.shape
    dev = A.device
    if keys is None:
        keys = torch.arange(S * n, device=dev, dtype=torch.int64).view(S, n)
    out = torch.empty(L, 2, S, H, n, d, dtype=torch.float16, device=dev)
    emb = E[tokens.to(torch.int64)].to(torch.float32)                         # [S][n][dm]
    for l in range(L):
        for a in range(2):
            for h in range(H):
                rows = emb @ A[l, a, h].to(torch.float32).t() + c[l, a, h].to(torch.float32)   # [S][n][d]
                if sigma:
                    rows = rows + sigma * hashed_normal(keys, (l * 2 + a) * H + h, d, seed)
                out[l, a, :, h] = rows.to(torch.float16)
    return out
