#!/usr/bin/env python
"""Benchmark of the predictive-delta-coding hot path (encode then decode of one synthetic batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama2-7b] [--impl own|reference]

A step = one pass of the whole path over one batch: top-K softmax, fused predict + quantise + rANS
encode of every (stream, position), then the decode of the same batch.  The metric is KV tokens per
second (a KV token = one token position of one session across all 2*L*H streams) that were both
encoded and decoded.  With N > 1 (torchrun) every rank runs its own batch (streams shard with no
exchange): weak scaling, value = tokens of all ranks / slowest rank's time.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "KV tokens/s encoded+decoded per B200"
UNIT = "KV tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        cmd = ["nvidia-smi", "-i", uuid, "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "200"]
        try:
            self.p = subprocess.Popen(cmd, stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.strip().split(",") for r in open(self.f.name) if r.strip()]
        os.unlink(self.f.name)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for nme, v in zip(names, r[3:7]):
                if v.strip().lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# DRAM bytes per vector of the fused kernels, from the ncu capture summarised in
# profiles/fused_kernels_mid_L4.md (dram__bytes_read.sum + dram__bytes_write.sum over 4.19 M vectors;
# traffic grows in proportion to the vectors).  Valid for the default workload and chunk size only.
NCU_DRAM_BYTES_PER_VECTOR = {"encode_kernel": 671.3, "decode_kernel": 431.9}


def max_over_ranks(ms, dist, device):
    """Slowest rank's time (the job's time); identity without a process group."""
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def job_value(world, tokens_per_rank_step, ms_per_step):
    """Whole-job KV tokens/s: every rank codes its own batch (weak scaling)."""
    return world * tokens_per_rank_step / (ms_per_step / 1e3)


def oracle_sample_rate(w, positions, layers):
    """Times the CPU oracle (encode + decode) on a slice of the workload: `positions` positions of
    session 0, `layers` layers, all heads.  Returns KV tokens/s (vectors / W / seconds)."""
    import oracle
    cfg = w["cfg"]
    H, d, V, K = cfg["H"], cfg["d"], cfg["V"], cfg["K"]
    Tn = w["T"][:layers].cpu().numpy()
    kvn = w["kv"][:layers, :, :1, :, :positions].cpu().numpy()
    lgn = w["logits"][:1, :positions].cpu().numpy()
    tkn = w["tokens"][:1, :positions].cpu().numpy()
    ocfg = oracle.Config(layers, H, d, V, K, cfg["delta"], 0.0, cfg["chunk_pos"], 0)
    t0 = time.perf_counter()
    enc = oracle.encode(ocfg, Tn, kvn, lgn, tkn)
    t1 = time.perf_counter()
    rc, out, _ = oracle.decode(ocfg, Tn, lgn, enc, kvn.shape)
    t2 = time.perf_counter()
    assert rc == 0
    W_full = 2 * cfg["L"] * H
    vecs = positions * 2 * layers * H
    return dict(value=vecs / W_full / (t2 - t0), encode=vecs / W_full / (t1 - t0), decode=vecs / W_full / (t2 - t1),
                seconds=t2 - t0, bytes=int(enc["stats"].payload_bytes), vectors=vecs,
                bits_per_component=8.0 * enc["stats"].payload_bytes / (vecs * d),
                ideal_bits_per_component=enc["stats"].ideal_bits / (vecs * d),        # sum of -log2(f/M) + raw bits
                token_bits_per_position=enc["stats"].token_bits / positions)          # sum of -log2 P(x_i | x_<i)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--chunk-pos", type=int, default=None)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-groups", type=int, default=4, help="layer groups (streams) of the host-buffer step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--set", action="append", default=[], help="override a workload field, e.g. --set L=4")
    ap.add_argument("--adaptive", type=int, default=0,
                    help="b0 > 0: surprisal-adaptive step (Def. 7) with hbar = log2(perplexity), cap b0 + 4")
    ap.add_argument("--variant", default="topk", choices=["topk", "dense", "linear"],
                    help="prediction: top-K gather (default), full-vocabulary bf16 tensor-core contraction, or the "
                         "linear-embedding model of Sec. 7.1 (two chained contractions; see --d-model)")
    ap.add_argument("--d-model", type=int, default=4096, help="embedding width of --variant linear")
    ap.add_argument("--rotq", type=int, default=0,
                    help="bits > 0: rotated fixed-rate quantiser on the residual (Prop. 3 step 3) instead of the entropy coder")
    ap.add_argument("--sigma-floor", type=float, default=0.0,
                    help="standard deviation added in quadrature to the mixture's before the scale class is taken")
    ap.add_argument("--zero-rate", type=float, default=0.0,
                    help="D > 0: zero-rate rule (Thm. 3), positions with mixture variance <= D carry no symbols")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    import torch
    from paper_2604_15356_b200 import workloads

    if args.impl == "reference":
        if rank != 0:
            return 0
        return reference_arm(args, workloads)

    import paper_2604_15356_b200 as plc
    plc.build()
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if args.workload == "append":
        return append_arm(args, torch, plc, workloads, dev)
    if args.workload == "dedup":
        return dedup_arm(args, torch, plc, workloads, dev)
    if args.rotq > 0:
        return rotq_arm(args, torch, plc, workloads, dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    over = {}
    for kvs in args.set:
        k, v = kvs.split("=")
        over[k] = float(v) if "." in v else int(v)
    if args.chunk_pos:
        over["chunk_pos"] = args.chunk_pos
    linear = args.variant == "linear"
    if linear:
        over["dm"] = args.d_model
    w = workloads.build(args.workload, dev, seed=20260415 + 1000 * rank, **over)
    cfg = w["cfg"]
    S, n, L, H, d, V, K = cfg["S"], cfg["n"], cfg["L"], cfg["H"], cfg["d"], cfg["V"], cfg["K"]
    W = 2 * L * H
    dense = args.variant == "dense"
    import math
    adaptive = (args.adaptive, 4, math.log2(cfg["pp"])) if args.adaptive > 0 else None
    tok = w["tokens"] if adaptive else None
    if linear:
        ctx = plc.Context.linear(w["E"], w["A"], w["c"], cfg["delta"], chunk_pos=cfg["chunk_pos"], out_dtype=plc.OUT_F16,
                                 zero_rate_D=args.zero_rate, sigma_floor=args.sigma_floor)
    else:
        ctx = plc.Context(w["T"], K, cfg["delta"], chunk_pos=cfg["chunk_pos"], out_dtype=plc.OUT_F16,
                          variant=plc.PRED_DENSE if dense else plc.PRED_TOPK, adaptive=adaptive, zero_rate_D=args.zero_rate,
                          sigma_floor=args.sigma_floor)
        ctx.reserve(S * n)
    ctx.set_profiling(True)
    mc = ctx.max_chunks(n)
    kv_bytes = w["kv"].numel() * 2
    st = plc.StreamSet(S * W, mc, int(0.70 * kv_bytes) + (1 << 20), dev)
    out = torch.empty_like(w["kv"])
    tokens_per_step = S * n

    def step():
        st.total_bytes.zero_()
        ctx.encode(w["kv"], w["logits"], st, tokens=tok)
        ctx.decode(st, w["logits"], out, tokens=tok)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 1)):
        step()
    barrier()
    assert ctx.sync_status() == plc.OK, "device status after warm-up"
    ctx.stats(reset=True)

    uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid)
    launches0 = plc.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3 * args.steps)]
    enc_k, dec_k, gemm_k = [], [], []
    barrier()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        st.total_bytes.zero_()
        ev[3 * i].record()
        ctx.encode(w["kv"], w["logits"], st, tokens=tok)
        ev[3 * i + 1].record()
        ctx.decode(st, w["logits"], out, tokens=tok)
        ev[3 * i + 2].record()
        enc_k.append(ctx.last_kernel_ms(0)); dec_k.append(ctx.last_kernel_ms(1))
        if dense or linear:
            gemm_k.append(ctx.last_kernel_ms(2))
    t_end.record()
    barrier()
    launches = plc.launch_count() - launches0
    clocks = sampler.stop()
    total_ms = t_start.elapsed_time(t_end)
    enc_ms = [ev[3 * i].elapsed_time(ev[3 * i + 1]) for i in range(args.steps)]
    dec_ms = [ev[3 * i + 1].elapsed_time(ev[3 * i + 2]) for i in range(args.steps)]
    assert ctx.sync_status() == plc.OK, "device status after the timed region"
    stats = ctx.stats()
    payload_per_step = stats.payload_bytes / args.steps
    chunks_per_step = stats.n_chunks / args.steps

    ms_per_step = max_over_ranks(total_ms, dist, dev) / args.steps
    value = job_value(world, tokens_per_step, ms_per_step)

    # spot check of the decoded batch (outside the timed region)
    sel = torch.randint(0, n, (64,), device=dev)
    err = float((out[:, :, :, :, sel].float() - w["kv"][:, :, :, :, sel].float()).abs().max())
    if not args.zero_rate:      # skipped positions are bounded in expectation only
        assert err <= cfg["delta"] * (2.0 ** (args.adaptive - 1) if adaptive else 1.0) / 2 + 1e-3 + 8 * 2 ** -11, err

    peak, peak_kind = measured_peaks()
    vecs = S * n * W
    ek, dk = statistics.mean(enc_k), statistics.mean(dec_k)
    gathered = vecs * K * d * 2
    bytes_ns = vecs * d * 2 + gathered + payload_per_step    # KV + T rows read + bitstream (either direction)
    bytes_c = vecs * d * 2 + (0 if linear else w["T"].numel() * 2) + payload_per_step
    dom_enc = ek >= dk
    dom_ms = ek if dom_enc else dk
    sm_mhz = clocks.get("sm_mhz") or 1965.0
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    fma_peak = sms * 128 * sm_mhz * 1e6                      # fp32 FMA/s at the sampled clock
    fma_ach = vecs * K * d / (dom_ms / 1e3)
    dom_name = "encode_kernel" if dom_enc else "decode_kernel"
    default_cfg = args.workload == "llama2-7b" and not over and not dense and not adaptive and not linear and not args.zero_rate and not args.sigma_floor
    traffic = NCU_DRAM_BYTES_PER_VECTOR[dom_name] * vecs if default_cfg else None
    roofline = {"kernel": dom_name, "bound": "hbm",
                "achieved": bytes_ns / (dom_ms / 1e3) / 1e9, "peak": peak, "unit": "GB/s",
                "frac": bytes_ns / (dom_ms / 1e3) / 1e9 / peak, "traffic": traffic, "peak_kind": peak_kind,
                "traffic_note": "ncu dram bytes of a 4-layer capture scaled by vectors; far below the algorithmic bytes "
                                "because gathered T rows are L1 / L2 hits, not HBM reads",
                "accounting": "KV + gathered T rows (K*d*2 B per vector, mostly served by L2) + bitstream, per launch",
                "bytes_per_launch": bytes_ns, "ms_per_launch": dom_ms,
                "compulsory": {"bytes_per_launch": bytes_c, "achieved": bytes_c / (dom_ms / 1e3) / 1e9,
                               "frac": bytes_c / (dom_ms / 1e3) / 1e9 / peak},
                "fp32_fma": {"achieved_gfma_s": fma_ach / 1e9, "peak_gfma_s": fma_peak / 1e9, "frac": fma_ach / fma_peak},
                "encode_kernel_ms": ek, "decode_kernel_ms": dk}

    if dense:
        # the contraction dominates: 2 * rows * V * (2H*d) flop per layer and direction
        gm = statistics.mean(gemm_k)
        flop = 2.0 * S * n * V * (2 * H * d)
        pk = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
        tpeak = float(pk.get("bf16_tflops_sustained", 1400.0))
        roofline = {"kernel": "dense_gemm_kernel", "bound": "tensor", "achieved": flop / (gm / 1e3) / 1e12, "peak": tpeak,
                    "unit": "TFLOP/s", "frac": flop / (gm / 1e3) / 1e12 / tpeak, "traffic": None,
                    "peak_kind": "measured sustained bf16" if pk else "fallback", "ms_per_launch": gm,
                    "flop_per_launch": flop, "launches_per_step": 2 * L,
                    "coder_kernels_ms_last_layer": {"encode": ek, "decode": dk}}
    if linear:
        # per layer: rows x (2H*d) x d_model; once per call: rows x d_model x V (Ebar) and rows x (L*2H) x V (variance)
        gm = statistics.mean(gemm_k)
        dm = args.d_model
        flop = 2.0 * S * n * dm * (2 * H * d)
        pk = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
        tpeak = float(pk.get("bf16_tflops_sustained", 1400.0))
        roofline = {"kernel": "dense_gemm_kernel", "bound": "tensor", "achieved": flop / (gm / 1e3) / 1e12, "peak": tpeak,
                    "unit": "TFLOP/s", "frac": flop / (gm / 1e3) / 1e12 / tpeak, "traffic": None,
                    "peak_kind": "measured sustained bf16" if pk else "fallback", "ms_per_launch": gm,
                    "flop_per_launch": flop, "launches_per_step": 2 * L,
                    "flop_per_step_all_contractions": 2 * (L * flop + 2.0 * S * n * V * dm + 2.0 * S * n * V * 256 * ((W + 255) // 256)),
                    "coder_kernels_ms_last_layer": {"encode": ek, "decode": dk}}
    e2e = None
    if not args.no_e2e and not linear:
        del out, st
        torch.cuda.empty_cache()

        def make_ctx(Tslice):
            return plc.Context(Tslice, K, cfg["delta"], chunk_pos=cfg["chunk_pos"], out_dtype=plc.OUT_F16,
                               variant=plc.PRED_DENSE if dense else plc.PRED_TOPK, adaptive=adaptive,
                               zero_rate_D=args.zero_rate, sigma_floor=args.sigma_floor)
        e2e = run_e2e(args, torch, plc, make_ctx, w, dev, world, dist, tokens_per_step, tok, args.e2e_groups)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not linear:
        layers, pos = min(L, 2), min(n, 256)
        r = oracle_sample_rate(w, pos, layers)
        cpu = {"value": r["value"], "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"session 0, first {pos} positions, {layers} of {L} layers, all heads ({r['vectors']} vectors, "
                         f"{r['seconds']:.1f} s encode+decode); rate scaled by W={W} vectors per KV token",
               "encode": r["encode"], "decode": r["decode"],
               "sample_bits_per_component": r["bits_per_component"],
               "sample_ideal_bits_per_component": r["ideal_bits_per_component"],
               "sample_token_bits_per_position": r["token_bits_per_position"]}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "S": S, "n": n, "L": L, "H": H, "d": d, "V": V, "K": K,
                       "delta": cfg["delta"], "chunk_pos": cfg["chunk_pos"], "perplexity": cfg["pp"],
                       "kv_dtype": "f16", "decode_out": "f16", "variant": args.variant, "adaptive_b0": args.adaptive, "zero_rate_D": args.zero_rate, "sigma_floor": args.sigma_floor,
                       "l2": "inputs larger than L2 (KV+logits %.1f GB per step)" % ((kv_bytes + w["logits"].numel() * 2) / 1e9)},
            "encode_tokens_s": tokens_per_step / (statistics.mean(enc_ms) / 1e3),
            "decode_tokens_s": tokens_per_step / (statistics.mean(dec_ms) / 1e3),
            "encode_ms": statistics.mean(enc_ms), "decode_ms": statistics.mean(dec_ms),
            "bits_per_token": 8 * (payload_per_step + 12 * chunks_per_step) / tokens_per_step,
            "bits_per_component": 8 * payload_per_step / (vecs * d),
            "paper_bound_bits_per_token": "3.3-4.3 at perplexity 10-20 (Cor. 1: theory for the token stream, not this synthetic KV)",
            "escapes_per_step": stats.n_escapes / args.steps,
            "skipped_vector_fraction": stats.skipped_vectors / max(stats.coded_vectors, 1),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def append_arm(args, torch, plc, workloads, dev):
    """Decode-time append: B sessions grow by one token per plc_append_step; per-step latency.
    `--steps` counts groups of 32 append steps (one chunk seal per group)."""
    from paper_2604_15356_b200 import synth
    over = {}
    for kvs in args.set:
        k, v = kvs.split("=")
        over[k] = float(v) if "." in v else int(v)
    cfg = dict(workloads.CONFIGS["append"]); cfg.update(over)
    B, L, H, d, V, K, CP = cfg["S"], cfg["L"], cfg["H"], cfg["d"], cfg["V"], cfg["K"], cfg["chunk_pos"]
    nsteps = CP * max(args.steps, 1)
    W = 2 * L * H
    seed = 20260419
    table = synth.markov_table(V, cfg["pp"], seed, device=dev)
    tokens = synth.sample_tokens(table, B, nsteps, seed + 1)
    logits = synth.position_logits(table, tokens)                       # [B][nsteps][V]
    T = synth.make_tables(L, H, V, d, seed + 2, device=dev)
    ctx = plc.Context(T, K, cfg["delta"], chunk_pos=CP)
    sb = ctx.new_session_batch(B, nsteps // CP + 1, int(nsteps * B * W * d * 1.4) + (1 << 20))
    g = torch.Generator(device=dev); g.manual_seed(seed + 3)
    lat = []
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nsteps)]
    launches0 = plc.launch_count()
    for i in range(nsteps):
        tok = tokens[:, i].to(torch.int64)
        kv_step = (T[:, :, :, tok, :].permute(0, 1, 3, 2, 4).float() +
                   cfg["sigma"] * torch.randn(L, 2, B, H, d, device=dev, generator=g)).to(torch.float16).contiguous()
        lg = logits[:, i, :].contiguous()
        torch.cuda.synchronize()
        ev[i][0].record()
        ctx.append_step(sb, kv_step, lg)
        ev[i][1].record()
    torch.cuda.synchronize()
    assert ctx.sync_status() == plc.OK
    lat = sorted(a.elapsed_time(b) for a, b in ev[CP:])                 # first chunk = warm-up
    seal = sorted(ev[i][0].elapsed_time(ev[i][1]) for i in range(CP, nsteps) if (i + 1) % CP == 0)
    st = ctx.stats()
    mean_ms = sum(lat) / len(lat)
    peak, kind = measured_peaks()
    gathered = B * W * K * d * 2
    line = {"metric": METRIC, "value": B / (mean_ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": nsteps - CP, "warmup": CP,
            "ms_per_step": mean_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": "append", "B": B, "L": L, "H": H, "d": d, "V": V, "K": K, "delta": cfg["delta"],
                       "chunk_pos": CP, "perplexity": cfg["pp"], "encode_only": True},
            "latency_ms": {"p50": lat[len(lat) // 2], "p99": lat[int(len(lat) * 0.99)], "max": lat[-1],
                           "seal_steps_mean": sum(seal) / max(len(seal), 1)},
            "bits_per_token": 8 * (st.payload_bytes + 12 * st.n_chunks) / max(st.coded_vectors / W, 1),
            "roofline": {"kernel": "append_quantise_kernel", "bound": "hbm", "achieved": gathered / (lat[len(lat) // 2] / 1e3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": gathered / (lat[len(lat) // 2] / 1e3) / 1e9 / peak,
                         "traffic": None, "peak_kind": kind,
                         "accounting": "random 256-byte T rows per step (B*W*K*d*2 bytes) over the median whole-step time"},
            "gpu_launches": plc.launch_count() - launches0}
    print(json.dumps(line))
    return 0


def dedup_arm(args, torch, plc, workloads, dev):
    """Prefix dedup followed by delta coding of the tails, at the shapes of `llama3-8b-dedup`: S
    sessions whose system prefixes come from a seeded 8-leaf prefix trie.  One step = log2 P of every
    token (top-K softmax kernel), batched LCP / trie metric / parents (plc_prefix_dedup), clusters
    (plc_prefix_clusters), then encode and decode of the non-shared tails, the sessions taken in
    batches of Sb (the logits of all sessions do not fit in memory at once).  Only library calls are
    timed (CUDA events around them); the synthetic inputs of a batch are generated between them.
    `--steps` repeats the whole pipeline; the first `--warmup` repetitions are not counted."""
    from paper_2604_15356_b200 import synth
    over = {}
    for kvs in args.set:
        k, v = kvs.split("=")
        over[k] = float(v) if "." in v else int(v)
    cfg = dict(workloads.CONFIGS["llama3-8b-dedup"]); cfg.update(over)
    S, n, L, H, d, V, K, CP = cfg["S"], cfg["n"], cfg["L"], cfg["H"], cfg["d"], cfg["V"], cfg["K"], cfg["chunk_pos"]
    Sb = int(cfg.get("Sb", 8))
    assert S % Sb == 0
    W = 2 * L * H
    seed = 20260417
    table = synth.markov_table(V, cfg["pp"], seed, alpha=cfg["alpha"], max_states=cfg.get("max_states", 4096), device=dev)
    seg_lo, seg_hi = int(cfg.get("seg_lo", 128)), int(cfg.get("seg_hi", 1024))
    tokens, keys, leaf, plen = synth.trie_sessions(table, S, n, seed + 1, seg_lo, seg_hi)
    T = synth.make_tables(L, H, V, d, seed + 2, device=dev)
    ctx = plc.Context(T, K, cfg["delta"], chunk_pos=CP, out_dtype=plc.OUT_F16)
    ctx.reserve(Sb * n)
    mc = ctx.max_chunks(n)
    kv = torch.empty(L, 2, Sb, H, n, d, dtype=torch.float16, device=dev)
    out = torch.empty_like(kv)
    st = plc.StreamSet(Sb * W, mc, int(0.70 * kv.numel() * 2) + (1 << 20), dev)
    lens = torch.full((S,), n, dtype=torch.int32, device=dev)
    logp2 = torch.empty(S, n, dtype=torch.float32, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    reps, stats_keep = [], None
    launches0 = plc.launch_count()
    for rep in range(args.warmup + args.steps):
        t = {"logp2": 0.0, "dedup": 0.0, "encode": 0.0, "decode": 0.0}
        spans = []

        def timed(key, fn):
            a, b = ev(), ev()
            a.record(); r = fn(); b.record()
            spans.append((key, a, b))
            return r
        for b0 in range(0, S, Sb):                                     # stage 1: edge weights of the trie
            lg = synth.position_logits(table, tokens[b0:b0 + Sb])
            o = timed("logp2", lambda: ctx.topk_softmax(lg, tokens[b0:b0 + Sb].reshape(-1), want=("logp2",)))
            logp2[b0:b0 + Sb] = o["logp2"].view(Sb, n)
            del lg
        lcp, dT, parent, shared = timed("dedup", lambda: ctx.prefix_dedup(tokens, lens, logp2))
        cl, ce, be = timed("dedup", lambda: ctx.prefix_clusters(lcp, dT, float(cfg.get("cluster_bits", 64.0))))
        ctx.stats(reset=True)
        worst = 0.0
        for b0 in range(0, S, Sb):                                     # stage 2: tails only
            tb = tokens[b0:b0 + Sb]
            lg = synth.position_logits(table, tb)
            synth.make_kv(T, tb, cfg["sigma"], seed + 3, keys=keys[b0:b0 + Sb], out=kv)
            pb, pe = shared[b0:b0 + Sb].contiguous(), lens[b0:b0 + Sb].contiguous()
            st.total_bytes.zero_()
            timed("encode", lambda: ctx.encode(kv, lg, st, pb, pe))
            out.zero_()
            timed("decode", lambda: ctx.decode(st, lg, out, pb, pe))
            torch.cuda.synchronize()
            assert ctx.sync_status() == plc.OK
            for s_ in range(Sb):                                       # decoded tails against the input
                m = int(pb[s_])
                if m < n:
                    worst = max(worst, float((out[:, :, s_, :, m:].float() - kv[:, :, s_, :, m:].float()).abs().max()))
            del lg
        torch.cuda.synchronize()
        for key, a, b in spans:
            t[key] += a.elapsed_time(b)
        assert worst <= cfg["delta"] / 2 + 1e-3 + 8 * 2 ** -11, worst
        if rep >= args.warmup:
            reps.append(t)
            stats_keep = ctx.stats()
    launches = plc.launch_count() - launches0
    mean = {k: sum(r[k] for r in reps) / len(reps) for k in reps[0]}
    total_ms = sum(mean.values())
    sh = shared.cpu().numpy().astype("int64")
    coded = int((n - sh).sum())
    peak, kind = measured_peaks()
    logits_bytes = 2.0 * S * n * V
    line = {"metric": METRIC, "value": coded / (total_ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": "dedup (llama3-8b-dedup shapes)", "S": S, "n": n, "L": L, "H": H, "d": d, "V": V, "K": K,
                       "delta": cfg["delta"], "chunk_pos": CP, "perplexity": cfg["pp"], "session_batch": Sb,
                       "prefix_trie": "15 segments of U[%d,%d] tokens, 8 leaves" % (seg_lo, seg_hi),
                       "value_counts": "coded (non-shared) token positions; shared prefixes cost no bits and no time"},
            "stage_ms": mean,
            "covered_tokens_s": S * n / (total_ms / 1e3),
            "shared_fraction": float(sh.sum()) / (S * n), "mean_shared_len": float(sh.mean()),
            "sessions_with_parent": int((parent.cpu().numpy() >= 0).sum()),
            "clusters_at_%g_bits" % float(cfg.get("cluster_bits", 64.0)): int(len(set(cl.cpu().numpy().tolist()))),
            "bits_per_token": 8 * (stats_keep.payload_bytes + 12 * stats_keep.n_chunks) / max(coded, 1),
            "bits_per_component": 8 * stats_keep.payload_bytes / max(stats_keep.coded_vectors * d, 1),
            "relative_storage_vs_no_dedup": coded / float(S * n),
            "roofline": {"kernel": "topk_softmax_kernel", "bound": "hbm", "achieved": logits_bytes / (mean["logp2"] / 1e3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": logits_bytes / (mean["logp2"] / 1e3) / 1e9 / peak,
                         "traffic": None, "peak_kind": kind,
                         "accounting": "logits read once (2*S*n*V bytes) over the summed log2 P launches; the encode and "
                                       "decode calls scan the logits of the coded positions once more each"},
            "gpu_launches": launches}
    print(json.dumps(line))
    return 0


def rotq_arm(args, torch, plc, workloads, dev):
    """Predict, rotate and quantise the residual to `--rotq` bits per component (fixed-size records),
    then decode; same workloads, same prediction kernels, no entropy coder."""
    over = {}
    for kvs in args.set:
        k, v = kvs.split("=")
        over[k] = float(v) if "." in v else int(v)
    w = workloads.build(args.workload, dev, seed=20260415, **over)
    cfg = w["cfg"]
    S, n, L, H, d, V, K = cfg["S"], cfg["n"], cfg["L"], cfg["H"], cfg["d"], cfg["V"], cfg["K"]
    W = 2 * L * H
    ctx = plc.Context(w["T"], K, cfg["delta"], chunk_pos=cfg["chunk_pos"], out_dtype=plc.OUT_F16)
    ctx.reserve(S * n)
    g = torch.Generator().manual_seed(7)
    params = ctx.rotq_params(args.rotq, torch.randint(0, 2, (d,), generator=g).tolist())
    rb = ctx.rotq_record_bytes(args.rotq)
    records = torch.empty(S * W * n * rb, dtype=torch.uint8, device=dev)
    out = torch.empty_like(w["kv"])
    for _ in range(max(args.warmup, 1)):
        ctx.encode_rotq(w["kv"], w["logits"], params, records)
        ctx.decode_rotq(records, w["logits"], params, out)
    torch.cuda.synchronize()
    assert ctx.sync_status() == plc.OK
    uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid)
    launches0 = plc.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps + 1)]
    ev[0].record()
    for i in range(args.steps):
        ctx.encode_rotq(w["kv"], w["logits"], params, records)
        ev[2 * i + 1].record()
        ctx.decode_rotq(records, w["logits"], params, out)
        ev[2 * i + 2].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = plc.launch_count() - launches0
    enc = statistics.mean(ev[2 * i].elapsed_time(ev[2 * i + 1]) for i in range(args.steps))
    dec = statistics.mean(ev[2 * i + 1].elapsed_time(ev[2 * i + 2]) for i in range(args.steps))
    ms = ev[0].elapsed_time(ev[-1]) / args.steps
    diff = out.float() - w["kv"].float()
    rms = float(diff.pow(2).mean().sqrt())
    peak, kind = measured_peaks()
    vecs = S * n * W
    bytes_ns = vecs * d * 2 + vecs * K * d * 2 + vecs * rb
    line = {"metric": METRIC, "value": S * n / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "S": S, "n": n, "L": L, "H": H, "d": d, "V": V, "K": K, "quantiser": "rotated, %d bits" % args.rotq,
                       "chunk_pos": cfg["chunk_pos"], "l2": "inputs larger than L2"},
            "encode_ms": enc, "decode_ms": dec, "bits_per_component": 8.0 * rb / d, "bits_per_token": 8.0 * rb * W,
            "rms_error": rms, "max_error": float(diff.abs().max()),
            "roofline": {"kernel": "rotq_kernel", "bound": "hbm", "achieved": bytes_ns / (max(enc, dec) / 1e3) / 1e9, "peak": peak,
                         "unit": "GB/s", "frac": bytes_ns / (max(enc, dec) / 1e3) / 1e9 / peak, "traffic": None, "peak_kind": kind,
                         "accounting": "KV + gathered T rows (K*d*2 B per vector, served by L1 / L2) + records, per call (top-K included)"},
            "gpu_launches": launches, "clocks": clocks}
    print(json.dumps(line))
    return 0


def run_e2e(args, torch, plc, make_ctx, w, dev, world, dist, tokens_per_step, tok=None, groups=4):
    """Same step with HOST buffers: pinned inputs are copied in, the coded bytes and index are
    copied out and back in, the decoded KV is copied out -- all inside the timed region.  The
    layers are cut into groups, each with its own context and CUDA stream, so that the copies of
    one group overlap the kernels and the opposite-direction copies of the others."""
    cfg = w["cfg"]
    S, n, L, H, d = cfg["S"], cfg["n"], cfg["L"], cfg["H"], cfg["d"]
    G = groups if (L % groups == 0 and args.variant == "topk") else 1
    Lg = L // G
    kv_h = w["kv"].cpu().pin_memory()
    lg_h = w["logits"].cpu().pin_memory()
    kvo_h = torch.empty_like(kv_h).pin_memory()
    kv_d, lg_d, out_d = torch.empty_like(w["kv"]), torch.empty_like(w["logits"]), torch.empty_like(w["kv"])
    ctxs, sts, pay_h, off_h, nby_h, tot_h, streams = [], [], [], [], [], [], []
    for g in range(G):
        c = make_ctx(w["T"][g * Lg:(g + 1) * Lg])
        c.reserve(S * n)
        ctxs.append(c)
        st = plc.StreamSet(S * c.W, c.max_chunks(n), int(0.70 * kv_h.numel() * 2 / G) + (1 << 20), dev)
        sts.append(st)
        pay_h.append(torch.empty(st.payload.numel(), dtype=torch.uint8).pin_memory())
        off_h.append(torch.empty_like(st.chunk_offset, device="cpu").pin_memory())
        nby_h.append(torch.empty_like(st.chunk_bytes, device="cpu").pin_memory())
        tot_h.append(torch.zeros(1, dtype=torch.int64).pin_memory())
        streams.append(torch.cuda.Stream(device=dev))
    ev0 = torch.cuda.Event()

    def step():
        main = torch.cuda.current_stream()
        lg_d.copy_(lg_h, non_blocking=True)
        ev0.record(main)
        for g in range(G):
            lo, hi = g * Lg, (g + 1) * Lg
            with torch.cuda.stream(streams[g]):
                streams[g].wait_event(ev0)
                kv_d[lo:hi].copy_(kv_h[lo:hi], non_blocking=True)
                sts[g].total_bytes.zero_()
                ctxs[g].encode(kv_d[lo:hi], lg_d, sts[g], tokens=tok)
                tot_h[g].copy_(sts[g].total_bytes, non_blocking=True)
        used_all = 0
        for g in range(G):
            lo, hi = g * Lg, (g + 1) * Lg
            streams[g].synchronize()                          # the byte count decides how much to copy out
            used = int(tot_h[g][0]); used_all += used
            st = sts[g]
            with torch.cuda.stream(streams[g]):
                pay_h[g][:used].copy_(st.payload[:used], non_blocking=True)
                off_h[g].copy_(st.chunk_offset, non_blocking=True); nby_h[g].copy_(st.chunk_bytes, non_blocking=True)
                st.payload[:used].copy_(pay_h[g][:used], non_blocking=True)
                st.chunk_offset.copy_(off_h[g], non_blocking=True); st.chunk_bytes.copy_(nby_h[g], non_blocking=True)
                ctxs[g].decode(st, lg_d, out_d[lo:hi], tokens=tok)
                kvo_h[lo:hi].copy_(out_d[lo:hi], non_blocking=True)
        for g in range(G):
            main.wait_stream(streams[g])
        return used_all

    used = step()
    torch.cuda.synchronize()
    for c in ctxs:
        assert c.sync_status() == plc.OK
    err = float((kvo_h[:, :, :, :, :64].float() - kv_h[:, :, :, :, :64].float()).abs().max())
    assert err <= cfg["delta"] * (2.0 ** (args.adaptive - 1) if args.adaptive > 0 else 1.0) / 2 + 1e-3 + 8 * 2 ** -11, err
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.e2e_steps):
        used = step()
    t1.record()
    torch.cuda.synchronize()
    ms = max_over_ranks(t0.elapsed_time(t1) / args.e2e_steps, dist, dev)
    idx_bytes = sum(o.numel() * 8 + b.numel() * 4 for o, b in zip(off_h, nby_h))
    return {"value": job_value(world, tokens_per_step, ms), "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": kv_h.numel() * 2 + lg_h.numel() * 2 + used + idx_bytes,
            "d2h_bytes_per_step": used + idx_bytes + 8 * G + kvo_h.numel() * 2, "steps": args.e2e_steps,
            "layer_groups": G}


def reference_arm(args, workloads):
    """The reference arm is the CPU oracle as it stands, on a bounded sample of the same workload."""
    cfg = dict(workloads.CONFIGS[args.workload])
    layers, pos = 1, min(cfg["n"], 64)
    # the sample is built on the CPU at the sample's own size (same recipe)
    w = workloads.build(args.workload, "cpu", seed=20260415, S=1, n=pos, L=layers, max_states=64)
    w["cfg"]["L"] = cfg["L"]                                  # the rate is scaled to the full number of streams
    for _ in range(min(args.warmup, 1)):
        oracle_sample_rate(w, pos, layers)
    rates = []
    t0 = time.perf_counter()
    for _ in range(args.steps):
        rates.append(oracle_sample_rate(w, pos, layers))
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = statistics.mean(r["value"] for r in rates)
    W = 2 * cfg["L"] * cfg["H"]
    sample = (f"1 session, {pos} positions, {layers} of {cfg['L']} layers, all heads "
              f"({rates[0]['vectors']} vectors per step); rate scaled by W={W} vectors per KV token")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
