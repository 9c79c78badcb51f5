"""Host-side logic of the multi-GPU benchmark path on CPU (gloo, world size 2): ranks code their
own batches with no data-path collective; only the timing is reduced (max over ranks)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    q.put((rank, ms, bench.job_value(world, 1000, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_time_is_max_over_ranks_and_value_is_whole_job():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29517, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 15.0                                    # the slower rank decides
        assert abs(value - 2 * 1000 / 15e-3) < 1e-6          # tokens of both ranks / that time


def _shard_worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    S, L, H, mc = 3, 5, 2, 4                                   # an odd layer count: the shards differ in size
    mine = bench.shard_slots(S, L, H, mc, world, rank)
    every = [None] * world
    dist.all_gather_object(every, sorted(mine))                # host-side bookkeeping only; no data-path collective
    total = torch.tensor([float(len(mine))])
    dist.all_reduce(total)                                     # the one reduction of the report (a count, like the byte total)
    q.put((rank, bench.shard_layers(L, world, rank), every, float(total[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_layer_shards_partition_the_single_gpu_slot_set():
    """--shard layers: rank r codes the streams of layers [rL/N, (r+1)L/N) of ONE batch.  The ranks'
    (session, table, chunk) slots are disjoint and their union is the single-GPU run's slot set."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, 29519, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import bench
    S, L, H, mc = 3, 5, 2, 4
    full = bench.shard_slots(S, L, H, mc, 1, 0)
    assert len(full) == S * 2 * L * H * mc
    assert [r[1] for r in res] == [(0, 2), (2, 5)]
    for rank, layers, every, total in res:
        a, b = set(map(tuple, every[0])), set(map(tuple, every[1]))
        assert not (a & b) and (a | b) == full and total == len(full)
        assert all(layers[0] * 2 * H <= t < layers[1] * 2 * H for _, t, _ in map(tuple, every[rank]))
    # any world size: contiguous, exhaustive, sizes within one of each other
    for world in (1, 2, 3, 4, 8):
        cuts = [bench.shard_layers(32, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == 32 and all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        assert max(hi - lo for lo, hi in cuts) - min(hi - lo for lo, hi in cuts) <= 1


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, None, torch.device("cpu")) == 7.5
    assert bench.job_value(1, 16384, 100.0) == 163840.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
