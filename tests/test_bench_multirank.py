"""The N > 1 logic of bench.py on CPU: two gloo ranks, max-over-ranks timing,
whole-job value for independent replicas; the reference arm prints on rank 0
only."""
from __future__ import annotations

import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + rank, 5.0 - rank]               # rank 1 is slower on the first timer
    got = bench.max_over_ranks(mine, "cpu")
    # a leg is entered only if every rank can (rank 1 cannot here)
    got.append(bench.all_ranks_ok(rank == 0, "cpu"))
    got.append(bench.all_ranks_ok(True, "cpu"))
    dist.barrier()
    q.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks():
    import bench
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0] == results[1] == [11.0, 5.0, False, True]
    # two replicas of 1e9 parameters at 11 ms per step
    assert bench.whole_job_value(2, 10 ** 9, 11.0) == 2 * 10 ** 9 / 11e-3


def test_reference_arm_prints_one_line_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "tiny", "--steps", "2", "--warmup", "1", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "tiny", "--steps", "2", "--warmup", "1", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["value"] > 0 and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["unit"] == "params/s" and line["n_gpus"] == 2


def _sharded_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200.sharded import ShardedAdamW

    class HP:
        lr, beta1, beta2, eps, weight_decay, max_grad_norm = 1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0

    shard = ShardedAdamW(10 * 512 + 7, 512, dry_run=True)
    for b in range(shard.info.n_buckets):
        B.so_debug_set_bucket_stats(shard.ctx, b, 4.0 if rank == 1 else 0.001, 0)
    decisions = bench.sharded_steps(shard, HP(), 3)
    q.put((rank, decisions, shard.info.n_buckets, B.so_get_step(shard.ctx), shard.exchange_bytes))
    shard.close()
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_bench_loop_with_two_gloo_ranks():
    """The loop `bench.py --sharded` times, on two CPU ranks in dry-run mode:
    bucket ranges per rank, one exchange per iteration, the same global verdict
    (rank 1's large gradients make both ranks clip)."""
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import build as so_build
    so_build.build_library()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 27500 + os.getpid() % 2000
    procs = [ctx.Process(target=_sharded_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = {r[0]: r[1:] for r in (q.get(timeout=180) for _ in procs)}
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][0] == got[1][0] == [B.SO_DECISION_CLIP_RESTEP] * 3
    assert got[0][1] + got[1][1] == 11 and abs(got[0][1] - got[1][1]) <= 1
    assert got[0][2] == got[1][2] == 3 and got[0][3] == 24
