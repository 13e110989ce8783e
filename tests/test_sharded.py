"""Optimizer states sharded by bucket ranges (Section 4.7): the only exchange
is one small all-reduce of the local sum of squares, NaN/Inf flag and error flag.  Host
logic with two gloo ranks on CPU; on the GPU two shards of one model are run
side by side in one process and compared with the unsharded run."""
from __future__ import annotations

import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_ranges_tile_the_parameter_space():
    from paper_2509_21271_b200.sharded import shard_range
    for total, bucket, world in [(1000, 256, 2), (1000, 256, 3), (1024, 256, 8), (5, 7, 2),
                                 (8_030_261_248, 200_000_000, 8)]:
        edges = [shard_range(total, bucket, r, world) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == total
        for (lo, hi), (lo2, _) in zip(edges, edges[1:]):
            assert lo <= hi == lo2
        for lo, hi in edges[:-1]:
            assert lo % bucket == 0 and (hi % bucket == 0 or hi == total)
        counts = [-(-(hi - lo) // bucket) for lo, hi in edges]
        assert max(counts) - min(counts) <= 1


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200.sharded import ShardedAdamW

    class HP:
        lr, beta1, beta2, eps, weight_decay, max_grad_norm = 1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0

    opt = ShardedAdamW(7 * 256 + 100, 256, dry_run=True)     # 8 buckets: 4 per rank
    out = []
    # iteration 1: small gradients everywhere -> COMMIT; 2: rank 1 is large -> both clip;
    # iteration 3: rank 0 sees an infinity -> both skip
    plans = [({0: 0.01, 1: 0.02}, None), ({0: 0.01, 1: 50.0}, None), ({0: 0.01, 1: 0.02}, 0)]
    for per_rank, bad_rank in plans:
        for b in range(opt.info.n_buckets):
            B.so_debug_set_bucket_stats(opt.ctx, b, per_rank[rank] / opt.info.n_buckets,
                                        1 if (bad_rank == rank and b == 1) else 0)
        r = opt.iteration(HP())
        out.append((r.decision, r.stats.sumsq, r.stats.norm, r.stats.nonfinite, r.step_after))
    q.put((rank, (opt.lo, opt.hi), out))
    opt.close()
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_global_verdict():
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import build as so_build
    so_build.build_library()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = {}
    for _ in procs:
        rank, rng, out = q.get(timeout=180)
        got[rank] = (rng, out)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][0] == (0, 1024) and got[1][0] == (1024, 7 * 256 + 100)
    a, b = got[0][1], got[1][1]
    assert a == b                                            # same global values on both ranks
    decisions = [x[0] for x in a]
    assert decisions == [B.SO_DECISION_COMMIT, B.SO_DECISION_CLIP_RESTEP, B.SO_DECISION_SKIP]
    assert a[0][1] == pytest.approx(0.03) and a[1][1] == pytest.approx(50.01)
    assert a[2][3] == 1 and [x[4] for x in a] == [1, 2, 2]


@pytest.mark.gpu
def test_two_shards_on_one_gpu_equal_the_unsharded_run():
    """Two shard contexts, stepped one after the other in one process (no
    kernel waits on another), with the combined sum handed to both: the union
    of their states is bit for bit the unsharded state."""
    import numpy as np
    from gpu_harness import hparams_of
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import workloads as W
    from paper_2509_21271_b200.optimizer import BucketedAdamW
    from paper_2509_21271_b200.sharded import shard_range

    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()
    w = W.tiny_ragged()
    hp = hparams_of(w)
    p0 = W.initial_master(w, device="cuda")
    whole = BucketedAdamW(w.numel, w.bucket_elems)
    whole.load_state(p0)
    whole.cast_params(stream=stream)
    ranges = [shard_range(w.total, w.bucket_elems, r, 2) for r in range(2)]
    shards = []
    for lo, hi in ranges:
        s = BucketedAdamW([hi - lo], w.bucket_elems)
        s.load_state(p0[lo:hi])
        s.cast_params(stream=stream)
        shards.append(s)
    for step in range(1, 9):
        g = W.gradients(w, step, device="cuda")
        whole.load_grads(g)
        ref = whole.iteration(hp, stream=stream)
        locals_ = []
        for s, (lo, hi) in zip(shards, ranges):
            s.load_grads(g[lo:hi])
            s.step_speculative(hp, B.SO_ALL, stream)
            locals_.append(s.grad_check(hp, B.SO_ALL, stream))
        total = locals_[0].sumsq + locals_[1].sumsq
        flag = locals_[0].nonfinite | locals_[1].nonfinite
        assert flag == ref.stats.nonfinite
        if not flag:
            assert total == pytest.approx(ref.stats.sumsq, rel=1e-14)
        for s in shards:
            # the unsharded sum is one valid order of the same global sum
            B.so_set_global_grad_stats(s.ctx, ref.stats.sumsq if not flag else total, flag)
            res = s.validate(hp, stream)
            assert (res.decision, res.step_after) == (ref.decision, ref.step_after)
            if not flag:
                assert res.stats.clip_coef == ref.stats.clip_coef
    torch.cuda.synchronize()
    ref_state = [x.cpu().numpy() for x in whole.gather_state()]
    ref_pb = whole.gather_param_bf16().view(torch.int16).cpu().numpy()
    for s, (lo, hi) in zip(shards, ranges):
        for a, b in zip([x.cpu().numpy() for x in s.gather_state()], ref_state):
            assert a.tobytes() == b[lo:hi].tobytes()
        assert np.array_equal(s.gather_param_bf16().view(torch.int16).cpu().numpy(), ref_pb[lo:hi])


def _failing_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200.sharded import ShardedAdamW, ShardFailure

    class HP:
        lr, beta1, beta2, eps, weight_decay, max_grad_norm = 1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0

    opt = ShardedAdamW(8 * 256, 256, dry_run=True)
    for b in range(opt.info.n_buckets):
        B.so_debug_set_bucket_stats(opt.ctx, b, 0.001, 0)
    log = []
    r = opt.iteration(HP())
    log.append(("ok", r.decision, r.step_after))
    # iteration 2: rank 1's device raises its status word (a kernel gave up a wait)
    if rank == 1:
        B.so_debug_set_bucket_stats(opt.ctx, B.SO_ALL, 0.0, 1)
    try:
        opt.iteration(HP())
        log.append(("ok",))
    except ShardFailure as e:
        log.append(("failed", e.failed_ranks, e.local_error is not None))
    # both ranks gave the iteration up the same way and can go on
    c = B.so_get_counters(opt.ctx)
    log.append((B.so_get_step(opt.ctx), B.so_pending_buckets(opt.ctx), c.timeouts, c.skips,
                [B.so_bucket_slot(opt.ctx, b) for b in range(opt.info.n_buckets)]))
    r = opt.iteration(HP())
    log.append(("ok", r.decision, r.step_after))
    q.put((rank, log))
    opt.close()
    dist.barrier()
    dist.destroy_process_group()


def test_a_failed_local_check_ends_the_iteration_on_every_rank():
    """One rank's local check fails; it still joins the exchange, every rank
    learns of it from the same all-reduce, gives the iteration up and raises;
    nobody is left waiting in a collective, and the next iteration runs."""
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import build as so_build
    so_build.build_library()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_failing_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank in (0, 1):
        log = got[rank]
        assert log[0] == ("ok", B.SO_DECISION_COMMIT, 1)
        assert log[1] == ("failed", 1, rank == 1)
        step, pending, timeouts, skips, slots = log[2]
        assert (step, pending, timeouts, skips) == (1, 4, 1, 0)
        assert sorted(slots) == [4, 5, 6, 7]            # the map of iteration 1, untouched
        assert log[3] == ("ok", B.SO_DECISION_COMMIT, 2)


def test_abandon_iteration_state_machine():
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import build as so_build
    so_build.build_library()

    class HP:
        lr, beta1, beta2, eps, weight_decay, max_grad_norm = 1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0

    ctx, _ = B.so_layout_init([1000], 256, B.SO_GRAD_BF16, 2)
    B.so_debug_set_dry_run(ctx, True)
    a = 0x10000000
    B.so_layout_bind(ctx, a, 2 * a, 3 * a, 4 * a, 5 * a, 6 * a)
    B.so_abandon_iteration(ctx)                              # idle: a no-op
    assert B.so_get_counters(ctx).timeouts == 0
    B.so_adam_step_speculative(ctx, HP(), B.SO_ALL)          # buckets 0, 1
    B.so_grad_check(ctx, None, 3)
    B.so_abandon_iteration(ctx)
    c = B.so_get_counters(ctx)
    assert c.timeouts == 1 and c.elems_cast == 512 and B.so_get_step(ctx) == 0
    assert B.so_pending_buckets(ctx) == 4
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [0, 1, 2, 3]
    B.so_adam_step_speculative(ctx, HP(), B.SO_ALL)
    B.so_grad_check(ctx, HP(), B.SO_ALL)
    B.so_abandon_iteration(ctx)                              # also after the check
    assert B.so_get_counters(ctx).timeouts == 2
    B.so_adam_step_speculative(ctx, HP(), 0)
    B.so_validate_begin(ctx, HP())
    with pytest.raises(B.SuperOffloadError) as err:
        B.so_abandon_iteration(ctx)                          # a begun validation must be collected
    assert err.value.status == B.SO_ERR_STATE
    r = B.so_validate_commit_or_rollback(ctx, HP())
    assert r.step_after == 1
    B.so_destroy(ctx)


@pytest.mark.gpu
def test_sharded_layer_on_a_real_process_group_against_the_oracle():
    """ShardedAdamW as it runs in production -- CUDA tensors through an NCCL
    all-reduce and all-gather -- on a one-rank group on cuda:0, through COMMIT,
    CLIP_RESTEP and SKIP, element by element against the oracle."""
    import numpy as np
    import oracle
    from gpu_harness import (Report, assert_bf16_consistent, bf16_to_numpy, check_stats,
                             compare_state, grads_to_numpy, hparams_of)
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import workloads as W
    from paper_2509_21271_b200.sharded import ShardedAdamW

    torch.cuda.set_device(0)
    port = 35500 + os.getpid() % 2000
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        w = W.tiny_ragged()
        w.sigma_g = 1.0
        w.target_norm = lambda step: 0.5 if step % 2 == 1 else 3.0
        w.faults = (W.Fault(step=3, flat_index=2 * 250_003 + 17, kind="inf"),)
        hp = hparams_of(w)
        stream = torch.cuda.current_stream()
        opt = ShardedAdamW(w.total, w.bucket_elems, undo_slots=3)
        assert (opt.lo, opt.hi) == (0, w.total) and opt.reduce_device.type == "cuda"
        p0 = W.initial_master(w, device="cuda")
        opt.local.load_state(p0)
        opt.local.cast_params(stream=stream)
        p = p0.cpu().numpy()
        m, v = np.zeros_like(p), np.zeros_like(p)
        pb = oracle.bf16_rne(p)
        rep, t = Report(), 0
        for step in range(1, 6):
            g = W.gradients(w, step, device="cuda")
            opt.local.load_grads(g)
            res = opt.iteration(hp, stream)
            torch.cuda.synchronize()
            forced = res.stats.clip_coef if res.decision == B.SO_DECISION_CLIP_RESTEP else None
            orc = oracle.iteration_stv(p, m, v, pb, grads_to_numpy(g), w.bucket_elems, t, hp,
                                       forced_coef=forced)
            assert res.decision == orc.decision
            check_stats(res.stats, orc, hp.max_grad_norm, rep)
            t = orc.step_after
            assert res.step_after == t
            rep.decisions.append(res.decision)
            dev = [x.cpu().numpy() for x in opt.local.gather_state()]
            full = opt.all_gather_param_bf16()
            assert full.numel() == w.total
            compare_state(dev, (p, m, v), rep)
            assert_bf16_consistent(bf16_to_numpy(full), dev[0], pb, p, rep)
            p, m, v, pb = dev[0], dev[1], dev[2], bf16_to_numpy(full)
        assert rep.decisions == [B.SO_DECISION_COMMIT, B.SO_DECISION_CLIP_RESTEP, B.SO_DECISION_SKIP,
                                 B.SO_DECISION_CLIP_RESTEP, B.SO_DECISION_COMMIT]
        opt.close()
    finally:
        dist.destroy_process_group()
