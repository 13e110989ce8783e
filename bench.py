#!/usr/bin/env python
"""Benchmark of the bucketized speculative AdamW step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A "step" is one pass of the whole hot path over one synthetic gradient batch:
speculative fused AdamW+cast step of every bucket, the global gradient check
(finalised from the tile sums the step left behind), and the validation
decision with whatever it entails (a commit on this workload).  Prints one JSON
line: optimizer params/s over all GPUs (`value`, inputs resident in HBM), the
same through the host-buffer entry point (`e2e`), the HBM roofline of the
fused step kernel, and the CPU oracle timed on a bounded sample.

With N > 1 (launched by torchrun) every rank runs an independent replica of
the workload on its own GPU -- the path has no exchange step on one node --
and the value is N x params / max-over-ranks time.

Side modes, each printing a JSON line of its own: --scan (the stand-alone
gradient check), --pack (one-launch flattening between per-tensor buffers and
the arenas), --placement (the paper's placement models fed with this box's
rates), --sharded (optimizer states sharded by bucket ranges over the ranks).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "optimizer_params_per_sec"
UNIT = "params/s"
BYTES_PER_PARAM = {"bf16": 28, "fp16": 28, "fp32": 30}      # algorithmic HBM bytes of the fused step
GRAD_BYTES = {"bf16": 2, "fp16": 2, "fp32": 4}
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0             # vendor figure for B200 HBM3e, quoted for context
# The largest configuration that fits one GPU: Llama-3-8B-shaped, 8.03 G
# parameters in 41 buckets of 200 M elements, 128.5 GB resident.
DEFAULT_WORKLOAD = "llama_8b"
# dram__bytes_read.sum + dram__bytes_write.sum per parameter of the fused step
# kernel (gpt2_small capture: 1.742 GB read + 1.688 GB written per launch of
# 124 439 808 parameters; profiles/adamw_step_tma_kernel_gpt2_small.md), scaled
# to the launch by the parameters it processes (traffic is proportional)
NCU_TRAFFIC_BYTES_PER_PARAM = 27.57


def _measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs:
    NVML polled from a thread every few milliseconds (the timed region of the
    default workload lasts tens of milliseconds), nvidia-smi as a fallback."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []                  # (sm_mhz, max_mhz, set of reason names)
        self.proc = None
        self.thread = None
        self._stop = threading.Event()
        self._nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self._nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read_smi, daemon=True)
        self.thread.start()

    def _physical_index(self) -> int:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        if vis:
            ids = [x.strip() for x in vis.split(",") if x.strip()]
            if self.index < len(ids) and ids[self.index].isdigit():
                return int(ids[self.index])
        return self.index

    def _poll_nvml(self):
        nv = self._nvml
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(self._handle, nv.NVML_CLOCK_SM)
                mx = nv.nvmlDeviceGetMaxClockInfo(self._handle, nv.NVML_CLOCK_SM)
                mask = get_reasons(self._handle)
                self.rows.append((float(sm), float(mx), {k for k, bit in names.items() if mask & bit}))
            except Exception:
                pass
            time.sleep(0.003)

    def _read_smi(self):
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) != 6:
                continue
            try:
                sm, mx = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            self.rows.append((sm, mx, {n for n, v in zip(names, parts[2:])
                                       if v.lower().startswith("active")}))

    def mark(self):
        """Number of samples so far (to cut out the timed region afterwards)."""
        return len(self.rows)

    def stop(self, first: int = 0, last: int = None):
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        rows = self.rows[first:last] or self.rows
        sm = sorted(r[0] for r in rows)
        reasons = set().union(*[r[2] for r in rows]) if rows else set()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None,
                "sm_max_mhz": rows[-1][1] if rows else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "source": "nvml" if self._nvml else "nvidia-smi"}


def max_over_ranks(values, device):
    """Element-wise maximum over all ranks of the default process group."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def all_ranks_ok(ok: bool, device) -> bool:
    """True only if `ok` holds on every rank of the default process group (a
    leg with barriers inside must be entered by all ranks or by none)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([1.0 if ok else 0.0], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MIN)
    return bool(t.item() == 1.0)


def whole_job_value(world: int, params_per_replica: int, ms_per_step: float) -> float:
    """Replicas only: every rank steps its own copy of the workload, so the
    job's throughput is world x params over the slowest rank's step time."""
    return world * params_per_replica / (ms_per_step * 1e-3)


def sharded_steps(shard, hp, steps: int, stream=None):
    """`steps` iterations of this rank's shard (speculative steps of the local
    buckets, local check, the one small all-reduce, validation on the global
    values).  Returns the decisions; all ranks see the same ones."""
    return [shard.iteration(hp, stream).decision for _ in range(steps)]


def run_sharded(args, w, torch, dist, rank, world, local_rank):
    """Optimizer states sharded by bucket ranges over the ranks (the paper's
    multi-Superchip mode): strong scaling of one model, one 24-byte all-reduce
    per iteration inside the timed region."""
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import workloads as W
    from paper_2509_21271_b200.sharded import ShardedAdamW

    hp = _hparams(w)
    stream = torch.cuda.current_stream()
    shard = ShardedAdamW(w.total, w.bucket_elems, w.grad_dtype, args.undo_slots if args.undo_slots >= 0
                         else B.SO_ALL)
    n_local = shard.hi - shard.lo
    mine = W.Workload(name=f"{w.name}_shard{rank}", numel=[n_local], bucket_elems=w.bucket_elems,
                      sigma_g=w.sigma_g, seed=w.seed + 17 * rank, max_grad_norm=w.max_grad_norm,
                      grad_dtype=w.grad_dtype, target_norm=w.target_norm)
    shard.local.load_state_stream(W.iter_initial_master(mine, device="cuda"))
    shard.local.cast_params(stream=stream)
    shard.local.load_grads_stream(W.iter_gradients(mine, 1, device="cuda"))
    torch.cuda.synchronize()
    sharded_steps(shard, hp, args.warmup, stream)
    torch.cuda.synchronize()
    dist.barrier()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    decisions = sharded_steps(shard, hp, args.steps, stream)
    t1.record(stream)
    torch.cuda.synchronize()
    dist.barrier()
    torch.cuda.synchronize()
    (elapsed_ms,) = max_over_ranks([t0.elapsed_time(t1)], "cuda")
    if rank == 0:
        ms = elapsed_ms / args.steps
        from paper_2509_21271_b200.binding import DECISION_NAMES
        print(json.dumps({
            "metric": METRIC, "value": w.total / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "params": w.total, "bucket_elems": w.bucket_elems,
                       "parallelism": "zero_buckets", "buckets_rank0": shard.info.n_buckets,
                       "exchange_bytes_per_step": shard.exchange_bytes,
                       "decisions": sorted({DECISION_NAMES[d] for d in decisions}),
                       "verdict": "global statistics combined on the host (one all-reduce), "
                                  "applied on the device"},
            "hbm_gbs_whole_step": BYTES_PER_PARAM[w.grad_dtype] * w.total / (ms * 1e-3) / 1e9}))
    shard.close()


def measure_link(torch, n_bytes: int = 1 << 30, repeats: int = 5):
    """Pinned host <-> device copy rates of this machine (one cudaMemcpyAsync of
    `n_bytes` each way, best of `repeats`, CUDA events), in bytes/s."""
    host = torch.empty(n_bytes, dtype=torch.uint8, pin_memory=True)
    dev = torch.empty(n_bytes, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    best = {}
    for name, dst, src in (("h2d", dev, host), ("d2h", host, dev)):
        times = []
        for _ in range(repeats + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            dst.copy_(src, non_blocking=True)
            e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        best[name] = n_bytes / (min(times[1:]) * 1e-3)
    # both directions at once (what overlapped iterations ask of the link): the
    # rate each way while the other is busy, from the time both copies took
    host2 = torch.empty(n_bytes, dtype=torch.uint8, pin_memory=True)
    dev2 = torch.empty(n_bytes, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    times = []
    for _ in range(repeats + 1):
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        side.wait_event(e0)
        dev.copy_(host, non_blocking=True)
        with torch.cuda.stream(side):
            host2.copy_(dev2, non_blocking=True)
            e2.record(side)
        stream.wait_event(e2)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    best["both"] = n_bytes / (min(times[1:]) * 1e-3)
    return best


PLACEMENT_CONFIGS = (("gpt2_small", 124_439_808, 25_000_000), ("llama_1b", 1_235_814_400, 100_000_000),
                     ("llama_8b", 8_030_261_248, 200_000_000))


def placement_table(step_gpu: float, step_cpu: float, h2d_bytes_s: float, d2h_bytes_s: float,
                    gemm_flops: float, seq: int = 1024, batches=(1, 4, 8)):
    """The paper's two placement models fed with rates measured on this machine.

    Section 4.3 (Eq. 4-5): n = buckets whose optimizer state should stay on the
    GPU so that the last offloaded bucket (gradient out, CPU step, parameters
    back) hides behind the backward pass and the GPU-side step of those n
    buckets; the backward pass costs 4 * bsz * seq FLOPs per parameter.
    Section 4.2 (Eq. 1-3): the smallest batch size at which streaming the
    low-precision weights in hides behind the forward pass (efficiency 60 %)."""
    from paper_2509_21271_b200 import placement_model as M
    rows = []
    for name, total, bucket in PLACEMENT_CONFIGS:
        nb = -(-total // bucket)
        for bsz in batches:
            rates = M.Rates(move_grad=d2h_bytes_s / 2.0, move_param=h2d_bytes_s / 2.0,
                            step_cpu=step_cpu, step_gpu=step_gpu,
                            bwd=gemm_flops / (4.0 * bsz * seq))
            rows.append({"workload": name, "n_buckets": nb, "bucket_elems": bucket, "batch": bsz,
                         "seq": seq, "n_gpu_resident": M.gpu_resident_buckets(bucket, nb, rates)})
    try:
        min_batch = M.min_batch_for_efficiency(0.6, seq, gemm_flops, h2d_bytes_s)
    except ValueError:
        min_batch = None
    return {"rows": rows, "min_batch_for_60pct_forward_efficiency": min_batch,
            "forward_efficiency_at_batch_4": M.forward_efficiency(1.0, 4, seq, gemm_flops, h2d_bytes_s)}


def run_placement(args, torch):
    """`--placement`: measure this box's rates and print what the paper's
    models make of them (one JSON line)."""
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import workloads as W
    from paper_2509_21271_b200.optimizer import BucketedAdamW

    link = measure_link(torch)
    w = W.by_name("llama_1b" if args.workload == DEFAULT_WORKLOAD else args.workload)
    hp = _hparams(w)
    stream = torch.cuda.current_stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, B.SO_ALL)
    opt.load_state_stream(W.iter_initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    opt.load_grads_stream(W.iter_gradients(w, 1, device="cuda"))
    for _ in range(3):
        opt.iteration(hp, stream=stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(10):
        opt.iteration(hp, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    step_gpu = w.total * 10 / (e0.elapsed_time(e1) * 1e-3)
    opt.close()
    cpu = _oracle_all_cores(w, 5.0)
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            gemm = float(json.load(fh)["bf16_tflops_sustained"]) * 1e12
        gemm_kind = "measured (sustained bf16 GEMM)"
    except Exception:
        gemm, gemm_kind = 1.4e15, "fallback"
    table = placement_table(step_gpu, cpu["value"], link["h2d"], link["d2h"], gemm)
    print(json.dumps({"placement": table,
                      "inputs": {"step_gpu_params_s": step_gpu, "step_gpu_workload": w.name,
                                 "step_cpu_params_s": cpu["value"], "cpu_cores": cpu["cores"],
                                 "cpu_model": cpu.get("cpu_model"),
                                 "h2d_gbs": link["h2d"] / 1e9, "d2h_gbs": link["d2h"] / 1e9,
                                 "gemm_flops": gemm, "gemm_kind": gemm_kind}}))


def run_pack(args, torch):
    """`--pack`: time the one-launch flattening (`so_layout_pack_grads`,
    `so_layout_unpack_params`) over the workload's tensor list, each tensor in a
    buffer of its own, against the per-tensor copies it replaces (one JSON
    line; bytes moved = 2 x element size x N per call)."""
    from paper_2509_21271_b200 import workloads as W
    from paper_2509_21271_b200.optimizer import BucketedAdamW

    w = W.by_name("llama_1b" if args.workload == DEFAULT_WORKLOAD else args.workload)
    stream = torch.cuda.current_stream()
    peak, peak_kind = _measured_peak()
    rows = []
    for off_grid in (False, True):
        opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 0)
        esz = opt.grad.element_size()
        grads, params = [], []
        for i, n in enumerate(w.numel):
            lead = (i % 2) * 3 if off_grid else 0          # every other tensor 3 elements off the 16-byte grid
            grads.append(torch.zeros(n + 8, dtype=opt.grad_torch_dtype, device="cuda")[lead:lead + n])
            params.append(torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda")[lead:lead + n])
        row = {"tensors_off_the_16_byte_grid": off_grid}
        for what, fn, bytes_moved in (("pack", lambda: opt.pack_grads(grads, stream), 2 * esz * w.total),
                                      ("unpack", lambda: opt.unpack_params(params, stream), 4 * w.total)):
            for _ in range(max(3, args.warmup)):
                fn()
            torch.cuda.synchronize()
            times = []
            for _ in range(max(5, args.steps)):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn()
                e1.record(stream)
                torch.cuda.synchronize()
                times.append(e0.elapsed_time(e1))
            times.sort()
            med = times[len(times) // 2]
            row[what] = {"ms_median": med, "gbs": bytes_moved / med / 1e6,
                         "frac": bytes_moved / med / 1e6 / peak}

        def per_tensor_copies():
            pos = 0
            for t in grads:
                opt._scatter(opt.grad, pos, t)
                pos += t.numel()
        for _ in range(2):
            per_tensor_copies()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        per_tensor_copies()
        e1.record(stream)
        torch.cuda.synchronize()
        row["per_tensor_copies_ms"] = e0.elapsed_time(e1)
        rows.append(row)
        opt.close()
        del grads, params
        torch.cuda.empty_cache()
    print(json.dumps({"pack": rows, "workload": w.name, "tensors": len(w.numel), "params": w.total,
                      "peak_gbs": peak, "peak_kind": peak_kind,
                      "timing": "CUDA events around each call (pointer upload and launch included)"}))


def run_scan(args, torch):
    """`--scan`: time the stand-alone gradient check (`so_grad_check(SO_ALL)`:
    one batched scan launch, the two-level reduction, the statistics sent to the
    host) over the workload's gradients, CUDA events around the call (one JSON
    line; algorithmic bytes = the gradient's element size x N)."""
    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import workloads as W
    from paper_2509_21271_b200.optimizer import BucketedAdamW

    w = W.by_name("llama_1b" if args.workload == DEFAULT_WORKLOAD else args.workload)
    hp = _hparams(w)
    stream = torch.cuda.current_stream()
    peak, peak_kind = _measured_peak()
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 0)
    if w.grad_dtype == "fp16":
        B.so_loss_scale_config(opt.ctx, w.loss_scale, w.ls_growth, w.ls_backoff, w.ls_interval)
    opt.load_grads_stream(W.iter_gradients(w, 1, device="cuda", loss_scale=w.loss_scale))
    torch.cuda.synchronize()
    times, stats = [], None
    for it in range(max(3, args.warmup) + max(5, args.steps)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        stats = B.so_grad_check(opt.ctx, hp, B.SO_ALL, stream)
        e1.record(stream)
        B.so_abandon_iteration(opt.ctx, stream)        # close the iteration without stepping
        torch.cuda.synchronize()
        if it >= max(3, args.warmup):
            times.append(e0.elapsed_time(e1))
    times.sort()
    med, best = times[len(times) // 2], times[0]
    n_bytes = w.total * opt.grad.element_size()
    print(json.dumps({"scan": {"ms_median": med, "ms_best": best, "gbs_median": n_bytes / med / 1e6,
                               "gbs_best": n_bytes / best / 1e6, "frac": n_bytes / med / 1e6 / peak,
                               "peak_gbs": peak, "peak_kind": peak_kind},
                      "workload": w.name, "params": w.total, "grad_dtype": w.grad_dtype,
                      "loss_scale": w.loss_scale, "norm": stats.norm,
                      "timing": "CUDA events around so_grad_check(SO_ALL): scan launch, reduction, "
                                "statistics to the host"}))
    opt.close()


def _hparams(w, oracle_mod=None):
    from paper_2509_21271_b200.binding import so_hparams
    return so_hparams(w.lr, w.beta1, w.beta2, w.eps, w.weight_decay, w.max_grad_norm)


ORACLE_SAMPLE_ELEMS = 64 << 20       # slice of the workload the CPU legs run on
ORACLE_THREAD_ELEMS = 4 << 20       # bucket each thread of the all-cores leg owns


def _oracle_inputs(w, n):
    """Seeded inputs of the first n parameters of the workload, as numpy."""
    import numpy as np
    import torch

    import oracle
    from paper_2509_21271_b200 import workloads as W

    sample = W.Workload(name=w.name + "_sample", numel=[n], bucket_elems=n, sigma_g=w.sigma_g,
                        seed=w.seed, max_grad_norm=w.max_grad_norm, grad_dtype=w.grad_dtype)
    hp = oracle.HParams(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                        weight_decay=w.weight_decay, max_grad_norm=w.max_grad_norm)
    p = W.initial_master(sample).numpy()
    g = W.gradients(sample, 1, loss_scale=w.loss_scale)
    g = g.view(torch.int16).numpy().view(np.uint16) if g.dtype == torch.bfloat16 else g.numpy()
    return p, g, hp


def _oracle_sample(w, steps, warmup):
    """The CPU oracle, as it stands (one thread), on a bounded slice of the
    workload: the first min(bucket, 64 Mi) parameters."""
    import numpy as np

    import oracle

    n = min(w.bucket_elems, w.total, ORACLE_SAMPLE_ELEMS)
    p, g, hp = _oracle_inputs(w, n)
    m, v = np.zeros_like(p), np.zeros_like(p)
    pb = oracle.bf16_rne(p)
    unscale = 1.0 / w.loss_scale
    t = 0
    for _ in range(warmup):
        t = oracle.iteration_ste(p, m, v, pb, g, n, t, hp, unscale=unscale).step_after
    t0 = time.perf_counter()
    for _ in range(steps):
        t = oracle.iteration_ste(p, m, v, pb, g, n, t, hp, unscale=unscale).step_after
    dt = time.perf_counter() - t0
    return {"value": n * steps / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {n} params of {w.name}, {steps} steps of check+AdamW+cast, "
                      f"single thread, {dt:.1f} s"}, dt / steps, n


def _cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def _oracle_all_cores(w, seconds: float = 8.0):
    """The same oracle loop, one bucket per thread on every host core: each
    thread owns a 4 Mi-parameter bucket (its own arrays) and repeats
    check+AdamW+cast on it until the time is up.  The oracle itself stays
    single-threaded C; the threads only run independent copies of it (ctypes
    releases the interpreter lock during the call)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor

    import oracle

    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    n = min(ORACLE_THREAD_ELEMS, w.total)
    p0, g, hp = _oracle_inputs(w, n)
    unscale = 1.0 / w.loss_scale

    def make():
        p = p0.copy()
        return p, np.zeros_like(p), np.zeros_like(p), oracle.bf16_rne(p)
    states = [make() for _ in range(cores)]
    deadline = [0.0]

    def work(i):
        p, m, v, pb = states[i]
        t, done = 0, 0
        while True:
            t = oracle.iteration_ste(p, m, v, pb, g, n, t, hp, unscale=unscale).step_after
            done += 1
            if time.perf_counter() >= deadline[0]:
                return done
    with ThreadPoolExecutor(max_workers=cores) as pool:
        t0 = time.perf_counter()
        deadline[0] = t0 + seconds
        counts = list(pool.map(work, range(cores)))
        dt = time.perf_counter() - t0
    return {"value": n * sum(counts) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "cpu_model": _cpu_model(),
            "sample": f"{cores} threads, one {n}-param bucket of {w.name} each, "
                      f"{sum(counts)} bucket steps of check+AdamW+cast in {dt:.1f} s"}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    base, per_step, n = _oracle_sample(w, args.steps, max(args.warmup, 1))
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": per_step * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sample_params": n, "bucket_elems": w.bucket_elems},
            "cpu_baseline": base,
            "cpu_baseline_all_cores": _oracle_all_cores(w, 5.0),
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_overlap(args, w, opt, hp, B, torch):
    """Speculative steps behind a synthetic bucket-by-bucket backward pass.

    The paper's speculation-then-validation schedule takes the optimizer off the
    critical path by stepping each bucket as soon as its gradients exist, while
    the backward pass goes on (critical path of an iteration: its Eq. 7 against
    Eq. 6).  Here both run on one GPU: the stand-in backward is a chain of bf16
    matmuls per bucket on one stream (library GEMMs: not part of the path, only
    something compute-bound to hide behind), the speculative step of bucket b
    waits on an event recorded after bucket b's matmuls and runs on a second
    stream, validation follows the last step.  Three timings over the same
    number of iterations: backward alone, steps + validation alone, both."""
    main = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    nb = opt.n_buckets
    dim = 4096
    a = torch.randn(dim, dim, device="cuda", dtype=torch.bfloat16)
    b = torch.randn(dim, dim, device="cuda", dtype=torch.bfloat16)
    out = torch.empty(dim, dim, device="cuda", dtype=torch.bfloat16)
    events = [torch.cuda.Event() for _ in range(nb)]

    def steps_only():
        for bk in range(nb):
            B.so_adam_step_speculative(opt.ctx, hp, bk, side)
        B.so_validate_commit_or_rollback(opt.ctx, hp, side)

    def timed(fn, iters):
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(main)
        side.wait_event(t0)
        for _ in range(iters):
            fn()
        done = torch.cuda.Event()
        done.record(side)
        main.wait_event(done)
        t1.record(main)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / iters

    for _ in range(3):
        steps_only()
    t_steps = timed(steps_only, args.steps)
    # matmuls per bucket so that the backward takes about bwd_ratio x the steps
    def backward_only(k):
        for bk in range(nb):
            for _ in range(k):
                torch.matmul(a, b, out=out)
            events[bk].record(main)
    backward_only(4)
    t_mm = timed(lambda: backward_only(4), 3) / (4 * nb)
    k = max(1, round(args.bwd_ratio * t_steps / (nb * t_mm)))
    backward_only(k)
    t_bwd = timed(lambda: backward_only(k), args.steps)

    def overlapped():
        for bk in range(nb):
            for _ in range(k):
                torch.matmul(a, b, out=out)
            events[bk].record(main)
            side.wait_event(events[bk])
            B.so_adam_step_speculative(opt.ctx, hp, bk, side)
        B.so_validate_commit_or_rollback(opt.ctx, hp, side)
    for _ in range(3):
        overlapped()
    t_both = timed(overlapped, args.steps)
    return {"ms_backward_alone": t_bwd, "ms_steps_and_validation_alone": t_steps,
            "ms_overlapped": t_both, "ms_exposed": t_both - t_bwd,
            "ms_serial_sum": t_bwd + t_steps,
            "ms_last_bucket_step": t_steps / nb,
            "matmuls_per_bucket": k, "matmul": f"{dim}x{dim}x{dim} bf16 (library GEMM stand-in)",
            "buckets": nb, "step_launches": "one per bucket, second stream"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--undo-slots", type=int, default=-1)
    ap.add_argument("--per-bucket", action="store_true",
                    help="one speculative-step call per bucket instead of one batched call")
    ap.add_argument("--order", default="stv", choices=["stv", "ste"],
                    help="stv: speculate, then validate (default); ste: gradient check first, "
                         "then the step and cast in place (the synchronous order the paper "
                         "starts from), for comparison")
    ap.add_argument("--overlap", action="store_true",
                    help="also time per-bucket speculative steps behind a synthetic backward pass")
    ap.add_argument("--bwd-ratio", type=float, default=4.0,
                    help="--overlap: length of the synthetic backward in units of the optimizer step")
    ap.add_argument("--sync-verdict", action="store_true",
                    help="collect every verdict on the host before the next iteration is enqueued "
                         "(default: one iteration late)")
    ap.add_argument("--placement", action="store_true",
                    help="measure this box's rates (fused step, pinned copies, all-cores oracle) and "
                         "print what the paper's placement models (Eq. 1-5) make of them")
    ap.add_argument("--scan", action="store_true",
                    help="time the stand-alone gradient check over the workload's gradients")
    ap.add_argument("--pack", action="store_true",
                    help="time the one-launch pack / unpack between per-tensor buffers and the arenas")
    ap.add_argument("--sharded", action="store_true",
                    help="shard the optimizer states by bucket ranges over the ranks (strong "
                         "scaling, one small all-reduce per iteration) instead of running replicas")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="no event pairs around speculative launches in the timed region (no roofline)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--step-variant", type=int, default=0,
                    help="0: chosen by launch size (default), 1: register-only step kernel, "
                         "2: bulk-copy pipeline")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    from paper_2509_21271_b200 import workloads as W
    w = W.by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch

    from paper_2509_21271_b200 import binding as B
    from paper_2509_21271_b200 import build as so_build
    from paper_2509_21271_b200.optimizer import BucketedAdamW

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        so_build.build_library()
    if dist is not None:
        dist.barrier()

    if args.placement or args.pack or args.scan:
        if rank == 0:
            (run_placement if args.placement else run_pack if args.pack else run_scan)(args, torch)
        if dist is not None:
            dist.destroy_process_group()
        return
    if args.sharded:
        if dist is None:
            import torch.distributed as dist
            dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29371", rank=0, world_size=1,
                                    device_id=torch.device("cuda", local_rank))
        run_sharded(args, w, torch, dist, rank, world, local_rank)
        dist.destroy_process_group()
        return

    hp = _hparams(w)
    stream = torch.cuda.current_stream()
    undo = args.undo_slots
    if undo < 0:
        # as many undo slots as fit next to the 16 B/param resident state
        stride = (w.bucket_elems + 63) // 64 * 64
        free_bytes, _ = torch.cuda.mem_get_info()
        gsz_arena = 4 if w.grad_dtype == "fp32" else 2
        resident = w.n_buckets * stride * (12 + gsz_arena + 2)
        room = free_bytes - resident - (6 << 30)
        undo = max(0, min(w.n_buckets, room // (12 * stride)))
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, undo,
                        step_variant=args.step_variant)
    opt.load_state_stream(W.iter_initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    if w.grad_dtype == "fp16":
        B.so_loss_scale_config(opt.ctx, w.loss_scale, w.ls_growth, w.ls_backoff, w.ls_interval)
    opt.load_grads_stream(W.iter_gradients(w, 1, device="cuda", loss_scale=w.loss_scale))
    torch.cuda.synchronize()
    N = w.total
    nb = opt.n_buckets

    def enqueue_steps(ev=None):
        """The speculative part of an iteration (nothing here waits for the GPU)."""
        if args.per_bucket:
            for b in range(nb):
                try:
                    B.so_adam_step_speculative(opt.ctx, hp, b, stream)
                except B.SuperOffloadError as e:
                    if e.status != B.SO_ERR_UNDO_EXHAUSTED:
                        raise
        else:
            if ev is not None:
                ev[0].record(stream)
            B.so_adam_step_speculative(opt.ctx, hp, B.SO_ALL, stream)
            if ev is not None:
                ev[1].record(stream)

    def one_step():
        """One iteration, verdict collected at once (warm-up, check-first order)."""
        if args.order == "ste":
            B.so_grad_check(opt.ctx, hp, B.SO_ALL, stream)
        else:
            enqueue_steps()
        return B.so_validate_commit_or_rollback(opt.ctx, hp, stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing ------------------------------------------
    for _ in range(args.warmup):
        one_step()
    # the fused step kernel is timed on every 4th step of the timed region (an
    # event pair costs a few microseconds of an iteration)
    sampled = set(range(0, args.steps, 4))
    kernel_events = {k: (torch.cuda.Event(enable_timing=True),
                         torch.cuda.Event(enable_timing=True)) for k in sampled}
    launches0 = opt.counters().kernel_launches
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.05)
    decisions = set()

    def timed_steps(marks=None, kernel_ev=None):
        """K iterations.  `marks`: an event after every iteration (per-step
        times); `kernel_ev`: event pairs around the speculative launch of some."""
        kernel_ev = kernel_ev or {}
        if args.order == "ste" or args.sync_verdict:
            for k in range(args.steps):
                if args.order == "ste":
                    decisions.add(one_step().decision)
                else:
                    enqueue_steps(kernel_ev.get(k))
                    decisions.add(B.so_validate_commit_or_rollback(opt.ctx, hp, stream).decision)
                if marks:
                    marks[k + 1].record(stream)
            return
        # The verdict is formed on the device and its follow-up is enqueued with
        # it; the host collects each verdict one iteration late, after it has
        # enqueued the next iteration's speculative steps (Section 4.4: the
        # result of the validation is consulted later, off the critical path).
        for k in range(args.steps):
            enqueue_steps(kernel_ev.get(k))
            if k > 0:
                decisions.add(B.so_validate_commit_or_rollback(opt.ctx, hp, stream).decision)
            B.so_validate_begin(opt.ctx, hp, stream)
            if marks:
                marks[k + 1].record(stream)
        decisions.add(B.so_validate_commit_or_rollback(opt.ctx, hp, stream).decision)

    # region 1, the headline: K iterations between two events; the speculative
    # launch of every 4th iteration carries an event pair for the roofline
    barrier()
    mark0 = sampler.mark()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    timed_steps(kernel_ev=None if args.no_kernel_events else kernel_events)
    t_end.record(stream)
    barrier()
    mark1 = sampler.mark()
    elapsed_ms = t_start.elapsed_time(t_end)
    launches = opt.counters().kernel_launches - launches0
    # region 2: the same K iterations with an event after each, for the spread
    # (the events themselves cost a few microseconds per iteration)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    marks[0].record(stream)
    timed_steps(marks=marks)
    barrier()
    per_step = sorted(marks[k].elapsed_time(marks[k + 1]) for k in range(args.steps))
    median_ms, best_ms = per_step[len(per_step) // 2], per_step[0]
    clocks = sampler.stop(mark0, mark1) if rank == 0 else None
    spec_buckets = min(nb, opt.info.undo_slots)
    spec_params = sum(opt.bucket_range(b)[1] - opt.bucket_range(b)[0] for b in range(spec_buckets))
    kernel_ms = None
    if not args.per_bucket and args.order == "stv" and not args.no_kernel_events:
        times = [a.elapsed_time(b) for a, b in kernel_events.values()]
        kernel_ms = sum(times) / len(times)

    # ---- end to end through the host-buffer entry point -------------------
    e2e = None
    if not args.no_e2e and args.order == "stv":
        gsz = 4 if w.grad_dtype == "fp32" else 2
        try:
            host_g = torch.empty(N, dtype=opt.grad_torch_dtype, pin_memory=True)
            host_p = torch.empty(N, dtype=torch.bfloat16, pin_memory=True)
        except RuntimeError as exc:       # the host refused to pin N * (gsz + 2) bytes
            host_g = host_p = None
            e2e = {"unavailable": f"could not pin {N * (gsz + 2)} bytes of host memory: "
                                  f"{str(exc).splitlines()[0][:120]}"}
        if dist is not None and not all_ranks_ok(host_g is not None, "cuda") and host_g is not None:
            host_g = host_p = None            # another rank could not pin its buffers: no rank runs the leg
            e2e = {"unavailable": "a rank could not pin its host buffers"}
        if host_g is not None:
            for start, piece in W.iter_gradients(w, 1, device="cuda", loss_scale=w.loss_scale):
                host_g[start:start + piece.numel()].copy_(piece)
            # Consecutive iterations overlap on the link: the parameters that can
            # only leave after the verdict travel while the next gradients arrive
            # (so_iteration_host_pipelined); the wait for the last copies is
            # inside the timed region.  Every step copies its gradients in and
            # its parameters out.
            n_warm = 3 if N < (1 << 31) else 1
            for _ in range(n_warm):
                B.so_iteration_host(opt.ctx, hp, host_g.data_ptr(), host_p.data_ptr(), stream)
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_e2e = max(3, min(args.steps, 10))
            e0.record(stream)
            for _ in range(n_e2e):
                B.so_iteration_host_pipelined(opt.ctx, hp, host_g.data_ptr(), host_p.data_ptr(), stream)
            B.so_iteration_host_wait(opt.ctx, stream)
            e1.record(stream)
            barrier()
            e2e_ms = e0.elapsed_time(e1) / n_e2e
            e2e = {"ms": e2e_ms, "h2d": N * gsz, "d2h": N * 2 + 40, "steps": n_e2e}
            del host_g, host_p
            e2e["link"] = measure_link(torch)

    # ---- max over ranks ----------------------------------------------------
    if dist is not None:
        have_e2e = bool(e2e) and "ms" in e2e
        elapsed_ms, e2e_ms, median_ms, best_ms = max_over_ranks(
            [elapsed_ms, e2e["ms"] if have_e2e else 0.0, median_ms, best_ms], "cuda")
        if have_e2e:
            e2e["ms"] = e2e_ms
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = elapsed_ms / args.steps
    value = whole_job_value(world, N, ms_per_step)
    peak, peak_kind = _measured_peak()
    bpp = BYTES_PER_PARAM[w.grad_dtype]
    roofline = None
    if kernel_ms:
        achieved = bpp * spec_params / (kernel_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "adamw_step_tma_kernel (fused speculative AdamW step + bf16 cast + tile sums)",
                    "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}",
                    "unit": "GB/s", "frac": achieved / peak,
                    "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                    "traffic": (NCU_TRAFFIC_BYTES_PER_PARAM * spec_params
                                if NCU_TRAFFIC_BYTES_PER_PARAM else None),
                    "bytes_per_param": bpp, "params_per_launch": spec_params,
                    "kernel_ms": kernel_ms, "launches_timed": len(kernel_events)}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "median_ms": median_ms,
        "best_ms": best_ms, "median_best_from": "a second pass of the same steps with an event after each",
        "timed_region_s": elapsed_ms * 1e-3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "params": N, "tensors": len(w.numel),
                   "bucket_elems": w.bucket_elems, "n_buckets": nb,
                   "undo_slots": opt.info.undo_slots, "grad_dtype": w.grad_dtype,
                   "max_grad_norm": w.max_grad_norm,
                   "decisions": sorted(B.DECISION_NAMES[d] for d in decisions),
                   "order": args.order,
                   "verdict": "on the device; collected by the host "
                              + ("at once" if (args.sync_verdict or args.order == "ste")
                                 else "one iteration late"),
                   "launch_mode": "per_bucket" if args.per_bucket else "batched",
                   "step_kernel": {0: "by launch size: bulk-copy pipeline, register kernel for launches "
                                       "of at most 3 Mi elements",
                                    1: "registers", 2: "bulk_copy_pipeline"}[args.step_variant],
                   "parallelism": "replicas" if world > 1 else "single",
                   "l2": f"working set {16 * N / 1e6:.0f} MB resident + undo slots, "
                         "larger than the 126 MB L2; no flush"},
        # check-first reads the gradients twice: once to check, once to step
        "hbm_gbs_whole_step": world * (bpp + (GRAD_BYTES[w.grad_dtype] if args.order == "ste" else 0))
                              * N / (ms_per_step * 1e-3) / 1e9,
        # bytes the step actually moves: buckets beyond the undo window are
        # scanned first (one more gradient read) and stepped in place afterwards
        "hbm_gbs_whole_step_moved": world * (bpp * N + GRAD_BYTES[w.grad_dtype] *
                                             (N if args.order == "ste" else N - spec_params))
                                    / (ms_per_step * 1e-3) / 1e9,
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if clocks and clocks.get("sm_mhz"):
        line["ms_per_step_x_sm_mhz"] = ms_per_step * clocks["sm_mhz"]
    if roofline:
        line["roofline"] = roofline
    if e2e and "ms" in e2e:
        line["e2e"] = {"value": world * N / (e2e["ms"] * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                       "ms_per_step": e2e["ms"], "steps": e2e["steps"],
                       "link_gbs_each_way": e2e["h2d"] / (e2e["ms"] * 1e-3) / 1e9,
                       # ceiling: both directions run at once, so a step cannot be
                       # shorter than the slower direction's copy at the measured rate
                       "pinned_h2d_gbs": e2e["link"]["h2d"] / 1e9,
                       "pinned_d2h_gbs": e2e["link"]["d2h"] / 1e9,
                       "pinned_each_way_when_both_gbs": e2e["link"]["both"] / 1e9,
                       "frac_of_link": max(e2e["h2d"] / e2e["link"]["h2d"],
                                           e2e["d2h"] / e2e["link"]["d2h"]) / (e2e["ms"] * 1e-3),
                       "frac_of_link_both_ways": max(e2e["h2d"], e2e["d2h"]) / e2e["link"]["both"]
                                                 / (e2e["ms"] * 1e-3)}
    elif e2e:
        line["e2e"] = e2e
    if args.overlap and world == 1:
        line["overlap"] = run_overlap(args, w, opt, hp, B, torch)
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = _oracle_sample(w, 10, 1)[0]
        line["cpu_baseline_all_cores"] = _oracle_all_cores(w)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
