"""The paper's closed-form placement models, fed with rates measured here.

Two small calculators, host-only arithmetic:

* the efficiency model of Section 4.2 (Eq. 1-3): the time to compute a forward
  pass against the time to stream the low-precision weights in,
  ``efficiency = comp / (comp + comm)``, with forward FLOPs ~ 2 * bsz * seq *
  params and 2 bytes moved per parameter;
* the bucket repartitioning inequality of Section 4.3 (Eq. 4-5): the number n
  of trailing buckets whose optimizer state should stay on the GPU so that the
  last offloaded bucket (gradient out, CPU step, parameters back) hides behind
  the backward pass and the GPU-side step of those n buckets.

They are models, not measurements: `step_gpu` is what this library measures
(params/s of the fused step), everything else is an input.
"""
from __future__ import annotations

from dataclasses import dataclass


def forward_efficiency(params: float, batch: float, seq: float, peak_flops: float,
                       link_bytes_per_s: float, bytes_per_param: float = 2.0) -> float:
    """Eq. 1-3: comp = 2*bsz*seq*params / peak, comm = bytes_per_param*params / bw."""
    comp = 2.0 * batch * seq * params / peak_flops
    comm = bytes_per_param * params / link_bytes_per_s
    return comp / (comp + comm)


def min_batch_for_efficiency(target: float, seq: float, peak_flops: float,
                             link_bytes_per_s: float, bytes_per_param: float = 2.0) -> int:
    """Smallest integer batch size whose forward efficiency reaches `target`
    (the model size cancels out of Eq. 3)."""
    b = 1
    while forward_efficiency(1.0, b, seq, peak_flops, link_bytes_per_s, bytes_per_param) < target:
        b += 1
        if b > 1 << 20:
            raise ValueError("target efficiency is not reachable")
    return b


@dataclass
class Rates:
    """Throughputs in elements (parameters) per second unless stated."""
    move_grad: float          # offloaded gradient bucket, GPU -> CPU
    move_param: float         # updated parameters, CPU -> GPU
    step_cpu: float           # optimizer step on the CPU
    step_gpu: float           # optimizer step on the GPU (this library)
    bwd: float                # parameters whose backward pass completes per second


def gpu_resident_buckets(bucket_elems: float, n_buckets: int, r: Rates) -> int:
    """Eq. 4-5: the smallest n with
        move(grad) + step_cpu(bucket) + move(param) <= bwd(n*bucket) + step_gpu(n*bucket),
    capped at n_buckets (everything stays on the GPU)."""
    exposed = bucket_elems / r.move_grad + bucket_elems / r.step_cpu + bucket_elems / r.move_param
    per_bucket_cover = bucket_elems / r.bwd + bucket_elems / r.step_gpu
    n = 0
    while n * per_bucket_cover < exposed and n < n_buckets:
        n += 1
    return n
