"""Optimizer states sharded by bucket ranges across the ranks of a process group.

Each rank owns a contiguous range of the global buckets and a
:class:`BucketedAdamW` over just that range (the paper's multi-Superchip mode,
Section 4.7: every process updates only its own subset of the parameters).
The element updates need nothing from the other ranks; the only exchange is
the global gradient check: one all-reduce of the local sum of squares (SUM)
and of the local NaN/Inf flag (MAX), 16 bytes, handed back to the library with
``so_set_global_grad_stats`` before validation.  An all-gather of the bf16
parameter shards is offered for callers that keep a full low-precision copy.

Plumbing only: ``torch.distributed`` moves two doubles; every step of the path
runs in the library's kernels.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist

from . import binding as B
from .optimizer import BucketedAdamW


def shard_range(total_elems: int, bucket_elems: int, rank: int, world: int) -> Tuple[int, int]:
    """Flat [lo, hi) owned by `rank`: buckets are dealt in contiguous runs, the
    first ``n_buckets % world`` ranks taking one bucket more."""
    n_buckets = -(-total_elems // bucket_elems)
    base, extra = divmod(n_buckets, world)
    first = rank * base + min(rank, extra)
    count = base + (1 if rank < extra else 0)
    lo = min(first * bucket_elems, total_elems)
    hi = min((first + count) * bucket_elems, total_elems)
    return lo, hi


class ShardedAdamW:
    """This rank's shard of a bucketized AdamW over `total_elems` parameters."""

    def __init__(self, total_elems: int, bucket_elems: int, grad_dtype: str = "bf16",
                 undo_slots: int = B.SO_ALL, device: str = "cuda",
                 group: Optional[dist.ProcessGroup] = None, dry_run: bool = False):
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.total_elems = total_elems
        self.lo, self.hi = shard_range(total_elems, bucket_elems, self.rank, self.world)
        self.dry_run = dry_run
        if dry_run:          # host logic only (CPU tests): no arenas, no launches
            gd = {"bf16": B.SO_GRAD_BF16, "fp32": B.SO_GRAD_FP32, "fp16": B.SO_GRAD_FP16}[grad_dtype]
            self.ctx, self.info = B.so_layout_init([self.hi - self.lo], bucket_elems, gd, undo_slots)
            B.so_debug_set_dry_run(self.ctx, True)
            a = 0x10000000
            B.so_layout_bind(self.ctx, a, 2 * a, 3 * a, 4 * a, 5 * a, 6 * a)
            self.local = None
            self.reduce_device = torch.device("cpu")
        else:
            self.local = BucketedAdamW([self.hi - self.lo], bucket_elems, grad_dtype, undo_slots,
                                       device=device)
            self.ctx, self.info = self.local.ctx, self.local.info
            self.reduce_device = self.local.device

    def iteration(self, hp, stream=None):
        """Speculate the local buckets, check locally, all-reduce the two
        scalars, validate on the global values."""
        B.so_adam_step_speculative(self.ctx, hp, B.SO_ALL, stream)
        local = B.so_grad_check(self.ctx, hp, B.SO_ALL, stream)
        sums = torch.tensor([local.sumsq], dtype=torch.float64, device=self.reduce_device)
        flag = torch.tensor([float(local.nonfinite)], dtype=torch.float64,
                            device=self.reduce_device)
        if self.world > 1:
            dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=self.group)
            dist.all_reduce(flag, op=dist.ReduceOp.MAX, group=self.group)
        B.so_set_global_grad_stats(self.ctx, float(sums.item()), int(flag.item() != 0.0))
        return B.so_validate_commit_or_rollback(self.ctx, hp, stream)

    def all_gather_param_bf16(self) -> torch.Tensor:
        """The full bf16 parameter vector, assembled from every rank's shard."""
        mine = self.local.gather_param_bf16()
        sizes = [shard_range(self.total_elems, self.info.bucket_elems, r, self.world)
                 for r in range(self.world)]
        longest = max(hi - lo for lo, hi in sizes)
        padded = torch.zeros(longest, dtype=torch.bfloat16, device=mine.device)
        padded[:mine.numel()] = mine
        parts = [torch.empty_like(padded) for _ in range(self.world)]
        if self.world > 1:
            dist.all_gather(parts, padded, group=self.group)
        else:
            parts = [padded]
        return torch.cat([p[:hi - lo] for p, (lo, hi) in zip(parts, sizes)])

    def close(self) -> None:
        if self.local is not None:
            self.local.close()
        elif self.ctx is not None:
            B.so_destroy(self.ctx)
        self.ctx = None
