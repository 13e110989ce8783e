"""Optimizer states sharded by bucket ranges across the ranks of a process group.

Each rank owns a contiguous range of the global buckets and a
:class:`BucketedAdamW` over just that range (the paper's multi-Superchip mode,
Section 4.7: every process updates only its own subset of the parameters).
The element updates need nothing from the other ranks; the only exchange is
the global gradient check: ONE all-reduce (SUM) of three doubles -- the local
sum of squares, the local NaN/Inf flag and a local error flag -- whose result
is handed back to the library with ``so_set_global_grad_stats`` before
validation.  The error flag keeps the ranks in step: a rank whose local check
failed (a kernel gave up a bounded wait, a CUDA error) still takes part in the
exchange, and when any rank reports an error every rank gives the iteration up
and raises, instead of the healthy ranks blocking in a collective the failed
one never joins.  An all-gather of the low-precision parameter shards is
offered for callers that keep a full copy.  Data lands in this rank's own
memory before any kernel reads it; no kernel is ever given a peer's pointer.

Plumbing only: ``torch.distributed`` moves three doubles; every step of the
path runs in the library's kernels.
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


class ShardFailure(RuntimeError):
    """Some rank's local gradient check failed; every rank gave the iteration up."""

    def __init__(self, failed_ranks: int, local_error: Optional[BaseException]):
        self.failed_ranks = failed_ranks
        self.local_error = local_error
        where = "this rank among them" if local_error is not None else "not this rank"
        super().__init__(f"{failed_ranks} rank(s) failed their local gradient check ({where}); "
                         "the iteration was given up on every rank")


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
        self.exchange_bytes = 24

    def iteration(self, hp, stream=None):
        """Speculate the local buckets, check locally, exchange three doubles
        in one all-reduce, validate on the global values."""
        failure = None
        sumsq = nonfinite = 0.0
        try:
            B.so_adam_step_speculative(self.ctx, hp, B.SO_ALL, stream)
            local = B.so_grad_check(self.ctx, hp, B.SO_ALL, stream)
            sumsq, nonfinite = local.sumsq, float(local.nonfinite)
        except B.SuperOffloadError as e:       # still take part in the exchange
            failure = e
        packed = torch.tensor([sumsq, nonfinite, 0.0 if failure is None else 1.0],
                              dtype=torch.float64, device=self.reduce_device)
        dist.all_reduce(packed, op=dist.ReduceOp.SUM, group=self.group)
        g_sumsq, g_nonfinite, g_errors = (float(x) for x in packed.tolist())
        if g_errors != 0.0:
            if failure is None or failure.status != B.SO_ERR_TIMEOUT:
                # the library has not ended this rank's iteration by itself
                try:
                    B.so_abandon_iteration(self.ctx, stream)
                except B.SuperOffloadError:
                    pass                       # a dead context stays dead; the caller learns below
            raise ShardFailure(int(g_errors), failure)
        B.so_set_global_grad_stats(self.ctx, g_sumsq, int(g_nonfinite != 0.0))
        return B.so_validate_commit_or_rollback(self.ctx, hp, stream)

    def all_gather_param_bf16(self) -> torch.Tensor:
        """The full low-precision parameter vector, assembled from every rank's shard."""
        mine = self.local.gather_param_bf16()
        sizes = [shard_range(self.total_elems, self.info.bucket_elems, r, self.world)
                 for r in range(self.world)]
        longest = max(hi - lo for lo, hi in sizes)
        padded = torch.zeros(longest, dtype=mine.dtype, device=mine.device)
        padded[:mine.numel()] = mine
        parts = [torch.empty_like(padded) for _ in range(self.world)]
        dist.all_gather(parts, padded, group=self.group)
        return torch.cat([p[:hi - lo] for p, (lo, hi) in zip(parts, sizes)])

    def close(self) -> None:
        if self.local is not None:
            self.local.close()
        elif self.ctx is not None:
            B.so_destroy(self.ctx)
        self.ctx = None
