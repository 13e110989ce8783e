"""Device-memory plumbing around the C-ABI calls.

``BucketedAdamW`` allocates the caller-owned arenas with torch (device memory
and streams are all torch is used for), binds them, and moves flat tensors in
and out of the slot layout.  It performs no arithmetic of the method: every
step of the path runs in the library's kernels.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding as B


def _guard(n_bytes: int) -> int:
    return (n_bytes + 255) // 256 * 256


class BucketedAdamW:
    """One optimizer context over a tensor list flattened into buckets."""

    GUARD = 4096            # bytes of sentinel before and after every arena
    # step kernel when the constructor is not told: 0 = chosen by launch size
    # (see so_debug_set_step_variant); the GPU tests set 2 so that the small
    # cases they run still go through the bulk-copy pipeline
    DEFAULT_STEP_VARIANT = 0

    def __init__(self, numel: Sequence[int], bucket_elems: int, grad_dtype: str = "bf16",
                 undo_slots: int = B.SO_ALL, device: str = "cuda", guard_bands: bool = False,
                 step_variant: Optional[int] = None, param_dtype: str = "bf16"):
        self.device = torch.device(device)
        gd = {"bf16": B.SO_GRAD_BF16, "fp32": B.SO_GRAD_FP32, "fp16": B.SO_GRAD_FP16}[grad_dtype]
        self.ctx, self.info = B.so_layout_init(list(numel), bucket_elems, gd, undo_slots)
        if step_variant is None:
            step_variant = self.DEFAULT_STEP_VARIANT
        if step_variant:
            B.so_debug_set_step_variant(self.ctx, step_variant)
        self.step_variant = step_variant
        self.grad_torch_dtype = {B.SO_GRAD_BF16: torch.bfloat16, B.SO_GRAD_FP32: torch.float32,
                                 B.SO_GRAD_FP16: torch.float16}[gd]
        self.guard_bands = guard_bands
        self.param_torch_dtype = {"bf16": torch.bfloat16, "fp16": torch.float16}[param_dtype]
        if param_dtype == "fp16":
            B.so_param_dtype_config(self.ctx, B.SO_PARAM_FP16)
        i = self.info
        self._raw = {}
        self.master = self._arena("master", i.bytes_master, torch.float32)
        self.m = self._arena("m", i.bytes_m, torch.float32)
        self.v = self._arena("v", i.bytes_v, torch.float32)
        self.grad = self._arena("grad", i.bytes_grad, self.grad_torch_dtype)
        self.param_bf16 = self._arena("param_bf16", i.bytes_param_bf16, self.param_torch_dtype)
        self.scratch = self._arena("scratch", i.bytes_scratch, torch.uint8)
        B.so_layout_bind(self.ctx, self.master.data_ptr(), self.m.data_ptr(), self.v.data_ptr(),
                         self.grad.data_ptr(), self.param_bf16.data_ptr(),
                         self.scratch.data_ptr())

    # ---- memory ---------------------------------------------------------
    def _arena(self, name: str, n_bytes: int, dtype: torch.dtype) -> torch.Tensor:
        body = _guard(max(int(n_bytes), 256))
        pad = self.GUARD if self.guard_bands else 0
        raw = torch.empty(body + 2 * pad, dtype=torch.uint8, device=self.device)
        if self.guard_bands:
            raw[:pad] = 0xA5
            raw[pad + body:] = 0xA5
        raw[pad:pad + body] = 0
        self._raw[name] = (raw, pad, body)
        view = raw[pad:pad + body].view(dtype)
        assert view.data_ptr() % 256 == 0
        return view

    def guard_bands_intact(self) -> bool:
        ok = True
        for raw, pad, body in self._raw.values():
            if pad:
                ok &= bool((raw[:pad] == 0xA5).all().item())
                ok &= bool((raw[pad + body:] == 0xA5).all().item())
        return ok

    def close(self) -> None:
        if self.ctx is not None:
            B.so_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- geometry -------------------------------------------------------
    @property
    def n_buckets(self) -> int:
        return self.info.n_buckets

    def bucket_range(self, b: int):
        lo = b * self.info.bucket_elems
        return lo, min(lo + self.info.bucket_elems, self.info.total_elems)

    def _slot_view(self, arena: torch.Tensor, slot: int, n: int) -> torch.Tensor:
        s = slot * self.info.slot_stride_elems
        return arena[s:s + n]

    # ---- moving flat tensors in and out of the slot layout --------------
    def load_state(self, p: torch.Tensor, m: Optional[torch.Tensor] = None,
                   v: Optional[torch.Tensor] = None) -> None:
        """Copy flat fp32 master (and moments, default zero) into the arenas."""
        for b in range(self.n_buckets):
            lo, hi = self.bucket_range(b)
            slot = B.so_bucket_slot(self.ctx, b)
            self._slot_view(self.master, slot, hi - lo).copy_(p[lo:hi])
            for arena, src in ((self.m, m), (self.v, v)):
                dst = self._slot_view(arena, slot, hi - lo)
                if src is None:
                    dst.zero_()
                else:
                    dst.copy_(src[lo:hi])

    def load_grads(self, g: torch.Tensor, non_blocking: bool = False) -> None:
        """Copy a flat gradient tensor (device or pinned host) into the arena."""
        stride, Bk = self.info.slot_stride_elems, self.info.bucket_elems
        if stride == Bk:
            self.grad[:g.numel()].copy_(g, non_blocking=non_blocking)
            return
        for b in range(self.n_buckets):
            lo, hi = self.bucket_range(b)
            self._slot_view(self.grad, b, hi - lo).copy_(g[lo:hi], non_blocking=non_blocking)

    def _scatter(self, arena: torch.Tensor, start: int, piece: torch.Tensor) -> None:
        """Copy a piece of the flat space starting at `start` into bucket slots."""
        Bk = self.info.bucket_elems
        pos, end = start, start + piece.numel()
        while pos < end:
            b = pos // Bk
            hi = min(end, (b + 1) * Bk)
            slot = b if arena is self.grad or arena is self.param_bf16 \
                else B.so_bucket_slot(self.ctx, b)
            off = slot * self.info.slot_stride_elems + (pos - b * Bk)
            arena[off:off + hi - pos].copy_(piece[pos - start:hi - start])
            pos = hi

    def load_state_stream(self, pieces) -> None:
        """Master weights from an iterator of (start, fp32 piece); m and v are
        left as they are (zero after construction)."""
        for start, piece in pieces:
            self._scatter(self.master, start, piece)

    def load_grads_stream(self, pieces) -> None:
        """Gradients from an iterator of (start, piece in the gradient dtype)."""
        for start, piece in pieces:
            self._scatter(self.grad, start, piece)

    def gather_state(self):
        """Flat (p, m, v) of the committed state, in parameter order."""
        N = self.info.total_elems
        out = [torch.empty(N, dtype=torch.float32, device=self.device) for _ in range(3)]
        for b in range(self.n_buckets):
            lo, hi = self.bucket_range(b)
            slot = B.so_bucket_slot(self.ctx, b)
            for dst, arena in zip(out, (self.master, self.m, self.v)):
                dst[lo:hi].copy_(self._slot_view(arena, slot, hi - lo))
        return out

    def gather_bucket(self, b: int):
        """(p, m, v, bf16 copy) views of one bucket's committed state."""
        lo, hi = self.bucket_range(b)
        slot = B.so_bucket_slot(self.ctx, b)
        return (self._slot_view(self.master, slot, hi - lo),
                self._slot_view(self.m, slot, hi - lo),
                self._slot_view(self.v, slot, hi - lo),
                self._slot_view(self.param_bf16, b, hi - lo))

    def gather_param_bf16(self) -> torch.Tensor:
        N = self.info.total_elems
        out = torch.empty(N, dtype=self.param_torch_dtype, device=self.device)
        for b in range(self.n_buckets):
            lo, hi = self.bucket_range(b)
            out[lo:hi].copy_(self._slot_view(self.param_bf16, b, hi - lo))
        return out

    def pack_grads(self, tensors, stream=None) -> None:
        """Gradients of the individual tensors -> gradient arena, one launch."""
        B.so_layout_pack_grads(self.ctx, [t.data_ptr() if t.numel() else 0 for t in tensors], stream)

    def unpack_params(self, tensors, stream=None) -> None:
        """Low-precision parameter arena -> the individual tensors, one launch."""
        B.so_layout_unpack_params(self.ctx, [t.data_ptr() if t.numel() else 0 for t in tensors],
                                  stream)

    # ---- the path -------------------------------------------------------
    def cast_params(self, bucket: int = B.SO_ALL, stream=None) -> None:
        B.so_cast_params(self.ctx, bucket, stream)

    def step_speculative(self, hp, bucket: int = B.SO_ALL, stream=None) -> None:
        B.so_adam_step_speculative(self.ctx, hp, bucket, stream)

    def grad_check(self, hp, bucket: int = B.SO_ALL, stream=None):
        return B.so_grad_check(self.ctx, hp, bucket, stream)

    def validate(self, hp, stream=None):
        return B.so_validate_commit_or_rollback(self.ctx, hp, stream)

    def validate_begin(self, hp, stream=None) -> None:
        """Enqueue the end of the iteration (verdict formed on the device)."""
        B.so_validate_begin(self.ctx, hp, stream)

    def iteration(self, hp, stream=None, speculative: bool = True):
        """One whole pass: speculate every bucket that fits, check, validate."""
        if speculative:
            self.step_speculative(hp, B.SO_ALL, stream)
        return self.validate(hp, stream)

    @property
    def step_count(self) -> int:
        return B.so_get_step(self.ctx)

    def counters(self):
        return B.so_get_counters(self.ctx)
