"""Thin ctypes binding of ``libsuperoffload.so`` (argument marshalling only).

Function names and argument order follow ``include/superoffload.h``.  Nothing
here computes: every step of the path runs in the CUDA kernels behind the C
ABI.  Loading fails loudly if the compiled library is missing -- there is no
fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

from .build import LIB_PATH

SO_OK = 0
SO_ERR_INVALID_ARG, SO_ERR_STATE, SO_ERR_CUDA = -1, -2, -3
SO_ERR_UNDO_EXHAUSTED, SO_ERR_NOMEM, SO_ERR_UNSUPPORTED = -4, -5, -6
SO_ERR_TIMEOUT = -7
SO_ERR_TOO_LARGE = -8
SO_STATIC_CHECK_MAX_ELEMS = 1 << 26
SO_GRAD_BF16, SO_GRAD_FP32, SO_GRAD_FP16 = 0, 1, 2
SO_PARAM_BF16, SO_PARAM_FP16 = 0, 1
SO_DECISION_COMMIT, SO_DECISION_SKIP, SO_DECISION_CLIP_RESTEP = 0, 1, 2
SO_ALL = -1
DECISION_NAMES = {0: "COMMIT", 1: "SKIP", 2: "CLIP_RESTEP"}


class so_hparams(C.Structure):
    _fields_ = [("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double),
                ("eps", C.c_double), ("weight_decay", C.c_double),
                ("max_grad_norm", C.c_double)]


class so_layout_info(C.Structure):
    _fields_ = [("total_elems", C.c_int64), ("bucket_elems", C.c_int64),
                ("slot_stride_elems", C.c_int64), ("last_bucket_elems", C.c_int64),
                ("n_buckets", C.c_int32), ("n_tensors", C.c_int32),
                ("n_state_slots", C.c_int32), ("undo_slots", C.c_int32),
                ("grad_dtype", C.c_int32), ("tile_elems", C.c_int32),
                ("tiles_per_slot", C.c_int64),
                ("bytes_master", C.c_uint64), ("bytes_m", C.c_uint64), ("bytes_v", C.c_uint64),
                ("bytes_grad", C.c_uint64), ("bytes_param_bf16", C.c_uint64),
                ("bytes_scratch", C.c_uint64)]


class so_grad_stats(C.Structure):
    _fields_ = [("sumsq", C.c_double), ("norm", C.c_double), ("clip_coef", C.c_double),
                ("nonfinite", C.c_int32), ("reserved", C.c_int32)]


class so_step_result(C.Structure):
    _fields_ = [("decision", C.c_int32), ("buckets_speculated", C.c_int32),
                ("step_after", C.c_int64), ("stats", so_grad_stats),
                ("loss_scale", C.c_double)]


class so_counters(C.Structure):
    _fields_ = [("commits", C.c_int64), ("skips", C.c_int64), ("clip_resteps", C.c_int64),
                ("kernel_launches", C.c_int64), ("elems_stepped", C.c_int64),
                ("elems_checked", C.c_int64), ("elems_cast", C.c_int64),
                ("timeouts", C.c_int64)]


class SuperOffloadError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = f"{where}: {strerror(status)} (status {status})"
        if cuda_error:
            msg += f", cudaError {cuda_error}"
        super().__init__(msg)


_lib = None

EXPORTS = ["so_layout_init", "so_layout_get_info", "so_layout_tensor", "so_layout_bind",
           "so_param_dtype_config", "so_layout_pack_grads", "so_layout_unpack_params",
           "so_debug_set_spin_limit", "so_abandon_iteration",
           "so_grad_check", "so_adam_step_speculative", "so_validate_commit_or_rollback",
           "so_validate_begin", "so_validate_poll", "so_set_global_grad_stats",
           "so_cast_params", "so_iteration_host", "so_iteration_host_pipelined",
           "so_iteration_host_wait", "so_grad_check_static",
           "so_loss_scale_config", "so_get_loss_scale", "so_state_export", "so_state_import",
           "so_bucket_slot", "so_get_step", "so_set_step", "so_pending_buckets",
           "so_get_counters", "so_last_cuda_error", "so_strerror", "so_destroy",
           "so_debug_set_dry_run", "so_debug_set_bucket_stats", "so_debug_set_step_variant"]


def lib() -> C.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2509_21271_b200.build` "
            "(or __graft_entry__.build()); there is no CPU or PyTorch fallback")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_double
    P = C.POINTER
    sig = {
        "so_layout_init": [P(vp), i32, P(i64), i64, i32, i32, P(so_layout_info)],
        "so_layout_get_info": [vp, P(so_layout_info)],
        "so_layout_tensor": [vp, i32, P(i64), P(i32), P(i32)],
        "so_layout_bind": [vp, vp, vp, vp, vp, vp, vp],
        "so_param_dtype_config": [vp, i32],
        "so_layout_pack_grads": [vp, P(vp), vp],
        "so_layout_unpack_params": [vp, P(vp), vp],
        "so_debug_set_spin_limit": [vp, i64],
        "so_abandon_iteration": [vp, vp],
        "so_grad_check": [vp, P(so_hparams), i32, vp, P(so_grad_stats)],
        "so_adam_step_speculative": [vp, P(so_hparams), i32, vp],
        "so_validate_commit_or_rollback": [vp, P(so_hparams), vp, P(so_step_result)],
        "so_validate_begin": [vp, P(so_hparams), vp],
        "so_validate_poll": [vp, P(i32)],
        "so_set_global_grad_stats": [vp, dbl, i32],
        "so_cast_params": [vp, i32, vp],
        "so_iteration_host": [vp, P(so_hparams), vp, vp, vp, P(so_step_result)],
        "so_iteration_host_pipelined": [vp, P(so_hparams), vp, vp, vp, P(so_step_result)],
        "so_iteration_host_wait": [vp, vp],
        "so_grad_check_static": [vp, i64, i32, dbl, vp, vp],
        "so_loss_scale_config": [vp, dbl, dbl, dbl, i64],
        "so_get_loss_scale": [vp, P(dbl)],
        "so_state_export": [vp, vp, vp, vp, vp],
        "so_state_import": [vp, vp, vp, vp, vp],
        "so_bucket_slot": [vp, i32, P(i32)],
        "so_get_step": [vp, P(i64)],
        "so_set_step": [vp, i64],
        "so_pending_buckets": [vp, P(i32)],
        "so_get_counters": [vp, P(so_counters)],
        "so_debug_set_dry_run": [vp, i32],
        "so_debug_set_bucket_stats": [vp, i32, dbl, i32],
        "so_debug_set_step_variant": [vp, i32],
    }
    for name, argtypes in sig.items():
        fn = getattr(L, name)
        fn.argtypes = argtypes
        fn.restype = i32
    L.so_last_cuda_error.argtypes = [vp]
    L.so_last_cuda_error.restype = i32
    L.so_strerror.argtypes = [i32]
    L.so_strerror.restype = C.c_char_p
    L.so_destroy.argtypes = [vp]
    L.so_destroy.restype = None
    _lib = L
    return L


def strerror(status: int) -> str:
    return lib().so_strerror(status).decode()


def _ok(ctx, status: int, where: str) -> None:
    if status != SO_OK:
        err = lib().so_last_cuda_error(ctx) if (ctx and status == SO_ERR_CUDA) else 0
        raise SuperOffloadError(status, where, err)


def _hp(hp) -> so_hparams:
    if isinstance(hp, so_hparams):
        return hp
    return so_hparams(hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay, hp.max_grad_norm)


def _stream(stream) -> C.c_void_p:
    if stream is None:
        return C.c_void_p(0)
    if isinstance(stream, int):
        return C.c_void_p(stream)
    return C.c_void_p(stream.cuda_stream)          # torch.cuda.Stream


# ---- the calls, one to one with the header --------------------------------

def so_layout_init(numel, bucket_elems: int, grad_dtype: int = SO_GRAD_BF16,
                   undo_slots: int = SO_ALL):
    """Returns (ctx handle, so_layout_info)."""
    n = len(numel)
    arr = (C.c_int64 * max(n, 1))(*numel)
    ctx = C.c_void_p()
    info = so_layout_info()
    st = lib().so_layout_init(C.byref(ctx), n, arr, bucket_elems, grad_dtype, undo_slots,
                              C.byref(info))
    _ok(None, st, "so_layout_init")
    return ctx, info


def so_layout_get_info(ctx) -> so_layout_info:
    info = so_layout_info()
    _ok(ctx, lib().so_layout_get_info(ctx, C.byref(info)), "so_layout_get_info")
    return info


def so_layout_tensor(ctx, i: int):
    """Returns (flat_offset, first_bucket, last_bucket)."""
    off, fb, lb = C.c_int64(), C.c_int32(), C.c_int32()
    _ok(ctx, lib().so_layout_tensor(ctx, i, C.byref(off), C.byref(fb), C.byref(lb)),
        "so_layout_tensor")
    return off.value, fb.value, lb.value


def so_layout_bind(ctx, master: int, m: int, v: int, grad: int, param_bf16: int,
                   scratch: int) -> None:
    """Arguments are raw device addresses (e.g. ``tensor.data_ptr()``)."""
    _ok(ctx, lib().so_layout_bind(ctx, master, m, v, grad, param_bf16, scratch),
        "so_layout_bind")


def so_param_dtype_config(ctx, param_dtype: int) -> None:
    _ok(ctx, lib().so_param_dtype_config(ctx, param_dtype), "so_param_dtype_config")


def _ptr_array(ptrs):
    return (C.c_void_p * max(len(ptrs), 1))(*[C.c_void_p(int(p) or None) for p in ptrs])


def so_layout_pack_grads(ctx, tensor_grads, stream=None) -> None:
    """`tensor_grads`: one raw device address per tensor, in layout order."""
    _ok(ctx, lib().so_layout_pack_grads(ctx, _ptr_array(tensor_grads), _stream(stream)),
        "so_layout_pack_grads")


def so_layout_unpack_params(ctx, tensor_params, stream=None) -> None:
    """`tensor_params`: one raw device address per tensor, in layout order."""
    _ok(ctx, lib().so_layout_unpack_params(ctx, _ptr_array(tensor_params), _stream(stream)),
        "so_layout_unpack_params")


def so_grad_check(ctx, hp, bucket: int = SO_ALL, stream=None):
    """Returns so_grad_stats for SO_ALL, None for a single bucket."""
    if bucket == SO_ALL:
        out = so_grad_stats()
        h = _hp(hp)
        _ok(ctx, lib().so_grad_check(ctx, C.byref(h), bucket, _stream(stream), C.byref(out)),
            "so_grad_check")
        return out
    _ok(ctx, lib().so_grad_check(ctx, None, bucket, _stream(stream), None), "so_grad_check")
    return None


def so_adam_step_speculative(ctx, hp, bucket: int = SO_ALL, stream=None) -> None:
    h = _hp(hp)
    _ok(ctx, lib().so_adam_step_speculative(ctx, C.byref(h), bucket, _stream(stream)),
        "so_adam_step_speculative")


def so_validate_commit_or_rollback(ctx, hp, stream=None) -> so_step_result:
    h = _hp(hp)
    out = so_step_result()
    _ok(ctx, lib().so_validate_commit_or_rollback(ctx, C.byref(h), _stream(stream),
                                                  C.byref(out)),
        "so_validate_commit_or_rollback")
    return out


def so_validate_begin(ctx, hp, stream=None) -> None:
    h = _hp(hp)
    _ok(ctx, lib().so_validate_begin(ctx, C.byref(h), _stream(stream)), "so_validate_begin")


def so_validate_poll(ctx) -> bool:
    ready = C.c_int32()
    _ok(ctx, lib().so_validate_poll(ctx, C.byref(ready)), "so_validate_poll")
    return bool(ready.value)


def so_set_global_grad_stats(ctx, global_sumsq: float, global_nonfinite: int) -> None:
    _ok(ctx, lib().so_set_global_grad_stats(ctx, global_sumsq, int(global_nonfinite)),
        "so_set_global_grad_stats")


def so_abandon_iteration(ctx, stream=None) -> None:
    _ok(ctx, lib().so_abandon_iteration(ctx, _stream(stream)), "so_abandon_iteration")


def so_cast_params(ctx, bucket: int = SO_ALL, stream=None) -> None:
    _ok(ctx, lib().so_cast_params(ctx, bucket, _stream(stream)), "so_cast_params")


def so_iteration_host(ctx, hp, host_grad: int, host_param_bf16: int, stream=None) -> so_step_result:
    """Host addresses (pinned memory); ``host_param_bf16`` may be 0 for no output."""
    h = _hp(hp)
    out = so_step_result()
    _ok(ctx, lib().so_iteration_host(ctx, C.byref(h), host_grad, host_param_bf16 or None,
                                     _stream(stream), C.byref(out)), "so_iteration_host")
    return out


def so_iteration_host_pipelined(ctx, hp, host_grad: int, host_param_bf16: int,
                                stream=None) -> so_step_result:
    """Like so_iteration_host, without the wait at the end (see the header)."""
    h = _hp(hp)
    out = so_step_result()
    _ok(ctx, lib().so_iteration_host_pipelined(ctx, C.byref(h), host_grad, host_param_bf16 or None,
                                               _stream(stream), C.byref(out)),
        "so_iteration_host_pipelined")
    return out


def so_iteration_host_wait(ctx, stream=None) -> None:
    _ok(ctx, lib().so_iteration_host_wait(ctx, _stream(stream)), "so_iteration_host_wait")


def so_grad_check_static(grad: int, n_elems: int, grad_dtype: int, max_grad_norm: float,
                         stream, out_device: int) -> None:
    """Gradient check without any allocation: `grad` and `out_device` are raw
    device addresses (a gradient buffer and a 32-byte so_grad_stats record)."""
    _ok(None, lib().so_grad_check_static(grad, n_elems, grad_dtype, max_grad_norm,
                                         _stream(stream), out_device), "so_grad_check_static")


def so_loss_scale_config(ctx, init_scale: float, growth: float = 2.0, backoff: float = 0.5,
                         interval: int = 0) -> None:
    _ok(ctx, lib().so_loss_scale_config(ctx, init_scale, growth, backoff, interval),
        "so_loss_scale_config")


def so_get_loss_scale(ctx) -> float:
    s = C.c_double()
    _ok(ctx, lib().so_get_loss_scale(ctx, C.byref(s)), "so_get_loss_scale")
    return s.value


def so_state_export(ctx, master: int, m: int, v: int, stream=None) -> None:
    """Flat fp32 arrays (device or host addresses, 0 to skip) <- committed state."""
    _ok(ctx, lib().so_state_export(ctx, master or None, m or None, v or None, _stream(stream)),
        "so_state_export")


def so_state_import(ctx, master: int, m: int, v: int, stream=None) -> None:
    """Committed state <- flat fp32 arrays (device or host addresses, 0 to skip)."""
    _ok(ctx, lib().so_state_import(ctx, master or None, m or None, v or None, _stream(stream)),
        "so_state_import")


def so_bucket_slot(ctx, bucket: int) -> int:
    s = C.c_int32()
    _ok(ctx, lib().so_bucket_slot(ctx, bucket, C.byref(s)), "so_bucket_slot")
    return s.value


def so_get_step(ctx) -> int:
    t = C.c_int64()
    _ok(ctx, lib().so_get_step(ctx, C.byref(t)), "so_get_step")
    return t.value


def so_set_step(ctx, t: int) -> None:
    _ok(ctx, lib().so_set_step(ctx, t), "so_set_step")


def so_pending_buckets(ctx) -> int:
    n = C.c_int32()
    _ok(ctx, lib().so_pending_buckets(ctx, C.byref(n)), "so_pending_buckets")
    return n.value


def so_get_counters(ctx) -> so_counters:
    out = so_counters()
    _ok(ctx, lib().so_get_counters(ctx, C.byref(out)), "so_get_counters")
    return out


def so_destroy(ctx) -> None:
    lib().so_destroy(ctx)


def so_debug_set_dry_run(ctx, on: bool) -> None:
    _ok(ctx, lib().so_debug_set_dry_run(ctx, int(on)), "so_debug_set_dry_run")


def so_debug_set_bucket_stats(ctx, bucket: int, sumsq: float, nonfinite: int) -> None:
    _ok(ctx, lib().so_debug_set_bucket_stats(ctx, bucket, sumsq, nonfinite),
        "so_debug_set_bucket_stats")


def so_debug_set_spin_limit(ctx, polls: int) -> None:
    _ok(ctx, lib().so_debug_set_spin_limit(ctx, polls), "so_debug_set_spin_limit")


def so_debug_set_step_variant(ctx, variant: int) -> None:
    _ok(ctx, lib().so_debug_set_step_variant(ctx, variant), "so_debug_set_step_variant")
