"""CPU oracle for the bucketized speculative AdamW step (test infrastructure).

This package is the slow, plain, single-threaded fp64 statement of what the
optimizer hot path computes.  Only the tests, the smoke check and the
CPU-baseline / reference leg of the benchmark may use it; it shares no code
with the CUDA library and never imports it.

The arithmetic lives in ``so_oracle.c`` (plain C, compiled here with
``gcc -O2 -ffp-contract=off``); this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "so_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

DECISION_COMMIT, DECISION_SKIP, DECISION_CLIP_RESTEP = 0, 1, 2
GRAD_BF16, GRAD_FP32, GRAD_FP16 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the C oracle into ``liboracle.so`` next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c99", "-shared",
           "-fPIC", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    vp, i64, i32, dbl = c.c_void_p, c.c_int64, c.c_int32, c.c_double
    pd, pi, pi64 = c.POINTER(c.c_double), c.POINTER(c.c_int), c.POINTER(c.c_int64)
    lib.orc_widen_bf16.restype = None
    lib.orc_widen_bf16.argtypes = [vp, vp, i64]
    lib.orc_widen_fp16.restype = None
    lib.orc_widen_fp16.argtypes = [vp, vp, i64]
    lib.orc_loss_scale_update.restype = None
    lib.orc_loss_scale_update.argtypes = [pd, pi64, c.c_int, dbl, dbl, i64]
    lib.orc_bf16_rne.restype = c.c_uint16
    lib.orc_bf16_rne.argtypes = [c.c_float]
    lib.orc_cast_params.restype = None
    lib.orc_cast_params.argtypes = [vp, vp, i64]
    lib.orc_fp16_rne.restype = c.c_uint16
    lib.orc_fp16_rne.argtypes = [c.c_float]
    lib.orc_cast_params_fp16.restype = None
    lib.orc_cast_params_fp16.argtypes = [vp, vp, i64]
    lib.orc_grad_check_range.restype = c.c_int
    lib.orc_grad_check_range.argtypes = [vp, c.c_int, i64, i64, dbl, pd]
    lib.orc_global_grad_check.restype = c.c_int
    lib.orc_global_grad_check.argtypes = [vp, c.c_int, i64, i64, dbl, pd, pd]
    lib.orc_clip_coef.restype = dbl
    lib.orc_clip_coef.argtypes = [dbl, dbl]
    lib.orc_decision.restype = c.c_int
    lib.orc_decision.argtypes = [c.c_int, dbl]
    lib.orc_adamw_step_range.restype = None
    lib.orc_adamw_step_range.argtypes = [vp, vp, vp, vp, c.c_int, i64, i64, dbl, dbl, i64,
                                         dbl, dbl, dbl, dbl, dbl]
    lib.orc_iteration_ste.restype = c.c_int
    lib.orc_iteration_ste.argtypes = [vp, vp, vp, vp, vp, c.c_int, i64, i64, pi64,
                                      dbl, dbl, dbl, dbl, dbl, dbl, dbl, pd, pd, pd, pi]
    lib.orc_iteration_stv.restype = c.c_int
    lib.orc_iteration_stv.argtypes = [vp, vp, vp, vp, vp, c.c_int, i64, i64, pi64,
                                      dbl, dbl, dbl, dbl, dbl, dbl, dbl, dbl, pd, pd, pd, pi]
    lib.orc_layout_offsets.restype = i64
    lib.orc_layout_offsets.argtypes = [pi64, i32, pi64]
    lib.orc_num_buckets.restype = i64
    lib.orc_num_buckets.argtypes = [i64, i64]
    lib.orc_resident_bytes.restype = i64
    lib.orc_resident_bytes.argtypes = [i64]
    _lib = lib
    return lib


@dataclass
class HParams:
    """AdamW hyper-parameters; ``max_grad_norm <= 0`` disables clipping."""
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    max_grad_norm: float = 1.0


@dataclass
class IterationResult:
    decision: int
    sumsq: float
    norm: float
    clip_coef: float
    nonfinite: int
    step_after: int


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _check(a: np.ndarray, dtype) -> np.ndarray:
    if a.dtype != dtype or not a.flags.c_contiguous:
        raise TypeError(f"expected contiguous {dtype}, got {a.dtype}")
    return a


def _grad_dtype(g: np.ndarray) -> int:
    if g.dtype == np.uint16:
        return GRAD_BF16
    if g.dtype == np.float32:
        return GRAD_FP32
    if g.dtype == np.float16:
        return GRAD_FP16
    raise TypeError("gradients must be uint16 (bf16 bit patterns), float16 or float32")


def bf16_rne(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    x = _check(np.ascontiguousarray(x), np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().orc_cast_params(_ptr(x), _ptr(out), x.size)
    return out


def fp16_rne(x: np.ndarray) -> np.ndarray:
    """fp32 -> IEEE binary16 bit patterns (uint16), round to nearest even."""
    x = _check(np.ascontiguousarray(x), np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().orc_cast_params_fp16(_ptr(x), _ptr(out), x.size)
    return out


def bf16_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32, exact (the defining shift)."""
    b = _check(np.ascontiguousarray(b), np.uint16)
    out = np.empty(b.shape, dtype=np.float32)
    _load().orc_widen_bf16(_ptr(b), _ptr(out), b.size)
    return out


def fp16_to_f32(h: np.ndarray) -> np.ndarray:
    """IEEE binary16 bit patterns (uint16) -> fp32, exact."""
    h = _check(np.ascontiguousarray(h), np.uint16)
    out = np.empty(h.shape, dtype=np.float32)
    _load().orc_widen_fp16(_ptr(h), _ptr(out), h.size)
    return out


def grad_check_range(g: np.ndarray, begin: int, end: int, unscale: float = 1.0):
    """(sum of squares in index order, non-finite flag) of unscale * g[begin:end]."""
    s = ctypes.c_double()
    flag = _load().orc_grad_check_range(_ptr(g), _grad_dtype(g), begin, end, unscale,
                                        ctypes.byref(s))
    return s.value, int(flag)


def global_grad_check(g: np.ndarray, bucket_elems: int, unscale: float = 1.0):
    """(sumsq, norm, nonfinite) over all of unscale * g, bucket partials in bucket order."""
    s, nrm = ctypes.c_double(), ctypes.c_double()
    flag = _load().orc_global_grad_check(_ptr(g), _grad_dtype(g), g.size, bucket_elems, unscale,
                                         ctypes.byref(s), ctypes.byref(nrm))
    return s.value, nrm.value, int(flag)


def loss_scale_update(scale: float, good_steps: int, nonfinite: int, growth: float = 2.0,
                      backoff: float = 0.5, interval: int = 2000):
    """One step of the dynamic loss-scale schedule: returns (scale, good_steps)."""
    s, gcount = ctypes.c_double(scale), ctypes.c_int64(good_steps)
    _load().orc_loss_scale_update(ctypes.byref(s), ctypes.byref(gcount), int(nonfinite),
                                  growth, backoff, interval)
    return s.value, gcount.value


def clip_coef(norm: float, max_norm: float) -> float:
    return _load().orc_clip_coef(norm, max_norm)


def decision(nonfinite: int, coef: float) -> int:
    return _load().orc_decision(int(nonfinite), coef)


def adamw_step_range(p, m, v, g, begin, end, scale, tt, hp: HParams,
                     unscale: float = 1.0) -> None:
    """In-place AdamW step of elements [begin, end) with step index ``tt``."""
    for a in (p, m, v):
        _check(a, np.float32)
    _load().orc_adamw_step_range(_ptr(p), _ptr(m), _ptr(v), _ptr(g), _grad_dtype(g),
                                 begin, end, unscale, scale, tt, hp.lr, hp.beta1, hp.beta2,
                                 hp.eps, hp.weight_decay)


def _iteration(fn_name, p, m, v, pb, g, bucket_elems, t, hp, forced_coef=None, unscale=1.0):
    for a in (p, m, v):
        _check(a, np.float32)
    _check(pb, np.uint16)
    lib = _load()
    tt = ctypes.c_int64(t)
    s, nrm, coef = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    flag = ctypes.c_int()
    args = [_ptr(p), _ptr(m), _ptr(v), _ptr(pb), _ptr(g), _grad_dtype(g), p.size,
            bucket_elems, ctypes.byref(tt), hp.lr, hp.beta1, hp.beta2, hp.eps,
            hp.weight_decay, hp.max_grad_norm, float(unscale)]
    if fn_name == "orc_iteration_stv":
        args.append(0.0 if forced_coef is None else float(forced_coef))
    args += [ctypes.byref(s), ctypes.byref(nrm), ctypes.byref(coef), ctypes.byref(flag)]
    d = getattr(lib, fn_name)(*args)
    if d < 0:
        raise MemoryError("oracle snapshot allocation failed")
    return IterationResult(d, s.value, nrm.value, coef.value, flag.value, tt.value)


def iteration_ste(p, m, v, pb, g, bucket_elems: int, t: int, hp: HParams,
                  unscale: float = 1.0) -> IterationResult:
    """Check every gradient, then step (or skip): the plain definition."""
    return _iteration("orc_iteration_ste", p, m, v, pb, g, bucket_elems, t, hp, None, unscale)


def iteration_stv(p, m, v, pb, g, bucket_elems: int, t: int, hp: HParams,
                  forced_coef: float | None = None, unscale: float = 1.0) -> IterationResult:
    """Speculate every bucket, validate, then commit / restore / re-step."""
    return _iteration("orc_iteration_stv", p, m, v, pb, g, bucket_elems, t, hp, forced_coef,
                      unscale)


def layout_offsets(numel):
    numel = np.ascontiguousarray(numel, dtype=np.int64)
    off = np.empty_like(numel)
    c = ctypes
    total = _load().orc_layout_offsets(numel.ctypes.data_as(c.POINTER(c.c_int64)),
                                       numel.size, off.ctypes.data_as(c.POINTER(c.c_int64)))
    return off, int(total)


def num_buckets(total: int, bucket_elems: int) -> int:
    return int(_load().orc_num_buckets(total, bucket_elems))


def resident_bytes(total: int) -> int:
    return int(_load().orc_resident_bytes(total))
