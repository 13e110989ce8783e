"""so_grad_check_static: the gradient check for callers that cannot allocate
device memory (its scratch is a fixed array inside the library).

This file is collected last on purpose: if the entry point misbehaves, a run
that stops at the first failure has already executed every other test.  It
compares the allocation-free entry point with the regular so_grad_check on the
same gradients, through the C ABI, on two calls in a row (the second call sees
whatever the first left in the shared array)."""
from __future__ import annotations

import ctypes

import numpy as np

import oracle
import pytest
import torch

from paper_2509_21271_b200 import binding as B
from paper_2509_21271_b200 import build as so_build

pytestmark = pytest.mark.gpu

NORM_RTOL = 1e-5        # the norm tolerance used by every GPU parity test


class HP:
    lr, beta1, beta2, eps, weight_decay = 1e-3, 0.9, 0.999, 1e-8, 0.01

    def __init__(self, max_grad_norm):
        self.max_grad_norm = max_grad_norm


@pytest.fixture(scope="module", autouse=True)
def _built():
    so_build.build_library()
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)


def _regular_check(g: torch.Tensor, bucket: int, max_norm: float):
    """The existing entry point: a context with caller-allocated scratch."""
    gd = B.SO_GRAD_BF16 if g.dtype == torch.bfloat16 else B.SO_GRAD_FP32
    ctx, info = B.so_layout_init([g.numel()], bucket, gd, 0)
    try:
        def arena(n_bytes):
            return torch.zeros(max(int(n_bytes), 256) + 256, dtype=torch.uint8, device="cuda")
        state = arena(info.bytes_master)
        grad = arena(info.bytes_grad)
        pb = arena(info.bytes_param_bf16)
        scratch = arena(info.bytes_scratch)
        assert info.slot_stride_elems == info.bucket_elems
        grad[:g.numel() * g.element_size()].copy_(g.view(torch.uint8))
        B.so_layout_bind(ctx, state.data_ptr(), state.data_ptr(), state.data_ptr(),
                         grad.data_ptr(), pb.data_ptr(), scratch.data_ptr())
        stats = B.so_grad_check(ctx, HP(max_norm), B.SO_ALL, torch.cuda.current_stream())
        return stats.sumsq, stats.norm, stats.clip_coef, stats.nonfinite
    finally:
        B.so_destroy(ctx)


def _static_check(g: torch.Tensor, max_norm: float, out: torch.Tensor):
    gd = B.SO_GRAD_BF16 if g.dtype == torch.bfloat16 else B.SO_GRAD_FP32
    B.so_grad_check_static(g.data_ptr(), g.numel(), gd, max_norm, torch.cuda.current_stream(),
                           out.data_ptr())
    torch.cuda.synchronize()
    raw = out.cpu().numpy().tobytes()
    rec = B.so_grad_stats.from_buffer_copy(raw)
    return rec.sumsq, rec.norm, rec.clip_coef, rec.nonfinite


def _close(a, b):
    return abs(a - b) <= NORM_RTOL * max(abs(b), 1e-300)


def _oracle_check(g: torch.Tensor, max_norm: float):
    """The CPU oracle on the same bits: (sumsq, norm, clip coefficient, flag)."""
    host = g.view(torch.int16).cpu().numpy().view(np.uint16) if g.dtype == torch.bfloat16 \
        else g.cpu().numpy()
    sumsq, norm, flag = oracle.global_grad_check(host, max(host.size, 1))
    return sumsq, norm, oracle.clip_coef(norm, max_norm), flag


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_check_matches_the_regular_check_on_two_calls_in_a_row(dtype):
    gen = torch.Generator(device="cuda").manual_seed(11)
    out = torch.zeros(ctypes.sizeof(B.so_grad_stats), dtype=torch.uint8, device="cuda")

    # call 1: a large ragged gradient, clipping active
    n1 = 3_000_017
    g1 = (torch.randn(n1, generator=gen, device="cuda") * 1e-2).to(dtype)
    got1 = _static_check(g1, 1.0, out)
    ref1 = _regular_check(g1, 1 << 20, 1.0)
    assert got1[3] == ref1[3] == 0
    assert _close(got1[0], ref1[0]) and _close(got1[1], ref1[1]) and _close(got1[2], ref1[2])
    assert got1[2] < 1.0                                        # norm ~ 17 > 1: clip active
    want1 = _oracle_check(g1, 1.0)                              # and against the CPU oracle itself
    assert got1[3] == want1[3] and all(_close(a, b) for a, b in zip(got1[:3], want1[:3]))

    # call 2, straight after, smaller: the array still holds call 1's tile sums
    # beyond this call's range, which must not leak into the result
    n2 = 70_001
    g2 = (torch.randn(n2, generator=gen, device="cuda") * 1e-3).to(dtype)
    got2 = _static_check(g2, 1.0, out)
    ref2 = _regular_check(g2, 1 << 16, 1.0)
    assert got2[3] == ref2[3] == 0
    assert _close(got2[0], ref2[0]) and _close(got2[1], ref2[1])
    assert got2[2] == ref2[2] == 1.0                            # norm ~ 0.26: no clip
    want2 = _oracle_check(g2, 1.0)
    assert want2[2] == 1.0 and _close(got2[0], want2[0]) and _close(got2[1], want2[1])

    # with a single bucket the two entry points fold in the same order: same bits
    one_bucket = _regular_check(g2, n2 + 63 - (n2 + 63) % 64, 1.0)
    assert got2[:3] == one_bucket[:3]

    # call 3: a non-finite value raises the flag in both
    g3 = g2.clone()
    g3[n2 - 1] = float("inf")
    got3 = _static_check(g3, 0.0, out)
    ref3 = _regular_check(g3, 1 << 16, 0.0)
    assert got3[3] == ref3[3] == _oracle_check(g3, 0.0)[3] == 1


def test_static_check_rejects_what_it_cannot_hold_and_handles_empty_input():
    out = torch.zeros(ctypes.sizeof(B.so_grad_stats), dtype=torch.uint8, device="cuda")
    g = torch.zeros(1024, dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream()
    with pytest.raises(B.SuperOffloadError) as err:
        B.so_grad_check_static(g.data_ptr(), B.SO_STATIC_CHECK_MAX_ELEMS + 1, B.SO_GRAD_BF16, 1.0,
                               stream, out.data_ptr())
    assert err.value.status == B.SO_ERR_TOO_LARGE
    assert "capacity" in str(err.value)
    with pytest.raises(B.SuperOffloadError) as err:
        B.so_grad_check_static(g.data_ptr() + 2, 16, B.SO_GRAD_BF16, 1.0, stream, out.data_ptr())
    assert err.value.status == B.SO_ERR_INVALID_ARG
    # an empty gradient is a valid input: norm 0, coefficient 1, no flag
    assert _static_check(g[:0], 1.0, out) == (0.0, 0.0, 1.0, 0)
    # exactly representable case: 1024 ones -> norm 32
    ones = torch.ones(1024, dtype=torch.bfloat16, device="cuda")
    assert _static_check(ones, 0.0, out) == (1024.0, 32.0, 1.0, 0)


@pytest.mark.parametrize("n", [5 * (1 << 20) + 1, B.SO_STATIC_CHECK_MAX_ELEMS])
def test_static_check_on_inputs_of_several_segments_and_at_its_capacity(n):
    """Beyond 4 Mi elements the regular check folds per segment first: the two
    entry points agree to rounding, and both with the oracle; the largest
    input the built-in array holds is accepted."""
    gen = torch.Generator(device="cuda").manual_seed(12)
    out = torch.zeros(ctypes.sizeof(B.so_grad_stats), dtype=torch.uint8, device="cuda")
    g = (torch.randn(n, generator=gen, device="cuda") * 1e-3).to(torch.bfloat16)
    got = _static_check(g, 1.0, out)
    ref = _regular_check(g, n + (-n) % 64, 1.0)
    want = _oracle_check(g, 1.0)
    assert got[3] == ref[3] == want[3] == 0
    for a, b, c in zip(got[:3], ref[:3], want[:3]):
        assert _close(a, b) and _close(a, c)
    again = _static_check(g, 1.0, out)                          # a second call in a row: same bits
    assert again == got


def test_static_check_refuses_fp16_gradients():
    out = torch.zeros(ctypes.sizeof(B.so_grad_stats), dtype=torch.uint8, device="cuda")
    g = torch.zeros(1024, dtype=torch.float16, device="cuda")
    with pytest.raises(B.SuperOffloadError) as err:
        B.so_grad_check_static(g.data_ptr(), 1024, B.SO_GRAD_FP16, 1.0, torch.cuda.current_stream(),
                               out.data_ptr())
    assert err.value.status == B.SO_ERR_INVALID_ARG
