"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Tolerances: fp32 master/m/v within 2 ulp per
element per step; global norm within 1e-5 relative; the bf16 copy is the exact
RNE cast of the device master; flags, decisions and rollbacks bit-exact."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
from gpu_harness import (Report, bf16_to_numpy, grads_to_numpy, hparams_of, run_lockstep)
from helpers import bf16_bits_to_f32, is_bf16_nan, ulp_distance
from paper_2509_21271_b200 import binding as B
from paper_2509_21271_b200 import build as so_build
from paper_2509_21271_b200 import workloads as W
from paper_2509_21271_b200.optimizer import BucketedAdamW

pytestmark = pytest.mark.gpu

C, S, R = B.SO_DECISION_COMMIT, B.SO_DECISION_SKIP, B.SO_DECISION_CLIP_RESTEP


@pytest.fixture(scope="module", autouse=True)
def _built():
    so_build.build_library()
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)


def _state_bytes(opt):
    return [x.cpu().numpy().tobytes() for x in opt.gather_state()] + \
        [bf16_to_numpy(opt.gather_param_bf16()).tobytes()]


# ---------------------------------------------------------------------------
# config "tiny": 1 Mi parameters, 4 buckets, clip every step, +inf on step 7
# ---------------------------------------------------------------------------

def test_tiny_ten_steps_lockstep():
    rep, opt = run_lockstep(W.tiny(), steps=10)
    assert rep.decisions == [R] * 6 + [S] + [R] * 3
    assert opt.step_count == 9
    c = opt.counters()
    assert (c.commits, c.skips, c.clip_resteps) == (0, 1, 9)
    # the moments follow the oracle's evaluation order: expected bit-identical
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0
    assert rep.n_diff["p"] <= 1e-5 * rep.n_elems


def test_tiny_ragged_tensors_and_odd_bucket_size():
    """Odd tensor sizes, a bucket size that is not a multiple of the vector
    width (slot stride != bucket size, partial quads and a partial tile)."""
    rep, opt = run_lockstep(W.tiny_ragged(), steps=8)
    assert rep.decisions[6] == S and set(rep.decisions) == {R, S}
    assert opt.info.slot_stride_elems != opt.info.bucket_elems


@pytest.mark.parametrize("name", ["tiny", "tiny_ragged"])
def test_register_variant_of_the_step_lockstep(name):
    """The step kernel that keeps everything in registers (no shared-memory
    staging) against the oracle."""
    rep, _ = run_lockstep(W.by_name(name), steps=8, step_variant=1)
    assert rep.decisions[6] == S
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0


@pytest.mark.parametrize("name", ["tiny", "tiny_ragged"])
def test_step_kernel_chosen_by_launch_size_lockstep(name):
    """The library's default: launches of at most 3 Mi elements take the register
    kernel (every launch of these small cases)."""
    rep, _ = run_lockstep(W.by_name(name), steps=8, step_variant=0)
    assert rep.decisions[6] == S
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0


def test_both_step_kernels_in_one_iteration_lockstep():
    """Buckets stepped one by one under the library's choice of kernel: two
    8 Mi-element buckets go through the bulk-copy pipeline, the last bucket
    (1 Mi + 77 elements) through the register kernel; one undo slot short, so
    one bucket is scanned and stepped in place; clip on the second step."""
    w = W.by_name("tiny")
    w.numel = [5 << 20, (12 << 20) + 77]
    w.bucket_elems = 8 << 20
    w.faults = ()
    w.target_norm = lambda step: 0.5 if step % 2 == 1 else 3.0

    def drive(opt, hp, stream, step):
        for b in (2, 0, 1):
            try:
                opt.step_speculative(hp, b, stream)
            except B.SuperOffloadError as e:
                assert e.status == B.SO_ERR_UNDO_EXHAUSTED
        return opt.validate(hp, stream)

    rep, _ = run_lockstep(w, steps=3, undo_slots=2, step_variant=0, drive=drive)
    assert rep.decisions == [C, R, C]
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0


def test_tiny_without_clipping_commits():
    w = W.tiny()
    w.max_grad_norm = 0.0
    w.faults = ()
    rep, opt = run_lockstep(w, steps=4)
    assert rep.decisions == [C] * 4
    assert opt.counters().elems_checked == 0          # sums came from the fused step


def test_tiny_fp32_gradients():
    w = W.tiny()
    w.grad_dtype = "fp32"
    rep, _ = run_lockstep(w, steps=8)
    assert rep.decisions[6] == S


@pytest.mark.parametrize("n,bucket", [(1, 64), (3, 1), (5, 7), (1023, 1024), (1025, 1024),
                                      (4096, 1024), (130_001, 2048), (70_000, 70_000)])
def test_small_and_degenerate_sizes(n, bucket):
    w = W.Workload(name="small", numel=[n], bucket_elems=bucket, sigma_g=1e-2, steps=3)
    rep, _ = run_lockstep(w, steps=3)
    assert len(rep.decisions) == 3


def test_empty_model_on_the_device():
    opt = BucketedAdamW([], 1024)
    hp = oracle.HParams()
    res = opt.iteration(hp, stream=torch.cuda.current_stream())
    assert res.decision == C and res.stats.norm == 0.0 and opt.step_count == 1


def test_empty_model_binds_without_any_device_memory():
    """An empty tensor list needs no arenas: all pointers may be NULL, bind
    touches no device memory, and the iteration is a valid no-op."""
    ctx, info = B.so_layout_init([], 1024)
    assert info.n_buckets == 0
    B.so_layout_bind(ctx, 0, 0, 0, 0, 0, 0)
    hp = oracle.HParams()
    stream = torch.cuda.current_stream()
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL, stream)
    B.so_validate_begin(ctx, hp, stream)
    assert B.so_validate_poll(ctx) is True
    res = B.so_validate_commit_or_rollback(ctx, hp, stream)
    assert res.decision == C and res.step_after == 1 and res.stats.norm == 0.0
    B.so_cast_params(ctx, B.SO_ALL, stream)
    assert B.so_get_counters(ctx).kernel_launches == 0
    B.so_destroy(ctx)


# ---------------------------------------------------------------------------
# exactness of speculation (Section 4.4) and of the rollback
# ---------------------------------------------------------------------------

def _run_device_only(w, steps, undo_slots, speculative, bucket_order=None, step_variant=None):
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, undo_slots,
                        step_variant=step_variant)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    trace = []
    for step in range(1, steps + 1):
        opt.load_grads(W.gradients(w, step, device="cuda"))
        if speculative and bucket_order is not None:
            for b in bucket_order:
                try:
                    opt.step_speculative(hp, b, stream)
                except B.SuperOffloadError as e:
                    assert e.status == B.SO_ERR_UNDO_EXHAUSTED
            res = opt.validate(hp, stream)
        else:
            res = opt.iteration(hp, stream=stream, speculative=speculative)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
    torch.cuda.synchronize()
    return trace, _state_bytes(opt)


@pytest.mark.parametrize("name", ["tiny", "tiny_ragged"])
def test_speculative_flow_is_bitwise_the_check_first_flow(name):
    """STV must reach exactly the result of synchronise-then-execute: state,
    bf16 copy, norm, coefficient and decisions, bit for bit -- whatever subset
    of buckets was speculated and in whatever order."""
    w = W.by_name(name)
    ref = _run_device_only(w, 9, undo_slots=0, speculative=False)
    full = _run_device_only(w, 9, undo_slots=B.SO_ALL, speculative=True)
    windowed = _run_device_only(w, 9, undo_slots=2, speculative=True)
    shuffled = _run_device_only(w, 9, undo_slots=3, speculative=True,
                                bucket_order=[3, 0, 2, 1] if name == "tiny" else [4, 1, 0, 3, 2])
    registers = _run_device_only(w, 9, undo_slots=B.SO_ALL, speculative=True, step_variant=1)
    # the kernel chosen by launch size (these launches are small: the register kernel)
    by_size = _run_device_only(w, 9, undo_slots=2, speculative=True, step_variant=0)
    assert ref[0] == full[0] == windowed[0] == shuffled[0] == registers[0] == by_size[0]
    assert ref[1] == full[1] == windowed[1] == shuffled[1] == registers[1] == by_size[1]


def test_repeat_runs_are_bitwise_identical():
    a = _run_device_only(W.tiny(), 5, B.SO_ALL, True)
    b = _run_device_only(W.tiny(), 5, B.SO_ALL, True)
    assert a == b


def test_elementwise_result_does_not_depend_on_bucket_size():
    outs = []
    for bucket in (262_144, 100_000, 1 << 20, 4096):
        w = W.tiny()
        w.bucket_elems, w.max_grad_norm, w.faults = bucket, 0.0, ()
        outs.append(_run_device_only(w, 3, B.SO_ALL, True)[1])
    assert all(o == outs[0] for o in outs)


@pytest.mark.parametrize("kind", ["inf", "-inf", "nan"])
@pytest.mark.parametrize("where", ["first", "last", "middle"])
def test_rollback_restores_the_prior_state_bit_for_bit(kind, where):
    w = W.tiny_ragged()
    w.faults = ()
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, guard_bands=True)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    opt.load_grads(W.gradients(w, 1, device="cuda"))
    assert opt.iteration(hp, stream=stream).decision == R       # some non-trivial m, v
    before = _state_bytes(opt)
    slots = [B.so_bucket_slot(opt.ctx, b) for b in range(opt.n_buckets)]
    g = W.gradients(w, 2, device="cuda")
    idx = {"first": 0, "last": w.total - 1, "middle": w.total // 2 + 1}[where]
    g[idx] = {"inf": float("inf"), "-inf": float("-inf"), "nan": float("nan")}[kind]
    opt.load_grads(g)
    opt.step_speculative(hp, B.SO_ALL, stream)
    torch.cuda.synchronize()
    during = bf16_to_numpy(opt.gather_param_bf16()).tobytes()
    assert during != before[3]                                  # the speculative copy is live
    res = opt.validate(hp, stream)
    torch.cuda.synchronize()
    assert res.decision == S and res.stats.nonfinite == 1 and res.step_after == 1
    assert _state_bytes(opt) == before
    assert [B.so_bucket_slot(opt.ctx, b) for b in range(opt.n_buckets)] == slots
    assert opt.guard_bands_intact()


# ---------------------------------------------------------------------------
# the gradient check alone
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_grad_check_against_the_oracle_norm(dtype):
    n, bucket = 3_000_017, 500_000
    gen = torch.Generator(device="cuda").manual_seed(5)
    z = torch.randn(n, generator=gen, device="cuda")
    # wide dynamic range, including magnitudes whose square leaves fp32
    expo = torch.randint(-40, 41, (n,), generator=gen, device="cuda").float()
    g = z * torch.pow(torch.tensor(2.0, device="cuda"), expo)
    g[17] = 3.0e38
    g[n - 1] = 1.0e-40
    g = g.to(torch.bfloat16 if dtype == "bf16" else torch.float32)
    opt = BucketedAdamW([n], bucket, grad_dtype=dtype, undo_slots=0)
    opt.load_grads(g)
    hp = oracle.HParams(max_grad_norm=1.0)
    stats = opt.grad_check(hp, stream=torch.cuda.current_stream())
    s, nrm, flag = oracle.global_grad_check(grads_to_numpy(g), bucket)
    assert flag == 0 and stats.nonfinite == 0                   # finite in, finite out
    assert stats.sumsq == pytest.approx(s, rel=1e-12)
    assert stats.norm == pytest.approx(nrm, rel=1e-12)
    assert stats.clip_coef == pytest.approx(oracle.clip_coef(nrm, 1.0), rel=1e-12)
    opt.validate(hp, torch.cuda.current_stream())


def test_nonfinite_flag_for_every_special_bf16_pattern_and_position():
    n, bucket = 5000, 1024
    specials = [0x7F80, 0xFF80, 0x7F81, 0x7FC0, 0xFFFF, 0x7FFF]
    finite_extremes = [0x7F7F, 0xFF7F, 0x0001, 0x8001, 0x0000, 0x8000]
    hp = oracle.HParams(max_grad_norm=0.0)
    opt = BucketedAdamW([n], bucket, undo_slots=0)
    base = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    for pos in (0, 1023, 1024, 4095, 4096, 4999):
        for pat, want in [(p, 1) for p in specials] + [(p, 0) for p in finite_extremes]:
            g = base.clone()
            g.view(torch.int16)[pos] = np.array(pat, dtype=np.uint16).view(np.int16).item()
            opt.load_grads(g)
            stats = opt.grad_check(hp, stream=torch.cuda.current_stream())
            assert stats.nonfinite == want, (hex(pat), pos)
            _, flag = oracle.grad_check_range(grads_to_numpy(g), 0, n)
            assert flag == want
            res = opt.validate(hp, torch.cuda.current_stream())
            assert res.decision == (S if want else C)


# ---------------------------------------------------------------------------
# the cast alone: every fp32 bit pattern
# ---------------------------------------------------------------------------

def test_cast_is_rne_for_all_2_to_32_patterns():
    chunk = 1 << 26
    opt = BucketedAdamW([chunk], 1 << 24, undo_slots=0)
    stream = torch.cuda.current_stream()
    for c in range((1 << 32) // chunk):
        pats = torch.arange(c * chunk, (c + 1) * chunk, dtype=torch.int64, device="cuda")
        bits = pats.to(torch.int32) if c < 32 else (pats - (1 << 32)).to(torch.int32)
        opt.master[:chunk].copy_(bits.view(torch.float32))
        opt.cast_params(stream=stream)
        got = opt.param_bf16[:chunk].view(torch.int16)
        host_in = bits.view(torch.float32).cpu().numpy()
        want = oracle.bf16_rne(host_in)
        want_t = torch.from_numpy(want.view(np.int16)).cuda()
        nan = torch.from_numpy(np.isnan(host_in)).cuda()
        assert torch.equal(got[~nan], want_t[~nan]), f"chunk {c}"
        if nan.any():
            got_nan = got[nan].cpu().numpy().view(np.uint16)
            assert is_bf16_nan(got_nan).all(), f"chunk {c}: NaN lost"


# ---------------------------------------------------------------------------
# GPT-2-small-shaped list: 124M parameters in 25M-element buckets
# ---------------------------------------------------------------------------

def test_gpt2_small_commit_path_lockstep():
    rep, opt = run_lockstep(W.gpt2_small(clip=False), steps=4, guard_bands=False)
    assert rep.decisions == [C] * 4
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0
    assert rep.max_norm_rel < 1e-12


def test_gpt2_small_clip_path_lockstep():
    rep, opt = run_lockstep(W.gpt2_small(clip=True), steps=3, guard_bands=False)
    assert rep.decisions == [R] * 3
    assert rep.max_ulp["p"] <= 2


# ---------------------------------------------------------------------------
# the host-fed, bucket-pipelined iteration
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("name,undo,dtype", [("tiny", B.SO_ALL, "bf16"), ("tiny_ragged", 2, "bf16"),
                                             ("tiny", 0, "bf16"), ("tiny_ragged", 3, "fp32")])
def test_host_fed_iteration_is_bitwise_the_device_fed_one(name, undo, dtype):
    """so_iteration_host (pinned gradients in, bf16 parameters out, copies
    overlapped per bucket) must leave exactly the state, statistics and
    decisions of the ordinary call sequence, and deliver the committed bf16
    parameters to the host -- through commits, clip re-steps and a skip."""
    w = W.by_name(name)
    w.grad_dtype = dtype
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    ref = _run_device_only(w, 8, undo_slots=undo, speculative=True)

    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, undo)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    host_g = torch.empty(w.total, dtype=opt.grad_torch_dtype, pin_memory=True)
    host_p = torch.empty(w.total, dtype=torch.bfloat16, pin_memory=True)
    trace = []
    for step in range(1, 9):
        host_g.copy_(W.gradients(w, step, device="cuda"))     # same bits as the reference run
        res = B.so_iteration_host(opt.ctx, hp, host_g.data_ptr(), host_p.data_ptr(), stream)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
        dev_pb = opt.gather_param_bf16().cpu()
        assert torch.equal(host_p.view(torch.int16), dev_pb.view(torch.int16)), step
    assert trace == ref[0]
    assert _state_bytes(opt) == ref[1]
    assert S in [t[0] for t in trace]


def test_pipelined_host_fed_iterations_overwrite_no_gradient_still_in_use():
    """Copies long enough (50 MB per bucket) that an incoming gradient which
    started too early would land under a kernel still reading the bucket: five
    buckets, two of them speculated, and a commit, a clip, a skip, a clip and a
    commit in a row, so that the next call follows every kind of verdict (after
    a commit the speculated buckets may be overwritten at once, after a skip all
    of them, after a clip none before the re-step has run)."""
    w = W.by_name("gpt2_small")
    w.max_grad_norm = 1.0
    w.target_norm = lambda step: 0.5 if step % 2 == 1 else 3.0
    w.faults = (W.Fault(step=3, flat_index=3 * w.bucket_elems + 12345, kind="inf"),)
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    ref = _run_device_only(w, 5, undo_slots=2, speculative=True)
    C, S, R = B.SO_DECISION_COMMIT, B.SO_DECISION_SKIP, B.SO_DECISION_CLIP_RESTEP
    assert [t[0] for t in ref[0]] == [C, R, S, R, C]
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 2)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    host_g = [torch.empty(w.total, dtype=opt.grad_torch_dtype, pin_memory=True) for _ in range(2)]
    host_p = torch.empty(w.total, dtype=torch.bfloat16, pin_memory=True)
    trace = []
    for step in range(1, 6):
        buf = host_g[step % 2]
        buf.copy_(W.gradients(w, step, device="cuda"))
        res = B.so_iteration_host_pipelined(opt.ctx, hp, buf.data_ptr(), host_p.data_ptr(), stream)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
    B.so_iteration_host_wait(opt.ctx, stream)
    assert trace == ref[0]
    assert _state_bytes(opt) == ref[1]
    assert torch.equal(host_p.view(torch.int16), opt.gather_param_bf16().cpu().view(torch.int16))


@pytest.mark.parametrize("name,undo", [("tiny", B.SO_ALL), ("tiny_ragged", 2), ("tiny_ragged", 0)])
def test_pipelined_host_fed_iterations_are_bitwise_the_blocking_ones(name, undo):
    """so_iteration_host_pipelined does not wait at its end: the parameters that
    leave after the verdict travel while the next call's gradients arrive.
    Two alternating gradient buffers (a buffer is refilled as soon as the call
    that read it has returned), one parameter buffer checked after the final
    wait and at every step through a blocking gather on the same stream."""
    w = W.by_name(name)
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    ref = _run_device_only(w, 8, undo_slots=undo, speculative=True)
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, undo)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    host_g = [torch.empty(w.total, dtype=opt.grad_torch_dtype, pin_memory=True) for _ in range(2)]
    host_p = torch.empty(w.total, dtype=torch.bfloat16, pin_memory=True)
    trace = []
    for step in range(1, 9):
        buf = host_g[step % 2]
        buf.copy_(W.gradients(w, step, device="cuda"))
        res = B.so_iteration_host_pipelined(opt.ctx, hp, buf.data_ptr(), host_p.data_ptr(), stream)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
    B.so_iteration_host_wait(opt.ctx, stream)
    assert trace == ref[0]
    assert _state_bytes(opt) == ref[1]
    dev_pb = opt.gather_param_bf16().cpu()
    assert torch.equal(host_p.view(torch.int16), dev_pb.view(torch.int16))
    B.so_iteration_host_wait(opt.ctx, stream)                  # nothing in flight: a no-op
    # a blocking call right after pipelined ones is ordered behind them
    host_g[0].copy_(W.gradients(w, 9, device="cuda"))
    B.so_iteration_host_pipelined(opt.ctx, hp, host_g[0].data_ptr(), host_p.data_ptr(), stream)
    host_g[1].copy_(W.gradients(w, 10, device="cuda"))
    B.so_iteration_host(opt.ctx, hp, host_g[1].data_ptr(), host_p.data_ptr(), stream)
    assert torch.equal(host_p.view(torch.int16), opt.gather_param_bf16().cpu().view(torch.int16))


def test_pipelined_host_fed_iterations_without_a_parameter_buffer():
    """No outgoing copies at all (host_param_bf16 = NULL): the calls still
    overlap their incoming copies with the previous iteration's follow-up, and
    the final wait still waits for the stream."""
    w = W.by_name("tiny_ragged")
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    ref = _run_device_only(w, 8, undo_slots=2, speculative=True)
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 2)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    host_g = [torch.empty(w.total, dtype=opt.grad_torch_dtype, pin_memory=True) for _ in range(2)]
    trace = []
    for step in range(1, 9):
        buf = host_g[step % 2]
        buf.copy_(W.gradients(w, step, device="cuda"))
        res = B.so_iteration_host_pipelined(opt.ctx, hp, buf.data_ptr(), 0, stream)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
    B.so_iteration_host_wait(opt.ctx, stream)
    assert trace == ref[0]
    assert _state_bytes(opt) == ref[1]


# ---------------------------------------------------------------------------
# fp16 gradients under dynamic loss scaling (the paper's own precision path)
# ---------------------------------------------------------------------------

def test_fp16_gradients_with_dynamic_loss_scale_lockstep():
    """Stored gradients are loss_scale * g in fp16.  The initial scale 2^23
    overflows (SKIP, scale halves) until the scaled gradients fit; then every
    step clips (norm ~ 10 > 1) and the scale doubles every 3 kept steps until
    it overflows again.  State, decisions and the scale schedule must follow
    the oracle."""
    rep, opt = run_lockstep(W.tiny_fp16(), steps=16)
    assert rep.decisions[0] == S and R in rep.decisions
    first_kept = rep.decisions.index(R)
    assert all(d == S for d in rep.decisions[:first_kept]) and first_kept >= 2
    assert S in rep.decisions[first_kept:]              # grew back into an overflow
    assert rep.loss_scales[first_kept - 1] == 2.0 ** (23 - first_kept)
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0
    assert opt.step_count == rep.decisions.count(R)


def test_fp16_static_scale_register_variant_and_check_first_flow():
    w = W.tiny_fp16()
    w.loss_scale, w.ls_interval = 2.0 ** 12, 0
    a, _ = run_lockstep(w, steps=4, step_variant=1)
    b, _ = run_lockstep(w, steps=4, undo_slots=0, speculative=False)
    assert a.decisions == b.decisions == [R] * 4
    assert a.loss_scales == b.loss_scales == [2.0 ** 12] * 4


# ---------------------------------------------------------------------------
# validation off the critical path; checkpoint and resume
# ---------------------------------------------------------------------------

def test_deferred_validation_gives_the_same_bits():
    """so_validate_begin, other work on the stream (a stand-in for the next
    forward pass), then the verdict: identical to validating at once."""
    w = W.tiny()
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    ref = _run_device_only(w, 8, undo_slots=B.SO_ALL, speculative=True)
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, B.SO_ALL)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    a = torch.randn(2048, 2048, device="cuda")
    trace = []
    for step in range(1, 9):
        opt.load_grads(W.gradients(w, step, device="cuda"))
        opt.step_speculative(hp, B.SO_ALL, stream)
        B.so_validate_begin(opt.ctx, hp, stream)
        for _ in range(4):
            a = torch.tanh(a @ a.t() * 1e-3)                 # "forward pass" behind the reduction
        polls = 0
        while not B.so_validate_poll(opt.ctx):
            polls += 1
            assert polls < 10_000_000
        res = opt.validate(hp, stream)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
    torch.cuda.synchronize()
    assert trace == ref[0] and _state_bytes(opt) == ref[1]


def test_checkpoint_export_import_resumes_bit_for_bit():
    w = W.tiny_ragged()
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    straight = _run_device_only(w, 6, undo_slots=B.SO_ALL, speculative=True)

    first = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, B.SO_ALL)
    first.load_state(W.initial_master(w, device="cuda"))
    first.cast_params(stream=stream)
    for step in (1, 2, 3):
        first.load_grads(W.gradients(w, step, device="cuda"))
        first.iteration(hp, stream=stream)
    n = w.total
    ckpt = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(2)]
    host_v = torch.empty(n, dtype=torch.float32, pin_memory=True)      # one array via the host
    B.so_state_export(first.ctx, ckpt[0].data_ptr(), ckpt[1].data_ptr(), host_v.data_ptr(), stream)
    torch.cuda.synchronize()
    t = first.step_count
    gathered = first.gather_state()
    assert torch.equal(ckpt[0], gathered[0]) and torch.equal(ckpt[1], gathered[1])
    assert torch.equal(host_v.cuda(), gathered[2])

    second = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 2)    # a different undo window
    B.so_state_import(second.ctx, ckpt[0].data_ptr(), ckpt[1].data_ptr(), host_v.data_ptr(), stream)
    B.so_set_step(second.ctx, t)
    second.cast_params(stream=stream)
    for step in (4, 5, 6):
        second.load_grads(W.gradients(w, step, device="cuda"))
        second.iteration(hp, stream=stream)
    torch.cuda.synchronize()
    assert second.step_count == straight[0][-1][5]
    assert _state_bytes(second) == straight[1]


# ---------------------------------------------------------------------------
# launch structure: batches of more than 128 buckets, several streams
# ---------------------------------------------------------------------------

def test_three_hundred_small_buckets_lockstep():
    """301 buckets of 4096 elements: a batched call splits into three launches
    (128 buckets each at most), each with its own tile counter."""
    w = W.Workload(name="many_buckets", numel=[300 * 4096 + 17], bucket_elems=4096,
                   sigma_g=1e-2, steps=4,
                   faults=(W.Fault(step=3, flat_index=200 * 4096 + 5, kind="nan"),))
    rep, opt = run_lockstep(w, steps=4)
    assert opt.n_buckets == 301 and rep.decisions == [R, R, S, R]
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0


def test_per_bucket_launches_on_two_streams_give_the_same_bits():
    """Buckets stepped one call at a time, alternating between two streams whose
    kernels may overlap on the GPU (each launch claims tiles from its own
    counter), against the single batched launch."""
    w = W.tiny_ragged()
    hp = hparams_of(w)
    ref = _run_device_only(w, 6, undo_slots=B.SO_ALL, speculative=True)
    main = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, B.SO_ALL)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=main)
    trace = []
    for step in range(1, 7):
        opt.load_grads(W.gradients(w, step, device="cuda"))
        side.wait_stream(main)
        for b in range(opt.n_buckets):
            opt.step_speculative(hp, b, side if b % 2 else main)
        main.wait_stream(side)
        res = opt.validate(hp, main)
        side.wait_stream(main)                      # re-steps / re-casts finish before reuse
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))
    torch.cuda.synchronize()
    assert trace == ref[0] and _state_bytes(opt) == ref[1]


# ---------------------------------------------------------------------------
# cancelling updates: p*(1 - lr*wd) and the Adam update nearly equal
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("t0,clip,dtype,undo", [(0, False, "bf16", B.SO_ALL), (0, True, "bf16", B.SO_ALL),
                                                (5, False, "bf16", B.SO_ALL), (5, True, "fp32", B.SO_ALL),
                                                (3, True, "fp16", B.SO_ALL),
                                                (5, False, "bf16", 0), (2, True, "fp32", 0)])
def test_cancelling_update_stays_within_tolerance(t0, clip, dtype, undo):
    """When the decayed parameter and the update cancel, the new parameter is
    orders of magnitude smaller than either, and an fp64 rounding error in the
    update that is harmless elsewhere becomes whole fp32 ulps of the result.
    Masters are placed next to the update (relative distance 2^-8 .. 2^-50
    before their own rounding to fp32), so most of the new parameters are
    1e-7 .. 1e-12 of the old ones.  The 2-ulp bound has to hold there too, and
    deep inside the zone the result has to be the oracle's bit for bit.
    undo = 0 takes the check-first route (steps in place); the 13 elements past
    the last full bucket take the kernels' guarded, non-staged path."""
    n, bucket = (1 << 20) + 13, 1 << 18
    rng = np.random.default_rng(11 + t0 + int(clip))
    hp = oracle.HParams(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
                        max_grad_norm=1.0 if clip else 0.0)
    loss_scale = 4096.0 if dtype == "fp16" else 1.0
    unscale = 1.0 / loss_scale
    g32 = (rng.standard_normal(n) * 1e-2 * loss_scale).astype(np.float32)
    torch_dtype = {"bf16": torch.bfloat16, "fp32": torch.float32, "fp16": torch.float16}[dtype]
    g_t = torch.from_numpy(g32).cuda().to(torch_dtype)
    g_host = grads_to_numpy(g_t)             # what the oracle takes: bf16 bits, or fp32 / fp16 values
    g = (bf16_bits_to_f32(g_host) if dtype == "bf16" else g_host).astype(np.float64) * unscale
    if t0:
        m0 = (rng.standard_normal(n) * 3e-3).astype(np.float32)
        v0 = (rng.random(n) * 1e-4 + 1e-8).astype(np.float32)
    else:
        m0 = np.zeros(n, np.float32)
        v0 = np.zeros(n, np.float32)
    coef = 1.0
    if clip:
        _, norm, _ = oracle.global_grad_check(g_host, bucket, unscale)
        coef = oracle.clip_coef(norm, hp.max_grad_norm)
        assert coef < 1.0
    # where the update will land (input construction only; the expected values
    # below come from the oracle)
    gs = g * coef
    m1 = hp.beta1 * m0 + (1 - hp.beta1) * gs
    v1 = hp.beta2 * v0 + (1 - hp.beta2) * gs * gs
    tt = t0 + 1
    u = hp.lr * (m1 / (1 - hp.beta1 ** tt)) / (np.sqrt(v1 / (1 - hp.beta2 ** tt)) + hp.eps)
    delta = np.ldexp(1.0, -rng.integers(8, 51, n)) * rng.choice([-1.0, 1.0], n)
    p0 = (u / (1 - hp.lr * hp.weight_decay) * (1 + delta)).astype(np.float32)

    stream = torch.cuda.current_stream()
    for variant in (2, 1):                 # the bulk-copy pipeline, the register kernel
        opt = BucketedAdamW([n], bucket, dtype, undo, step_variant=variant)
        opt.load_state(torch.from_numpy(p0).cuda(), torch.from_numpy(m0).cuda(),
                       torch.from_numpy(v0).cuda())
        B.so_set_step(opt.ctx, t0)
        if dtype == "fp16":
            B.so_loss_scale_config(opt.ctx, loss_scale, 2.0, 0.5, 1000)
        opt.cast_params(stream=stream)
        opt.load_grads(g_t)
        res = opt.iteration(hp, stream=stream)
        torch.cuda.synchronize()
        assert res.decision == (R if clip else C)

        p, m, v = p0.copy(), m0.copy(), v0.copy()
        pb = oracle.bf16_rne(p)
        orc = oracle.iteration_stv(p, m, v, pb, g_host, bucket, t0, hp,
                                   forced_coef=res.stats.clip_coef if clip else None,
                                   unscale=unscale)
        assert orc.decision == res.decision
        dev = [x.cpu().numpy() for x in opt.gather_state()]
        ratio = np.abs(p.astype(np.float64)) / np.abs(p0.astype(np.float64))
        # with a clip, the device's coefficient differs from the one the masters
        # were placed with by ~1e-13 relative, which bounds the cancellation
        assert np.count_nonzero(ratio < 2.0 ** -24) > n // 4     # the zone is populated
        d = ulp_distance(dev[0], p)
        assert d.max() <= 2, f"variant {variant}: p {d.max()} ulp from the oracle"
        deep = ratio < 2.0 ** -17
        assert np.array_equal(dev[0][deep].view(np.uint32), p[deep].view(np.uint32))
        assert dev[1].tobytes() == m.tobytes() and dev[2].tobytes() == v.tobytes()
        assert np.array_equal(bf16_to_numpy(opt.gather_param_bf16()), oracle.bf16_rne(dev[0]))
        opt.close()


# ---------------------------------------------------------------------------
# random call sequences: any legal order and granularity gives the oracle's result
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("seed,undo,dtype", [(0, B.SO_ALL, "bf16"), (1, 5, "bf16"),
                                             (2, 0, "fp32"), (3, 11, "fp32")])
def test_random_call_sequences_lockstep(seed, undo, dtype):
    """22 ragged buckets; per iteration the buckets are visited in random order
    and each is stepped speculatively, scanned, or left to validation; the
    check is finished by so_grad_check(SO_ALL), so_validate_begin, or validation
    itself; norms fall on both sides of the clip threshold and two iterations
    carry a non-finite gradient.  Every iteration is compared with the oracle."""
    import random
    rng = random.Random(seed)
    w = W.tiny_ragged()
    w.name = f"random_walk_{seed}"
    w.bucket_elems = 50_003
    w.grad_dtype = dtype
    w.seed = 100 + seed
    w.target_norm = lambda step: (0.4, 2.5, 0.9, 7.0)[(step * 7 + seed) % 4]
    w.faults = (W.Fault(step=4, flat_index=3 * 50_003 + 11, kind="nan"),
                W.Fault(step=9, flat_index=w.total - 1, kind="-inf"))
    exhausted = [0]

    def drive(opt, hp, stream, step):
        order = list(range(opt.n_buckets))
        rng.shuffle(order)
        for b in order:
            r = rng.random()
            try:
                if r < 0.6:
                    B.so_adam_step_speculative(opt.ctx, hp, b, stream)
                elif r < 0.8:
                    B.so_grad_check(opt.ctx, None, b, stream)
            except B.SuperOffloadError as e:
                assert e.status == B.SO_ERR_UNDO_EXHAUSTED
                exhausted[0] += 1
        mode = rng.random()
        if mode < 0.3:
            B.so_validate_begin(opt.ctx, hp, stream)
        elif mode < 0.5:
            B.so_grad_check(opt.ctx, hp, B.SO_ALL, stream)
        return B.so_validate_commit_or_rollback(opt.ctx, hp, stream)

    rep, opt = run_lockstep(w, steps=12, undo_slots=undo, drive=drive)
    assert {C, S, R} <= set(rep.decisions), rep.decisions
    assert rep.decisions[3] == S and rep.decisions[8] == S
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0
    assert opt.step_count == 10
    if undo not in (B.SO_ALL,):
        assert exhausted[0] > 0
    opt.close()


# ---------------------------------------------------------------------------
# verdict on the device, host one iteration behind
# ---------------------------------------------------------------------------

def _mixed_outcome_workload():
    """Ragged tensors, norm alternating below / above the clip threshold, one
    +inf and one NaN: COMMIT, CLIP_RESTEP and SKIP all occur."""
    w = W.tiny_ragged()
    w.name = "tiny_ragged_mixed"
    w.sigma_g = 1.0
    w.target_norm = lambda step: 0.5 if step % 2 == 1 else 3.0
    w.faults = (W.Fault(step=3, flat_index=2 * 250_003 + 17, kind="inf"),
                W.Fault(step=6, flat_index=5, kind="nan"))
    return w


@pytest.mark.parametrize("undo,per_bucket", [(B.SO_ALL, False), (2, False), (3, True)])
def test_pipelined_iterations_with_the_verdict_on_the_device_lockstep(undo, per_bucket):
    """The next iteration's speculative steps are enqueued before the host has
    collected the previous verdict; windowed undo; every outcome."""
    from gpu_harness import run_lockstep_pipelined
    rep, opt = run_lockstep_pipelined(_mixed_outcome_workload(), steps=9, undo_slots=undo,
                                      per_bucket=per_bucket)
    assert rep.decisions == [C, R, S, R, C, S, C, R, C]
    assert opt.step_count == 7
    assert rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0
    # the same trajectory as collecting every verdict at once, bit for bit
    ref, ref_opt = run_lockstep(_mixed_outcome_workload(), steps=9, undo_slots=undo)
    assert ref.decisions == rep.decisions
    assert _state_bytes(opt) == _state_bytes(ref_opt)


def test_pipelined_fp16_gradients_pick_the_loss_scale_on_the_device():
    """Dynamic loss scaling: the scale of iteration k+1 depends on how
    iteration k ended, which its kernels read on the device."""
    from gpu_harness import run_lockstep_pipelined
    w = W.tiny_fp16()
    rep, opt = run_lockstep_pipelined(w, steps=12, undo_slots=3)
    ref, ref_opt = run_lockstep(W.tiny_fp16(), steps=12, undo_slots=3)
    assert rep.decisions == ref.decisions and S in rep.decisions and R in rep.decisions
    assert rep.loss_scales == ref.loss_scales
    assert _state_bytes(opt) == _state_bytes(ref_opt)


def test_a_kernel_that_gives_up_its_wait_ends_the_iteration_cleanly():
    """The bulk-copy step kernel polls a bounded number of times for a chunk's
    loads.  With the limit at zero every warp gives up at once (its copies are
    still waited for, with the full limit, before the block exits): the device
    raises its status word, the validation reports SO_ERR_TIMEOUT, the committed
    state is untouched, and the same iteration then runs normally."""
    w = W.tiny()
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 3, guard_bands=True)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    g = W.gradients(w, 1, device="cuda")
    opt.load_grads(g)
    torch.cuda.synchronize()
    before = _state_bytes(opt)
    B.so_debug_set_spin_limit(opt.ctx, 0)
    opt.step_speculative(hp, B.SO_ALL, stream)           # buckets 0..2, all warps give up
    B.so_debug_set_spin_limit(opt.ctx, 1 << 20)
    with pytest.raises(B.SuperOffloadError) as err:
        opt.validate(hp, stream)
    assert err.value.status == B.SO_ERR_TIMEOUT
    torch.cuda.synchronize()
    c = opt.counters()
    assert c.timeouts == 1 and (c.commits, c.skips, c.clip_resteps) == (0, 0, 0)
    assert opt.step_count == 0 and B.so_pending_buckets(opt.ctx) == 4
    assert _state_bytes(opt) == before                    # fp32 state and the re-derived bf16 copy
    # the status was consumed: the iteration is repeated and matches the oracle
    res = opt.iteration(hp, stream=stream)
    torch.cuda.synchronize()
    p = W.initial_master(w, device="cuda").cpu().numpy()
    m, v = np.zeros_like(p), np.zeros_like(p)
    pb = oracle.bf16_rne(p)
    ref = oracle.iteration_stv(p, m, v, pb, grads_to_numpy(g), w.bucket_elems, 0, hp,
                               forced_coef=res.stats.clip_coef)
    assert res.decision == ref.decision == R and opt.step_count == 1
    dev = [x.cpu().numpy() for x in opt.gather_state()]
    for a, b in zip(dev, (p, m, v)):
        assert ulp_distance(a, b).max() <= 2
    assert opt.counters().timeouts == 1 and opt.guard_bands_intact()


def test_a_give_up_inside_pipelined_host_fed_iterations_leaves_nothing_in_flight():
    """The same bounded wait running out in the middle of overlapped host-fed
    iterations: the failing call reports SO_ERR_TIMEOUT after waiting for every
    copy it or its predecessor started, the committed state is the one before
    it, and the iteration, given again, continues the sequence bit for bit."""
    w = W.by_name("tiny_ragged")
    hp = hparams_of(w)
    stream = torch.cuda.current_stream()
    ref = _run_device_only(w, 4, undo_slots=2, speculative=True)
    opt = BucketedAdamW(w.numel, w.bucket_elems, w.grad_dtype, 2, guard_bands=True)
    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    host_g = [torch.empty(w.total, dtype=opt.grad_torch_dtype, pin_memory=True) for _ in range(2)]
    host_p = torch.empty(w.total, dtype=torch.bfloat16, pin_memory=True)
    trace = []

    def call(step):
        buf = host_g[step % 2]
        buf.copy_(W.gradients(w, step, device="cuda"))
        res = B.so_iteration_host_pipelined(opt.ctx, hp, buf.data_ptr(), host_p.data_ptr(), stream)
        trace.append((res.decision, res.stats.sumsq, res.stats.norm, res.stats.clip_coef,
                      res.stats.nonfinite, res.step_after))

    call(1)
    call(2)
    B.so_debug_set_spin_limit(opt.ctx, 0)
    with pytest.raises(B.SuperOffloadError) as err:
        call(3)
    assert err.value.status == B.SO_ERR_TIMEOUT
    B.so_debug_set_spin_limit(opt.ctx, 1 << 20)
    assert opt.step_count == 2 and opt.counters().timeouts == 1
    B.so_iteration_host_wait(opt.ctx, stream)                 # nothing left to wait for
    call(3)
    call(4)
    B.so_iteration_host_wait(opt.ctx, stream)
    assert trace == ref[0]
    assert _state_bytes(opt) == ref[1]
    assert torch.equal(host_p.view(torch.int16), opt.gather_param_bf16().cpu().view(torch.int16))
    assert opt.guard_bands_intact()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_second_moments_that_overflow_fp32_follow_the_oracle(dtype):
    """Finite gradients around 1e21 with clipping off: (1 - beta2) g^2 exceeds
    the fp32 range, the stored second moment becomes +Inf, and the update of
    those elements is exactly the decay term, on both sides, from then on."""
    w = W.Workload(name="huge_grads", numel=[5000], bucket_elems=2048, sigma_g=1e21, steps=3,
                   max_grad_norm=0.0, grad_dtype=dtype)
    rep, opt = run_lockstep(w, steps=3)
    assert rep.decisions == [C] * 3
    v = opt.gather_state()[2]
    assert torch.isinf(v).any() and not torch.isnan(opt.gather_state()[0]).any()
    assert rep.max_ulp["p"] <= 2 and rep.n_diff["v"] == 0


# ---------------------------------------------------------------------------
# binary16 parameter copy (the paper's FP16 runs)
# ---------------------------------------------------------------------------

def _is_fp16_nan(bits):
    b = bits.astype(np.uint32)
    return ((b & 0x7C00) == 0x7C00) & ((b & 0x03FF) != 0)


def test_fp16_cast_is_rne_for_all_2_to_32_patterns():
    chunk = 1 << 26
    opt = BucketedAdamW([chunk], 1 << 24, undo_slots=0, param_dtype="fp16")
    stream = torch.cuda.current_stream()
    for c in range((1 << 32) // chunk):
        pats = torch.arange(c * chunk, (c + 1) * chunk, dtype=torch.int64, device="cuda")
        bits = pats.to(torch.int32) if c < 32 else (pats - (1 << 32)).to(torch.int32)
        opt.master[:chunk].copy_(bits.view(torch.float32))
        opt.cast_params(stream=stream)
        got = opt.param_bf16[:chunk].view(torch.int16)
        host_in = bits.view(torch.float32).cpu().numpy()
        want = oracle.fp16_rne(host_in)
        want_t = torch.from_numpy(want.view(np.int16)).cuda()
        nan = torch.from_numpy(np.isnan(host_in)).cuda()
        assert torch.equal(got[~nan], want_t[~nan]), f"chunk {c}"
        if nan.any():
            got_nan = got[nan].cpu().numpy().view(np.uint16)
            assert _is_fp16_nan(got_nan).all(), f"chunk {c}: NaN lost"


@pytest.mark.parametrize("name", ["tiny_ragged", "tiny_fp16"])
def test_fp16_parameter_copy_lockstep(name):
    """The fused step writes binary16 parameters (with fp16 gradients and loss
    scaling this is the paper's own precision recipe)."""
    rep, opt = run_lockstep(W.by_name(name), steps=8, undo_slots=3, param_dtype="fp16")
    assert S in rep.decisions and rep.n_diff["m"] == 0 and rep.n_diff["v"] == 0
    assert opt.param_bf16.dtype == torch.float16


# ---------------------------------------------------------------------------
# flattening on the device: tensor list <-> bucket arenas in one launch
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("name,dtype", [("tiny_ragged", "bf16"), ("tiny_ragged", "fp32"),
                                        ("gpt2_small", "bf16")])
def test_pack_and_unpack_match_the_per_tensor_copies(name, dtype):
    w = W.by_name(name)
    w.grad_dtype = dtype
    stream = torch.cuda.current_stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, dtype, 0, guard_bands=True)
    flat = W.gradients(w, 1, device="cuda")
    # every tensor in a buffer of its own, starting at an odd element offset for
    # every other one (no 16-byte alignment to rely on)
    tensors, pos = [], 0
    for i, n in enumerate(w.numel):
        buf = torch.empty(n + 8, dtype=flat.dtype, device="cuda")
        t = buf[(i % 2) * 3:(i % 2) * 3 + n]
        t.copy_(flat[pos:pos + n])
        tensors.append(t)
        pos += n
    opt.pack_grads(tensors, stream)
    torch.cuda.synchronize()
    packed = opt.grad.clone()
    opt.grad.zero_()
    opt.load_grads(flat)                                   # the per-bucket torch copies
    torch.cuda.synchronize()
    assert torch.equal(packed.view(torch.uint8), opt.grad.view(torch.uint8))

    opt.load_state(W.initial_master(w, device="cuda"))
    opt.cast_params(stream=stream)
    want = opt.gather_param_bf16()
    outs = []
    for i, n in enumerate(w.numel):
        buf = torch.full((n + 8,), 7.0, dtype=torch.bfloat16, device="cuda")
        outs.append((buf, buf[(i % 2) * 5:(i % 2) * 5 + n]))
    opt.unpack_params([t for _, t in outs], stream)
    torch.cuda.synchronize()
    pos = 0
    for i, (buf, t) in enumerate(outs):
        n = w.numel[i]
        assert torch.equal(t.view(torch.int16), want[pos:pos + n].view(torch.int16)), i
        lead = (i % 2) * 5
        assert (buf[:lead] == 7.0).all() and (buf[lead + n:] == 7.0).all()     # nothing around it
        pos += n
    assert opt.guard_bands_intact()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("bucket", [100_000, 100_003])
def test_pack_and_unpack_at_every_offset_from_the_16_byte_grid(dtype, bucket):
    """Tensors that start 0, 1, ... 7 elements into their buffers (every offset
    from the 16-byte grid the element size allows), long enough that whole runs
    lie inside one tensor, against aligned and unaligned bucket starts."""
    w = W.by_name("tiny")
    w.numel = [50_000 + 37 * i for i in range(16)]
    w.bucket_elems = bucket
    w.grad_dtype = dtype
    stream = torch.cuda.current_stream()
    opt = BucketedAdamW(w.numel, w.bucket_elems, dtype, 0, guard_bands=True)
    total = sum(w.numel)
    gen = torch.Generator(device="cuda").manual_seed(11)
    flat = torch.randn(total, device="cuda", generator=gen).to(opt.grad_torch_dtype)
    tensors, pos = [], 0
    for i, n in enumerate(w.numel):
        buf = torch.empty(n + 8, dtype=flat.dtype, device="cuda")
        t = buf[i % 8:i % 8 + n]
        t.copy_(flat[pos:pos + n])
        tensors.append(t)
        pos += n
    opt.pack_grads(tensors, stream)
    torch.cuda.synchronize()
    packed = opt.grad.clone()
    opt.grad.zero_()
    opt.load_grads(flat)
    torch.cuda.synchronize()
    assert torch.equal(packed.view(torch.uint8), opt.grad.view(torch.uint8))

    master = torch.randn(total, device="cuda", generator=gen)
    opt.load_state(master)
    opt.cast_params(stream=stream)
    want = opt.gather_param_bf16()
    outs = []
    for i, n in enumerate(w.numel):
        lead = (3 * i + 1) % 8
        buf = torch.full((n + 8,), 7.0, dtype=torch.bfloat16, device="cuda")
        outs.append((buf, lead, buf[lead:lead + n]))
    opt.unpack_params([t for _, _, t in outs], stream)
    torch.cuda.synchronize()
    pos = 0
    for i, (buf, lead, t) in enumerate(outs):
        n = w.numel[i]
        assert torch.equal(t.view(torch.int16), want[pos:pos + n].view(torch.int16)), i
        assert (buf[:lead] == 7.0).all() and (buf[lead + n:] == 7.0).all(), i
        pos += n
    assert opt.guard_bands_intact()
