"""CPU-only tests of the library's host side: it loads, exports what the header
declares, does the layout arithmetic, and runs the slot map / per-iteration
state machine (in dry-run mode, where nothing is launched)."""
from __future__ import annotations

import math
import os
import re

import pytest

import oracle
from paper_2509_21271_b200 import binding as B
from paper_2509_21271_b200 import build as so_build
from paper_2509_21271_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    so_build.build_library()


class HP:
    lr, beta1, beta2, eps, weight_decay, max_grad_norm = 1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0

    def __init__(self, **kw):
        for k, v in kw.items():
            setattr(self, k, v)


def _dry_ctx(numel, bucket, undo=B.SO_ALL, gd=B.SO_GRAD_BF16):
    ctx, info = B.so_layout_init(numel, bucket, gd, undo)
    B.so_debug_set_dry_run(ctx, True)
    base = 0x10000000
    B.so_layout_bind(ctx, base, base * 2, base * 3, base * 4, base * 5, base * 6)
    return ctx, info


def _status(fn, *a):
    try:
        fn(*a)
        return B.SO_OK
    except B.SuperOffloadError as e:
        return e.status


def test_library_exports_every_declared_symbol():
    with open(os.path.join(ROOT, "include", "superoffload.h")) as fh:
        text = re.sub(r"/\*.*?\*/", "", fh.read(), flags=re.S)
    declared = set(re.findall(r"\b(so_[a-z_]+)\s*\(", text))
    assert {"so_layout_init", "so_grad_check", "so_adam_step_speculative",
            "so_validate_commit_or_rollback", "so_cast_params"} <= declared
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_layout_matches_the_oracle_arithmetic():
    for w in (W.tiny(), W.tiny_ragged(), W.gpt2_small(), W.llama_1b(), W.llama_8b()):
        ctx, info = B.so_layout_init(w.numel, w.bucket_elems)
        off, total = oracle.layout_offsets(w.numel)
        assert info.total_elems == total == w.total
        assert info.n_buckets == oracle.num_buckets(total, w.bucket_elems) == w.n_buckets
        assert info.n_tensors == len(w.numel)
        assert info.slot_stride_elems % 64 == 0
        assert 0 <= info.slot_stride_elems - w.bucket_elems < 64
        assert info.last_bucket_elems == total - (info.n_buckets - 1) * w.bucket_elems
        for i in sorted({0, min(1, len(w.numel) - 1), len(w.numel) // 2, len(w.numel) - 1}):
            o, fb, lb = B.so_layout_tensor(ctx, i)
            assert o == off[i]
            assert fb == off[i] // w.bucket_elems
            assert lb == (off[i] + w.numel[i] - 1) // w.bucket_elems
        # arena sizes: state has n_buckets + undo slots; grads/bf16 have n_buckets
        s = info.slot_stride_elems
        assert info.n_state_slots == 2 * info.n_buckets
        assert info.bytes_master == info.bytes_m == info.bytes_v == info.n_state_slots * s * 4
        assert info.bytes_grad == info.n_buckets * s * 2
        assert info.bytes_param_bf16 == info.n_buckets * s * 2
        assert info.bytes_scratch >= info.n_buckets * (info.tiles_per_slot * 8 + 16)
        B.so_destroy(ctx)
    # known bucket counts of the paper-shaped workloads
    assert W.gpt2_small().n_buckets == 5 and W.llama_1b().n_buckets == 13
    assert W.llama_8b().n_buckets == 41


def test_resident_bytes_without_undo_follow_the_16_bytes_per_parameter_accounting():
    ctx, info = B.so_layout_init([1 << 20], 262_144, B.SO_GRAD_BF16, 0)
    resident = (info.bytes_master + info.bytes_m + info.bytes_v + info.bytes_grad
                + info.bytes_param_bf16)
    assert resident == oracle.resident_bytes(1 << 20)      # 2 + 2 + 12 per parameter
    B.so_destroy(ctx)


def test_empty_tensor_and_tensor_straddling_buckets():
    ctx, info = B.so_layout_init([5, 0, 7, 1, 100], 10)
    assert info.n_buckets == 12 and info.last_bucket_elems == 3
    assert B.so_layout_tensor(ctx, 1) == (5, 0, -1)            # empty: first > last
    assert B.so_layout_tensor(ctx, 2) == (5, 0, 1)             # straddles buckets 0 and 1
    assert B.so_layout_tensor(ctx, 4) == (13, 1, 11)
    B.so_destroy(ctx)
    ctx, info = B.so_layout_init([], 10)
    assert info.n_buckets == 0 and info.total_elems == 0
    B.so_destroy(ctx)


def test_layout_init_rejects_bad_arguments():
    bad = B.SO_ERR_INVALID_ARG
    assert _status(B.so_layout_init, [4], 0) == bad
    assert _status(B.so_layout_init, [4], (1 << 30) + 1) == bad
    assert _status(B.so_layout_init, [-1], 4) == bad
    assert _status(B.so_layout_init, [4], 4, 7) == bad
    assert _status(B.so_layout_init, [40], 4, B.SO_GRAD_BF16, 11) == bad
    assert _status(B.so_layout_init, [40], 4, B.SO_GRAD_BF16, -2) == bad


def test_bind_rejects_misaligned_or_null_pointers():
    ctx, _ = B.so_layout_init([1024], 256)
    B.so_debug_set_dry_run(ctx, True)
    a = 0x10000000
    assert _status(B.so_layout_bind, ctx, a, a, a, a, a, a + 8) == B.SO_ERR_INVALID_ARG
    assert _status(B.so_layout_bind, ctx, a, a, 0, a, a, a) == B.SO_ERR_INVALID_ARG
    assert _status(B.so_adam_step_speculative, ctx, HP(), 0) == B.SO_ERR_STATE   # not bound
    B.so_destroy(ctx)


def test_commit_repoints_buckets_and_recycles_slots():
    ctx, info = _dry_ctx([1000], 256)                      # 4 buckets, 4 undo slots
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [0, 1, 2, 3]
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 0.01, 0)
    hp = HP()
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
    assert B.so_pending_buckets(ctx) == 0
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_COMMIT and r.step_after == 1
    assert r.buckets_speculated == 4
    assert r.stats.sumsq == pytest.approx(0.04) and r.stats.norm == pytest.approx(0.2)
    first = [B.so_bucket_slot(ctx, b) for b in range(4)]
    assert sorted(first) == [4, 5, 6, 7]
    # next iteration lands back in the recycled slots
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.step_after == 2
    assert sorted(B.so_bucket_slot(ctx, b) for b in range(4)) == [0, 1, 2, 3]
    c = B.so_get_counters(ctx)
    assert (c.commits, c.skips, c.clip_resteps) == (2, 0, 0)
    # per iteration: the batched step, the reduction (which decides on the device)
    # and two follow-up launches that read the verdict and return at once on a
    # commit (the re-cast a skip would need, the re-step a clip would need)
    assert c.kernel_launches == 8 and c.elems_stepped == 2000 and c.elems_checked == 0
    B.so_destroy(ctx)


def test_skip_keeps_the_slot_map_and_the_step_count():
    ctx, _ = _dry_ctx([1000], 256)
    hp = HP()
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 0.01, 1 if b == 2 else 0)
    B.so_adam_step_speculative(ctx, hp, 1)
    B.so_adam_step_speculative(ctx, hp, 3)
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_SKIP and r.step_after == 0 and r.stats.nonfinite == 1
    assert r.buckets_speculated == 2
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [0, 1, 2, 3]
    c = B.so_get_counters(ctx)
    assert c.skips == 1 and c.elems_cast == 256 + (1000 - 768)   # re-cast of buckets 1 and 3
    assert c.elems_checked == 512                                # buckets 0 and 2 were only scanned
    # all four slots are free again
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 0.0, 0)
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
    assert B.so_pending_buckets(ctx) == 0
    B.so_destroy(ctx)


def test_clip_resteps_every_bucket_and_commits():
    ctx, _ = _dry_ctx([1000], 256)
    hp = HP(max_grad_norm=1.0)
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 25.0, 0)             # norm 10
    B.so_adam_step_speculative(ctx, hp, 0)
    B.so_adam_step_speculative(ctx, hp, 2)
    st = B.so_grad_check(ctx, hp, B.SO_ALL)
    assert st.norm == 10.0 and st.clip_coef == 1.0 / (10.0 + 1e-6)
    assert st.clip_coef == oracle.clip_coef(10.0, 1.0)
    before = B.so_get_counters(ctx).elems_stepped
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_CLIP_RESTEP and r.step_after == 1
    assert B.so_get_counters(ctx).elems_stepped - before == 1000  # every element re-stepped
    slots = [B.so_bucket_slot(ctx, b) for b in range(4)]
    assert slots[1] == 1 and slots[3] == 3 and slots[0] >= 4 and slots[2] >= 4
    B.so_destroy(ctx)


def test_windowed_undo_and_exhaustion():
    ctx, info = _dry_ctx([1000], 256, undo=2)
    assert info.n_state_slots == 6
    hp = HP(max_grad_norm=0.0)
    B.so_adam_step_speculative(ctx, hp, 3)
    B.so_adam_step_speculative(ctx, hp, 0)
    assert _status(B.so_adam_step_speculative, ctx, hp, 1) == B.SO_ERR_UNDO_EXHAUSTED
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)               # nothing fits: still OK
    assert B.so_pending_buckets(ctx) == 2
    B.so_grad_check(ctx, None, 1)                               # scan one of the rest by hand
    r = B.so_validate_commit_or_rollback(ctx, hp)               # scans 2, steps 1 and 2 in place
    assert r.decision == B.SO_DECISION_COMMIT and r.buckets_speculated == 2
    c = B.so_get_counters(ctx)
    assert c.elems_checked == 512 and c.elems_stepped == 1000
    assert [B.so_bucket_slot(ctx, b) for b in (1, 2)] == [1, 2]
    B.so_destroy(ctx)


def test_no_undo_slots_is_the_plain_check_then_step_flow():
    ctx, info = _dry_ctx([1000], 256, undo=0)
    hp = HP()
    assert _status(B.so_adam_step_speculative, ctx, hp, 0) == B.SO_ERR_UNDO_EXHAUSTED
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_COMMIT and r.step_after == 1
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [0, 1, 2, 3]
    B.so_destroy(ctx)


def test_state_machine_errors_leave_the_context_usable():
    ctx, _ = _dry_ctx([1000], 256)
    hp = HP()
    B.so_adam_step_speculative(ctx, hp, 1)
    assert _status(B.so_adam_step_speculative, ctx, hp, 1) == B.SO_ERR_STATE      # twice
    assert _status(B.so_grad_check, ctx, None, 1) == B.SO_ERR_STATE               # already covered
    assert _status(B.so_cast_params, ctx) == B.SO_ERR_STATE                       # mid-iteration
    assert _status(B.so_set_step, ctx, 5) == B.SO_ERR_STATE
    assert _status(B.so_adam_step_speculative, ctx, HP(lr=2e-3), 2) == B.SO_ERR_INVALID_ARG
    assert _status(B.so_adam_step_speculative, ctx, hp, 9) == B.SO_ERR_INVALID_ARG
    assert _status(B.so_adam_step_speculative, ctx, HP(beta1=1.0), 2) == B.SO_ERR_INVALID_ARG
    assert _status(B.so_adam_step_speculative, ctx, HP(lr=math.nan), 2) == B.SO_ERR_INVALID_ARG
    B.so_grad_check(ctx, hp, B.SO_ALL)
    assert _status(B.so_adam_step_speculative, ctx, hp, 2) == B.SO_ERR_STATE      # after the check
    assert _status(B.so_grad_check, ctx, hp, B.SO_ALL) == B.SO_ERR_STATE
    assert _status(B.so_validate_commit_or_rollback, ctx, HP(lr=2e-3)) == B.SO_ERR_INVALID_ARG
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.step_after == 1
    B.so_cast_params(ctx)                                                         # idle again
    B.so_set_step(ctx, 41)
    assert B.so_get_step(ctx) == 41
    B.so_destroy(ctx)


def test_empty_model_is_a_valid_no_op():
    ctx, info = _dry_ctx([], 256)
    hp = HP()
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_COMMIT and r.stats.norm == 0.0 and r.step_after == 1
    assert B.so_get_counters(ctx).kernel_launches == 0
    B.so_destroy(ctx)


def test_batches_of_more_than_128_buckets_are_split_into_several_launches():
    ctx, info = _dry_ctx([300 * 64], 64)
    assert info.n_buckets == 300
    hp = HP(max_grad_norm=0.0)
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
    assert B.so_get_counters(ctx).kernel_launches == 3
    B.so_validate_commit_or_rollback(ctx, hp)
    # the reduction and 3 predicated re-cast launches; clipping is off and every
    # bucket was speculated, so no step can follow the verdict
    assert B.so_get_counters(ctx).kernel_launches == 3 + 1 + 3
    B.so_destroy(ctx)


def test_strerror_is_defined_for_every_status():
    for s in range(-6, 1):
        assert B.strerror(s) and B.strerror(s) != "unknown status"
    assert B.strerror(-99) == "unknown status"


def test_loss_scale_schedule_follows_the_oracle():
    ctx, _ = _dry_ctx([1000], 256, gd=B.SO_GRAD_FP16)
    hp = HP(max_grad_norm=0.0)
    B.so_loss_scale_config(ctx, 65536.0, 2.0, 0.5, 3)
    scale, good = 65536.0, 0
    for bad in [0, 0, 0, 0, 1, 0, 0, 1, 1, 0, 0, 0]:
        for b in range(4):
            B.so_debug_set_bucket_stats(ctx, b, 1e-4, 1 if (bad and b == 2) else 0)
        B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
        r = B.so_validate_commit_or_rollback(ctx, hp)
        scale, good = oracle.loss_scale_update(scale, good, bad, 2.0, 0.5, 3)
        assert r.loss_scale == scale == B.so_get_loss_scale(ctx)
        assert r.decision == (B.SO_DECISION_SKIP if bad else B.SO_DECISION_COMMIT)
    assert B.so_get_step(ctx) == 9
    B.so_destroy(ctx)


def test_loss_scale_is_only_for_fp16_contexts_and_validates_its_arguments():
    ctx, _ = _dry_ctx([1000], 256)
    assert _status(B.so_loss_scale_config, ctx, 1024.0) == B.SO_ERR_UNSUPPORTED
    B.so_destroy(ctx)
    ctx, info = _dry_ctx([1000], 256, gd=B.SO_GRAD_FP16)
    assert info.bytes_grad == 4 * 256 * 2
    bad = B.SO_ERR_INVALID_ARG
    assert _status(B.so_loss_scale_config, ctx, 0.0) == bad
    assert _status(B.so_loss_scale_config, ctx, 1024.0, 0.5, 0.5, 10) == bad     # growth < 1
    assert _status(B.so_loss_scale_config, ctx, 1024.0, 2.0, 1.5, 10) == bad     # backoff > 1
    assert _status(B.so_loss_scale_config, ctx, 1024.0, 2.0, 0.5, -1) == bad
    B.so_loss_scale_config(ctx, 1024.0)                                          # static scale
    B.so_adam_step_speculative(ctx, HP(), 0)
    assert _status(B.so_loss_scale_config, ctx, 2048.0) == B.SO_ERR_STATE        # mid-iteration
    B.so_destroy(ctx)


def test_deferred_validation_state_machine():
    ctx, _ = _dry_ctx([1000], 256)
    hp = HP(max_grad_norm=0.0)
    assert _status(B.so_validate_poll, ctx) == B.SO_ERR_STATE           # nothing in flight
    B.so_adam_step_speculative(ctx, hp, 0)
    B.so_validate_begin(ctx, hp)                                         # scans buckets 1..3
    assert B.so_get_counters(ctx).elems_checked == 1000 - 256
    assert B.so_validate_poll(ctx) is True
    assert _status(B.so_validate_begin, ctx, hp) == B.SO_ERR_STATE       # already begun
    assert _status(B.so_cast_params, ctx) == B.SO_ERR_STATE              # verdict not collected
    assert _status(B.so_set_step, ctx, 3) == B.SO_ERR_STATE
    st = B.so_grad_check(ctx, hp, B.SO_ALL)                              # its statistics: allowed
    assert st.nonfinite == 0
    assert B.so_validate_poll(ctx) is True
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_COMMIT and r.step_after == 1
    B.so_validate_begin(ctx, hp)                                         # check-first flow, deferred
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.step_after == 2 and r.buckets_speculated == 0
    B.so_destroy(ctx)


def test_next_iteration_may_be_assembled_while_a_verdict_is_pending():
    """The verdict is formed on the device; the host may run one iteration
    ahead of its own bookkeeping.  Collecting validates the older iteration
    and leaves the newer one open."""
    ctx, _ = _dry_ctx([1000], 256, undo=2)
    hp = HP(max_grad_norm=1.0)
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 0.01, 0)
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)            # buckets 0, 1 speculated
    B.so_validate_begin(ctx, hp)                              # 2, 3 scanned; verdict pending
    before = [B.so_bucket_slot(ctx, b) for b in range(4)]
    assert before == [0, 1, 2, 3]                             # host map not yet updated
    # iteration 2 is assembled on top of the pending verdict
    B.so_adam_step_speculative(ctx, hp, 3)
    B.so_grad_check(ctx, None, 0)
    assert B.so_pending_buckets(ctx) == 2
    assert _status(B.so_adam_step_speculative, ctx, hp, 3) == B.SO_ERR_STATE     # twice
    assert _status(B.so_grad_check, ctx, hp, B.SO_ALL) == B.SO_ERR_STATE         # a new iteration is open
    assert _status(B.so_validate_begin, ctx, hp) == B.SO_ERR_STATE               # collect first
    r = B.so_validate_commit_or_rollback(ctx, hp)             # collects iteration 1
    assert r.decision == B.SO_DECISION_COMMIT and r.step_after == 1 and r.buckets_speculated == 2
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [4, 5, 2, 3]
    assert B.so_pending_buckets(ctx) == 2                     # iteration 2 untouched
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 25.0, 0)          # norm 10: clip
    r = B.so_validate_commit_or_rollback(ctx, hp)             # now validates iteration 2
    assert r.decision == B.SO_DECISION_CLIP_RESTEP and r.step_after == 2 and r.buckets_speculated == 1
    # bucket 3 took spare index 0, which held slot 0 after the first commit
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [4, 5, 2, 0]
    c = B.so_get_counters(ctx)
    assert (c.commits, c.clip_resteps) == (1, 1)
    # iteration 1: 512 speculated + 488 in place; iteration 2: 232 speculated + 1000 re-stepped
    assert c.elems_stepped == 512 + 488 + 232 + 1000
    B.so_destroy(ctx)


def test_device_timeout_gives_the_iteration_up_and_leaves_the_context_usable():
    """A raised device status word (a kernel gave up a bounded wait) must end
    the iteration as if it had not happened: slots released, slot map, step
    count and loss scale unchanged, bf16 of the speculated buckets re-derived,
    and the same iteration can be run again."""
    ctx, _ = _dry_ctx([1000], 256, undo=3)
    hp = HP()
    for b in range(4):
        B.so_debug_set_bucket_stats(ctx, b, 0.01, 0)
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)            # buckets 0..2 speculated
    B.so_debug_set_bucket_stats(ctx, B.SO_ALL, 0.0, 1)       # status word of the next check
    assert _status(B.so_validate_commit_or_rollback, ctx, hp) == B.SO_ERR_TIMEOUT
    assert [B.so_bucket_slot(ctx, b) for b in range(4)] == [0, 1, 2, 3]
    assert B.so_get_step(ctx) == 0 and B.so_pending_buckets(ctx) == 4
    c = B.so_get_counters(ctx)
    assert c.timeouts == 1 and (c.commits, c.skips, c.clip_resteps) == (0, 0, 0)
    assert c.elems_cast == 768                               # bf16 of buckets 0..2 again
    # the status was consumed; the iteration runs again, all three slots free
    B.so_adam_step_speculative(ctx, hp, B.SO_ALL)
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_COMMIT and r.buckets_speculated == 3 and r.step_after == 1
    # also on the blocking check and on the deferred path
    B.so_debug_set_bucket_stats(ctx, B.SO_ALL, 0.0, 1)
    assert _status(B.so_grad_check, ctx, hp, B.SO_ALL) == B.SO_ERR_TIMEOUT
    B.so_adam_step_speculative(ctx, hp, 0)
    B.so_validate_begin(ctx, hp)
    B.so_debug_set_bucket_stats(ctx, B.SO_ALL, 0.0, 1)
    assert _status(B.so_validate_commit_or_rollback, ctx, hp) == B.SO_ERR_TIMEOUT
    assert B.so_get_step(ctx) == 1 and B.so_get_counters(ctx).timeouts == 3
    r = B.so_validate_commit_or_rollback(ctx, hp)
    assert r.decision == B.SO_DECISION_COMMIT and r.step_after == 2
    B.so_destroy(ctx)


def test_header_is_plain_c_and_a_c_program_can_drive_the_library(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 with no CUDA or
    C++ in sight, and a program written in C must be able to link against the
    shared library and run the host-side calls (dry run: no GPU needed)."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    src = tmp_path / "drive.c"
    src.write_text(r'''
#include <stdio.h>
#include <stdint.h>
#include "superoffload.h"
int main(void) {
    int64_t numel[3] = {1000, 0, 537};
    so_ctx *ctx = 0;
    so_layout_info info;
    if (so_layout_init(&ctx, 3, numel, 256, SO_GRAD_BF16, SO_ALL, &info) != SO_OK) return 1;
    if (info.n_buckets != 7 || info.total_elems != 1537) return 2;
    if (so_debug_set_dry_run(ctx, 1) != SO_OK) return 3;
    char *base = (char *)0x10000000;
    if (so_layout_bind(ctx, base, base + 0x1000000, base + 0x2000000, base + 0x3000000,
                       base + 0x4000000, base + 0x5000000) != SO_OK) return 4;
    so_hparams hp = {1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0};
    for (int b = 0; b < 7; ++b) so_debug_set_bucket_stats(ctx, b, 1.0, 0);
    if (so_adam_step_speculative(ctx, &hp, SO_ALL, 0) != SO_OK) return 5;
    so_step_result r;
    if (so_validate_commit_or_rollback(ctx, &hp, 0, &r) != SO_OK) return 6;
    printf("%d %d %lld %.6f\n", (int)r.decision, (int)r.buckets_speculated,
           (long long)r.step_after, r.stats.norm);
    so_destroy(ctx);
    return 0;
}
''')
    inc = os.path.join(ROOT, "include")
    exe = tmp_path / "drive"
    subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-pedantic", "-fsyntax-only",
                    "-I", inc, "-x", "c", os.path.join(inc, "superoffload.h")], check=True)
    libdir = os.path.dirname(so_build.LIB_PATH)
    subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-I", inc, str(src), "-o", str(exe),
                    "-L", libdir, "-lsuperoffload", f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert out == [str(B.SO_DECISION_CLIP_RESTEP), "7", "1", f"{7 ** 0.5:.6f}"]


def test_binding_structs_have_the_c_layout(tmp_path):
    """ctypes mirrors of the header's structs: same size, same field offsets."""
    import ctypes
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    structs = {"so_hparams": B.so_hparams, "so_layout_info": B.so_layout_info,
               "so_grad_stats": B.so_grad_stats, "so_step_result": B.so_step_result,
               "so_counters": B.so_counters}
    lines = []
    for name, cls in structs.items():
        lines.append(f'printf("{name} %zu\\n", sizeof({name}));')
        for field, _ in cls._fields_:
            lines.append(f'printf("{name}.{field} %zu\\n", offsetof({name}, {field}));')
    src = tmp_path / "layout.c"
    src.write_text("#include <stdio.h>\n#include <stddef.h>\n#include \"superoffload.h\"\n"
                   "int main(void) {\n" + "\n".join(lines) + "\nreturn 0; }\n")
    exe = tmp_path / "layout"
    subprocess.run([gcc, "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)],
                   check=True)
    got = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True,
                                                 text=True).stdout.splitlines())
    for name, cls in structs.items():
        assert int(got[name]) == ctypes.sizeof(cls), name
        for field, _ in cls._fields_:
            assert int(got[f"{name}.{field}"]) == getattr(cls, field).offset, (name, field)
