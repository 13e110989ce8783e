"""Randomised walk over the library's per-iteration state machine (dry-run mode,
no GPU) against a small model written from the header's description of the
calls: which calls are accepted when, and what a verdict does to the slot map, the
step count and the work counters."""
from __future__ import annotations

import random

import pytest

from paper_2509_21271_b200 import binding as B
from paper_2509_21271_b200 import build as so_build

C_, S_, R_ = B.SO_DECISION_COMMIT, B.SO_DECISION_SKIP, B.SO_DECISION_CLIP_RESTEP


@pytest.fixture(scope="module", autouse=True)
def _built():
    so_build.build_library()


class HP:
    lr, beta1, beta2, eps, weight_decay = 1e-3, 0.9, 0.999, 1e-8, 0.01

    def __init__(self, max_grad_norm):
        self.max_grad_norm = max_grad_norm


def _status(fn, *a):
    try:
        return B.SO_OK, fn(*a)
    except B.SuperOffloadError as e:
        return e.status, None


class Model:
    """What the header promises, in a few lines."""

    def __init__(self, total, bucket, undo):
        self.nb = -(-total // bucket) if total else 0
        self.elems = [min(bucket, total - b * bucket) for b in range(self.nb)]
        self.undo = self.nb if undo == B.SO_ALL else undo
        self.t = 0
        self.stepped = self.checked = self.cast = 0
        self.commits = self.skips = self.resteps = 0
        self.new_iteration()

    def new_iteration(self):
        self.cover = ["none"] * self.nb
        self.free = self.undo
        self.verdict_known = False

    def speculate(self, b):
        if self.verdict_known or self.cover[b] != "none":
            return B.SO_ERR_STATE
        if self.free == 0:
            return B.SO_ERR_UNDO_EXHAUSTED
        self.free -= 1
        self.cover[b] = "spec"
        self.stepped += self.elems[b]
        return B.SO_OK

    def speculate_all(self):
        if self.verdict_known:
            return B.SO_ERR_STATE
        for b in range(self.nb):
            if self.cover[b] == "none" and self.free > 0:
                self.speculate(b)
        return B.SO_OK

    def scan(self, b):
        if self.verdict_known or self.cover[b] != "none":
            return B.SO_ERR_STATE
        self.cover[b] = "scan"
        self.checked += self.elems[b]
        return B.SO_OK

    def scan_rest(self):
        if self.verdict_known:
            return B.SO_ERR_STATE
        for b in range(self.nb):
            if self.cover[b] == "none":
                self.scan(b)
        self.verdict_known = True
        return B.SO_OK

    def validate(self, nonfinite, coef):
        if not self.verdict_known:
            self.scan_rest()
        spec = [b for b in range(self.nb) if self.cover[b] == "spec"]
        moved = []
        if nonfinite:
            decision = S_
            self.cast += sum(self.elems[b] for b in spec)
            self.skips += 1
        else:
            decision = R_ if coef < 1.0 else C_
            for b in range(self.nb):
                if decision == R_ or self.cover[b] != "spec":
                    self.stepped += self.elems[b]
            moved = spec
            self.t += 1
            if decision == R_:
                self.resteps += 1
            else:
                self.commits += 1
        n_spec = len(spec)
        self.new_iteration()
        return decision, n_spec, moved


@pytest.mark.parametrize("seed", range(12))
def test_random_walk_matches_the_model(seed):
    rng = random.Random(seed)
    bucket = rng.choice([64, 100, 256])
    nb = rng.choice([1, 2, 3, 7, 20, 150])
    total = (nb - 1) * bucket + rng.randint(1, bucket)
    undo = rng.choice([B.SO_ALL, 0, 1, max(1, nb // 2), nb])
    ctx, info = B.so_layout_init([total], bucket, B.SO_GRAD_BF16, undo)
    B.so_debug_set_dry_run(ctx, True)
    a = 0x10000000
    B.so_layout_bind(ctx, a, 2 * a, 3 * a, 4 * a, 5 * a, 6 * a)
    m = Model(total, bucket, undo)
    assert info.n_buckets == m.nb and info.n_state_slots == m.nb + m.undo
    slots = [B.so_bucket_slot(ctx, b) for b in range(m.nb)]
    assert slots == list(range(m.nb))

    for it in range(40):
        max_norm = rng.choice([0.0, 1.0])
        hp = HP(max_norm)
        # this iteration's gradients, as the per-bucket records a scan would return
        nonfinite_bucket = rng.randrange(m.nb) if rng.random() < 0.2 else -1
        big = rng.random() < 0.4
        sumsq = []
        for b in range(m.nb):
            s = rng.random() * (10.0 if big else 0.5 / m.nb)
            sumsq.append(s)
            B.so_debug_set_bucket_stats(ctx, b, s, 1 if b == nonfinite_bucket else 0)
        norm = sum(sumsq) ** 0.5
        coef = min(1.0, max_norm / (norm + 1e-6)) if max_norm > 0 else 1.0

        for _ in range(rng.randint(0, 2 * m.nb + 2)):
            op = rng.random()
            if op < 0.45:
                b = rng.randrange(m.nb)
                assert _status(B.so_adam_step_speculative, ctx, hp, b)[0] == m.speculate(b)
            elif op < 0.7:
                b = rng.randrange(m.nb)
                assert _status(B.so_grad_check, ctx, None, b)[0] == m.scan(b)
            elif op < 0.85:
                assert _status(B.so_adam_step_speculative, ctx, hp, B.SO_ALL)[0] == m.speculate_all()
            elif op < 0.92:
                st, stats = _status(B.so_grad_check, ctx, hp, B.SO_ALL)
                assert st == m.scan_rest()
                if st == B.SO_OK:
                    assert stats.nonfinite == (1 if nonfinite_bucket >= 0 else 0)
                    assert stats.sumsq == pytest.approx(sum(sumsq), rel=1e-12)
            else:
                # calls that are only legal between iterations
                idle = all(c == "none" for c in m.cover) and not m.verdict_known
                assert _status(B.so_cast_params, ctx)[0] == (B.SO_OK if idle else B.SO_ERR_STATE)
                if idle:
                    m.cast += total
            pending = sum(1 for c in m.cover if c == "none")
            assert B.so_pending_buckets(ctx) == pending

        before = [B.so_bucket_slot(ctx, b) for b in range(m.nb)]
        r = B.so_validate_commit_or_rollback(ctx, hp)
        decision, n_spec, moved = m.validate(nonfinite_bucket >= 0, coef)
        assert (r.decision, r.buckets_speculated, r.step_after) == (decision, n_spec, m.t)
        assert r.stats.clip_coef == pytest.approx(coef, rel=1e-12)
        after = [B.so_bucket_slot(ctx, b) for b in range(m.nb)]
        assert len(set(after)) == m.nb and all(0 <= s < m.nb + m.undo for s in after)
        for b in range(m.nb):
            if b in moved:
                assert after[b] != before[b] and after[b] not in before
            else:
                assert after[b] == before[b]
        c = B.so_get_counters(ctx)
        assert (c.commits, c.skips, c.clip_resteps) == (m.commits, m.skips, m.resteps)
        assert (c.elems_stepped, c.elems_checked, c.elems_cast) == (m.stepped, m.checked, m.cast)
        assert B.so_get_step(ctx) == m.t and B.so_pending_buckets(ctx) == m.nb
    B.so_destroy(ctx)
