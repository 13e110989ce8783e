"""Pins for the CPU oracle: every check here is against something other than
the oracle itself -- exact rational arithmetic, closed forms of Adam, brute
force, hand-worked bit tables, or an independent library routine."""
from __future__ import annotations

import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import HParams
from helpers import (bf16_bits_to_f32, f32_from_fraction, is_bf16_nan, ulp_distance)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bf16_bits(rng, n, sigma):
    g = torch.from_numpy(rng.normal(0.0, sigma, n).astype(np.float32)).to(torch.bfloat16)
    return g.view(torch.int16).numpy().view(np.uint16).copy()


def _fr(x) -> Fraction:
    return Fraction(float(x))


# ---------------------------------------------------------------------------
# Adam: closed forms (Kingma & Ba Alg. 1 with m0 = v0 = 0; decoupled decay)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("scale", [1.0, 0.09765625, 0.3141592653589793])
@pytest.mark.parametrize("grad_kind", ["bf16", "fp32"])
def test_first_step_matches_exact_rational_closed_form(scale, grad_kind):
    """t=1, m=v=0: m1=(1-b1)g~, v1=(1-b2)g~^2, p1=p0(1-lr*wd)-lr*g~/(|g~|+eps),
    evaluated in exact rationals and rounded once to fp32."""
    rng = np.random.default_rng(1)
    n = 600
    hp = HParams(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    if grad_kind == "bf16":
        g = _rand_bf16_bits(rng, n, 1e-2)
        gval = bf16_bits_to_f32(g)
    else:
        g = rng.normal(0, 1e-2, n).astype(np.float32)
        gval = g
    # a few awkward gradients: zero, tiny, huge, comparable to eps
    special = np.array([0.0, 1e-30, 3e4, 1e-8, -1e-8, 2.5e-9], dtype=np.float32)
    if grad_kind == "bf16":
        sb = torch.from_numpy(special).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        g[:special.size] = sb
        gval = bf16_bits_to_f32(g)
    else:
        g[:special.size] = special
        gval = g
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    oracle.adamw_step_range(p, m, v, g, 0, n, scale, 1, hp)

    lr, b1, b2, eps, wd = map(_fr, (hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay))
    exp_p, exp_m, exp_v = (np.empty(n, np.float32) for _ in range(3))
    for i in range(n):
        gs = _fr(gval[i]) * _fr(scale)
        exp_m[i] = f32_from_fraction((1 - b1) * gs)
        exp_v[i] = f32_from_fraction((1 - b2) * gs * gs)
        exp_p[i] = f32_from_fraction(_fr(p0[i]) * (1 - lr * wd) - lr * gs / (abs(gs) + eps))
    for name, got, exp in (("p", p, exp_p), ("m", m, exp_m), ("v", v, exp_v)):
        d = ulp_distance(got, exp)
        assert d.max() <= 1, (name, int(d.max()))
        assert (d == 0).mean() > 0.98, name     # double rounding may move a rare tie


def _sqrt_fraction(x: Fraction, bits: int = 200) -> Fraction:
    """sqrt of a non-negative rational to `bits` fractional bits (integer square root)."""
    from math import isqrt
    scaled = (x.numerator << (2 * bits)) // x.denominator
    return Fraction(isqrt(scaled), 1 << bits)


@pytest.mark.parametrize("tt", [2, 7, 1000])
@pytest.mark.parametrize("scale", [1.0, 0.3141592653589793])
def test_later_step_with_moments_matches_high_precision_arithmetic(tt, scale):
    """A step from non-zero moments (bias corrections 1 - beta^t with t > 1),
    evaluated in rationals with a 200-bit square root and rounded once to fp32:
    m' = b1 m + (1-b1) g~,  v' = b2 v + (1-b2) g~^2,
    p' = p (1 - lr wd) - lr (m'/(1-b1^t)) / (sqrt(v'/(1-b2^t)) + eps)."""
    rng = np.random.default_rng(100 + tt)
    n = 400
    hp = HParams(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    m0 = rng.normal(0, 3e-3, n).astype(np.float32)
    v0 = (rng.random(n) * 1e-4).astype(np.float32)
    v0[:5] = 0.0                                   # a cold second moment among warm ones
    g = _rand_bf16_bits(rng, n, 1e-2)
    gval = bf16_bits_to_f32(g)
    p, m, v = p0.copy(), m0.copy(), v0.copy()
    oracle.adamw_step_range(p, m, v, g, 0, n, scale, tt, hp)

    lr, b1, b2, eps, wd = map(_fr, (hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay))
    bc1, bc2 = 1 - b1 ** tt, 1 - b2 ** tt
    exp_p, exp_m, exp_v = (np.empty(n, np.float32) for _ in range(3))
    for i in range(n):
        gs = _fr(gval[i]) * _fr(scale)
        m1 = b1 * _fr(m0[i]) + (1 - b1) * gs
        v1 = b2 * _fr(v0[i]) + (1 - b2) * gs * gs
        u = lr * (m1 / bc1) / (_sqrt_fraction(v1 / bc2) + eps)
        exp_m[i] = f32_from_fraction(m1)
        exp_v[i] = f32_from_fraction(v1)
        exp_p[i] = f32_from_fraction(_fr(p0[i]) * (1 - lr * wd) - u)
    for name, got, exp in (("p", p, exp_p), ("m", m, exp_m), ("v", v, exp_v)):
        d = ulp_distance(got, exp)
        assert d.max() <= 1, (name, int(d.max()))
        # With beta = 0.9 the exact b1*m + (1-b1)*g sits within 1e-16 of an fp32
        # tie for a few percent of these inputs; the fp64 evaluation then rounds
        # either way.  Anything but a last-place difference is a wrong formula.
        assert (d == 0).mean() > 0.9, name


def test_constant_gradient_many_steps_tracks_t():
    """Constant g, wd=0: in exact arithmetic mhat_t=g and vhat_t=g^2 for all t,
    so p_t = p0 - t*lr*g/(|g|+eps).  Catches an off-by-one in the bias
    correction or the step counter."""
    hp = HParams(lr=1e-3, weight_decay=0.0, max_grad_norm=0.0)
    n, steps = 64, 40
    rng = np.random.default_rng(2)
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = _rand_bf16_bits(rng, n, 1e-2)
    gval = bf16_bits_to_f32(g).astype(np.float64)
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    pb = oracle.bf16_rne(p)
    t = 0
    for k in range(1, steps + 1):
        r = oracle.iteration_ste(p, m, v, pb, g, 16, t, hp)
        t = r.step_after
        assert t == k and r.decision == oracle.DECISION_COMMIT
        expect = p0.astype(np.float64) - k * hp.lr * gval / (np.abs(gval) + hp.eps)
        # fp32 storage rounds p, m, v once per step: allow ~1 ulp(p) per step
        reach = (np.abs(p0) + np.float32(k * hp.lr)).astype(np.float32)
        tol = (k + 2) * np.spacing(reach).astype(np.float64) + k * 2e-7 * hp.lr
        assert np.all(np.abs(p.astype(np.float64) - expect) <= tol), k
        # bias-corrected moments equal g and g^2 up to fp32 storage rounding
        bc1, bc2 = 1 - hp.beta1 ** k, 1 - hp.beta2 ** k
        np.testing.assert_allclose(m / bc1, gval, rtol=1e-6 / bc1 * 1.0 + 1e-6)
        np.testing.assert_allclose(v / bc2, gval ** 2, rtol=5e-6)


def test_skip_does_not_advance_t_or_touch_state():
    """An iteration with a non-finite gradient leaves p, m, v, bf16 copy and t
    exactly as they were (rollback scenario 1, Section 4.4)."""
    hp = HParams()
    rng = np.random.default_rng(3)
    n = 1000
    p = rng.normal(0, 0.02, n).astype(np.float32)
    m = rng.normal(0, 1e-3, n).astype(np.float32)
    v = (rng.normal(0, 1e-3, n) ** 2).astype(np.float32)
    pb = oracle.bf16_rne(p)
    for bad in (0x7F80, 0xFF80, 0x7FC0, 0x7F81):
        for fn in (oracle.iteration_ste, oracle.iteration_stv):
            g = _rand_bf16_bits(rng, n, 1e-2)
            g[777] = bad
            q, mm, vv, qb = p.copy(), m.copy(), v.copy(), pb.copy()
            r = fn(q, mm, vv, qb, g, 256, 5, hp)
            assert r.decision == oracle.DECISION_SKIP and r.nonfinite == 1
            assert r.step_after == 5
            for a, b in ((q, p), (mm, m), (vv, v)):
                assert a.tobytes() == b.tobytes()
            assert qb.tobytes() == pb.tobytes()


def test_constant_gradient_with_a_skipped_iteration():
    """After a SKIP the next kept step must reuse the same step index."""
    hp = HParams(lr=1e-3, weight_decay=0.0, max_grad_norm=0.0)
    n = 32
    rng = np.random.default_rng(4)
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = _rand_bf16_bits(rng, n, 1e-2)
    gval = bf16_bits_to_f32(g).astype(np.float64)
    bad = g.copy(); bad[3] = 0x7F80
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    pb = oracle.bf16_rne(p)
    t = 0
    for it in range(1, 7):
        r = oracle.iteration_stv(p, m, v, pb, bad if it == 3 else g, 8, t, hp)
        t = r.step_after
    assert t == 5
    expect = p0.astype(np.float64) - 5 * hp.lr * gval / (np.abs(gval) + hp.eps)
    assert np.all(np.abs(p - expect) <= 8 * np.spacing(np.abs(p0) + np.float32(0.005)) + 1e-9)


def test_decay_only_and_zero_lr():
    """g=0, m=v=0: p' = fl32(p*(1-lr*wd)) exactly, m and v stay 0; lr=0 leaves
    p bit-identical."""
    rng = np.random.default_rng(5)
    n = 500
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = np.zeros(n, np.uint16)
    hp = HParams(lr=3e-3, weight_decay=0.1)
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    oracle.adamw_step_range(p, m, v, g, 0, n, 1.0, 1, hp)
    factor = 1 - _fr(hp.lr) * _fr(hp.weight_decay)
    exp = np.array([f32_from_fraction(_fr(x) * factor) for x in p0], np.float32)
    assert ulp_distance(p, exp).max() <= 1 and (p == exp).mean() > 0.98
    assert not m.any() and not v.any()

    hp0 = HParams(lr=0.0, weight_decay=0.1)
    p = p0.copy()
    gg = _rand_bf16_bits(rng, n, 1e-2)
    oracle.adamw_step_range(p, m, v, gg, 0, n, 1.0, 1, hp0)
    assert p.tobytes() == p0.tobytes()


def test_clip_on_first_step_scales_moments_not_the_update():
    """Adam's first step is sign-like: with coef << 1 the parameter moves
    almost as far as without clipping, while m scales by coef and v by
    coef^2.  Separates 'scaled gradient' from 'scaled update' mistakes."""
    hp = HParams(weight_decay=0.0)
    n = 256
    rng = np.random.default_rng(6)
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = _rand_bf16_bits(rng, n, 1.0)
    coef = 1.0 / 64
    pa, ma, va = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    pc, mc, vc = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    oracle.adamw_step_range(pa, ma, va, g, 0, n, 1.0, 1, hp)
    oracle.adamw_step_range(pc, mc, vc, g, 0, n, coef, 1, hp)
    assert np.array_equal(mc, ma * np.float32(coef))          # power of two: exact
    assert np.array_equal(vc, va * np.float32(coef * coef))
    big = np.abs(bf16_bits_to_f32(g)) > 1e-3
    np.testing.assert_allclose((pc - p0)[big], (pa - p0)[big], rtol=1e-3)


def test_step_against_torch_adamw_in_float64():
    """Library cross-check: torch.optim.AdamW on fp64 CPU tensors, one step at
    a time from the oracle's own fp32 state (so storage rounding is shared)."""
    rng = np.random.default_rng(7)
    n = 4096
    hp = HParams(lr=2e-3, beta1=0.85, beta2=0.97, eps=1e-7, weight_decay=0.05)
    p = rng.normal(0, 0.02, n).astype(np.float32)
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for tt in range(1, 6):
        g = _rand_bf16_bits(rng, n, 1e-2)
        gval = bf16_bits_to_f32(g)
        param = torch.nn.Parameter(torch.from_numpy(p.astype(np.float64)))
        opt = torch.optim.AdamW([param], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps,
                                weight_decay=hp.weight_decay, foreach=False)
        opt.state[param] = {"step": torch.tensor(float(tt - 1)),
                            "exp_avg": torch.from_numpy(m.astype(np.float64)),
                            "exp_avg_sq": torch.from_numpy(v.astype(np.float64))}
        param.grad = torch.from_numpy(gval.astype(np.float64))
        opt.step()
        oracle.adamw_step_range(p, m, v, g, 0, n, 1.0, tt, hp)
        st = opt.state[param]
        for got, ref in ((p, param.detach()), (m, st["exp_avg"]), (v, st["exp_avg_sq"])):
            d = ulp_distance(got, ref.numpy().astype(np.float32))
            assert d.max() <= 1
            # torch forms m as m + (1-b1)*(g-m); with decimal betas the exact
            # value (17m+3g)/20 often sits on an fp32 tie, which the two
            # evaluation orders break differently: a fraction of a percent of
            # the m entries legitimately differ by one ulp.
            assert (d == 0).mean() > 0.99


# ---------------------------------------------------------------------------
# gradient norm, coefficient, flags, decisions
# ---------------------------------------------------------------------------

def test_norm_textbook_values():
    three_four = np.array([3.0, 4.0], np.float32)
    s, nrm, flag = oracle.global_grad_check(three_four, 1)
    assert (s, nrm, flag) == (25.0, 5.0, 0)
    ones = np.full(1 << 20, 0x3F80, np.uint16)             # bf16 1.0
    s, nrm, flag = oracle.global_grad_check(ones, 262_144)
    assert (s, nrm, flag) == (float(1 << 20), 1024.0, 0)


@pytest.mark.parametrize("kind", ["bf16", "fp32"])
def test_norm_against_exact_brute_force(kind):
    """Sum of squares vs the exactly rounded sum (math.fsum of exact squares)."""
    rng = np.random.default_rng(8)
    n = 5000
    if kind == "bf16":
        g = _rand_bf16_bits(rng, n, 1e-2)
        vals = bf16_bits_to_f32(g).astype(np.float64)
    else:
        g = (rng.normal(0, 1, n) * 10.0 ** rng.uniform(-12, 12, n)).astype(np.float32)
        vals = g.astype(np.float64)
    exact = Fraction(0)
    for x in vals:
        exact += Fraction(float(x)) ** 2
    for bucket in (n, 1024, 7):
        s, nrm, flag = oracle.global_grad_check(g, bucket)
        assert flag == 0
        assert abs(Fraction(s) - exact) <= exact * Fraction(n, 2 ** 52)
        assert nrm == pytest.approx(math.sqrt(float(exact)), rel=1e-13)


def test_norm_of_iid_normal_is_sigma_sqrt_n():
    rng = np.random.default_rng(9)
    g = _rand_bf16_bits(rng, 1 << 20, 1e-2)
    _, nrm, _ = oracle.global_grad_check(g, 262_144)
    assert nrm == pytest.approx(1e-2 * math.sqrt(1 << 20), rel=5e-3)     # ~ 10.24


def test_square_does_not_overflow_for_finite_gradients():
    """|g| >= 2^64 squares past fp32 range; a finite gradient must stay finite."""
    g = np.array([0x7F7F, 0x7F7F, 0x0001], np.uint16)       # max bf16 twice, min denormal
    s, nrm, flag = oracle.global_grad_check(g, 2)
    assert flag == 0 and math.isfinite(s) and s > 1e76
    gf = np.array([3.4e38, 1e-45], np.float32)
    s, nrm, flag = oracle.global_grad_check(gf, 2)
    assert flag == 0 and math.isfinite(nrm)


def test_nonfinite_flag_over_every_bf16_pattern():
    """Exhaustive: the flag of a one-element range is 'not finite', for all
    65 536 bf16 patterns, judged by numpy on the widened value."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = ~np.isfinite(bf16_bits_to_f32(bits))
    assert want.sum() == 2 * 128                            # exponent all-ones
    for b in range(65536):
        _, flag = oracle.grad_check_range(bits, b, b + 1)
        assert bool(flag) == bool(want[b]), hex(b)


def test_nonfinite_fp32_gradients():
    for bad in (np.inf, -np.inf, np.nan):
        g = np.array([1.0, bad, 2.0], np.float32)
        assert oracle.global_grad_check(g, 2)[2] == 1
    assert oracle.global_grad_check(np.array([1.0, 2.0], np.float32), 2)[2] == 0


def test_clip_coefficient_properties():
    assert oracle.clip_coef(10.0, 0.0) == 1.0 and oracle.clip_coef(10.0, -1.0) == 1.0
    assert oracle.clip_coef(0.5, 1.0) == 1.0
    assert oracle.clip_coef(1.0 - 1e-6, 1.0) == 1.0         # norm + 1e-6 <= max_norm
    assert oracle.clip_coef(1.0, 1.0) < 1.0                 # the 1e-6 makes this clip
    c = oracle.clip_coef(10.24, 1.0)
    assert c == 1.0 / (10.24 + 1e-6)
    # scaled norm = max_norm * norm / (norm + 1e-6)
    assert c * 10.24 == pytest.approx(1.0 * 10.24 / (10.24 + 1e-6), rel=1e-15)


def test_clip_against_torch_clip_grad_norm():
    """Library cross-check of norm and coefficient."""
    rng = np.random.default_rng(10)
    g = _rand_bf16_bits(rng, 10000, 1e-1)
    gv = torch.from_numpy(bf16_bits_to_f32(g).astype(np.float64))
    prm = torch.nn.Parameter(torch.zeros_like(gv))
    prm.grad = gv.clone()
    total = torch.nn.utils.clip_grad_norm_([prm], max_norm=1.0, foreach=False)
    _, nrm, _ = oracle.global_grad_check(g, 4096)
    assert nrm == pytest.approx(float(total), rel=1e-13)
    coef = oracle.clip_coef(nrm, 1.0)
    np.testing.assert_allclose(prm.grad.numpy(), gv.numpy() * coef, rtol=1e-13)


def test_decision_table():
    C, S, R = oracle.DECISION_COMMIT, oracle.DECISION_SKIP, oracle.DECISION_CLIP_RESTEP
    assert oracle.decision(0, 1.0) == C
    assert oracle.decision(0, 0.999) == R
    assert oracle.decision(1, 1.0) == S
    assert oracle.decision(1, 0.1) == S                     # non-finite wins over clip
    # through the whole iteration, clip on / off x finite / inf / nan
    rng = np.random.default_rng(11)
    n = 512
    for max_norm, fault, want in ((1.0, None, R), (0.0, None, C), (100.0, None, C),
                                  (1.0, 0x7F80, S), (0.0, 0x7FC0, S), (100.0, 0xFF80, S)):
        g = _rand_bf16_bits(rng, n, 1.0)
        if fault is not None:
            g[100] = fault
        p = rng.normal(0, 0.02, n).astype(np.float32)
        m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
        pb = oracle.bf16_rne(p)
        r = oracle.iteration_ste(p, m, v, pb, g, 128, 0, HParams(max_grad_norm=max_norm))
        assert r.decision == want
        assert r.step_after == (0 if want == S else 1)


# ---------------------------------------------------------------------------
# speculation-then-validation is exact (Section 4.4)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("max_norm", [0.0, 1.0])
@pytest.mark.parametrize("grad_kind", ["bf16", "fp32"])
def test_stv_equals_ste_bitwise(max_norm, grad_kind):
    rng = np.random.default_rng(12)
    n, bucket = 10_007, 1024
    hp = HParams(max_grad_norm=max_norm)
    p = rng.normal(0, 0.02, n).astype(np.float32)
    state_a = [p.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32), oracle.bf16_rne(p)]
    state_b = [a.copy() for a in state_a]
    ta = tb = 0
    for it in range(1, 9):
        if grad_kind == "bf16":
            g = _rand_bf16_bits(rng, n, 1e-2 if it % 2 else 1e-4)
            if it == 5:
                g[n - 1] = 0x7F80
        else:
            g = rng.normal(0, 1e-2 if it % 2 else 1e-4, n).astype(np.float32)
            if it == 5:
                g[n - 1] = np.nan
        ra = oracle.iteration_ste(*state_a, g, bucket, ta, hp)
        rb = oracle.iteration_stv(*state_b, g, bucket, tb, hp)
        ta, tb = ra.step_after, rb.step_after
        assert (ra.decision, ra.norm, ra.clip_coef, ta) == (rb.decision, rb.norm, rb.clip_coef, tb) \
            or (it == 5 and ra.decision == rb.decision == oracle.DECISION_SKIP)
        for a, b in zip(state_a, state_b):
            assert a.tobytes() == b.tobytes()
        assert state_a[3].tobytes() == oracle.bf16_rne(state_a[0]).tobytes()
    assert ta == 7


def test_elementwise_result_does_not_depend_on_bucket_size():
    rng = np.random.default_rng(13)
    n = 5000
    hp = HParams(max_grad_norm=0.0)
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = _rand_bf16_bits(rng, n, 1e-2)
    outs = []
    for bucket in (n, 1000, 64, 7):
        st = [p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32), oracle.bf16_rne(p0)]
        oracle.iteration_stv(*st, g, bucket, 0, hp)
        outs.append(b"".join(a.tobytes() for a in st))
    assert all(o == outs[0] for o in outs)


# ---------------------------------------------------------------------------
# the bf16 cast (Section 4.5)
# ---------------------------------------------------------------------------

def _golden_cast_rows():
    rows = []
    with open(os.path.join(GOLDEN, "bf16_rne_table.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if len(line) == 2:
                rows.append((int(line[0], 16), line[1]))
    return rows


def test_bf16_rne_golden_table():
    rows = _golden_cast_rows()
    assert len(rows) >= 25
    src = np.array([r[0] for r in rows], np.uint32).view(np.float32)
    got = oracle.bf16_rne(src)
    for (pattern, want), out in zip(rows, got):
        if want == "nan":
            assert is_bf16_nan(np.array([out]))[0], hex(pattern)
        else:
            assert out == int(want, 16), (hex(pattern), hex(out))


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if len(line) == 2:
                rows.append((int(line[0], 16), line[1]))
    return rows


def _is_fp16_nan(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.uint32)
    return ((b & 0x7C00) == 0x7C00) & ((b & 0x03FF) != 0)


def test_fp16_rne_golden_table():
    rows = _golden_rows("fp16_rne_table.txt")
    assert len(rows) >= 35
    src = np.array([r[0] for r in rows], np.uint32).view(np.float32)
    got = oracle.fp16_rne(src)
    for (pattern, want), out in zip(rows, got):
        if want == "nan":
            assert _is_fp16_nan(np.array([out]))[0], hex(pattern)
        else:
            assert out == int(want, 16), (hex(pattern), hex(out))


def test_fp16_rne_against_numpy_conversion():
    """Library cross-check: numpy's float32 -> float16 conversion (IEEE round
    to nearest even) on every upper half x lower halves that decide a rounding
    at each possible cut (the cut moves down the word in the subnormal range),
    plus eight million random patterns."""
    rng = np.random.default_rng(15)
    hi = np.arange(65536, dtype=np.uint32) << 16
    lows = np.array([0, 1, 0x0FFF, 0x1000, 0x1001, 0x1FFF, 0x2000, 0x2FFF, 0x3000, 0x3001,
                     0x7FFF, 0x8000, 0x8001, 0xEFFF, 0xF000, 0xFFFF], np.uint32)
    pats = np.concatenate([(hi[:, None] | lows[None, :]).reshape(-1),
                           rng.integers(0, 1 << 32, 1 << 23, dtype=np.uint64).astype(np.uint32),
                           # dense around the subnormal range and the overflow threshold
                           rng.integers(0x32000000, 0x39000000, 1 << 21, dtype=np.uint64).astype(np.uint32),
                           rng.integers(0x477F0000, 0x47810000, 1 << 18, dtype=np.uint64).astype(np.uint32)])
    x = pats.view(np.float32)
    got = oracle.fp16_rne(x)
    with np.errstate(over="ignore", invalid="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    nan = np.isnan(x)
    assert _is_fp16_nan(got[nan]).all()
    assert np.array_equal(got[~nan], ref[~nan])
    # the sign of a NaN is kept
    assert np.array_equal(got[nan] >> 15, (pats[nan] >> 31).astype(np.uint16))


def test_fp16_rne_round_trip_and_monotonicity():
    """Every binary16 value widened to fp32 casts back to itself, and the cast
    never decreases when its argument increases (both fix the rounding
    direction of every interval without reference to another implementation)."""
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    finite_or_inf = ~_is_fp16_nan(h)
    wide = oracle.fp16_to_f32(h)
    back = oracle.fp16_rne(wide)
    assert np.array_equal(back[finite_or_inf], h[finite_or_inf])
    pats = np.sort(np.random.default_rng(16).integers(0, 0x7F800000, 1 << 20, dtype=np.uint64)
                   .astype(np.uint32))
    out = oracle.fp16_rne(pats.view(np.float32)).astype(np.int64)
    assert (np.diff(out) >= 0).all()
    # halfway points between neighbours go to the neighbour with the even pattern
    lo = np.arange(0, 0x7BFF, dtype=np.uint32).astype(np.uint16)
    a = oracle.fp16_to_f32(lo).astype(np.float64)
    b = oracle.fp16_to_f32((lo + 1).astype(np.uint16)).astype(np.float64)
    mid = ((a + b) / 2).astype(np.float32)          # exact: 12 significant bits
    assert np.array_equal(mid.astype(np.float64), (a + b) / 2)
    want = np.where(lo % 2 == 0, lo, lo + 1).astype(np.uint16)
    assert np.array_equal(oracle.fp16_rne(mid), want)


def test_bf16_rne_against_torch_conversion():
    """Library cross-check on every upper half x the decisive lower halves,
    plus four million random patterns."""
    rng = np.random.default_rng(14)
    hi = np.arange(65536, dtype=np.uint32) << 16
    lows = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF], np.uint32)
    pats = np.concatenate([(hi[:, None] | lows[None, :]).reshape(-1),
                           rng.integers(0, 1 << 32, 1 << 22, dtype=np.uint64).astype(np.uint32)])
    x = pats.view(np.float32)
    got = oracle.bf16_rne(x)
    ref = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(x)
    assert np.array_equal(is_bf16_nan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])


def test_bf16_widening_is_the_shift_for_all_patterns():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle.bf16_to_f32(bits)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).float().numpy()
    assert got.view(np.uint32).tobytes() == ref.view(np.uint32).tobytes()
    # and widening then rounding is the identity on non-NaN patterns
    back = oracle.bf16_rne(got)
    nan = is_bf16_nan(bits)
    assert np.array_equal(back[~nan], bits[~nan])


# ---------------------------------------------------------------------------
# layout and the paper's memory accounting
# ---------------------------------------------------------------------------

def test_layout_offsets_and_bucket_count():
    numel = [5, 0, 7, 1, 100]
    off, total = oracle.layout_offsets(numel)
    assert list(off) == [0, 5, 5, 12, 13] and total == 113
    assert oracle.num_buckets(113, 10) == 12 and oracle.num_buckets(110, 10) == 11
    assert oracle.num_buckets(0, 10) == 0 and oracle.num_buckets(1, 10) == 1
    assert oracle.num_buckets(8_030_261_248, 200_000_000) == 41


def test_resident_bytes_follow_the_papers_accounting():
    parts = {}
    with open(os.path.join(GOLDEN, "memory_accounting.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if len(line) == 2:
                parts[line[0]] = int(line[1])
    assert sum(v for k, v in parts.items() if k != "total") == parts["total"] == 16
    assert oracle.resident_bytes(1_000_000) == parts["total"] * 1_000_000


# ---------------------------------------------------------------------------
# fp16 gradients and loss scaling (the paper's own precision path)
# ---------------------------------------------------------------------------

def test_fp16_widening_for_all_patterns_against_numpy():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle.fp16_to_f32(bits)
    ref = bits.view(np.float16).astype(np.float32)
    nan = np.isnan(ref)
    assert nan.sum() == 2 * 1023
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got.view(np.uint32)[~nan], ref.view(np.uint32)[~nan])
    # hand-checked anchors: 1.0, smallest subnormal, largest finite, -2.0, +inf
    anchors = {0x3C00: 1.0, 0x0001: 2.0 ** -24, 0x7BFF: 65504.0, 0xC000: -2.0, 0x7C00: np.inf}
    for pat, val in anchors.items():
        assert got[pat] == np.float32(val), hex(pat)


@pytest.mark.parametrize("unscale", [2.0 ** -16, 1.0 / 3000.0])
@pytest.mark.parametrize("scale", [1.0, 0.25])
def test_first_step_with_fp16_gradients_and_unscale_matches_exact_rationals(unscale, scale):
    """Stored gradient g_s = S*g: the step must see g = unscale*g_s, then the
    clip scale; closed form of the first Adam step in exact rationals."""
    rng = np.random.default_rng(21)
    n = 400
    hp = HParams()
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = (rng.normal(0, 1e-2, n) / unscale).astype(np.float16)
    assert np.isfinite(g).all()
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    oracle.adamw_step_range(p, m, v, g, 0, n, scale, 1, hp, unscale=unscale)
    lr, b1, b2, eps, wd = map(_fr, (hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay))
    for i in range(n):
        gs = _fr(g[i]) * _fr(unscale) * _fr(scale)
        exp_m = f32_from_fraction((1 - b1) * gs)
        exp_v = f32_from_fraction((1 - b2) * gs * gs)
        exp_p = f32_from_fraction(_fr(p0[i]) * (1 - lr * wd) - lr * gs / (abs(gs) + eps))
        assert ulp_distance(np.array([m[i]]), np.array([exp_m]))[0] <= 1
        assert ulp_distance(np.array([v[i]]), np.array([exp_v]))[0] <= 1
        assert ulp_distance(np.array([p[i]]), np.array([exp_p]))[0] <= 1


def test_power_of_two_unscale_scales_the_norm_exactly():
    rng = np.random.default_rng(22)
    g = (rng.normal(0, 1.0, 20000) * 500).astype(np.float16)
    s1, n1, f1 = oracle.global_grad_check(g, 4096)
    s2, n2, f2 = oracle.global_grad_check(g, 4096, unscale=2.0 ** -12)
    assert f1 == f2 == 0
    assert s2 == s1 * 2.0 ** -24 and n2 == n1 * 2.0 ** -12
    # an fp16 overflow in the stored gradient is a non-finite gradient
    g[77] = np.float16(np.inf)
    assert oracle.global_grad_check(g, 4096, unscale=2.0 ** -12)[2] == 1
    # whole iteration: unscale folded into the step equals stepping on pre-divided fp32 gradients
    g[77] = np.float16(3.0)
    hp = HParams(max_grad_norm=0.0)
    n = g.size
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    a = [p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32), oracle.bf16_rne(p0)]
    b = [x.copy() for x in a]
    oracle.iteration_ste(*a, g, 4096, 0, hp, unscale=2.0 ** -12)
    g32 = (g.astype(np.float32) * np.float32(2.0 ** -12))          # exact: power of two
    oracle.iteration_ste(*b, g32, 4096, 0, hp)
    for x, y in zip(a, b):
        assert x.tobytes() == y.tobytes()


def test_loss_scale_schedule():
    """Back off on overflow, grow after `interval` clean steps, counter resets."""
    scale, good = 65536.0, 0
    seen = []
    for bad in [0, 0, 0, 0, 1, 0, 0, 1, 1, 0, 0, 0]:
        scale, good = oracle.loss_scale_update(scale, good, bad, 2.0, 0.5, 3)
        seen.append(scale)
    assert seen == [65536, 65536, 131072, 131072, 65536, 65536, 65536, 32768, 16384,
                    16384, 16384, 32768]
    # a static scale never moves
    assert oracle.loss_scale_update(1024.0, 0, 1, 2.0, 0.5, 0) == (1024.0, 0)
    assert oracle.loss_scale_update(1024.0, 0, 0, 2.0, 0.5, 0) == (1024.0, 0)
