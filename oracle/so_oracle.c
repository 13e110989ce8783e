/*
 * CPU oracle for the bucketized mixed-precision AdamW step with
 * speculation-then-validation (STV).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain statement of what
 * the optimizer hot path must compute, used only by the tests, the smoke check
 * and the CPU-baseline leg of the benchmark.  It shares no code with the CUDA
 * library and is never on the product path.
 *
 * Conventions
 *   - single-threaded, index-order loops, `double` arithmetic, compiled with
 *     -ffp-contract=off so that no multiply-add is fused;
 *   - state is stored as fp32 (master weight p, first moment m, second moment
 *     v) and rounded to nearest-even after every step, denormals kept;
 *   - gradients arrive as bf16 bit patterns (uint16_t), as fp32, or as IEEE
 *     binary16 bit patterns (the paper's own FP16 path), the latter normally
 *     multiplied by a loss scale that `unscale` = 1/scale takes out again;
 *   - a "bucket" is the contiguous flat range [b*B, min((b+1)*B, N)).
 *
 * What follows which passage of the paper
 *   - memory accounting 2+2+12 bytes per parameter: Section 2 ("mixed
 *     precision training" paragraph);
 *   - global gradient norm and NaN/Inf check as the synchronisation that
 *     precedes the step: Section 4.4, first paragraph;
 *   - speculative step, in-place rollback and its two scenarios (skip on
 *     NaN/Inf, revert + re-execute with clipped gradients): Section 4.4;
 *   - exactness of STV (same result as synchronise-then-execute): Section 4.4;
 *   - casting on the GPU side of the move: Section 4.5;
 *   - Adam itself is only cited by the paper: the update below is Algorithm 1
 *     of Kingma & Ba (bias-corrected moments, epsilon added outside the square
 *     root) with the decoupled weight decay of Loshchilov & Hutter in the
 *     p*(1 - lr*wd) convention; norm clipping is Pascanu et al.'s
 *     g <- g * min(1, max_norm / (norm + 1e-6)).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_DECISION_COMMIT = 0, ORC_DECISION_SKIP = 1, ORC_DECISION_CLIP_RESTEP = 2 };
enum { ORC_GRAD_BF16 = 0, ORC_GRAD_FP32 = 1, ORC_GRAD_FP16 = 2 };

/* ---- bit views ---------------------------------------------------------- */

static uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }
static float bits_f32(uint32_t u) { float x; memcpy(&x, &u, 4); return x; }

/* bf16 is the upper half of an fp32 pattern: widening is a shift (exact). */
float orc_bf16_to_f32(uint16_t b) { return bits_f32((uint32_t)b << 16); }

void orc_widen_bf16(const uint16_t *b, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_bf16_to_f32(b[i]);
}

/*
 * IEEE binary16 -> fp32 (exact): 1 sign, 5 exponent (bias 15), 10 mantissa
 * bits; exponent 0 is zero or a subnormal (mantissa * 2^-24), exponent 31 is
 * infinity (mantissa 0) or NaN.  This is the gradient format of the paper's
 * mixed-precision runs (Section 4.5).
 */
float orc_fp16_to_f32(uint16_t h)
{
    const int sign = (h >> 15) & 1;
    const int exponent = (h >> 10) & 0x1F;
    const int mantissa = h & 0x3FF;
    double v;
    if (exponent == 0) v = ldexp((double)mantissa, -24);
    else if (exponent == 31) v = mantissa ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)mantissa / 1024.0, exponent - 15);
    return (float)(sign ? -v : v);
}

void orc_widen_fp16(const uint16_t *h, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_fp16_to_f32(h[i]);
}

/*
 * fp32 -> bf16, round to nearest, ties to even (Section 4.5: the cast that
 * produces the low-precision parameter copy).  Integer definition: keep the
 * upper 16 bits; look at the 16 dropped bits; round up when they exceed half,
 * or equal half and the kept lsb is odd.  NaN stays NaN (quiet, sign kept).
 * A carry out of the mantissa correctly bumps the exponent, and the largest
 * finite values round to infinity.
 */
uint16_t orc_bf16_rne(float x)
{
    uint32_t u = f32_bits(x);
    uint32_t exponent = (u >> 23) & 0xFFu;
    uint32_t mantissa = u & 0x7FFFFFu;
    if (exponent == 0xFFu && mantissa != 0u)
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t kept = u >> 16;
    uint32_t dropped = u & 0xFFFFu;
    if (dropped > 0x8000u || (dropped == 0x8000u && (kept & 1u)))
        kept += 1u;
    return (uint16_t)kept;
}

void orc_cast_params(const float *p, uint16_t *pb, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) pb[i] = orc_bf16_rne(p[i]);
}

/*
 * fp32 -> IEEE binary16, round to nearest, ties to even (Section 4.5 names the
 * FP32 <-> FP16 casts of the paper's own mixed-precision runs).  Written out on
 * the bit fields: binary16 keeps 10 mantissa bits and exponents -14..15; below
 * 2^-14 its numbers are the multiples of 2^-24 (subnormals); a value that
 * rounds to 2^16 or more becomes infinity (65520, halfway between the largest
 * finite 65504 and 2^16, is the first such value: the tie goes to the even
 * neighbour, which is 2^16).  NaN maps to a quiet NaN with the sign kept.
 */
uint16_t orc_fp16_rne(float x)
{
    const uint32_t u = f32_bits(x);
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    const uint32_t magnitude = u & 0x7FFFFFFFu;
    const int exponent = (int)(magnitude >> 23) - 127;         /* unbiased, of a normal fp32 */
    if (magnitude > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);       /* NaN */
    if (magnitude == 0x7F800000u) return (uint16_t)(sign | 0x7C00u);      /* infinity */
    if (exponent < -26) return sign;          /* below 2^-26 (fp32 subnormals included): under half of 2^-24 */
    {
        /* 24-bit significand with its leading one; the result keeps its top
         * bits down to the binary16 quantum: 2^(exponent-10) for a normal
         * result, 2^-24 below 2^-14 */
        const uint32_t significand = (magnitude & 0x7FFFFFu) | 0x800000u;
        const int shift = exponent >= -14 ? 13 : 13 + (-14 - exponent);
        uint32_t kept = significand >> shift;
        const uint32_t dropped = significand & ((1u << shift) - 1u);
        const uint32_t half = 1u << (shift - 1);
        uint32_t bits;
        if (dropped > half || (dropped == half && (kept & 1u))) kept += 1u;
        if (exponent >= -14)
            bits = ((uint32_t)(exponent + 14) << 10) + kept;   /* kept includes the leading one: +1 on the exponent field */
        else
            bits = kept;                                       /* subnormal, or 0x400 = 2^-14 after rounding up */
        if (bits >= 0x7C00u) bits = 0x7C00u;                   /* rounded past the largest finite value */
        return (uint16_t)(sign | bits);
    }
}

void orc_cast_params_fp16(const float *p, uint16_t *ph, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) ph[i] = orc_fp16_rne(p[i]);
}

/* ---- gradient check (Section 4.4: global norm + NaN/Inf check) ---------- */

static double grad_at(const void *g, int grad_dtype, int64_t i)
{
    if (grad_dtype == ORC_GRAD_BF16)
        return (double)orc_bf16_to_f32(((const uint16_t *)g)[i]);
    if (grad_dtype == ORC_GRAD_FP16)
        return (double)orc_fp16_to_f32(((const uint16_t *)g)[i]);
    return (double)((const float *)g)[i];
}

/* Sum of squares of one range in index order, and whether any element is
 * NaN or +-Inf.  Each stored gradient is first multiplied by `unscale` (1 when
 * no loss scaling is in use, 1/loss_scale otherwise), so the norm is that of
 * the true gradient.  The square is taken in double, so it cannot overflow for
 * a finite fp32/bf16/fp16 input. */
int orc_grad_check_range(const void *g, int grad_dtype, int64_t begin, int64_t end,
                         double unscale, double *sumsq_out)
{
    double s = 0.0;
    int nonfinite = 0;
    for (int64_t i = begin; i < end; ++i) {
        double x = grad_at(g, grad_dtype, i) * unscale;
        if (!isfinite(x)) nonfinite = 1;
        s += x * x;
    }
    *sumsq_out = s;
    return nonfinite;
}

/* Per-bucket partials in index order, then the sum over buckets in bucket
 * order; norm = sqrt(sum). */
int orc_global_grad_check(const void *g, int grad_dtype, int64_t n, int64_t bucket_elems,
                          double unscale, double *sumsq_out, double *norm_out)
{
    double total = 0.0;
    int nonfinite = 0;
    for (int64_t b0 = 0; b0 < n; b0 += bucket_elems) {
        int64_t b1 = b0 + bucket_elems < n ? b0 + bucket_elems : n;
        double s;
        if (orc_grad_check_range(g, grad_dtype, b0, b1, unscale, &s)) nonfinite = 1;
        total += s;
    }
    *sumsq_out = total;
    *norm_out = sqrt(total);
    return nonfinite;
}

/* Clip coefficient: min(1, max_norm / (norm + 1e-6)); clipping is disabled
 * for max_norm <= 0.  "Clip active" means coef < 1. */
double orc_clip_coef(double norm, double max_norm)
{
    if (!(max_norm > 0.0)) return 1.0;
    double c = max_norm / (norm + 1e-6);
    return c < 1.0 ? c : 1.0;
}

/* Section 4.4's two rollback scenarios as a decision: a non-finite gradient
 * skips the iteration (and wins over clipping); otherwise an active clip
 * means "revert and re-execute with clipped gradients"; otherwise keep. */
int orc_decision(int nonfinite, double coef)
{
    if (nonfinite) return ORC_DECISION_SKIP;
    if (coef < 1.0) return ORC_DECISION_CLIP_RESTEP;
    return ORC_DECISION_COMMIT;
}

/* ---- AdamW element update ----------------------------------------------- */

/*
 * One AdamW step over the flat range [begin, end) with step index tt (1-based)
 * and gradient scale `scale` (1 for an unclipped step, the clip coefficient
 * otherwise).  Kingma & Ba, Algorithm 1, with decoupled decay:
 *     g~   = scale * (unscale * g_stored)
 *     m    = beta1*m + (1-beta1)*g~
 *     v    = beta2*v + (1-beta2)*g~^2
 *     mhat = m / (1 - beta1^tt),   vhat = v / (1 - beta2^tt)
 *     p    = p*(1 - lr*wd) - lr * mhat / (sqrt(vhat) + eps)
 * all in double; p, m, v are then rounded to fp32.
 */
void orc_adamw_step_range(float *p, float *m, float *v, const void *g, int grad_dtype,
                          int64_t begin, int64_t end, double unscale, double scale, int64_t tt,
                          double lr, double beta1, double beta2, double eps, double wd)
{
    const double bc1 = 1.0 - pow(beta1, (double)tt);
    const double bc2 = 1.0 - pow(beta2, (double)tt);
    for (int64_t i = begin; i < end; ++i) {
        double gs = (grad_at(g, grad_dtype, i) * unscale) * scale;
        double m64 = beta1 * (double)m[i] + (1.0 - beta1) * gs;
        double v64 = beta2 * (double)v[i] + (1.0 - beta2) * (gs * gs);
        double mhat = m64 / bc1;
        double vhat = v64 / bc2;
        double u = lr * (mhat / (sqrt(vhat) + eps));
        double p64 = (double)p[i] * (1.0 - lr * wd) - u;
        p[i] = (float)p64;
        m[i] = (float)m64;
        v[i] = (float)v64;
    }
}

/* ---- one training iteration, plain (synchronise-then-execute) ----------- */

/*
 * Check all gradients, decide, then either leave everything untouched (SKIP)
 * or step every element with the clip coefficient and re-derive the bf16 copy.
 * *t is the number of committed steps and advances only when a step is kept.
 * Returns the decision.
 */
int orc_iteration_ste(float *p, float *m, float *v, uint16_t *pb, const void *g,
                      int grad_dtype, int64_t n, int64_t bucket_elems, int64_t *t,
                      double lr, double beta1, double beta2, double eps, double wd,
                      double max_norm, double unscale, double *sumsq_out, double *norm_out,
                      double *coef_out, int *nonfinite_out)
{
    double sumsq, norm;
    int nonfinite = orc_global_grad_check(g, grad_dtype, n, bucket_elems, unscale, &sumsq, &norm);
    double coef = orc_clip_coef(norm, max_norm);
    int decision = orc_decision(nonfinite, coef);
    if (decision != ORC_DECISION_SKIP) {
        orc_adamw_step_range(p, m, v, g, grad_dtype, 0, n, unscale, coef, *t + 1,
                             lr, beta1, beta2, eps, wd);
        orc_cast_params(p, pb, n);
        *t += 1;
    }
    *sumsq_out = sumsq; *norm_out = norm; *coef_out = coef; *nonfinite_out = nonfinite;
    return decision;
}

/* ---- one training iteration, speculation-then-validation view ----------- */

/*
 * The same iteration the way Section 4.4 schedules it: every bucket is stepped
 * first, assuming finite gradients and no clipping (scale 1), with the prior
 * fp32 state kept; validation follows; then COMMIT keeps the result, SKIP puts
 * the prior state back, CLIP_RESTEP puts it back and steps again with the
 * coefficient.  `forced_coef`, when > 0, replaces the coefficient computed
 * here (tests use it to replay the coefficient another implementation found,
 * so that element results can be compared in lock-step).  Returns the
 * decision, or -1 if the snapshot could not be allocated.
 */
int orc_iteration_stv(float *p, float *m, float *v, uint16_t *pb, const void *g,
                      int grad_dtype, int64_t n, int64_t bucket_elems, int64_t *t,
                      double lr, double beta1, double beta2, double eps, double wd,
                      double max_norm, double unscale, double forced_coef, double *sumsq_out,
                      double *norm_out, double *coef_out, int *nonfinite_out)
{
    size_t fbytes = (size_t)n * sizeof(float);
    float *p0 = malloc(fbytes ? fbytes : 1), *m0 = malloc(fbytes ? fbytes : 1),
          *v0 = malloc(fbytes ? fbytes : 1);
    uint16_t *pb0 = malloc(n ? (size_t)n * 2 : 1);
    if (!p0 || !m0 || !v0 || !pb0) { free(p0); free(m0); free(v0); free(pb0); return -1; }
    memcpy(p0, p, fbytes); memcpy(m0, m, fbytes); memcpy(v0, v, fbytes);
    memcpy(pb0, pb, (size_t)n * 2);

    /* speculation: bucket by bucket, scale 1 */
    for (int64_t b0 = 0; b0 < n; b0 += bucket_elems) {
        int64_t b1 = b0 + bucket_elems < n ? b0 + bucket_elems : n;
        orc_adamw_step_range(p, m, v, g, grad_dtype, b0, b1, unscale, 1.0, *t + 1,
                             lr, beta1, beta2, eps, wd);
        orc_cast_params(p + b0, pb + b0, b1 - b0);
    }

    /* validation */
    double sumsq, norm;
    int nonfinite = orc_global_grad_check(g, grad_dtype, n, bucket_elems, unscale, &sumsq, &norm);
    double coef = orc_clip_coef(norm, max_norm);
    if (forced_coef > 0.0) coef = forced_coef;
    int decision = orc_decision(nonfinite, coef);

    if (decision == ORC_DECISION_COMMIT) {
        *t += 1;
    } else {
        memcpy(p, p0, fbytes); memcpy(m, m0, fbytes); memcpy(v, v0, fbytes);
        memcpy(pb, pb0, (size_t)n * 2);
        if (decision == ORC_DECISION_CLIP_RESTEP) {
            orc_adamw_step_range(p, m, v, g, grad_dtype, 0, n, unscale, coef, *t + 1,
                                 lr, beta1, beta2, eps, wd);
            orc_cast_params(p, pb, n);
            *t += 1;
        }
    }
    free(p0); free(m0); free(v0); free(pb0);
    *sumsq_out = sumsq; *norm_out = norm; *coef_out = coef; *nonfinite_out = nonfinite;
    return decision;
}

/* ---- dynamic loss scaling (the paper's FP16 runs; Section 4.4's NaN/Inf check
 *      is this scaler's overflow test) ------------------------------------- */

/*
 * The loss-scale schedule of mixed-precision training (Micikevicius et al.,
 * which the paper cites for its NaN/Inf check): after an iteration that found
 * a non-finite gradient (and was therefore skipped) the scale is multiplied by
 * `backoff` (< 1); after `interval` consecutive clean iterations it is
 * multiplied by `growth` (> 1).  interval <= 0 keeps the scale fixed.
 */
void orc_loss_scale_update(double *scale, int64_t *good_steps, int nonfinite,
                           double growth, double backoff, int64_t interval)
{
    if (interval <= 0) return;
    if (nonfinite) {
        *scale *= backoff;
        *good_steps = 0;
    } else {
        *good_steps += 1;
        if (*good_steps == interval) {
            *scale *= growth;
            *good_steps = 0;
        }
    }
}

/* ---- layout (Section 4.3: flat model states cut into fixed-size buckets) - */

/* Tensor i starts at the sum of the sizes before it; the number of buckets is
 * ceil(N / B).  Writes n_tensors offsets and returns N, or -1 on bad input. */
int64_t orc_layout_offsets(const int64_t *numel, int32_t n_tensors, int64_t *offsets)
{
    int64_t total = 0;
    for (int32_t i = 0; i < n_tensors; ++i) {
        if (numel[i] < 0) return -1;
        offsets[i] = total;
        total += numel[i];
    }
    return total;
}

int64_t orc_num_buckets(int64_t total, int64_t bucket_elems)
{
    if (bucket_elems <= 0 || total < 0) return -1;
    return (total + bucket_elems - 1) / bucket_elems;
}

/* Bytes resident per the paper's accounting: 2 (low-precision parameter) +
 * 2 (low-precision gradient) + 12 (fp32 master, m, v) per parameter. */
int64_t orc_resident_bytes(int64_t total) { return total * (2 + 2 + 12); }
