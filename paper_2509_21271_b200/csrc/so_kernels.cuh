// Device code of the bucketized speculative AdamW library (sm_100a).
//
// Everything here is a streaming, HBM-bound pass: no reuse, no contraction, no
// tensor cores.  The design rules are the ones that matter for such passes on
// B200: perfectly coalesced 128-bit (fp32) and 64-bit (bf16) accesses, enough
// independent bytes in flight per SM to cover DRAM latency, streaming cache
// policy (nothing is read twice), a persistent grid sized from the SM count,
// and no block-level synchronisation at all (the reduction is per warp).
//
// Work decomposition.  A bucket is cut into *tiles* of 1024 consecutive
// elements; one warp owns one tile at a time (dealt round-robin to all warps
// of the grid here, claimed from a counter in the bulk-copy step kernel).
// Inside a tile a warp sweeps 8 *rows* of 128 elements; lane l owns the *quad*
// of elements [4l, 4l+4) of each row, so a warp-wide fp32 access is one
// contiguous 512-byte line set and a bf16 access one contiguous 256-byte one.  The sum of squares of a tile is accumulated
// per lane in four chains (one per quad position, each in row order), combined
// pairwise, folded across lanes with an xor-shuffle tree and stored as one
// double per tile; a second tiny kernel folds the tiles of each bucket in a
// fixed order.  The summation order therefore depends on nothing but the data
// and the bucket geometry: the same bits come out whatever the grid size, and
// whether the sums were produced by the fused step kernel or by the
// stand-alone check kernel.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <type_traits>

#include "so_types.h"

namespace so {

// Gradient element types: uint16_t carries bf16 bit patterns, half_t IEEE
// binary16 bit patterns (the only type that is used with a loss scale), float
// plain fp32.
struct half_t { uint16_t bits; };

template <typename GradT> struct grad_traits { static constexpr bool kUnscale = false; };
template <> struct grad_traits<half_t> { static constexpr bool kUnscale = true; };

// Every kernel of the library may be launched as a programmatic dependent of
// the kernel before it in the stream (its blocks are set up while that kernel
// drains): nothing written by an earlier kernel may be read before this returns.
__device__ __forceinline__ void wait_for_prior_kernels()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void allow_dependent_launch()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Which of the prepared constant sets applies: a launch enqueued while the
// previous validation was still pending reads how it ended from the device.
__device__ __forceinline__ int outcome_index(int32_t pick, const Verdict *verdict)
{
    if (!pick) return kAfterKept;
    const int32_t d = __ldcg(&verdict->decision);
    return d == kDecisionSkip ? kAfterSkipped : d == kDecisionAbandon ? kAfterAbandoned : kAfterKept;
}

// Copy the verdict in scratch into mapped host memory: the fields, one
// system-wide fence, then the stamp -- a host that sees the stamp sees the rest.
// One thread does it (the first thread of a step kernel that was enqueued while
// the verdict was pending, else a one-thread kernel of its own).
__device__ __forceinline__ void verdict_to_host(const Verdict *src, Verdict *host)
{
    volatile Verdict *dst = host;
    dst->sumsq = __ldcg(&src->sumsq);
    dst->norm = __ldcg(&src->norm);
    dst->coef = __ldcg(&src->coef);
    dst->nonfinite = __ldcg(&src->nonfinite);
    dst->decision = __ldcg(&src->decision);
    dst->status = __ldcg(&src->status);
    const int32_t seq = __ldcg(&src->seq);
    __threadfence_system();
    dst->seq = seq;
}

// The slot tables and the verdict are rewritten by one kernel and read by the
// next, which may already be resident when they change (dependent launches):
// they are always read from L2 (ld.global.cg), never from an SM's L1.
struct ResolvedEntry { int32_t bucket, src_slot, dst_slot; };

// Slots of a speculative step: read the committed slot, write the spare one.
__device__ __forceinline__ ResolvedEntry resolve_speculative(const SlotTables &t, BucketEntry e)
{
    return ResolvedEntry{e.bucket, __ldcg(&t.slot_of[e.bucket]), __ldcg(&t.free_slot[e.free_idx])};
}

// Slots of a step that follows a kept verdict, whose slot swap has already
// happened: a speculated bucket is stepped again from its prior state (now in
// the spare slot) into its committed slot (clip re-step); a bucket that was
// only checked is stepped in place.
__device__ __forceinline__ ResolvedEntry resolve_after_verdict(const SlotTables &t, BucketEntry e)
{
    const int32_t cur = __ldcg(&t.slot_of[e.bucket]);
    return ResolvedEntry{e.bucket, e.free_idx >= 0 ? __ldcg(&t.free_slot[e.free_idx]) : cur, cur};
}

// ---------------------------------------------------------------------------
// streaming loads / stores of one quad (4 consecutive elements)
// ---------------------------------------------------------------------------

__device__ __forceinline__ void load_quad(const float *base, uint32_t idx, uint32_t n, float (&x)[4])
{
    if (idx + 4 <= n) {
        const float4 q = __ldcs(reinterpret_cast<const float4 *>(base + idx));
        x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) x[j] = (idx + j < n) ? __ldcs(base + idx + j) : 0.0f;
    }
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

__device__ __forceinline__ void load_quad(const uint16_t *base, uint32_t idx, uint32_t n, float (&x)[4])
{
    if (idx + 4 <= n) {
        const uint2 q = __ldcs(reinterpret_cast<const uint2 *>(base + idx));
        x[0] = __uint_as_float(q.x << 16);
        x[1] = __uint_as_float(q.x & 0xFFFF0000u);
        x[2] = __uint_as_float(q.y << 16);
        x[3] = __uint_as_float(q.y & 0xFFFF0000u);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            x[j] = (idx + j < n) ? bf16_bits_to_float(__ldcs(base + idx + j)) : 0.0f;
    }
}

// two packed 16-bit gradients -> two floats (element at the lower address first)
template <typename GradT>
__device__ __forceinline__ void unpack2(uint32_t w, float &lo, float &hi);

template <>
__device__ __forceinline__ void unpack2<uint16_t>(uint32_t w, float &lo, float &hi)
{
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xFFFF0000u);
}

template <>
__device__ __forceinline__ void unpack2<half_t>(uint32_t w, float &lo, float &hi)
{
    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w));
    lo = f.x;
    hi = f.y;
}

__device__ __forceinline__ void load_quad(const half_t *base, uint32_t idx, uint32_t n, float (&x)[4])
{
    if (idx + 4 <= n) {
        const uint2 q = __ldcs(reinterpret_cast<const uint2 *>(base + idx));
        unpack2<half_t>(q.x, x[0], x[1]);
        unpack2<half_t>(q.y, x[2], x[3]);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            x[j] = (idx + j < n)
                       ? __half2float(__ushort_as_half(
                             __ldcs(reinterpret_cast<const uint16_t *>(base) + idx + j)))
                       : 0.0f;
    }
}

template <typename T>
__device__ __forceinline__ float4 load_quad4(const T *base, uint32_t idx, uint32_t n)
{
    float x[4];
    load_quad(base, idx, n, x);
    return make_float4(x[0], x[1], x[2], x[3]);
}

__device__ __forceinline__ void store_quad(float *base, uint32_t idx, uint32_t n, const float (&x)[4])
{
    if (idx + 4 <= n) {
        __stcs(reinterpret_cast<float4 *>(base + idx), make_float4(x[0], x[1], x[2], x[3]));
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (idx + j < n) __stcs(base + idx + j, x[j]);
    }
}

// fp32 pair -> packed bf16 pair, round to nearest even (hardware cvt; NaN maps
// to the canonical quiet NaN, denormals are kept).  `lo` lands in bits 0..15.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// fp32 pair -> packed IEEE binary16 pair, round to nearest even (overflow goes
// to infinity, subnormals are kept).
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// The low-precision parameter copy is bf16 or, for the paper's FP16 runs, binary16.
__device__ __forceinline__ uint32_t pack_lp(float lo, float hi, bool fp16)
{
    return fp16 ? pack_f16x2(lo, hi) : pack_bf16x2(lo, hi);
}

__device__ __forceinline__ void store_quad_lp(uint16_t *base, uint32_t idx, uint32_t n,
                                              const float (&x)[4], bool fp16)
{
    const uint32_t w0 = pack_lp(x[0], x[1], fp16);
    const uint32_t w1 = pack_lp(x[2], x[3], fp16);
    if (idx + 4 <= n) {
        __stcs(reinterpret_cast<uint2 *>(base + idx), make_uint2(w0, w1));
    } else {
        const uint16_t h[4] = {(uint16_t)(w0 & 0xFFFFu), (uint16_t)(w0 >> 16),
                               (uint16_t)(w1 & 0xFFFFu), (uint16_t)(w1 >> 16)};
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (idx + j < n) __stcs(base + idx + j, h[j]);
    }
}

// Sum of a tile, fixed order.  A lane keeps four running sums, one per
// position in its quad, each advanced in row order (four independent chains
// instead of one 32-long one: the adds have a long latency); they are combined
// as (s0 + s1) + (s2 + s3) and then folded across the warp with an xor tree.
__device__ __forceinline__ double warp_fold(double x);
__device__ __forceinline__ double tile_fold(const double (&acc)[4])
{
    return warp_fold(__dadd_rn(__dadd_rn(acc[0], acc[1]), __dadd_rn(acc[2], acc[3])));
}

// Fold a per-lane double across the warp with a fixed xor tree.
__device__ __forceinline__ double warp_fold(double x)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        x = __dadd_rn(x, __shfl_xor_sync(0xFFFFFFFFu, x, off));
    return x;
}

// ---------------------------------------------------------------------------
// AdamW on one element, in double (Kingma & Ba Alg. 1 + decoupled decay)
// ---------------------------------------------------------------------------
//
//   g~ = scale*g;  m' = b1*m + (1-b1)*g~;  v' = b2*v + (1-b2)*g~^2
//   p' = p*(1 - lr*wd) - (lr/bc1) * m' / (sqrt(v')/sqrt(bc2) + eps)
//
// m' and v' are formed with separately rounded products and one add (no fused
// multiply-add): with decimal betas the exact value often sits on an fp32
// rounding tie, and only this evaluation order reproduces the reference
// rounding of the stored moments bit for bit.  The parameter update hoists the
// bias corrections into per-step scalars (one division and one square root per
// element); it agrees with the textbook order to a few 1e-16 relative -- of the
// two terms.  Where p*(1 - lr*wd) and the update cancel, that is no longer small
// against the difference: a new parameter 2^-24 of the old one would be off by
// whole fp32 ulps.  So a result below 2^-16 of the old parameter is formed again
// in the textbook order with correctly rounded IEEE operations (about one element
// in a million for N(0, 0.02) weights and lr = 1e-3); above that ratio the two
// orders differ by less than 1 % of half an fp32 ulp of the result.

// sqrt(x) for x >= 0 in double, to within an ulp or two: hardware reciprocal-
// square-root seed (about 20 bits, from the upper word) and one third-order
// step on it (fewer double-precision operations than two Newton steps: on a
// power-capped part the arithmetic's energy, not its time, is what costs
// bandwidth), applied to x times the seed.  Straight-line code: the library
// routine's range checks and slow path are not needed here (x is a finite,
// non-negative, never subnormal second moment).  The seed is taken of
// x + 1e-300: every non-zero second moment is at least 1e-93 (the square of the
// smallest fp32 denormal times 1 - beta2), so the addition returns x itself,
// and for x = 0 it keeps the seed finite so that 0 * (refined seed) = 0 comes
// out exactly.  (Flooring the upper word with an integer maximum instead of the
// addition measured the same.)  For x = +Inf (a second moment that overflowed
// fp32) the result is NaN (Inf * 0); the caller then forms the element again
// with IEEE operations.
__device__ __forceinline__ double sqrt_nonneg(double x)
{
    double y;
    const double xs = __dadd_rn(x, 1e-300);
    asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(xs));
    // one third-order step: with e = 1 - x y^2 (about 2^-20 from the seed),
    // sqrt(x) = x y (1 + e/2 + 3 e^2/8 + O(e^3)); the remainder is below 2^-58.
    // a = x y is sqrt(x) to the seed's accuracy already and the correction is
    // applied to it (the rounding of a enters e and is half taken out again).
    const double a = __dmul_rn(x, y);
    const double e = __fma_rn(-a, y, 1.0);
    const double t = __dmul_rn(e, __fma_rn(e, 0.375, 0.5));
    return __fma_rn(a, t, a);
}

// 1 / b for finite, normal b > 0, to within an ulp or two: reciprocal seed
// (about 20 bits) and one third-order step, 1/b = y (1 + e + e^2 + O(e^3)) with
// e = 1 - b y.
__device__ __forceinline__ double rcp_pos(double b)
{
    double y;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(b));
    const double e = __fma_rn(-b, y, 1.0);
    return __fma_rn(y, __fma_rn(e, e, e), y);
}

// One element, fast order.  Returns true when the new parameter came out below
// 2^-16 of the old one (or not a number), i.e. when the caller has to replace it by
// adamw_exact_p() of the ORIGINAL inputs (the check costs a multiply and a
// compare; taking the branch here, per element, would stop the compiler from
// interleaving the four dependent chains of a quad).
template <bool kScaled, bool kUnscale>
__device__ __forceinline__ bool adamw_element(float g, float &p, float &m, float &v,
                                              const AdamScalars &k, double scale, double &sumsq)
{
    const double gd = kUnscale ? __dmul_rn((double)g, k.unscale) : (double)g;
    const double gs = kScaled ? __dmul_rn(gd, scale) : gd;
    const double sq = __dmul_rn(gs, gs);
    if (!kScaled) sumsq = __dadd_rn(sumsq, sq);
    const double m64 = __dadd_rn(__dmul_rn(k.beta1, (double)m), __dmul_rn(k.omb1, gs));
    const double v64 = __dadd_rn(__dmul_rn(k.beta2, (double)v), __dmul_rn(k.omb2, sq));
    const double denom = __fma_rn(sqrt_nonneg(v64), k.rsqrt_bc2, k.eps);
    const double u = __dmul_rn(__dmul_rn(k.step_size, m64), rcp_pos(denom));
    const double p64 = __fma_rn((double)p, k.decay, -u);
    // negated >=, so that a NaN here (a second moment that reached +Inf makes the
    // straight-line square root produce one) also takes the textbook order,
    // whose IEEE operations handle infinities
    // (the comparison is made on the rounded result, in single precision: the
    // threshold is a margin, not a boundary that has to be exact)
    const float p_new = __double2float_rn(p64);
    const bool cancelled = !(fabsf(p_new) >= __fmul_rn(fabsf(p), 0x1p-16f));
    p = p_new;
    m = __double2float_rn(m64);
    v = __double2float_rn(v64);
    return cancelled;
}

// p' of one element from its original inputs, in the order of Kingma & Ba's
// Algorithm 1 with decoupled decay, every operation correctly rounded:
// mhat = m'/bc1, vhat = v'/bc2, p' = p*(1 - lr*wd) - lr*(mhat/(sqrt(vhat) + eps)).
template <bool kScaled, bool kUnscale>
__device__ __forceinline__ float adamw_exact_p(float g, float p, float m, float v,
                                               const AdamScalars &k, double scale)
{
    const double gd = kUnscale ? __dmul_rn((double)g, k.unscale) : (double)g;
    const double gs = kScaled ? __dmul_rn(gd, scale) : gd;
    const double m64 = __dadd_rn(__dmul_rn(k.beta1, (double)m), __dmul_rn(k.omb1, gs));
    const double v64 = __dadd_rn(__dmul_rn(k.beta2, (double)v), __dmul_rn(k.omb2, __dmul_rn(gs, gs)));
    const double mhat = __ddiv_rn(m64, k.bc1);
    const double vhat = __ddiv_rn(v64, k.bc2);
    const double u = __dmul_rn(k.lr, __ddiv_rn(mhat, __dadd_rn(__dsqrt_rn(vhat), k.eps)));
    return __double2float_rn(__dsub_rn(__dmul_rn((double)p, k.decay), u));
}

// The same for a whole quad, out of line: it runs for about one quad in a
// quarter of a million.  All four elements take the textbook order (a padding
// element past the end of a bucket is all zeros and stays zero).
template <bool kScaled, bool kUnscale>
static __device__ __noinline__ float4 adamw_exact_quad(float4 g, float4 p, float4 m, float4 v,
                                                       const AdamScalars &k, double scale)
{
    float4 r;
    r.x = adamw_exact_p<kScaled, kUnscale>(g.x, p.x, m.x, v.x, k, scale);
    r.y = adamw_exact_p<kScaled, kUnscale>(g.y, p.y, m.y, v.y, k, scale);
    r.z = adamw_exact_p<kScaled, kUnscale>(g.z, p.z, m.z, v.z, k, scale);
    r.w = adamw_exact_p<kScaled, kUnscale>(g.w, p.w, m.w, v.w, k, scale);
    return r;
}

// The same, fetching the original inputs itself from global memory (they have
// not been overwritten there yet): the call site passes four pointers and an
// index instead of sixteen values.
template <typename GradT, bool kScaled>
static __device__ __noinline__ float4 adamw_exact_quad_at(const GradT *g, const float *p,
                                                          const float *m, const float *v,
                                                          uint32_t idx, uint32_t n,
                                                          const AdamScalars &k, double scale)
{
    return adamw_exact_quad<kScaled, grad_traits<GradT>::kUnscale>(
        load_quad4(g, idx, n), load_quad4(p, idx, n), load_quad4(m, idx, n), load_quad4(v, idx, n), k,
        scale);
}

// The four elements of a lane's quad; `reload` forms the quad again in the
// textbook order from its original inputs (they have been overwritten in
// registers by then) and is only called when one of the four cancelled.
template <bool kScaled, bool kUnscale, typename Reload>
__device__ __forceinline__ void adamw_quad(const float (&gq)[4], float (&pq)[4], float (&mq)[4],
                                           float (&vq)[4], const AdamScalars &k, double scale,
                                           double (&acc)[4], Reload reload)
{
    bool redo = false;
#pragma unroll
    for (int q = 0; q < 4; ++q)
        redo |= adamw_element<kScaled, kUnscale>(gq[q], pq[q], mq[q], vq[q], k, scale, acc[q]);
    if (__builtin_expect(redo, false)) {
        const float4 e = reload();
        pq[0] = e.x; pq[1] = e.y; pq[2] = e.z; pq[3] = e.w;
    }
}

// ---------------------------------------------------------------------------
// fused step: g, p, m, v in -> p', m', v', bf16(p') out (+ tile sums of g^2)
// ---------------------------------------------------------------------------
//
// kSpec = true : speculative step (scale 1, tile sums written, new state into
//                the bucket's spare slot).
// kSpec = false: the step that follows a verdict, with the scale the verdict
//                fixed and no sums: after a clip every bucket of the launch
//                (speculated ones from their prior state, the others in
//                place), after a commit only the buckets that were merely
//                checked, after a skip nothing (the low-precision copy of the
//                speculated buckets is then derived again by the cast kernel).
// Source and destination slots may be the same slot (in-place): every element
// is read and written by the same thread, reads first.

// What a follow-up launch does, read from the device verdict.
struct FollowUp { bool step_all, step_inplace; double scale; };

__device__ __forceinline__ FollowUp follow_up_of(const Verdict *verdict)
{
    const int32_t d = __ldcg(&verdict->decision);
    FollowUp f;
    f.step_all = d == kDecisionClip;
    f.step_inplace = d == kDecisionCommit;
    f.scale = d == kDecisionClip ? __ldcg(&verdict->coef) : 1.0;
    return f;
}

template <typename GradT, bool kSpec, int kRowsInFlight>
__global__ void __launch_bounds__(kThreads, 2) adamw_step_kernel(const __grid_constant__ StepArgs a)
{
    wait_for_prior_kernels();
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t tps = a.geo.tiles_per_slot;
    const uint32_t total_tiles = (uint32_t)a.n_entries * tps;
    const AdamScalars &k = a.k[outcome_index(a.pick, a.tab.verdict)];
    const bool fp16 = a.param_fp16 != 0;
    if (a.publish_to != nullptr && blockIdx.x == 0 && threadIdx.x == 0)
        verdict_to_host(a.tab.verdict, a.publish_to);

    FollowUp f{};
    f.scale = 1.0;
    if constexpr (kSpec) {
        if (blockIdx.x == 0 && (int)threadIdx.x < a.n_entries)
            a.tab.spec_idx[a.e[threadIdx.x].bucket] = a.e[threadIdx.x].free_idx;
    } else {
        f = follow_up_of(a.tab.verdict);
        if (!f.step_all && !f.step_inplace) return;      // skipped: nothing is stepped
    }

    for (uint32_t tile = warp; tile < total_tiles; tile += n_warps) {
        const uint32_t j = tile / tps;
        const uint32_t lt = tile - j * tps;
        if (!kSpec && !f.step_all && a.e[j].free_idx >= 0) continue;    // kept as speculated
        const ResolvedEntry e = kSpec ? resolve_speculative(a.tab, a.e[j])
                                      : resolve_after_verdict(a.tab, a.e[j]);
        const uint32_t n = (e.bucket == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
        const uint32_t base = lt * kTileElems;
        if (base >= n) continue;

        const GradT *g = static_cast<const GradT *>(a.grad) + (int64_t)e.bucket * a.geo.stride;
        const int64_t src = (int64_t)e.src_slot * a.geo.stride;
        const int64_t dst = (int64_t)e.dst_slot * a.geo.stride;
        const float *p_in = a.master + src, *m_in = a.mom + src, *v_in = a.var + src;
        float *p_out = a.master + dst, *m_out = a.mom + dst, *v_out = a.var + dst;
        uint16_t *pb = a.param_lp + (int64_t)e.bucket * a.geo.stride;

        double acc[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll 1
        for (int r0 = 0; r0 < kRowsPerTile; r0 += kRowsInFlight) {
            if (base + r0 * kRowElems >= n) break;
            float gq[kRowsInFlight][4], pq[kRowsInFlight][4], mq[kRowsInFlight][4],
                vq[kRowsInFlight][4];
#pragma unroll
            for (int u = 0; u < kRowsInFlight; ++u) {
                const uint32_t idx = base + (r0 + u) * kRowElems + lane * 4;
                load_quad(g, idx, n, gq[u]);
                load_quad(p_in, idx, n, pq[u]);
                load_quad(m_in, idx, n, mq[u]);
                load_quad(v_in, idx, n, vq[u]);
            }
#pragma unroll
            for (int u = 0; u < kRowsInFlight; ++u) {
                const uint32_t idx = base + (r0 + u) * kRowElems + lane * 4;
                adamw_quad<!kSpec, grad_traits<GradT>::kUnscale>(
                    gq[u], pq[u], mq[u], vq[u], k, f.scale, acc,
                    [&]() {                    // not stored yet: still the inputs
                        return adamw_exact_quad_at<GradT, !kSpec>(g, p_in, m_in, v_in, idx, n, k,
                                                                  f.scale);
                    });
                if (idx < n) {
                    store_quad(p_out, idx, n, pq[u]);
                    store_quad(m_out, idx, n, mq[u]);
                    store_quad(v_out, idx, n, vq[u]);
                    store_quad_lp(pb, idx, n, pq[u], fp16);
                }
            }
        }
        if (kSpec) {
            const double tile_sum = tile_fold(acc);
            if (lane == 0) a.partials[(int64_t)e.bucket * tps + lt] = tile_sum;
        }
    }
}

// ---------------------------------------------------------------------------
// stand-alone gradient scan: tile sums of g^2 (same order as the fused kernel)
// ---------------------------------------------------------------------------//
// Read-only, 2 (4) bytes per element: all that matters is bytes in flight.  A
// warp keeps the eight row loads of its *next* tile in flight while it sums the
// current one (two register buffers of raw quads).
template <typename GradT> struct raw_quad { typedef uint2 type; };
template <> struct raw_quad<float> { typedef float4 type; };

template <typename GradT>
__device__ __forceinline__ void unpack_quad(const typename raw_quad<GradT>::type &q, float (&x)[4])
{
    if constexpr (sizeof(GradT) == 2) {
        unpack2<GradT>(q.x, x[0], x[1]);
        unpack2<GradT>(q.y, x[2], x[3]);
    } else {
        x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
    }
}

// A tile of the scan: `n` = elements in its bucket (0: no tile), `base` = its
// first element within the bucket.
struct CheckTile { uint32_t n, base; int32_t bucket; };

// Resident blocks per SM the scan is compiled for (its two register buffers of
// raw quads are twice as large with 4-byte gradients).
template <typename GradT> struct check_shape { static constexpr int kBlocksPerSm = 4; };
template <> struct check_shape<float> { static constexpr int kBlocksPerSm = 2; };

template <typename GradT>
__global__ void __launch_bounds__(kThreads, check_shape<GradT>::kBlocksPerSm)
grad_check_kernel(const __grid_constant__ CheckArgs a)
{
    using Raw = typename raw_quad<GradT>::type;
    constexpr bool kUnscale = grad_traits<GradT>::kUnscale;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t tps = a.geo.tiles_per_slot;
    const uint32_t n_entries = (uint32_t)a.n_entries;
    const GradT *grad = static_cast<const GradT *>(a.grad);
    wait_for_prior_kernels();
    const double unscale = a.unscale[outcome_index(a.pick, a.verdict)];

    // Position of the next tile to fetch, kept as (entry, tile within the slot)
    // and advanced by the grid's stride without a division.
    uint32_t ent = warp / tps, lt = warp - ent * tps;

    // Describe the tile at the position (skipping slot padding), issue its
    // vector loads (a ragged end is read later, guarded), start the tile this
    // warp takes after it on its way from DRAM into L2 (no registers held for
    // it), and move the position on.
    auto fetch_next = [&](CheckTile &t, Raw (&raw)[kRowsPerTile]) {
        for (;;) {
            if (ent >= n_entries) { t.n = 0; return; }
            const int32_t b = a.bucket[ent];
            const uint32_t n = (b == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
            const uint32_t base = lt * kTileElems;
            if (base < n) {
                t.n = n; t.base = base; t.bucket = b;
                const GradT *slot = grad + (int64_t)b * a.geo.stride;
                const GradT *g = slot + base + lane * 4;
                if (base + kTileElems <= n) {
#pragma unroll
                    for (int r = 0; r < kRowsPerTile; ++r)
                        raw[r] = __ldcs(reinterpret_cast<const Raw *>(g + r * kRowElems));
                } else {
#pragma unroll
                    for (int r = 0; r < kRowsPerTile; ++r)
                        if (base + r * kRowElems + lane * 4 + 4 <= n)
                            raw[r] = __ldcs(reinterpret_cast<const Raw *>(g + r * kRowElems));
                }
                constexpr uint32_t kLines = kTileElems * sizeof(GradT) / 128;
                const uint64_t ahead = (uint64_t)(lt + n_warps) * kTileElems;
                if (ahead + kTileElems <= n && lane < kLines)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(
                        reinterpret_cast<const char *>(slot + ahead) + lane * 128));
            }
            lt += n_warps;
            while (lt >= tps) { lt -= tps; ++ent; }
            if (base < n) return;
        }
    };
    // The square of a bf16 or fp32 value has at most 48 significant bits: it is
    // exact in double, so one fused multiply-add rounds exactly like the
    // multiply and the add it replaces.  The same holds for a binary16 value
    // times a power of two (the usual loss scales); with any other scale the
    // unscaled value has a full double mantissa and keeps the two separately
    // rounded operations.
    // With a power-of-two scale the factor is also taken out of the loop: the
    // stored values are squared and summed as they are and the tile's sum is
    // multiplied by the scale's square once -- scaling every term of a sum by a
    // power of two scales every rounding with it, so the bits are those of the
    // sum of the unscaled squares.
    const bool exact_square = !kUnscale || (__double2loint(unscale) == 0 &&
                                            (__double2hiint(unscale) & 0x000FFFFF) == 0);
    const double sum_scale = (kUnscale && exact_square) ? __dmul_rn(unscale, unscale) : 1.0;
    // (the choice is made once per tile, outside the unrolled element loop)
    auto consume_as = [&](auto exact, const CheckTile &t, const Raw (&raw)[kRowsPerTile]) {
        constexpr bool kExact = decltype(exact)::value;
        auto square_add = [&](double stored, double &acc) {
            if constexpr (kExact) {
                acc = __fma_rn(stored, stored, acc);
            } else {
                const double gd = __dmul_rn(stored, unscale);
                acc = __dadd_rn(acc, __dmul_rn(gd, gd));
            }
        };
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        if (t.base + kTileElems <= t.n) {
            // the usual case, straight-line: no bounds to check
#pragma unroll
            for (int r = 0; r < kRowsPerTile; ++r) {
                float x[4];
                unpack_quad<GradT>(raw[r], x);
#pragma unroll
                for (int q = 0; q < 4; ++q) square_add((double)x[q], acc[q]);
            }
        } else {
            const GradT *g = grad + (int64_t)t.bucket * a.geo.stride;
#pragma unroll
            for (int r = 0; r < kRowsPerTile; ++r) {
                const uint32_t idx = t.base + r * kRowElems + lane * 4;
                float x[4];
                if (idx + 4 <= t.n) unpack_quad<GradT>(raw[r], x);
                else load_quad(g, idx, t.n, x);                 // guarded: zeros past the end
#pragma unroll
                for (int q = 0; q < 4; ++q) square_add((double)x[q], acc[q]);
            }
        }
        const double tile_sum = tile_fold(acc);
        if (lane == 0)
            a.partials[(int64_t)t.bucket * tps + t.base / kTileElems] =
                kUnscale ? __dmul_rn(tile_sum, sum_scale) : tile_sum;
    };
    auto consume = [&](const CheckTile &t, const Raw (&raw)[kRowsPerTile]) {
        if constexpr (!kUnscale) {
            consume_as(std::true_type{}, t, raw);
        } else {
            if (exact_square) consume_as(std::true_type{}, t, raw);
            else consume_as(std::false_type{}, t, raw);
        }
    };

    // Two register buffers used alternately: while one tile is summed the loads
    // of the next are in flight and the one after that is coming into L2.
    CheckTile t0, t1;
    Raw buf0[kRowsPerTile], buf1[kRowsPerTile];
    fetch_next(t0, buf0);
    while (t0.n) {
        fetch_next(t1, buf1);
        consume(t0, buf0);
        if (!t1.n) break;
        fetch_next(t0, buf0);
        consume(t1, buf1);
    }
}

// ---------------------------------------------------------------------------
// per-bucket fold of the tile sums (fixed order) + non-finite flag + verdict
// ---------------------------------------------------------------------------
//
// g^2 is formed in double, so it cannot overflow for a finite fp32/bf16 input,
// and a sum of non-negative finite doubles this long cannot overflow either: a
// tile sum is Inf or NaN exactly when the tile holds a NaN or an infinity.
//
// A bucket's tile sums are cut into segments of 4096 tiles.  One block folds
// one segment (each thread adds up to 8 strided tile sums, then a shared-memory
// tree); the block that finishes a bucket's last outstanding segment folds the
// tree).  The block that arrives last (one counter for the whole launch) does
// the rest alone: per bucket the segment sums, then the bucket sums, each added
// one after the other in index order; then the verdict (norm, clip coefficient,
// decision); if the iteration is kept it re-points the speculated buckets at
// their new slots; the verdict stays in scratch for the kernels that follow.
// Segment boundaries and all fold orders are fixed, so the result does not
// depend on which block happens to come last.  The arrival counter starts at
// zero (bind) and is put back to zero by that last block.

// Fold `count` doubles starting at src (stride 1) in the fixed block order.
__device__ __forceinline__ void block_fold(const double *src, uint32_t count, double *s_sum,
                                           int *s_bad, double &sum_out, int &bad_out)
{
    double acc = 0.0;
    int bad = 0;
    for (uint32_t i = threadIdx.x; i < count; i += kReduceThreads) {
        const double x = src[i];
        const uint32_t hi = (uint32_t)__double2hiint(x);
        bad |= ((hi & 0x7FF00000u) == 0x7FF00000u);
        acc = __dadd_rn(acc, x);
    }
    s_sum[threadIdx.x] = acc;
    s_bad[threadIdx.x] = bad;
    __syncthreads();
    for (int s = kReduceThreads / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) {
            s_sum[threadIdx.x] = __dadd_rn(s_sum[threadIdx.x], s_sum[threadIdx.x + s]);
            s_bad[threadIdx.x] |= s_bad[threadIdx.x + s];
        }
        __syncthreads();
    }
    sum_out = s_sum[0];
    bad_out = s_bad[0];
    __syncthreads();
}

// Norm, clip coefficient and decision from the global sum and flag.  Square
// root, addition and division are IEEE correctly rounded, so a host that does
// the same three operations on the same sum gets the same bits.
__device__ __forceinline__ Verdict make_verdict(double sumsq, int nonfinite, int status,
                                                double max_grad_norm, int32_t seq)
{
    Verdict v;
    v.sumsq = sumsq;
    v.norm = __dsqrt_rn(sumsq);
    v.coef = 1.0;
    if (max_grad_norm > 0.0) {
        const double c = __ddiv_rn(max_grad_norm, __dadd_rn(v.norm, 1e-6));
        v.coef = c < 1.0 ? c : 1.0;
    }
    v.nonfinite = nonfinite != 0;
    v.decision = status != 0       ? kDecisionAbandon
                 : v.nonfinite     ? kDecisionSkip
                 : v.coef < 1.0    ? kDecisionClip
                                   : kDecisionCommit;
    v.status = status;
    v.seq = seq;
    v.pad[0] = v.pad[1] = 0;
    return v;
}

// Executed by one whole block of kReduceThreads threads: act on the verdict
// (a kept iteration swaps every speculated bucket's committed and spare slot;
// any verdict clears the speculation marks), then leave it in scratch for the
// kernels that follow.
__device__ __forceinline__ void publish_verdict(const Verdict &v, const SlotTables &tab,
                                                int32_t n_buckets)
{
    const bool kept = v.decision == kDecisionCommit || v.decision == kDecisionClip;
    for (int32_t b = threadIdx.x; b < n_buckets; b += kReduceThreads) {
        const int32_t j = __ldcg(&tab.spec_idx[b]);
        if (j >= 0) {
            if (kept) {
                const int32_t old_slot = __ldcg(&tab.slot_of[b]);
                tab.slot_of[b] = __ldcg(&tab.free_slot[j]);
                tab.free_slot[j] = old_slot;
            }
            tab.spec_idx[b] = -1;
        }
    }
    if (threadIdx.x == 0) *const_cast<Verdict *>(tab.verdict) = v;
}

static __global__ void __launch_bounds__(kReduceThreads) bucket_reduce_kernel(const ReduceArgs a)
{
    __shared__ double s_sum[kReduceThreads];
    __shared__ int s_bad[kReduceThreads];
    __shared__ int s_last;
    __shared__ Verdict s_verdict;
    wait_for_prior_kernels();
    allow_dependent_launch();      // the kernel after this one waits for our completion itself
    const int32_t b = (int32_t)(blockIdx.x / a.segs_per_slot);
    const uint32_t seg = blockIdx.x - (uint32_t)b * a.segs_per_slot;
    const uint32_t n = (b == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
    const uint32_t n_tiles = (n + kTileElems - 1) / kTileElems;
    const uint32_t n_segs = (n_tiles + kSegTiles - 1) / kSegTiles;
    if (seg >= n_segs) return;
    const uint32_t lo = seg * kSegTiles;
    const uint32_t count = n_tiles - lo < (uint32_t)kSegTiles ? n_tiles - lo : (uint32_t)kSegTiles;

    // first level: this block's segment of tile sums
    double sum;
    int bad;
    block_fold(a.partials + (int64_t)b * a.geo.tiles_per_slot + lo, count, s_sum, s_bad, sum, bad);
    if (threadIdx.x == 0) {
        SegSum *mine = a.seg + (int64_t)b * a.segs_per_slot + seg;
        mine->sum = sum;
        mine->bad = bad;
        __threadfence();
        s_last = (atomicAdd(a.blocks_done, 1u) == a.n_active_blocks - 1u);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // The last block to arrive does the rest.  Second level: one thread per
    // bucket adds that bucket's segment sums one after the other in index order
    // and writes the bucket's record.  Third level: the bucket sums, again one
    // after the other in index order, by one thread (records pass through shared
    // memory in runs of 512).  Segment sums of other blocks are read from L2.
    double total = 0.0;
    int flag = 0;
    for (int32_t first = 0; first < a.n_buckets; first += kReduceThreads) {
        const int32_t i = first + (int32_t)threadIdx.x;
        __syncthreads();
        if (i < a.n_buckets) {
            const uint32_t ni = (i == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
            const uint32_t segs_i = ((ni + kTileElems - 1) / kTileElems + kSegTiles - 1) / kSegTiles;
            const SegSum *segs = a.seg + (int64_t)i * a.segs_per_slot;
            double acc = 0.0;
            int any_bad = 0;
            for (uint32_t q = 0; q < segs_i; ++q) {
                acc = __dadd_rn(acc, __ldcg(&segs[q].sum));
                any_bad |= __ldcg(&segs[q].bad);
            }
            BucketStats r;
            r.sumsq = acc;
            r.nonfinite = any_bad;
            r.pad = 0;
            a.stats[i] = r;
            s_sum[threadIdx.x] = acc;
            s_bad[threadIdx.x] = any_bad;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const int32_t m = a.n_buckets - first < kReduceThreads ? a.n_buckets - first : kReduceThreads;
            for (int32_t q = 0; q < m; ++q) {
                total = __dadd_rn(total, s_sum[q]);
                flag |= (s_bad[q] != 0);
            }
        }
    }
    if (threadIdx.x == 0) {
        *a.blocks_done = 0;
        const int status = atomicExch(a.status, 0);
        s_verdict = make_verdict(total, flag, status, a.max_grad_norm, a.seq);
        if (!a.decide) s_verdict.decision = -1;
    }
    __syncthreads();
    if (a.decide) publish_verdict(s_verdict, a.tab, a.n_buckets);
    else if (threadIdx.x == 0) *const_cast<Verdict *>(a.tab.verdict) = s_verdict;
}

static __global__ void publish_to_host_kernel(const Verdict *src, Verdict *host)
{
    wait_for_prior_kernels();
    if (threadIdx.x == 0) verdict_to_host(src, host);
}

// The verdict from a sum and a flag the host supplies: after so_grad_check(SO_ALL)
// (whose reduction did not decide), or with the statistics of all ranks when the
// optimizer states are sharded.  One block.
static __global__ void __launch_bounds__(kReduceThreads) apply_verdict_kernel(const VerdictArgs a)
{
    __shared__ Verdict s_verdict;
    wait_for_prior_kernels();
    allow_dependent_launch();
    if (threadIdx.x == 0)
        s_verdict = make_verdict(a.sumsq, a.nonfinite, a.abandon, a.max_grad_norm, a.seq);
    __syncthreads();
    publish_verdict(s_verdict, a.tab, a.n_buckets);
}

// ---------------------------------------------------------------------------
// stand-alone cast: committed fp32 master -> low-precision copy of the bucket
// ---------------------------------------------------------------------------
static __global__ void __launch_bounds__(kThreads) cast_params_kernel(const __grid_constant__ CastArgs a)
{
    wait_for_prior_kernels();
    if (a.only_after_skip) {
        // the follow-up of a validation: after a skip (or a give-up) the copy of
        // the speculated buckets is derived again from their untouched master
        const int32_t d = __ldcg(&a.tab.verdict->decision);
        if (d != kDecisionSkip && d != kDecisionAbandon) return;
    }
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t tps = a.geo.tiles_per_slot;
    const uint32_t total_tiles = (uint32_t)a.n_entries * tps;
    const bool fp16 = a.param_fp16 != 0;

    for (uint32_t tile = warp; tile < total_tiles; tile += n_warps) {
        const uint32_t j = tile / tps;
        const uint32_t lt = tile - j * tps;
        const int32_t b = a.bucket[j];
        const uint32_t n = (b == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
        const uint32_t base = lt * kTileElems;
        if (base >= n) continue;
        const float *p = a.master + (int64_t)__ldcg(&a.tab.slot_of[b]) * a.geo.stride;
        uint16_t *pb = a.param_lp + (int64_t)b * a.geo.stride;

        float pq[kRowsPerTile][4];
#pragma unroll
        for (int r = 0; r < kRowsPerTile; ++r) {
            const uint32_t idx = base + r * kRowElems + lane * 4;
            if (idx < n) load_quad(p, idx, n, pq[r]);
        }
#pragma unroll
        for (int r = 0; r < kRowsPerTile; ++r) {
            const uint32_t idx = base + r * kRowElems + lane * 4;
            if (idx < n) store_quad_lp(pb, idx, n, pq[r], fp16);
        }
    }
}

}  // namespace so
