// Fused AdamW step with bulk-copy (TMA) staging of its inputs through shared
// memory and dynamic tile scheduling.
//
// Same arithmetic, same tile/row/quad ownership and same summation order as
// adamw_step_kernel; only the data movement and the work distribution differ.
//
// Data movement.  The register version keeps a warp's loads in flight only
// while that warp is not computing, which leaves both DRAM and the issue slots
// half idle.  Here every warp runs a private software pipeline over *chunks*
// (4 rows of a tile), consumed two rows at a time:
//
//   global --cp.async.bulk--> shared (kStagesIn chunks ahead, completion on an
//   mbarrier) --> registers --> fp64 AdamW --> 128-bit streaming stores --> global
//
// One lane issues the copies; the bytes in flight no longer depend on where
// the warp is in its arithmetic.  The results leave straight from registers:
// staging them through shared memory for bulk stores as well cost the issuing
// lane four more copies, a commit and a wait per chunk (a tenth of all warp
// instructions, executed with one lane active) and 70 KB of shared memory per
// block, and was slower wherever a power cap holds the clock down (-1.1 % per
// iteration on 8 B parameters, -1.3 % on 1.2 B, equal on 124 M).  Pipelines
// are private to a warp, so there is no block-wide synchronisation and the
// deterministic per-tile reduction is unchanged.
// Bulk copies need 16-byte aligned addresses and sizes: slots are 256-byte
// aligned and chunk starts are multiples of 128 elements, so only a chunk
// whose valid length is not a multiple of 8 elements (the ragged end of a
// bucket) takes the guarded register path instead.
//
// Work distribution.  Tiles are not dealt out statically: each warp claims its
// next tile from a global counter (one atomicAdd per 1024 elements, issued one
// tile ahead of need).  With a static round-robin the SMs drift apart and the
// set of DRAM pages being touched spreads; claiming in order keeps every SM
// working inside one compact, advancing window, which on B200 is worth about
// 10 % of HBM throughput for this 4-in / 4-out stream pattern (measured with a
// copy-only kernel: 5.9-6.3 TB/s static, 6.8-6.9 TB/s dynamic).  Which warp
// processes a tile has no influence on any result: tile sums are per tile.
// The counter lives in a small control block in scratch; the last warp to
// finish puts it back to zero for the next launch.
//
// Every wait on an mbarrier is bounded: on expiry the kernel raises a status
// word for the host, drains what it can with bounded waits, and returns.
#pragma once

#include "so_kernels.cuh"

namespace so {

// Shape of the per-warp pipeline: rows (of 128 elements) per chunk, warps per
// block (one block per SM), chunks in flight ahead of the arithmetic.
template <int kRows_, int kWarps_, int kStagesIn_>
struct PipeShape {
    static constexpr int kRows = kRows_;
    static constexpr int kWarps = kWarps_;
    static constexpr int kStagesIn = kStagesIn_;
    static constexpr int kChunkElems = kRows_ * kRowElems;
    static constexpr int kChunksPerTile = kTileElems / kChunkElems;
    static constexpr int kThreads = kWarps_ * 32;
};

// What a pipeline stage holds, written by the issuing lane and read by the
// whole warp when the chunk is consumed.
struct ChunkDesc {
    uint32_t start;        // first element of the chunk within its bucket
    uint32_t len;          // valid elements (0 marks the end of the warp's work)
    uint32_t n;            // elements in the bucket
    uint32_t tile_in_bucket;
    int32_t bucket, src_slot, dst_slot;
    uint32_t flags;        // kLastOfTile | kRagged
};
constexpr uint32_t kLastOfTile = 1u, kRagged = 2u;

template <typename GradT, typename S>
struct TmaLayout {
    static constexpr int kGradBytes = S::kChunkElems * (int)sizeof(GradT);
    static constexpr int kF32Bytes = S::kChunkElems * 4;
    static constexpr int kInStage = 3 * kF32Bytes + kGradBytes;            // p, m, v, g
    static constexpr int kWarpBytes = S::kStagesIn * kInStage;
    // per warp and input stage: one mbarrier (8 B) and one descriptor (32 B);
    // then the launch's buckets with their slots resolved, and their count
    static constexpr int kEntriesOffset = S::kWarps * S::kStagesIn * 40;
    static constexpr int kHeaderBytes =
        128 * ((kEntriesOffset + kMaxBatch * (int)sizeof(ResolvedEntry) + 16 + 127) / 128);
    static constexpr int kSmemBytes = kHeaderBytes + S::kWarps * kWarpBytes;
};

// ---- PTX wrappers -----------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// Bounded wait; returns false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit)
{
    for (uint32_t it = 0; it < limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes,
                                          uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1], %2, [%3], %4;" ::"r"(dst_smem),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- the kernel ---------------------------------------------------------------

template <typename GradT, bool kSpec, typename S>
__global__ void __launch_bounds__(S::kThreads, 1)
adamw_step_tma_kernel(const __grid_constant__ StepArgs a, ControlBlock *ctrl, int pair)
{
    using L = TmaLayout<GradT, S>;
    constexpr int kStagesIn = S::kStagesIn;
    constexpr int kChunkRows = S::kRows, kTmaWarps = S::kWarps;
    extern __shared__ __align__(128) unsigned char smem[];

    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wib = threadIdx.x >> 5;
    const uint32_t n_warps = gridDim.x * kTmaWarps;
    const uint32_t tps = a.geo.tiles_per_slot;

    const uint32_t bars = smem_u32(smem) + wib * kStagesIn * 8;
    ChunkDesc *descs = reinterpret_cast<ChunkDesc *>(smem + kTmaWarps * kStagesIn * 8) +
                       wib * kStagesIn;
    ResolvedEntry *entries = reinterpret_cast<ResolvedEntry *>(smem + L::kEntriesOffset);
    int32_t *n_active_smem = reinterpret_cast<int32_t *>(entries + kMaxBatch);
    unsigned char *wbase = smem + L::kHeaderBytes + wib * L::kWarpBytes;
    uint32_t *next_tile = &ctrl->counters[pair][0];
    uint32_t *done_warps = &ctrl->counters[pair][1];

    // ---- which buckets, which slots, which constants ----
    wait_for_prior_kernels();
    const AdamScalars &k = a.k[outcome_index(a.pick, a.tab.verdict)];
    const bool fp16 = a.param_fp16 != 0;
    double scale = 1.0;
    // the verdict this launch was enqueued behind sets out for the host from here
    if (a.publish_to != nullptr && blockIdx.x == 0 && threadIdx.x == 0)
        verdict_to_host(a.tab.verdict, a.publish_to);
    if constexpr (kSpec) {
        for (int i = threadIdx.x; i < a.n_entries; i += S::kThreads) {
            entries[i] = resolve_speculative(a.tab, a.e[i]);
            if (blockIdx.x == 0) a.tab.spec_idx[a.e[i].bucket] = a.e[i].free_idx;
        }
        if (threadIdx.x == 0) *n_active_smem = a.n_entries;
    } else {
        const FollowUp f = follow_up_of(a.tab.verdict);
        if (!f.step_all && !f.step_inplace) return;      // skipped: nothing is stepped
        scale = f.scale;
        if (threadIdx.x == 0) {
            int32_t n = 0;
            for (int i = 0; i < a.n_entries; ++i)
                if (f.step_all || a.e[i].free_idx < 0) entries[n++] = resolve_after_verdict(a.tab, a.e[i]);
            *n_active_smem = n;
        }
    }
    __syncthreads();
    // nothing to do (a commit with every bucket speculated): the same in every
    // block, so no warp of the launch touches the tile counters
    if (*n_active_smem == 0) return;
    const uint32_t total_tiles = (uint32_t)*n_active_smem * tps;

    const uint64_t policy = l2_evict_first_policy();
    const int64_t stride = a.geo.stride;

    // ---- producer state: meaningful in lane 0 only ----
    uint32_t cur_tile = 0, claimed = 0;        // tile being cut into chunks; tile claimed ahead
    uint32_t cur_sub = 0, cur_n = 0, cur_base = 0, cur_lt = 0;
    int32_t cur_bucket = 0, cur_src = 0, cur_dst = 0;
    bool cur_valid = false;

    // take the tile claimed earlier, claim the next one (its value is not
    // needed until this tile is used up), skip tiles past a partial bucket's end
    auto next_tile_for_lane0 = [&]() {
        for (;;) {
            cur_tile = claimed;
            claimed = atomicAdd(next_tile, 1u);
            if (cur_tile >= total_tiles) {
                cur_valid = false;
                return;
            }
            const uint32_t j = cur_tile / tps;
            const uint32_t lt = cur_tile - j * tps;
            const ResolvedEntry e = entries[j];
            const uint32_t n =
                (e.bucket == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
            if (lt * kTileElems < n) {
                cur_n = n;
                cur_lt = lt;
                cur_base = lt * kTileElems;
                cur_bucket = e.bucket;
                cur_src = e.src_slot;
                cur_dst = e.dst_slot;
                cur_sub = 0;
                cur_valid = true;
                return;
            }
        }
    };

    // describe the next chunk in stage s and start its loads (lane 0 only)
    auto produce = [&](int s) {
        ChunkDesc d;
        if (!cur_valid) {
            d.start = d.len = d.n = d.tile_in_bucket = d.flags = 0;
            d.bucket = d.src_slot = d.dst_slot = 0;
            descs[s] = d;
            return;
        }
        const uint32_t start = cur_base + cur_sub * S::kChunkElems;
        const uint32_t left = cur_n - start;
        const uint32_t len = left < (uint32_t)S::kChunkElems ? left : (uint32_t)S::kChunkElems;
        const bool last = cur_sub + 1 == (uint32_t)S::kChunksPerTile ||
                          start + S::kChunkElems >= cur_n;
        const bool ragged = (len & 7u) != 0;
        d.start = start;
        d.len = len;
        d.n = cur_n;
        d.tile_in_bucket = cur_lt;
        d.bucket = cur_bucket;
        d.src_slot = cur_src;
        d.dst_slot = cur_dst;
        d.flags = (last ? kLastOfTile : 0u) | (ragged ? kRagged : 0u);
        descs[s] = d;
        if (!ragged) {
            const int64_t src = (int64_t)cur_src * stride + start;
            const uint32_t bar = bars + s * 8;
            const uint32_t dst = smem_u32(wbase + s * L::kInStage);
            const uint32_t fbytes = len * 4u, gbytes = len * (uint32_t)sizeof(GradT);
            mbar_expect_tx(bar, 3u * fbytes + gbytes);
            bulk_load(dst, a.master + src, fbytes, bar, policy);
            bulk_load(dst + L::kF32Bytes, a.mom + src, fbytes, bar, policy);
            bulk_load(dst + 2 * L::kF32Bytes, a.var + src, fbytes, bar, policy);
            bulk_load(dst + 3 * L::kF32Bytes,
                      static_cast<const GradT *>(a.grad) + (int64_t)cur_bucket * stride + start,
                      gbytes, bar, policy);
        }
        if (last) next_tile_for_lane0();
        else cur_sub += 1;
    };

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStagesIn; ++s) mbar_init(bars + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
        claimed = atomicAdd(next_tile, 1u);
        next_tile_for_lane0();
#pragma unroll 1
        for (int s = 0; s < kStagesIn; ++s) produce(s);
    }
    __syncwarp();

    uint32_t phases = 0;               // parity bit per input stage
    int stage = 0;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    bool failed = false;

#pragma unroll 1
    for (;;) {
        const ChunkDesc d = descs[stage];
        if (d.len == 0) break;
        const uint32_t len = d.len, start = d.start;
        const bool bulk = (d.flags & kRagged) == 0;
        const int64_t dst = (int64_t)d.dst_slot * stride;
        uint16_t *pb = a.param_lp + (int64_t)d.bucket * stride;

        if (bulk) {
            // every lane polls the same barrier; the verdict is made warp-wide so
            // that no lane leaves the loop while others go on to a __syncwarp
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(bars + stage * 8, (phases >> stage) & 1u,
                                                           a.spin_limit))) {
                failed = true;
                break;
            }
            phases ^= 1u << stage;
            const unsigned char *in = wbase + stage * L::kInStage;
            float *p_out = a.master + dst + start, *m_out = a.mom + dst + start,
                  *v_out = a.var + dst + start;
            uint16_t *lp_out = pb + start;
            // Two rows (8 elements per lane) in flight at a time: the eight
            // dependent chains of conversions, seeds and fp64 operations
            // interleave, which is what hides their latency with only ten warps
            // per SM when a power cap holds the SM clock down.
            auto load_row = [&](uint32_t off, float (&gq)[4], float (&pq)[4], float (&mq)[4],
                                float (&vq)[4]) {
                const float4 p4 = *reinterpret_cast<const float4 *>(in + off * 4);
                const float4 m4 = *reinterpret_cast<const float4 *>(in + L::kF32Bytes + off * 4);
                const float4 v4 = *reinterpret_cast<const float4 *>(in + 2 * L::kF32Bytes + off * 4);
                pq[0] = p4.x; pq[1] = p4.y; pq[2] = p4.z; pq[3] = p4.w;
                mq[0] = m4.x; mq[1] = m4.y; mq[2] = m4.z; mq[3] = m4.w;
                vq[0] = v4.x; vq[1] = v4.y; vq[2] = v4.z; vq[3] = v4.w;
                if constexpr (sizeof(GradT) == 2) {
                    const uint2 g2 = *reinterpret_cast<const uint2 *>(in + 3 * L::kF32Bytes + off * 2);
                    unpack2<GradT>(g2.x, gq[0], gq[1]);
                    unpack2<GradT>(g2.y, gq[2], gq[3]);
                } else {
                    const float4 g4 = *reinterpret_cast<const float4 *>(in + 3 * L::kF32Bytes + off * 4);
                    gq[0] = g4.x; gq[1] = g4.y; gq[2] = g4.z; gq[3] = g4.w;
                }
            };
            // the quad again in the textbook order, from its inputs in the stage
            // (which is refilled only after the chunk)
            auto redo_row = [&](uint32_t off) {
                float g0[4], p0[4], m0[4], v0[4];
                load_row(off, g0, p0, m0, v0);
                return adamw_exact_quad<!kSpec, grad_traits<GradT>::kUnscale>(
                    make_float4(g0[0], g0[1], g0[2], g0[3]), make_float4(p0[0], p0[1], p0[2], p0[3]),
                    make_float4(m0[0], m0[1], m0[2], m0[3]), make_float4(v0[0], v0[1], v0[2], v0[3]), k,
                    scale);
            };
            // (a chunk that takes this path starts on a 16-byte boundary in
            // every arena and its valid length is a multiple of 8 elements, so
            // every quad below it is whole and aligned)
            auto store_row = [&](uint32_t off, const float (&pq)[4], const float (&mq)[4],
                                 const float (&vq)[4]) {
                __stcs(reinterpret_cast<float4 *>(p_out + off), make_float4(pq[0], pq[1], pq[2], pq[3]));
                __stcs(reinterpret_cast<float4 *>(m_out + off), make_float4(mq[0], mq[1], mq[2], mq[3]));
                __stcs(reinterpret_cast<float4 *>(v_out + off), make_float4(vq[0], vq[1], vq[2], vq[3]));
                __stcs(reinterpret_cast<uint2 *>(lp_out + off),
                       make_uint2(pack_lp(pq[0], pq[1], fp16), pack_lp(pq[2], pq[3], fp16)));
            };
            constexpr int kAtOnce = 2;     // four at once spill (168 registers + 80 bytes of stack)
            static_assert(kChunkRows % kAtOnce == 0, "rows are taken in groups");
#pragma unroll 1
            for (int r = 0; r < kChunkRows; r += kAtOnce) {
                const uint32_t off0 = r * kRowElems + lane * 4;    // element within the chunk
                if (off0 >= len) break;
                float gq[kAtOnce][4], pq[kAtOnce][4], mq[kAtOnce][4], vq[kAtOnce][4];
                if (off0 + (kAtOnce - 1) * kRowElems < len) {
#pragma unroll
                    for (int u = 0; u < kAtOnce; ++u)
                        load_row(off0 + u * kRowElems, gq[u], pq[u], mq[u], vq[u]);
                    // (the sums still take the rows in order: same order as ever)
#pragma unroll
                    for (int u = 0; u < kAtOnce; ++u)
                        adamw_quad<!kSpec, grad_traits<GradT>::kUnscale>(
                            gq[u], pq[u], mq[u], vq[u], k, scale, acc,
                            [&]() { return redo_row(off0 + u * kRowElems); });
#pragma unroll
                    for (int u = 0; u < kAtOnce; ++u)
                        store_row(off0 + u * kRowElems, pq[u], mq[u], vq[u]);
                } else {
                    // the ragged end of a chunk: row by row
                    for (int u = 0; u < kAtOnce; ++u) {
                        const uint32_t off = off0 + u * kRowElems;
                        if (off >= len) break;
                        load_row(off, gq[0], pq[0], mq[0], vq[0]);
                        adamw_quad<!kSpec, grad_traits<GradT>::kUnscale>(
                            gq[0], pq[0], mq[0], vq[0], k, scale, acc, [&]() { return redo_row(off); });
                        store_row(off, pq[0], mq[0], vq[0]);
                    }
                }
            }
            // every lane is done with the input stage: refill it
            __syncwarp();
            if (lane == 0) produce(stage);
        } else {
            const GradT *g = static_cast<const GradT *>(a.grad) + (int64_t)d.bucket * stride;
            const int64_t src = (int64_t)d.src_slot * stride;
#pragma unroll 1
            for (int r = 0; r < kChunkRows; ++r) {
                const uint32_t idx = start + r * kRowElems + lane * 4;
                float gq[4], pq[4], mq[4], vq[4];
                load_quad(g, idx, d.n, gq);
                load_quad(a.master + src, idx, d.n, pq);
                load_quad(a.mom + src, idx, d.n, mq);
                load_quad(a.var + src, idx, d.n, vq);
                adamw_quad<!kSpec, grad_traits<GradT>::kUnscale>(
                    gq, pq, mq, vq, k, scale, acc,
                    [&]() {                    // not stored yet: still the inputs
                        return adamw_exact_quad_at<GradT, !kSpec>(g, a.master + src, a.mom + src,
                                                                  a.var + src, idx, d.n, k, scale);
                    });
                if (idx < d.n) {
                    store_quad(a.master + dst, idx, d.n, pq);
                    store_quad(a.mom + dst, idx, d.n, mq);
                    store_quad(a.var + dst, idx, d.n, vq);
                    store_quad_lp(pb, idx, d.n, pq, fp16);
                }
            }
            __syncwarp();
            if (lane == 0) produce(stage);
        }

        if (d.flags & kLastOfTile) {
            if (kSpec) {
                const double tile_sum = tile_fold(acc);
                if (lane == 0) a.partials[(int64_t)d.bucket * tps + d.tile_in_bucket] = tile_sum;
            }
            acc[0] = acc[1] = acc[2] = acc[3] = 0.0;
        }
        stage = (stage + 1 == kStagesIn) ? 0 : stage + 1;
    }

    // this warp has no more tiles to claim: a dependent kernel may be set up
    allow_dependent_launch();

    if (failed) {
        // a copy did not complete in time: tell the host, then wait (bounded,
        // with the full limit) for every chunk whose loads are in flight --
        // all stages hold a produced, unconsumed chunk at this point -- so
        // that nothing lands in this block's shared memory after it is released
        if (lane == 0) atomicExch(&ctrl->status, 1);
        for (int s = 0; s < kStagesIn; ++s) {
            const ChunkDesc pending = descs[s];
            if (pending.len != 0 && (pending.flags & kRagged) == 0)
                mbar_wait_bounded(bars + s * 8, (phases >> s) & 1u, kSpinLimit);
        }
    }
    if (lane == 0) {
        // The last warp of the launch to get here re-arms the counters.  The
        // fence orders this warp's tile claims (including the look-ahead claim
        // whose value is never used) before its arrival, so no claim can land
        // after the reset.
        __threadfence();
        if (atomicAdd(done_warps, 1u) == n_warps - 1) {
            *next_tile = 0;
            *done_warps = 0;
        }
    }
    __syncwarp();
}

}  // namespace so
