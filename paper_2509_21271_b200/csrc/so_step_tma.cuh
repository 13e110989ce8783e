// Fused AdamW step with bulk-copy (TMA) staging through shared memory.
//
// Same arithmetic, same tile/row/quad ownership and same summation order as
// adamw_step_kernel; only the data movement differs.  The register version
// keeps a warp's loads in flight only while that warp is not computing, which
// leaves both DRAM and the issue slots half idle.  Here every warp runs a
// private software pipeline over *chunks* of 256 elements:
//
//   global --cp.async.bulk--> shared (kStagesIn chunks ahead, completion on an
//   mbarrier) --> registers --> fp64 AdamW --> shared --cp.async.bulk--> global
//
// One lane issues the copies; the bytes in flight no longer depend on where
// the warp is in its arithmetic, and stores leave through the async proxy as
// well.  Pipelines are private to a warp, so there is no block-wide
// synchronisation and the deterministic per-tile reduction is unchanged.
// Bulk copies need 16-byte aligned addresses and sizes: slots are 256-byte
// aligned and chunk starts are multiples of 256 elements, so only a chunk
// whose valid length is not a multiple of 8 elements (the ragged end of a
// bucket) takes the guarded register path instead.
//
// Every wait on an mbarrier is bounded: on expiry the kernel raises a status
// word for the host, drains what it can with bounded waits, and returns.
#pragma once

#include "so_kernels.cuh"

namespace so {

constexpr uint32_t kSpinLimit = 1u << 20;              // bounded mbarrier polling

// Shape of the per-warp pipeline: rows (of 128 elements) per chunk, warps per
// block (one block per SM), chunks in flight ahead of the arithmetic, and
// output staging buffers.
template <int kRows_, int kWarps_, int kStagesIn_, int kStagesOut_>
struct PipeShape {
    static constexpr int kRows = kRows_;
    static constexpr int kWarps = kWarps_;
    static constexpr int kStagesIn = kStagesIn_;
    static constexpr int kStagesOut = kStagesOut_;
    static constexpr int kChunkElems = kRows_ * kRowElems;
    static constexpr int kChunksPerTile = kTileElems / kChunkElems;
    static constexpr int kThreads = kWarps_ * 32;
};

template <typename GradT, typename S>
struct TmaLayout {
    static constexpr int kGradBytes = S::kChunkElems * (int)sizeof(GradT);
    static constexpr int kF32Bytes = S::kChunkElems * 4;
    static constexpr int kInStage = 3 * kF32Bytes + kGradBytes;            // p, m, v, g
    static constexpr int kOutStage = 3 * kF32Bytes + S::kChunkElems * 2;   // p, m, v, bf16
    static constexpr int kWarpBytes = S::kStagesIn * kInStage + S::kStagesOut * kOutStage;
    static constexpr int kBarrierBytes = 128 * ((S::kWarps * S::kStagesIn * 8 + 127) / 128);
    static constexpr int kSmemBytes = kBarrierBytes + S::kWarps * kWarpBytes;
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

// Bounded wait; returns false if the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it)
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

__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes,
                                           uint64_t policy)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::
                     "l"(dst),
                 "r"(src_smem), "r"(bytes), "l"(policy)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

template <int kPending>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kPending) : "memory");
}

__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- cursor over the chunks a warp owns -------------------------------------
//
// Tiles are dealt to warps round-robin (tile = warp, warp + n_warps, ...); a
// tile holds up to 4 chunks.  The cursor walks the warp's chunks in order and
// skips tiles that lie beyond the end of a partial last bucket.
struct ChunkCursor {
    uint32_t tile;       // index in the launch's tile space
    uint32_t sub;        // chunk within the tile
    uint32_t n;          // elements in the tile's bucket
    uint32_t base;       // first element of the tile within the bucket
    int32_t bucket, src_slot, dst_slot;
    bool valid;
};

__device__ __forceinline__ void cursor_seek(ChunkCursor &c, const StepArgs &a, uint32_t n_warps)
{
    const uint32_t tps = a.geo.tiles_per_slot;
    const uint32_t total = (uint32_t)a.n_entries * tps;
    while (c.tile < total) {
        const uint32_t j = c.tile / tps;
        const uint32_t lt = c.tile - j * tps;
        const BucketEntry e = a.e[j];
        const uint32_t n = (e.bucket == a.geo.last_bucket) ? a.geo.last_elems : a.geo.bucket_elems;
        if (lt * kTileElems < n) {
            c.n = n;
            c.base = lt * kTileElems;
            c.bucket = e.bucket;
            c.src_slot = e.src_slot;
            c.dst_slot = e.dst_slot;
            c.sub = 0;
            c.valid = true;
            return;
        }
        c.tile += n_warps;
    }
    c.valid = false;
}

template <typename S>
__device__ __forceinline__ void cursor_next(ChunkCursor &c, const StepArgs &a, uint32_t n_warps)
{
    c.sub += 1;
    if (c.sub < (uint32_t)S::kChunksPerTile && c.base + c.sub * S::kChunkElems < c.n) return;
    c.tile += n_warps;
    cursor_seek(c, a, n_warps);
}

template <typename S>
__device__ __forceinline__ uint32_t chunk_start(const ChunkCursor &c)
{
    return c.base + c.sub * S::kChunkElems;
}

template <typename S>
__device__ __forceinline__ uint32_t chunk_len(const ChunkCursor &c)
{
    const uint32_t left = c.n - chunk_start<S>(c);
    return left < (uint32_t)S::kChunkElems ? left : (uint32_t)S::kChunkElems;
}

template <typename S>
__device__ __forceinline__ bool chunk_is_last_of_tile(const ChunkCursor &c)
{
    return c.sub + 1 == (uint32_t)S::kChunksPerTile ||
           c.base + (c.sub + 1) * S::kChunkElems >= c.n;
}

// ---- the kernel ---------------------------------------------------------------

template <typename GradT, bool kSpec, typename S>
__global__ void __launch_bounds__(S::kThreads, 1)
adamw_step_tma_kernel(const __grid_constant__ StepArgs a, int32_t *status)
{
    using L = TmaLayout<GradT, S>;
    constexpr int kStagesIn = S::kStagesIn, kStagesOut = S::kStagesOut;
    constexpr int kChunkRows = S::kRows, kTmaWarps = S::kWarps;
    extern __shared__ __align__(128) unsigned char smem[];

    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wib = threadIdx.x >> 5;
    const uint32_t warp = blockIdx.x * kTmaWarps + wib;
    const uint32_t n_warps = gridDim.x * kTmaWarps;
    const uint32_t tps = a.geo.tiles_per_slot;

    const uint32_t bars = smem_u32(smem) + wib * kStagesIn * 8;
    unsigned char *wbase = smem + L::kBarrierBytes + wib * L::kWarpBytes;
    unsigned char *out_base = wbase + kStagesIn * L::kInStage;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStagesIn; ++s) mbar_init(bars + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncwarp();

    const uint64_t policy = l2_evict_first_policy();
    const int64_t stride = a.geo.stride;

    // issue the four bulk loads of the chunk under `c` into stage s (lane 0 only)
    auto issue_load = [&](const ChunkCursor &c, int s) {
        const uint32_t len = chunk_len<S>(c);
        if ((len & 7u) != 0) return;                       // ragged chunk: register path
        const uint32_t start = chunk_start<S>(c);
        const int64_t src = (int64_t)c.src_slot * stride + start;
        const uint32_t bar = bars + s * 8;
        const uint32_t dst = smem_u32(wbase + s * L::kInStage);
        const uint32_t fbytes = len * 4u, gbytes = len * (uint32_t)sizeof(GradT);
        mbar_expect_tx(bar, 3u * fbytes + gbytes);
        bulk_load(dst, a.master + src, fbytes, bar, policy);
        bulk_load(dst + L::kF32Bytes, a.mom + src, fbytes, bar, policy);
        bulk_load(dst + 2 * L::kF32Bytes, a.var + src, fbytes, bar, policy);
        bulk_load(dst + 3 * L::kF32Bytes,
                  static_cast<const GradT *>(a.grad) + (int64_t)c.bucket * stride + start, gbytes,
                  bar, policy);
    };

    ChunkCursor ld;                    // next chunk to load
    ld.tile = warp;
    cursor_seek(ld, a, n_warps);
    ChunkCursor cs = ld;               // next chunk to consume

    // prologue: fill the pipeline
#pragma unroll 1
    for (int s = 0; s < kStagesIn; ++s) {
        if (!ld.valid) break;
        if (lane == 0) issue_load(ld, s);
        cursor_next<S>(ld, a, n_warps);
    }

    uint32_t phases = 0;               // parity bit per input stage
    int stage = 0, ostage = 0;
    double acc = 0.0;
    bool failed = false;

#pragma unroll 1
    while (cs.valid) {
        const uint32_t len = chunk_len<S>(cs);
        const uint32_t start = chunk_start<S>(cs);
        const bool bulk = (len & 7u) == 0;
        float gq[kChunkRows][4], pq[kChunkRows][4], mq[kChunkRows][4], vq[kChunkRows][4];

        if (bulk) {
            if (!mbar_wait_bounded(bars + stage * 8, (phases >> stage) & 1u)) {
                failed = true;
                break;
            }
            phases ^= 1u << stage;
            const unsigned char *in = wbase + stage * L::kInStage;
#pragma unroll
            for (int r = 0; r < kChunkRows; ++r) {
                const uint32_t off = r * kRowElems + lane * 4;     // element within the chunk
                if (off < len) {
                    const float4 p4 = *reinterpret_cast<const float4 *>(in + off * 4);
                    const float4 m4 = *reinterpret_cast<const float4 *>(in + L::kF32Bytes + off * 4);
                    const float4 v4 =
                        *reinterpret_cast<const float4 *>(in + 2 * L::kF32Bytes + off * 4);
                    pq[r][0] = p4.x; pq[r][1] = p4.y; pq[r][2] = p4.z; pq[r][3] = p4.w;
                    mq[r][0] = m4.x; mq[r][1] = m4.y; mq[r][2] = m4.z; mq[r][3] = m4.w;
                    vq[r][0] = v4.x; vq[r][1] = v4.y; vq[r][2] = v4.z; vq[r][3] = v4.w;
                    if (sizeof(GradT) == 2) {
                        const uint2 g2 = *reinterpret_cast<const uint2 *>(in + 3 * L::kF32Bytes +
                                                                          off * 2);
                        gq[r][0] = __uint_as_float(g2.x << 16);
                        gq[r][1] = __uint_as_float(g2.x & 0xFFFF0000u);
                        gq[r][2] = __uint_as_float(g2.y << 16);
                        gq[r][3] = __uint_as_float(g2.y & 0xFFFF0000u);
                    } else {
                        const float4 g4 = *reinterpret_cast<const float4 *>(
                            in + 3 * L::kF32Bytes + off * 4);
                        gq[r][0] = g4.x; gq[r][1] = g4.y; gq[r][2] = g4.z; gq[r][3] = g4.w;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q) gq[r][q] = pq[r][q] = mq[r][q] = vq[r][q] = 0.0f;
                }
            }
        } else {
            const GradT *g = static_cast<const GradT *>(a.grad) + (int64_t)cs.bucket * stride;
            const int64_t src = (int64_t)cs.src_slot * stride;
#pragma unroll
            for (int r = 0; r < kChunkRows; ++r) {
                const uint32_t idx = start + r * kRowElems + lane * 4;
                load_quad(g, idx, cs.n, gq[r]);
                load_quad(a.master + src, idx, cs.n, pq[r]);
                load_quad(a.mom + src, idx, cs.n, mq[r]);
                load_quad(a.var + src, idx, cs.n, vq[r]);
            }
        }
        // every lane has copied its part of the stage: refill it
        __syncwarp();
        if (ld.valid) {
            if (lane == 0) issue_load(ld, stage);
            cursor_next<S>(ld, a, n_warps);
        }

#pragma unroll
        for (int r = 0; r < kChunkRows; ++r)
#pragma unroll
            for (int q = 0; q < 4; ++q)
                adamw_element<!kSpec>(gq[r][q], pq[r][q], mq[r][q], vq[r][q], a.k, acc);

        const int64_t dst = (int64_t)cs.dst_slot * stride;
        uint16_t *pb = a.param_bf16 + (int64_t)cs.bucket * stride;
        if (bulk) {
            // the output stage is free once the bulk stores issued from it
            // kStagesOut chunks ago have finished reading shared memory
            if (lane == 0) bulk_wait_read<kStagesOut - 1>();
            __syncwarp();
            unsigned char *out = out_base + ostage * L::kOutStage;
#pragma unroll
            for (int r = 0; r < kChunkRows; ++r) {
                const uint32_t off = r * kRowElems + lane * 4;
                if (off < len) {
                    *reinterpret_cast<float4 *>(out + off * 4) =
                        make_float4(pq[r][0], pq[r][1], pq[r][2], pq[r][3]);
                    *reinterpret_cast<float4 *>(out + L::kF32Bytes + off * 4) =
                        make_float4(mq[r][0], mq[r][1], mq[r][2], mq[r][3]);
                    *reinterpret_cast<float4 *>(out + 2 * L::kF32Bytes + off * 4) =
                        make_float4(vq[r][0], vq[r][1], vq[r][2], vq[r][3]);
                    *reinterpret_cast<uint2 *>(out + 3 * L::kF32Bytes + off * 2) =
                        make_uint2(pack_bf16x2(pq[r][0], pq[r][1]), pack_bf16x2(pq[r][2], pq[r][3]));
                }
            }
            fence_async_smem();        // generic writes -> visible to the async proxy
            __syncwarp();
            if (lane == 0) {
                const uint32_t src_s = smem_u32(out);
                const uint32_t fbytes = len * 4u;
                bulk_store(a.master + dst + start, src_s, fbytes, policy);
                bulk_store(a.mom + dst + start, src_s + L::kF32Bytes, fbytes, policy);
                bulk_store(a.var + dst + start, src_s + 2 * L::kF32Bytes, fbytes, policy);
                bulk_store(pb + start, src_s + 3 * L::kF32Bytes, len * 2u, policy);
                bulk_commit();
            }
            ostage = (ostage + 1 == kStagesOut) ? 0 : ostage + 1;
        } else {
#pragma unroll
            for (int r = 0; r < kChunkRows; ++r) {
                const uint32_t idx = start + r * kRowElems + lane * 4;
                if (idx < cs.n) {
                    store_quad(a.master + dst, idx, cs.n, pq[r]);
                    store_quad(a.mom + dst, idx, cs.n, mq[r]);
                    store_quad(a.var + dst, idx, cs.n, vq[r]);
                    store_quad_bf16(pb, idx, cs.n, pq[r]);
                }
            }
        }

        if (chunk_is_last_of_tile<S>(cs)) {
            if (kSpec) {
                const double tile_sum = warp_fold(acc);
                if (lane == 0)
                    a.partials[(int64_t)cs.bucket * tps + cs.base / kTileElems] = tile_sum;
            }
            acc = 0.0;
        }
        cursor_next<S>(cs, a, n_warps);
        stage = (stage + 1 == kStagesIn) ? 0 : stage + 1;
    }

    if (failed) {
        // a copy never completed: tell the host, then give the copies that are
        // still in flight a bounded chance to land before this block's shared
        // memory is released
        if (lane == 0) atomicExch(status, 1);
        for (int s = 0; s < kStagesIn; ++s) mbar_wait_bounded(bars + s * 8, (phases >> s) & 1u);
    }
    if (lane == 0) bulk_wait_all();
    __syncwarp();
}

}  // namespace so
