// Flattening on the device: one launch moves every tensor of the caller's
// list between its own buffer and the bucket arena (gradients in, low-precision
// parameters out), in place of one copy per tensor and bucket boundary.
//
// The flat parameter space [0, N) is cut into runs of 2048 elements; a block
// takes 32 consecutive runs, four per warp.  A lane moves groups of 16
// bytes (8 two-byte or 4 four-byte elements).  A group that lies inside one
// tensor and one bucket is one 128-bit load and one 128-bit store where the
// addresses are 16-byte aligned (a tensor that starts at an odd element offset
// is read or written on its own side in the largest aligned pieces its address
// allows); a group with a tensor or bucket boundary inside it is moved element
// by element.  Which
// tensor holds a flat index is found by bisection over the tensors' flat
// offsets once per lane and run, then by walking forward.
//
// Most runs lie inside one tensor and one bucket with both addresses aligned:
// those are copied straight, eight 128-bit loads in flight per lane before the
// first store (the per-group path keeps one), which is what fills the memory
// pipeline at four blocks of 256 threads per SM.
#pragma once

#include "so_kernels.cuh"

namespace so {

// Index of the tensor that holds flat element f (tensors with no elements are
// passed over): the last tensor whose offset is <= f and that is not empty.
__device__ __forceinline__ int32_t tensor_of(const PackTensor *t, int32_t n_tensors, int64_t f)
{
    int32_t lo = 0, hi = n_tensors - 1;
    while (lo < hi) {
        const int32_t mid = (lo + hi + 1) >> 1;
        if (t[mid].flat_offset <= f) lo = mid; else hi = mid - 1;
    }
    // empty tensors share their offset with the next non-empty one; the
    // bisection lands on the last of them, which is the non-empty one unless
    // trailing tensors are empty
    while (lo > 0 && t[lo].numel == 0) --lo;
    return lo;
}

// ---- 16 bytes to or from an address that is not 16-byte aligned ------------
//
// The bytes of a group sit in four 32-bit words w[0..3] (little endian).  With
// kA = address & 15 known (even, non-zero), the group is moved in the largest
// naturally aligned pieces the address allows -- 2, 4 or 8 bytes, at most four
// of them -- instead of element by element.

// The 32 bits that start at byte kPos (even, kPos + 4 <= 16) of the group.
template <int kPos>
__device__ __forceinline__ uint32_t word_at(const uint32_t (&w)[4])
{
    if constexpr ((kPos & 2) != 0) return __byte_perm(w[kPos >> 2], w[(kPos >> 2) + 1], 0x5432);
    else return w[kPos >> 2];
}

template <int kA, int kPos>
struct PieceAt {
    static constexpr int kAddr = kA + kPos;
    static constexpr int kSize = (kAddr % 8 == 0 && kPos + 8 <= 16) ? 8 : (kAddr % 4 == 0 && kPos + 4 <= 16) ? 4 : 2;
};

template <int kA, int kPos = 0>
__device__ __forceinline__ void store_pieces(char *dst, const uint32_t (&w)[4])
{
    if constexpr (kPos < 16) {
        constexpr int kSize = PieceAt<kA, kPos>::kSize;
        if constexpr (kSize == 8) {
            __stcs(reinterpret_cast<uint2 *>(dst + kPos), make_uint2(word_at<kPos>(w), word_at<kPos + 4>(w)));
        } else if constexpr (kSize == 4) {
            __stcs(reinterpret_cast<uint32_t *>(dst + kPos), word_at<kPos>(w));
        } else {
            const uint32_t x = w[kPos >> 2];
            __stcs(reinterpret_cast<uint16_t *>(dst + kPos), (uint16_t)((kPos & 2) ? x >> 16 : x & 0xFFFFu));
        }
        store_pieces<kA, kPos + kSize>(dst, w);
    }
}

// 32 bits into the group at byte kPos; w starts as zeros and pieces arrive in
// ascending order, so or-ing is enough.
template <int kPos>
__device__ __forceinline__ void put_word(uint32_t (&w)[4], uint32_t x)
{
    if constexpr ((kPos & 2) != 0) {
        w[kPos >> 2] |= x << 16;
        w[(kPos >> 2) + 1] |= x >> 16;
    } else {
        w[kPos >> 2] |= x;
    }
}

template <int kA, int kPos = 0>
__device__ __forceinline__ void load_pieces(const char *src, uint32_t (&w)[4])
{
    if constexpr (kPos < 16) {
        constexpr int kSize = PieceAt<kA, kPos>::kSize;
        if constexpr (kSize == 8) {
            const uint2 x = __ldcs(reinterpret_cast<const uint2 *>(src + kPos));
            put_word<kPos>(w, x.x);
            put_word<kPos + 4>(w, x.y);
        } else if constexpr (kSize == 4) {
            put_word<kPos>(w, __ldcs(reinterpret_cast<const uint32_t *>(src + kPos)));
        } else {
            const uint32_t x = __ldcs(reinterpret_cast<const uint16_t *>(src + kPos));
            w[kPos >> 2] |= (kPos & 2) ? x << 16 : x;
        }
        load_pieces<kA, kPos + kSize>(src, w);
    }
}

// One run (kGroups groups per lane, 512 bytes apart) with exactly one side off
// the 16-byte grid by kA bytes: 128-bit access on the aligned side, pieces on
// the other, four groups in flight per lane.
template <int kA, bool kSrcAligned, int kGroups>
__device__ __forceinline__ void copy_run_pieces(const char *src, char *dst)
{
    constexpr int kInFlight = 4;
#pragma unroll 1
    for (int g0 = 0; g0 < kGroups; g0 += kInFlight) {
        uint32_t w[kInFlight][4];
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) {
            const char *from = src + (g0 + k) * 512;
            if constexpr (kSrcAligned) {
                const uint4 q = __ldcs(reinterpret_cast<const uint4 *>(from));
                w[k][0] = q.x; w[k][1] = q.y; w[k][2] = q.z; w[k][3] = q.w;
            } else {
                w[k][0] = w[k][1] = w[k][2] = w[k][3] = 0u;
                load_pieces<kA>(from, w[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) {
            char *to = dst + (g0 + k) * 512;
            if constexpr (kSrcAligned) store_pieces<kA>(to, w[k]);
            else __stcs(reinterpret_cast<uint4 *>(to), make_uint4(w[k][0], w[k][1], w[k][2], w[k][3]));
        }
    }
}

template <bool kSrcAligned, int kGroups>
__device__ __forceinline__ void copy_run_pieces_any(uint32_t off_by, const char *src, char *dst)
{
    switch (off_by >> 1) {                  // uniform over the warp
    case 1: copy_run_pieces<2, kSrcAligned, kGroups>(src, dst); break;
    case 2: copy_run_pieces<4, kSrcAligned, kGroups>(src, dst); break;
    case 3: copy_run_pieces<6, kSrcAligned, kGroups>(src, dst); break;
    case 4: copy_run_pieces<8, kSrcAligned, kGroups>(src, dst); break;
    case 5: copy_run_pieces<10, kSrcAligned, kGroups>(src, dst); break;
    case 6: copy_run_pieces<12, kSrcAligned, kGroups>(src, dst); break;
    default: copy_run_pieces<14, kSrcAligned, kGroups>(src, dst); break;
    }
}

template <typename ElemT, bool kPack>
__global__ void __launch_bounds__(kThreads, 4) pack_kernel(const PackArgs a)
{
    wait_for_prior_kernels();
    constexpr int kVec = 16 / (int)sizeof(ElemT);          // elements per 16-byte group
    constexpr int kGroupsPerLane = kPackTileElems / (32 * kVec);
    constexpr int kBatch = 8;                              // 128-bit loads in flight per lane
    static_assert(kGroupsPerLane % kBatch == 0, "a run is a whole number of batches");
    const uint32_t lane = threadIdx.x & 31u;
    const int64_t n_tiles = (a.total + kPackTileElems - 1) / kPackTileElems;
    ElemT *arena = static_cast<ElemT *>(a.arena);

    // A block owns kPackRunsPerWarp x 8 consecutive runs and its warps take them
    // interleaved, so that what the block touches at any time is one contiguous
    // stretch; blocks are handed out in index order by the hardware, which keeps
    // the whole grid's accesses advancing together through memory (a persistent
    // grid-stride loop lets the SMs drift apart and loses a tenth of the
    // bandwidth).
    const int64_t first = (int64_t)blockIdx.x * (kWarpsPerBlock * kPackRunsPerWarp) + (threadIdx.x >> 5);
#pragma unroll 1
    for (int r = 0; r < kPackRunsPerWarp; ++r) {
        const int64_t tile = first + (int64_t)r * kWarpsPerBlock;
        if (tile >= n_tiles) break;
        const int64_t tile_base = tile * kPackTileElems;
        int32_t ti = tensor_of(a.tensors, a.n_tensors, tile_base);
        {
            // the whole run inside one tensor and one bucket (a run is 4 KB or
            // 8 KB long, so its groups share the alignment of its first element)
            const PackTensor t = a.tensors[ti];
            const int64_t bucket = tile_base / a.bucket_elems;
            const int64_t in_bucket = tile_base - bucket * a.bucket_elems;
            ElemT *slot = arena + bucket * a.stride + in_bucket;
            ElemT *own = static_cast<ElemT *>(t.ptr) + (tile_base - t.flat_offset);
            const bool in_one = tile_base + kPackTileElems <= t.flat_offset + t.numel &&
                                in_bucket + kPackTileElems <= a.bucket_elems;
            const uint32_t src_off = (uint32_t)(reinterpret_cast<uintptr_t>(kPack ? own : slot) & 15u);
            const uint32_t dst_off = (uint32_t)(reinterpret_cast<uintptr_t>(kPack ? slot : own) & 15u);
            if (in_one && (src_off == 0) != (dst_off == 0)) {
                // one side off the 16-byte grid (a tensor that starts at an odd
                // offset): that side in aligned pieces, the other in 128-bit words
                const char *src = reinterpret_cast<const char *>(kPack ? own : slot) + lane * 16;
                char *dst = reinterpret_cast<char *>(kPack ? slot : own) + lane * 16;
                if (src_off == 0) copy_run_pieces_any<true, kGroupsPerLane>(dst_off, src, dst);
                else copy_run_pieces_any<false, kGroupsPerLane>(src_off, src, dst);
                continue;
            }
            if (in_one && src_off == 0 && dst_off == 0) {
                const uint4 *src = reinterpret_cast<const uint4 *>(kPack ? own : slot) + lane;
                uint4 *dst = reinterpret_cast<uint4 *>(kPack ? slot : own) + lane;
#pragma unroll 1
                for (int g0 = 0; g0 < kGroupsPerLane; g0 += kBatch) {
                    uint4 q[kBatch];
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) q[k] = __ldcs(src + (g0 + k) * 32);
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) __stcs(dst + (g0 + k) * 32, q[k]);
                }
                continue;
            }
        }
#pragma unroll 1
        for (int g = 0; g < kGroupsPerLane; ++g) {
            const int64_t f = tile_base + ((int64_t)g * 32 + lane) * kVec;
            if (f >= a.total) break;
            while (f >= a.tensors[ti].flat_offset + a.tensors[ti].numel) ++ti;
            const PackTensor t = a.tensors[ti];
            const int64_t bucket = f / a.bucket_elems;
            const int64_t in_bucket = f - bucket * a.bucket_elems;
            ElemT *slot = arena + bucket * a.stride + in_bucket;
            ElemT *own = static_cast<ElemT *>(t.ptr) + (f - t.flat_offset);
            const bool whole = f + kVec <= t.flat_offset + t.numel && in_bucket + kVec <= a.bucket_elems;
            const bool slot_ok = (reinterpret_cast<uintptr_t>(slot) & 15u) == 0;
            const bool own_ok = (reinterpret_cast<uintptr_t>(own) & 15u) == 0;
            if (whole && (slot_ok || own_ok)) {
                // the group lies in one tensor and one bucket: 128-bit access on
                // every side whose address allows it, elements on the other
                const ElemT *src = kPack ? own : slot;
                ElemT *dst = kPack ? slot : own;
                const bool src_ok = kPack ? own_ok : slot_ok;
                const bool dst_ok = kPack ? slot_ok : own_ok;
                union { uint4 q; ElemT e[kVec]; } g;
                if (src_ok) {
                    g.q = __ldcs(reinterpret_cast<const uint4 *>(src));
                } else {
#pragma unroll
                    for (int k = 0; k < kVec; ++k) g.e[k] = __ldcs(src + k);
                }
                if (dst_ok) {
                    __stcs(reinterpret_cast<uint4 *>(dst), g.q);
                } else {
#pragma unroll
                    for (int k = 0; k < kVec; ++k) __stcs(dst + k, g.e[k]);
                }
            } else {
                int32_t tj = ti;
                for (int k = 0; k < kVec; ++k) {
                    const int64_t fk = f + k;
                    if (fk >= a.total) break;
                    while (fk >= a.tensors[tj].flat_offset + a.tensors[tj].numel) ++tj;
                    const int64_t bk = fk / a.bucket_elems;
                    ElemT *s = arena + bk * a.stride + (fk - bk * a.bucket_elems);
                    ElemT *o = static_cast<ElemT *>(a.tensors[tj].ptr) + (fk - a.tensors[tj].flat_offset);
                    if (kPack) *s = *o; else *o = *s;
                }
            }
        }
    }
}

}  // namespace so
