// Flattening on the device: one launch moves every tensor of the caller's
// list between its own buffer and the bucket arena (gradients in, low-precision
// parameters out), in place of one copy per tensor and bucket boundary.
//
// The flat parameter space [0, N) is cut into runs of 2048 elements dealt
// round-robin to the warps of a persistent grid.  A lane moves groups of 16
// bytes (8 two-byte or 4 four-byte elements).  A group that lies inside one
// tensor and one bucket is one 128-bit load and one 128-bit store where the
// addresses are 16-byte aligned (a tensor that starts at an odd element offset
// is read or written element by element on its own side only); a group with a
// tensor or bucket boundary inside it is moved element by element.  Which
// tensor holds a flat index is found by bisection over the tensors' flat
// offsets once per lane and run, then by walking forward.
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

template <typename ElemT, bool kPack>
__global__ void __launch_bounds__(kThreads, 8) pack_kernel(const PackArgs a)
{
    wait_for_prior_kernels();
    constexpr int kVec = 16 / (int)sizeof(ElemT);          // elements per 16-byte group
    constexpr int kGroupsPerLane = kPackTileElems / (32 * kVec);
    const uint32_t lane = threadIdx.x & 31u;
    const int64_t warp = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kWarpsPerBlock;
    const int64_t n_tiles = (a.total + kPackTileElems - 1) / kPackTileElems;
    ElemT *arena = static_cast<ElemT *>(a.arena);

    for (int64_t tile = warp; tile < n_tiles; tile += n_warps) {
        const int64_t tile_base = tile * kPackTileElems;
        int32_t ti = -1;
#pragma unroll 1
        for (int g = 0; g < kGroupsPerLane; ++g) {
            const int64_t f = tile_base + ((int64_t)g * 32 + lane) * kVec;
            if (f >= a.total) break;
            if (ti < 0) ti = tensor_of(a.tensors, a.n_tensors, f);
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
