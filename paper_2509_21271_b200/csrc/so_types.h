// Plain data shared by the host code and the kernels of the bucketized
// speculative AdamW library: launch arguments, the records kept in scratch
// memory, and the few constants both sides must agree on.  No device code.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace so {

constexpr int kTileElems = 1024;          // elements per warp tile
constexpr int kRowElems = 128;            // 32 lanes x 4 elements
constexpr int kRowsPerTile = kTileElems / kRowElems;
constexpr int kThreads = 256;             // threads per block (8 warps)
constexpr int kWarpsPerBlock = kThreads / 32;
constexpr int kMaxBatch = 128;            // buckets per launch
constexpr int kReduceThreads = 512;
constexpr int kSegTiles = 4096;           // tile sums folded by one block of the reduction
constexpr uint32_t kSpinLimit = 1u << 20; // bounded mbarrier polling

// Launches of one context that may be outstanding at a time (enqueued and not
// yet finished, on whatever streams).  A launch takes the next pair of the ring;
// within one stream a pair's previous user has finished and re-armed it long
// before it comes round again, and across streams the ring is long enough that
// one stream would have to run 4096 launches ahead of another for two running
// kernels to meet on a pair.
constexpr int kCounterPairs = 4096;

struct Geometry {
    int64_t stride;                       // elements between slots
    uint32_t tiles_per_slot;
    uint32_t bucket_elems;
    uint32_t last_elems;                  // elements in the last bucket
    int32_t last_bucket;                  // its index (-1 if none)
};

// Per-step constants, all derived on the host in double precision.
struct AdamScalars {
    double beta1, omb1;                   // beta1, 1 - beta1
    double beta2, omb2;
    double rsqrt_bc2;                     // 1 / sqrt(1 - beta2^t)
    double step_size;                     // lr / (1 - beta1^t)
    double decay;                         // 1 - lr * wd
    double eps;
    double lr, bc1, bc2;                  // unhoisted: lr, 1 - beta1^t, 1 - beta2^t
    double unscale;                       // 1 / loss scale (fp16 gradients), else 1
};                                        // (the clip scale comes from the verdict on the device)

// Outcome of an iteration as the device records it.  The first three are the
// SO_DECISION_* values of the C ABI; kDecisionAbandon marks an iteration given
// up because a kernel's bounded wait ran out (treated like a skip on the device).
constexpr int32_t kDecisionCommit = 0, kDecisionSkip = 1, kDecisionClip = 2, kDecisionAbandon = 3;

// The verdict of the latest validation.  One copy lives in scratch memory for
// the kernels that follow, one in mapped host memory for the host's
// bookkeeping; `seq` is written last on the host copy.
struct Verdict {
    double sumsq, norm, coef;
    int32_t nonfinite;
    int32_t decision;                     // kDecision*
    int32_t status;                       // device status word this validation saw (0 = fine)
    int32_t seq;                          // stamp of the reduction that produced it
    int32_t pad[2];
};

// Where the fp32 state of the buckets lives, kept on the device so that kernels
// can be enqueued before the host knows how the iteration before ended.
//   slot_of[b]    slot of the state arenas holding bucket b's committed state
//   free_slot[j]  the j-th spare slot (j < undo_slots); the i-th bucket an
//                 iteration speculates writes its new state there
//   spec_idx[b]   j while bucket b holds a speculative result, else -1
// A kept iteration swaps slot_of[b] with free_slot[spec_idx[b]] for every
// speculated bucket; a skipped one only clears spec_idx.
struct SlotTables {
    int32_t *slot_of;
    int32_t *free_slot;
    int32_t *spec_idx;
    const Verdict *verdict;
};

// A bucket in a launch: free_idx >= 0 names the spare slot of a speculated
// bucket, free_idx < 0 a bucket that is stepped (or cast) in place.
struct BucketEntry { int32_t bucket, free_idx; };

// Index into StepArgs::k / CheckArgs::unscale when the launch was enqueued
// before the previous verdict was known to the host: what the step index and
// the loss scale are depends on how that iteration ended.
constexpr int kAfterKept = 0, kAfterSkipped = 1, kAfterAbandoned = 2;

struct StepArgs {
    const void *grad;
    float *master, *mom, *var;
    uint16_t *param_lp;                   // low-precision parameter copy (bf16 or fp16 bits)
    double *partials;
    Geometry geo;
    AdamScalars k[3];                     // by outcome of the pending validation; k[0] if none
    SlotTables tab;
    int32_t pick;                         // 1: choose k[] by the device verdict, 0: k[0]
    int32_t param_fp16;                   // low-precision copy is IEEE binary16 instead of bf16
    uint32_t spin_limit;                  // polls of the wait for a chunk's loads
    Verdict *publish_to;                  // mapped host memory: the first thread of the launch copies
                                          // the (pending) verdict there before it starts; else nullptr
    int32_t n_entries;
    BucketEntry e[kMaxBatch];
};

struct CheckArgs {
    const void *grad;
    double *partials;
    double unscale[3];                    // 1 / loss scale (fp16 gradients), else 1; indexed like StepArgs::k
    const Verdict *verdict;
    int32_t pick;
    Geometry geo;
    int32_t n_entries;
    int32_t bucket[kMaxBatch];
};

struct CastArgs {
    const float *master;
    uint16_t *param_lp;
    Geometry geo;
    SlotTables tab;
    int32_t param_fp16;
    int32_t only_after_skip;              // 1: do nothing unless the device verdict is a skip / give-up
    int32_t n_entries;
    int32_t bucket[kMaxBatch];
};

struct BucketStats { double sumsq; int32_t nonfinite; int32_t pad; };

struct SegSum { double sum; int32_t bad; int32_t pad; };

// Control block in scratch (zeroed once at bind time): a status word and a
// ring of {next tile, finished warps} counter pairs, one pair per launch.
struct ControlBlock {
    int32_t status;
    uint32_t blocks_done;                 // arrival counter of the bucket reduction
    int32_t pad[2];
    uint32_t counters[kCounterPairs][2];
};

struct ReduceArgs {
    const double *partials;               // tile sums
    SegSum *seg;                          // n_buckets x segs_per_slot
    BucketStats *stats;                   // device copy of the records (a Verdict follows them)
    int32_t *status;                      // device status word: read, reported and cleared
    uint32_t *blocks_done;                // arrival counter over the launch's blocks (starts and ends at zero)
    uint32_t n_active_blocks;             // blocks that fold a segment (sum over buckets of their segments)
    SlotTables tab;                       // tab.verdict is the device record to write
    double max_grad_norm;
    int32_t decide;                       // 1: form the verdict and re-point the slots here
    int32_t seq;                          // stamp of this reduction, written last
    Geometry geo;
    uint32_t segs_per_slot;
    int32_t n_buckets;
};

// Arguments of the stand-alone verdict kernel (the host supplies the global
// sum and flag: after so_grad_check(SO_ALL), or combined over ranks).
struct VerdictArgs {
    SlotTables tab;
    double sumsq, max_grad_norm;
    int32_t nonfinite;
    int32_t abandon;                      // 1: the host gives the iteration up
    int32_t seq;
    int32_t n_buckets;
};

// One tensor of the caller's list, as the pack / unpack kernels see it.  The
// pointer comes first: a call uploads only the pointers (strided copy).
struct PackTensor {
    void *ptr;                            // the tensor's own buffer (device)
    int64_t flat_offset;                  // its first element in the flat parameter space
    int64_t numel;
};

constexpr int kPackTileElems = 2048;      // flat elements one warp moves at a time
constexpr int kPackRunsPerWarp = 4;       // such runs per warp of a pack / unpack block

struct PackArgs {
    const PackTensor *tensors;            // device table, flat offsets ascending
    int32_t n_tensors;
    void *arena;                          // gradient arena (pack) or low-precision parameter arena (unpack)
    int64_t total;                        // N
    int64_t bucket_elems;                 // B
    int64_t stride;                       // elements between slots of the arena
};

// The gradient scan is compiled once (with the other kernels) and launched
// from there on behalf of every translation unit.
cudaError_t launch_grad_check(const CheckArgs &a, int grad_dtype, unsigned grid, cudaStream_t stream);
cudaError_t grad_check_occupancy(int grad_dtype, int *blocks_per_sm);

}  // namespace so
