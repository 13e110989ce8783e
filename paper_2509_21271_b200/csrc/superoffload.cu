// Host side of the bucketized speculative AdamW library: layout arithmetic,
// the slot map, the per-iteration state machine, and the kernel launches.
// The C ABI is documented in include/superoffload.h.
//
// How an iteration runs without a host round trip.  The slot map (which slot
// of the state arenas holds which bucket) lives on the device.  The bucket
// reduction's last block forms the verdict there -- norm, clip coefficient,
// decision -- and re-points the speculated buckets if the iteration is kept;
// one follow-up launch, enqueued right behind it, reads that verdict and does
// whatever it entails (nothing after a plain commit, the in-place step of
// buckets that were only checked, the re-step of every bucket after a clip,
// the re-cast of the speculated buckets after a skip).  The host reads the same
// verdict from mapped memory afterwards, only for its own bookkeeping (step
// count, loss scale, counters, its mirror of the slot map), and may enqueue the
// next iteration's speculative steps before it has done so: those launches carry
// the constants for every way the pending iteration can have ended and pick on
// the device.
#include "superoffload.h"

#include <cmath>
#include <cstdlib>
#include <chrono>
#include <cstring>
#include <atomic>
#include <new>
#include <utility>
#include <vector>

#include "so_kernels.cuh"
#include "so_step_tma.cuh"
#include "so_pack.cuh"

using namespace so;

namespace {

enum Phase { kIdle = 0, kOpen = 1, kChecked = 2 };
enum Cover : uint8_t { kNone = 0, kCheckedOnly = 1, kSpeculated = 2 };

// One iteration as the host sees it: which buckets have been covered how.
struct IterRec {
    std::vector<uint8_t> cover;
    std::vector<int32_t> free_idx;      // spare slot index of a speculated bucket
    int32_t n_covered = 0, n_speculated = 0;
    bool have_hp = false;
    so_hparams hp{};
    int phase = kIdle;

    void reset()
    {
        std::fill(cover.begin(), cover.end(), (uint8_t)kNone);
        std::fill(free_idx.begin(), free_idx.end(), -1);
        n_covered = n_speculated = 0;
        have_hp = false;
        phase = kIdle;
    }
};

// Step count and loss-scale state.
struct Progress {
    int64_t t = 0;
    double loss_scale = 1.0;
    int64_t good_steps = 0;
};

}  // namespace

struct so_ctx {
    // ---- layout (immutable after init) ----
    std::vector<int64_t> numel, offsets;
    int64_t total = 0, bucket_elems = 0, stride = 0, last_elems = 0, tiles_per_slot = 0;
    int32_t n_buckets = 0, undo_slots = 0, n_slots = 0, grad_dtype = SO_GRAD_BF16;
    int32_t param_dtype = SO_PARAM_BF16;
    // ---- binding ----
    bool bound = false;
    int device = -1, num_sms = 0;
    float *master = nullptr, *mom = nullptr, *var = nullptr;
    void *grad = nullptr;
    uint16_t *param_lp = nullptr;
    double *d_partials = nullptr;
    BucketStats *d_stats = nullptr;     // n_buckets records, then the device Verdict
    Verdict *d_verdict = nullptr;
    ControlBlock *d_ctrl = nullptr;
    SegSum *d_seg = nullptr;            // per-bucket segment sums of the reduction
    int32_t *d_slot_of = nullptr, *d_free_slot = nullptr, *d_spec_idx = nullptr;
    PackTensor *d_tensors = nullptr;    // per-tensor (pointer, flat offset, numel) for pack / unpack
    uint64_t *h_ptr_stage = nullptr;    // pinned staging of a tensor pointer list
    cudaEvent_t ptrs_uploaded = nullptr;    // behind the latest upload from it
    int64_t segs_per_slot = 1;
    uint32_t launch_seq = 0;            // picks the counter pair of each pipeline launch
    int step_variant = 0;               // 0: by launch size, 1: register kernel, 2: bulk-copy pipeline
    uint32_t spin_limit = kSpinLimit;   // polls a step kernel waits for a chunk (debug hook)
    Verdict *h_verdict = nullptr;       // host copy of the verdict
    Verdict *h_verdict_dev = nullptr;   // device view of it when it is mapped pinned memory
    bool h_verdict_pinned = false;
    int32_t reduce_seq = 0;             // stamp of the latest reduction (never 0)
    cudaEvent_t reduce_done = nullptr;  // completion of the copy-back when the host copy is not mapped
    int occ_step = 0, occ_check = 0, occ_cast = 0;
    // ---- slot map (host mirror of the device tables) ----
    std::vector<int32_t> slot_of;       // committed slot of each bucket
    std::vector<int32_t> free_slot;     // the spare slots, by index
    // ---- iterations ----
    IterRec cur;                        // the iteration being assembled
    IterRec pend;                       // an iteration whose validation has been enqueued
    bool pending = false;               //   ... and whose verdict the host has not applied yet
    bool pend_known = false;            // its verdict was formed from host-supplied statistics
    Verdict pend_verdict{};             //   (then this is it)
    cudaStream_t pend_stream = nullptr;
    bool pend_published = false;        // something that sends its verdict to the host is enqueued
    cudaStream_t pend_wait_stream = nullptr;   // stream whose completion implies the verdict is in
    so_grad_stats stats{};              // result of the last completed check
    Progress prog;
    double ls_growth = 2.0, ls_backoff = 0.5;
    int64_t ls_interval = 0;            // clean iterations before growth; 0 = static scale
    // ---- bookkeeping ----
    so_counters counters{};
    int32_t last_cuda_error = 0;
    bool dry_run = false;
    std::vector<BucketStats> injected;
    int32_t injected_status = 0;
    // ---- host-fed iteration: copy streams and ordering events (lazy) ----
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    std::vector<cudaEvent_t> events;
    bool copies_in_flight = false;      // a pipelined call's outgoing parameters may still be travelling
    // After a pipelined call, which gradient buckets its kernels are done with
    // (everything that reads them ran before the verdict the call waited for)
    // and an event behind the kernels that still read the others.
    bool after_pipelined = false;
    std::vector<uint8_t> grad_done;
    cudaEvent_t grads_read = nullptr;
};

namespace {

Geometry geometry_of(const so_ctx *c)
{
    Geometry g;
    g.stride = c->stride;
    g.tiles_per_slot = (uint32_t)c->tiles_per_slot;
    g.bucket_elems = (uint32_t)c->bucket_elems;
    g.last_elems = (uint32_t)c->last_elems;
    g.last_bucket = c->n_buckets - 1;
    return g;
}

SlotTables tables_of(const so_ctx *c)
{
    SlotTables t;
    t.slot_of = c->d_slot_of;
    t.free_slot = c->d_free_slot;
    t.spec_idx = c->d_spec_idx;
    t.verdict = c->d_verdict;
    return t;
}

Verdict *host_verdict_of(const so_ctx *c) { return c->h_verdict; }

int64_t elems_of(const so_ctx *c, int32_t b)
{
    return b == c->n_buckets - 1 ? c->last_elems : c->bucket_elems;
}

so_status cuda_fail(so_ctx *c, cudaError_t e)
{
    c->last_cuda_error = (int32_t)e;
    return SO_ERR_CUDA;
}

bool hparams_ok(const so_hparams *hp)
{
    if (!hp) return false;
    const double vals[] = {hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay,
                           hp->max_grad_norm};
    for (double x : vals)
        if (!std::isfinite(x)) return false;
    return hp->lr >= 0.0 && hp->beta1 >= 0.0 && hp->beta1 < 1.0 && hp->beta2 >= 0.0 &&
           hp->beta2 < 1.0 && hp->eps >= 2.3e-308 && hp->weight_decay >= 0.0;
}

bool hparams_equal(const so_hparams &a, const so_hparams &b)
{
    return std::memcmp(&a, &b, sizeof(so_hparams)) == 0;
}

AdamScalars scalars_for(const so_hparams &hp, int64_t step_index, double unscale)
{
    const double bc1 = 1.0 - std::pow(hp.beta1, (double)step_index);
    const double bc2 = 1.0 - std::pow(hp.beta2, (double)step_index);
    AdamScalars k;
    k.beta1 = hp.beta1;
    k.omb1 = 1.0 - hp.beta1;
    k.beta2 = hp.beta2;
    k.omb2 = 1.0 - hp.beta2;
    k.rsqrt_bc2 = 1.0 / std::sqrt(bc2);
    k.step_size = hp.lr / bc1;
    k.decay = 1.0 - hp.lr * hp.weight_decay;
    k.eps = hp.eps;
    k.lr = hp.lr;
    k.bc1 = bc1;
    k.bc2 = bc2;
    k.unscale = unscale;
    return k;
}

double clip_coef_of(double norm, double max_norm)
{
    if (!(max_norm > 0.0)) return 1.0;
    const double c = max_norm / (norm + 1e-6);
    return c < 1.0 ? c : 1.0;
}

// The verdict as the device forms it (make_verdict), restated for the host:
// used where no device takes part (dry run) and where the host already holds
// the global sum and flag.  Same three IEEE operations, same bits.
Verdict verdict_of(double sumsq, int nonfinite, int status, double max_grad_norm, int32_t seq)
{
    Verdict v;
    std::memset(&v, 0, sizeof(v));
    v.sumsq = sumsq;
    v.norm = std::sqrt(sumsq);
    v.coef = clip_coef_of(v.norm, max_grad_norm);
    v.nonfinite = nonfinite != 0;
    v.decision = status != 0 ? kDecisionAbandon
                 : v.nonfinite ? kDecisionSkip
                 : v.coef < 1.0 ? kDecisionClip
                                : kDecisionCommit;
    v.status = status;
    v.seq = seq;
    return v;
}

// Step count and loss scale after an iteration that ended in `outcome`
// (kAfterKept / kAfterSkipped / kAfterAbandoned).  Dynamic loss scaling: back
// off after an overflow, grow after a run of clean iterations.
Progress progress_after(const so_ctx *c, int outcome)
{
    Progress p = c->prog;
    if (outcome == kAfterKept) {
        p.t += 1;
        if (c->ls_interval > 0 && ++p.good_steps == c->ls_interval) {
            p.loss_scale *= c->ls_growth;
            p.good_steps = 0;
        }
    } else if (outcome == kAfterSkipped) {
        if (c->ls_interval > 0) {
            p.loss_scale *= c->ls_backoff;
            p.good_steps = 0;
        }
    }
    return p;
}

// Persistent grid: enough blocks to fill every SM at the kernel's occupancy,
// never more than there are tiles to hand out.
unsigned grid_for(const so_ctx *c, int64_t total_tiles, int blocks_per_sm)
{
    int64_t want = (total_tiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
    int64_t cap = (int64_t)c->num_sms * (blocks_per_sm > 0 ? blocks_per_sm : 1);
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    return (unsigned)want;
}

so_status after_launch(so_ctx *c, cudaError_t launch_error = cudaSuccess)
{
    c->counters.kernel_launches += 1;
    if (c->dry_run) return SO_OK;
    if (launch_error != cudaSuccess) return cuda_fail(c, launch_error);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SO_OK : cuda_fail(c, e);
}

// ---- launches --------------------------------------------------------------

// Every kernel is launched as a programmatic dependent of whatever precedes it
// in the stream: its blocks may be set up while that kernel drains, and each of
// them waits (griddepcontrol.wait, first thing) for its completion and memory
// flush before reading anything.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                             cudaStream_t stream, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Launches of at most this many elements take the register kernel (measured
// crossover between 2 Mi and 4 Mi elements per launch).
constexpr int64_t kSmallLaunchElems = (int64_t)3 << 20;

// Shape of the bulk-copy pipeline: rows per chunk, warps per block (one block
// per SM), input stages.  It came out of sweeps on B200: 512-element chunks
// halve the per-chunk bookkeeping, and two input stages of 7 KB (8 KB with fp32
// gradients) per warp keep 140-160 KB of loads in flight per SM.  Twelve warps,
// or a third stage, fit as well since the results no longer pass through shared
// memory; twelve warps measured 0.2 % better on 8 B parameters under the power
// cap and 1 % worse on 124 M at full clock, a third stage 0.3-0.5 % worse on both.
using ShapeBf16 = PipeShape<4, 10, 2>;
using ShapeFp32 = PipeShape<4, 10, 2>;

template <typename GradT, typename S>
cudaError_t launch_tma(so_ctx *c, const StepArgs &a, int n, bool speculative, cudaStream_t stream)
{
    int64_t blocks = ((int64_t)n * a.geo.tiles_per_slot + S::kWarps - 1) / S::kWarps;
    if (blocks > c->num_sms) blocks = c->num_sms;
    const unsigned grid = (unsigned)(blocks < 1 ? 1 : blocks);
    // launches that may overlap in time (other streams) must not share a tile counter
    const int pair = (int)(c->launch_seq++ % kCounterPairs);
    const size_t sm = TmaLayout<GradT, S>::kSmemBytes;
    if (speculative)
        return launch_dependent(adamw_step_tma_kernel<GradT, true, S>, grid, S::kThreads, sm, stream,
                                a, c->d_ctrl, pair);
    return launch_dependent(adamw_step_tma_kernel<GradT, false, S>, grid, S::kThreads, sm, stream, a,
                            c->d_ctrl, pair);
}

template <typename GradT>
cudaError_t launch_registers(const StepArgs &a, unsigned grid, bool speculative, cudaStream_t stream)
{
    if (speculative)
        return launch_dependent(adamw_step_kernel<GradT, true, 2>, grid, kThreads, 0, stream, a);
    return launch_dependent(adamw_step_kernel<GradT, false, 2>, grid, kThreads, 0, stream, a);
}

// The bulk-copy kernels stage through more than 48 KB of shared memory.
template <typename GradT, typename S>
cudaError_t allow_smem()
{
    static_assert(TmaLayout<GradT, S>::kSmemBytes <= 227 * 1024, "pipeline does not fit");
    const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = cudaFuncSetAttribute(adamw_step_tma_kernel<GradT, true, S>, attr,
                                         TmaLayout<GradT, S>::kSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(adamw_step_tma_kernel<GradT, false, S>, attr,
                                 TmaLayout<GradT, S>::kSmemBytes);
    return e;
}

// Step the listed buckets.  speculative: scale 1, new state into the spare
// slot, tile sums written.  Otherwise the launch follows a verdict and does
// what the verdict on the device says (see adamw_step_kernel).
// A speculative launch enqueued while a validation is pending carries the
// constants for each way that validation can end.
so_status launch_steps(so_ctx *c, const std::vector<BucketEntry> &entries, const so_hparams &hp,
                       bool speculative, cudaStream_t stream)
{
    const Geometry geo = geometry_of(c);
    for (size_t first = 0; first < entries.size(); first += kMaxBatch) {
        const int n = (int)std::min<size_t>(kMaxBatch, entries.size() - first);
        StepArgs a;
        a.grad = c->grad;
        a.master = c->master;
        a.mom = c->mom;
        a.var = c->var;
        a.param_lp = c->param_lp;
        a.partials = c->d_partials;
        a.geo = geo;
        a.tab = tables_of(c);
        a.pick = c->pending ? 1 : 0;
        for (int o = 0; o < 3; ++o) {
            const Progress p = c->pending ? progress_after(c, o) : c->prog;
            a.k[o] = scalars_for(hp, p.t + 1, 1.0 / p.loss_scale);
        }
        a.param_fp16 = c->param_dtype == SO_PARAM_FP16;
        a.spin_limit = c->spin_limit;
        a.publish_to = nullptr;
        if (c->pending && !c->pend_known && !c->pend_published && c->h_verdict_dev && !c->dry_run) {
            // the pending verdict rides to the host with this launch
            a.publish_to = c->h_verdict_dev;
            c->pend_published = true;
            c->pend_wait_stream = stream;
        }
        a.n_entries = n;
        for (int i = 0; i < n; ++i) a.e[i] = entries[first + i];
        for (int i = n; i < kMaxBatch; ++i) a.e[i] = BucketEntry{0, -1};
        cudaError_t e = cudaSuccess;
        if (!c->dry_run) {
            const int dt = c->grad_dtype;
            const unsigned grid = grid_for(c, (int64_t)n * geo.tiles_per_slot, c->occ_step);
            // A small launch takes the register kernel: no pipeline to fill and
            // drain, no 146 KB of shared memory per block to set up (a launch of
            // 1 Mi elements: 14.3 us against 15.8 us; from 4 Mi elements on the
            // pipeline is ahead, by 26 % at 8 Mi).
            int64_t launch_elems = 0;
            for (int i = 0; i < n; ++i) launch_elems += elems_of(c, a.e[i].bucket);
            const bool registers = c->step_variant == 1 ||
                                   (c->step_variant == 0 && launch_elems <= kSmallLaunchElems);
            if (!registers) {
                if (dt == SO_GRAD_BF16) e = launch_tma<uint16_t, ShapeBf16>(c, a, n, speculative, stream);
                else if (dt == SO_GRAD_FP16) e = launch_tma<half_t, ShapeBf16>(c, a, n, speculative, stream);
                else e = launch_tma<float, ShapeFp32>(c, a, n, speculative, stream);
            } else {
                if (dt == SO_GRAD_BF16) e = launch_registers<uint16_t>(a, grid, speculative, stream);
                else if (dt == SO_GRAD_FP16) e = launch_registers<half_t>(a, grid, speculative, stream);
                else e = launch_registers<float>(a, grid, speculative, stream);
            }
        }
        const so_status s = after_launch(c, e);
        if (s != SO_OK) return s;
    }
    return SO_OK;
}

so_status launch_checks(so_ctx *c, const std::vector<int32_t> &buckets, cudaStream_t stream)
{
    const Geometry geo = geometry_of(c);
    for (size_t first = 0; first < buckets.size(); first += kMaxBatch) {
        const int n = (int)std::min<size_t>(kMaxBatch, buckets.size() - first);
        CheckArgs a;
        a.grad = c->grad;
        a.partials = c->d_partials;
        for (int o = 0; o < 3; ++o)
            a.unscale[o] = 1.0 / (c->pending ? progress_after(c, o) : c->prog).loss_scale;
        a.verdict = c->d_verdict;
        a.pick = c->pending ? 1 : 0;
        a.geo = geo;
        a.n_entries = n;
        for (int i = 0; i < n; ++i) {
            a.bucket[i] = buckets[first + i];
            c->counters.elems_checked += elems_of(c, a.bucket[i]);
        }
        for (int i = n; i < kMaxBatch; ++i) a.bucket[i] = 0;
        cudaError_t e = cudaSuccess;
        if (!c->dry_run) {
            const unsigned grid = grid_for(c, (int64_t)n * geo.tiles_per_slot, c->occ_check);
            e = launch_grad_check(a, c->grad_dtype, grid, stream);
        }
        const so_status s = after_launch(c, e);
        if (s != SO_OK) return s;
    }
    return SO_OK;
}

// only_after_skip: the follow-up of a validation, which casts only if the
// device verdict is a skip (its elements are counted when the verdict is known).
so_status launch_casts(so_ctx *c, const std::vector<int32_t> &buckets, cudaStream_t stream,
                       bool only_after_skip = false)
{
    const Geometry geo = geometry_of(c);
    for (size_t first = 0; first < buckets.size(); first += kMaxBatch) {
        const int n = (int)std::min<size_t>(kMaxBatch, buckets.size() - first);
        CastArgs a;
        a.master = c->master;
        a.param_lp = c->param_lp;
        a.geo = geo;
        a.tab = tables_of(c);
        a.param_fp16 = c->param_dtype == SO_PARAM_FP16;
        a.only_after_skip = only_after_skip ? 1 : 0;
        a.n_entries = n;
        for (int i = 0; i < n; ++i) {
            a.bucket[i] = buckets[first + i];
            if (!only_after_skip) c->counters.elems_cast += elems_of(c, a.bucket[i]);
        }
        for (int i = n; i < kMaxBatch; ++i) a.bucket[i] = 0;
        cudaError_t e = cudaSuccess;
        if (!c->dry_run) {
            const unsigned grid = grid_for(c, (int64_t)n * geo.tiles_per_slot, c->occ_cast);
            e = launch_dependent(cast_params_kernel, grid, kThreads, 0, stream, a);
        }
        const so_status s = after_launch(c, e);
        if (s != SO_OK) return s;
    }
    return SO_OK;
}

// Scan whatever the open iteration has not covered yet.
so_status scan_uncovered(so_ctx *c, cudaStream_t stream)
{
    std::vector<int32_t> todo;
    for (int32_t b = 0; b < c->n_buckets; ++b)
        if (c->cur.cover[b] == kNone) todo.push_back(b);
    if (todo.empty()) return SO_OK;
    const so_status s = launch_checks(c, todo, stream);
    if (s != SO_OK) return s;
    for (int32_t b : todo) c->cur.cover[b] = kCheckedOnly;
    c->cur.n_covered = c->n_buckets;
    return SO_OK;
}

// The per-bucket reduction; with `decide` its last block also forms the verdict
// and re-points the slots.
so_status launch_reduce(so_ctx *c, double max_grad_norm, bool decide, cudaStream_t stream)
{
    c->reduce_seq = c->reduce_seq == 0x7FFFFFFF ? 1 : c->reduce_seq + 1;
    if (c->n_buckets == 0) return SO_OK;
    cudaError_t e = cudaSuccess;
    if (!c->dry_run) {
        ReduceArgs r;
        r.partials = c->d_partials;
        r.seg = c->d_seg;
        r.stats = c->d_stats;
        r.status = &c->d_ctrl->status;
        r.blocks_done = &c->d_ctrl->blocks_done;
        int64_t active = 0;
        for (int32_t b = 0; b < c->n_buckets; ++b)
            active += ((elems_of(c, b) + kTileElems - 1) / kTileElems + kSegTiles - 1) / kSegTiles;
        r.n_active_blocks = (uint32_t)active;
        r.tab = tables_of(c);
        r.max_grad_norm = max_grad_norm;
        r.decide = decide ? 1 : 0;
        r.seq = c->reduce_seq;
        r.geo = geometry_of(c);
        r.segs_per_slot = (uint32_t)c->segs_per_slot;
        r.n_buckets = c->n_buckets;
        const int64_t blocks = (int64_t)c->n_buckets * c->segs_per_slot;
        e = launch_dependent(bucket_reduce_kernel, (unsigned)blocks, kReduceThreads, 0, stream, r);
    }
    return after_launch(c, e);
}

// Send the verdict of the latest reduction to the host with a kernel of its
// own (used when no step kernel is there to carry it).
so_status publish_to_host(so_ctx *c, cudaStream_t stream)
{
    if (c->dry_run || c->n_buckets == 0) return SO_OK;
    cudaError_t e = cudaSuccess;
    c->pend_wait_stream = stream;
    if (c->h_verdict_dev) {
        e = launch_dependent(publish_to_host_kernel, 1u, 32u, 0, stream,
                             static_cast<const Verdict *>(c->d_verdict), c->h_verdict_dev);
        return after_launch(c, e);
    }
    e = cudaMemcpyAsync(c->h_verdict, c->d_verdict, sizeof(Verdict), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess && !c->reduce_done)
        e = cudaEventCreateWithFlags(&c->reduce_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventRecord(c->reduce_done, stream);
    return e == cudaSuccess ? SO_OK : cuda_fail(c, e);
}

// The verdict from statistics the host holds (after so_grad_check(SO_ALL), or
// global ones from so_set_global_grad_stats), applied on the device.
so_status launch_verdict(so_ctx *c, const Verdict &v, double max_grad_norm, cudaStream_t stream)
{
    if (c->n_buckets == 0) return SO_OK;
    cudaError_t e = cudaSuccess;
    if (!c->dry_run) {
        VerdictArgs a;
        a.tab = tables_of(c);
        a.sumsq = v.sumsq;
        a.max_grad_norm = max_grad_norm;
        a.nonfinite = v.nonfinite;
        a.abandon = v.decision == kDecisionAbandon ? 1 : 0;
        a.seq = v.seq;
        a.n_buckets = c->n_buckets;
        e = launch_dependent(apply_verdict_kernel, 1u, kReduceThreads, 0, stream, a);
    }
    return after_launch(c, e);
}

// What is enqueued behind a verdict; the kernels read on the device what there
// is to do.  After a skip the low-precision copy of the speculated buckets is
// derived again (a light kernel that returns at once otherwise).  The step
// kernel is launched only when the verdict can call for it: buckets that were
// merely checked take their step in place after a commit or a clip, and with
// clipping enabled a clip re-steps every bucket.
so_status launch_follow_up(so_ctx *c, const so_hparams &hp, cudaStream_t stream)
{
    std::vector<BucketEntry> all;
    std::vector<int32_t> speculated;
    all.reserve((size_t)c->n_buckets);
    for (int32_t b = 0; b < c->n_buckets; ++b) {
        const bool spec = c->cur.cover[b] == kSpeculated;
        all.push_back(BucketEntry{b, spec ? c->cur.free_idx[b] : -1});
        if (spec) speculated.push_back(b);
    }
    if (!speculated.empty()) {
        const so_status s = launch_casts(c, speculated, stream, /*only_after_skip=*/true);
        if (s != SO_OK) return s;
    }
    const bool may_step = speculated.size() < all.size() || hp.max_grad_norm > 0.0;
    if (all.empty() || !may_step) return SO_OK;
    return launch_steps(c, all, hp, /*speculative=*/false, stream);
}

// ---- validation ------------------------------------------------------------

// Have the records of the latest reduction reached the host?  Never blocks.
bool reduction_arrived(so_ctx *c)
{
    if (c->dry_run || c->n_buckets == 0) return true;
    if (c->h_verdict_dev) {
        const volatile int32_t *stamp = &host_verdict_of(c)->seq;
        return *stamp == c->reduce_seq;
    }
    return cudaEventQuery(c->reduce_done) == cudaSuccess;
}

// Wait (bounded spinning on the stamp, then a stream synchronisation that also
// surfaces any error) until the latest reduction's records are in host memory.
so_status wait_for_reduction(so_ctx *c, cudaStream_t stream)
{
    if (c->dry_run || c->n_buckets == 0) return SO_OK;
    cudaError_t e = cudaSuccess;
    if (c->h_verdict_dev) {
        // The verdict arrives in mapped host memory; watching for the stamp
        // that follows them is several microseconds quicker than waiting for
        // the stream's completion to be signalled.
        const auto t0 = std::chrono::steady_clock::now();
        bool arrived = false;
        for (uint32_t spins = 0;; ++spins) {
            if (reduction_arrived(c)) { arrived = true; break; }
            if ((spins & 0xFFFu) == 0xFFFu &&
                std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2))
                break;
        }
        std::atomic_thread_fence(std::memory_order_acquire);
        if (!arrived) {
            e = cudaStreamSynchronize(stream);
            if (e != cudaSuccess) return cuda_fail(c, e);
            if (!reduction_arrived(c)) return cuda_fail(c, cudaErrorUnknown);
        }
    } else {
        e = cudaStreamSynchronize(stream);
        if (e != cudaSuccess) return cuda_fail(c, e);
    }
    return SO_OK;
}

// Dry run: the records a device would have produced, from the injected values.
// `consume_status` false leaves the injected status word for a later call.
void inject_records(so_ctx *c, double max_grad_norm, bool decide, bool consume_status)
{
    double sumsq = 0.0;
    int flag = 0;
    for (int32_t b = 0; b < c->n_buckets; ++b) {
        sumsq += c->injected[b].sumsq;
        flag |= c->injected[b].nonfinite != 0;
    }
    Verdict v = verdict_of(sumsq, flag, c->injected_status, max_grad_norm, c->reduce_seq);
    if (!decide) v.decision = -1;
    if (consume_status) c->injected_status = 0;
    *host_verdict_of(c) = v;
}

so_status note_hparams(const IterRec &it, const so_hparams *hp)
{
    if (!hparams_ok(hp)) return SO_ERR_INVALID_ARG;
    if (it.have_hp && !hparams_equal(it.hp, *hp)) return SO_ERR_INVALID_ARG;
    return SO_OK;
}

void make_pending(so_ctx *c, const so_hparams &hp, cudaStream_t stream)
{
    if (!c->cur.have_hp) { c->cur.hp = hp; c->cur.have_hp = true; }
    std::swap(c->cur, c->pend);
    c->cur.reset();
    c->pending = true;
    c->pend_stream = stream;
}

// Enqueue the end of the open iteration: scan what is uncovered, reduce and
// decide on the device, follow up.  The iteration becomes the pending one.
// publish_now: the caller is about to wait for the verdict, so it is sent to the
// host straight behind the reduction, ahead of the follow-up launches (which can
// be the step of every bucket beyond the undo window): the host learns it
// without waiting for them.
so_status begin_validation(so_ctx *c, const so_hparams &hp, cudaStream_t stream, bool publish_now)
{
    so_status s = scan_uncovered(c, stream);
    if (s != SO_OK) return s;
    s = launch_reduce(c, hp.max_grad_norm, /*decide=*/true, stream);
    if (s != SO_OK) return s;
    if (publish_now && (s = publish_to_host(c, stream)) != SO_OK) return s;
    s = launch_follow_up(c, hp, stream);
    if (s != SO_OK) return s;
    make_pending(c, hp, stream);
    c->pend_known = false;
    // otherwise the next step launch carries it, or whoever asks first sends it
    c->pend_published = publish_now && !c->dry_run;
    return SO_OK;
}

// The same with a verdict the host already holds (the check has completed,
// possibly with global statistics handed in): the device applies it, nothing
// is waited for.
so_status begin_validation_known(so_ctx *c, const so_hparams &hp, const Verdict &v,
                                 cudaStream_t stream)
{
    so_status s = launch_verdict(c, v, hp.max_grad_norm, stream);
    if (s != SO_OK) return s;
    s = launch_follow_up(c, hp, stream);
    if (s != SO_OK) return s;
    make_pending(c, hp, stream);
    c->pend_known = true;
    c->pend_verdict = v;
    return SO_OK;
}

// The pending iteration's verdict, waiting for it if it is still on its way.
so_status pending_verdict(so_ctx *c, Verdict *v, bool consume_status)
{
    if (c->pend_known) {
        *v = c->pend_verdict;
        return SO_OK;
    }
    if (c->dry_run) {
        inject_records(c, c->pend.hp.max_grad_norm, /*decide=*/true, consume_status);
    } else {
        so_status s = SO_OK;
        if (!c->pend_published) {
            s = publish_to_host(c, c->pend_stream);
            if (s != SO_OK) return s;
            c->pend_published = true;
        }
        s = wait_for_reduction(c, c->pend_wait_stream);
        if (s != SO_OK) return s;
    }
    if (c->n_buckets > 0) std::memcpy(v, host_verdict_of(c), sizeof(*v));
    else *v = verdict_of(0.0, 0, 0, c->pend.hp.max_grad_norm, c->reduce_seq);
    return SO_OK;
}

// Learn the pending iteration's verdict and bring the host's books in line
// with what the device has done.
so_status collect_validation(so_ctx *c, so_step_result *out)
{
    Verdict v;
    const so_status got = pending_verdict(c, &v, /*consume_status=*/true);
    if (got != SO_OK) return got;
    const IterRec &it = c->pend;
    const int outcome = v.decision == kDecisionAbandon ? kAfterAbandoned
                        : v.decision == kDecisionSkip  ? kAfterSkipped
                                                       : kAfterKept;
    const bool clip = v.decision == kDecisionClip;
    for (int32_t b = 0; b < c->n_buckets; ++b) {
        const int64_t n = elems_of(c, b);
        if (it.cover[b] == kSpeculated) {
            if (outcome == kAfterKept) {
                std::swap(c->slot_of[b], c->free_slot[it.free_idx[b]]);
                if (clip) c->counters.elems_stepped += n;
            } else {
                c->counters.elems_cast += n;     // low-precision copy derived again from the old master
            }
        } else if (outcome == kAfterKept) {
            c->counters.elems_stepped += n;       // stepped in place with the validated scale
        }
    }
    c->prog = progress_after(c, outcome);
    if (outcome == kAfterKept) {
        if (clip) c->counters.clip_resteps += 1; else c->counters.commits += 1;
    } else if (outcome == kAfterSkipped) {
        c->counters.skips += 1;
    } else {
        c->counters.timeouts += 1;
    }
    c->stats.sumsq = v.sumsq;
    c->stats.norm = v.norm;
    c->stats.clip_coef = v.coef;
    c->stats.nonfinite = v.nonfinite;
    c->stats.reserved = 0;
    if (out && outcome != kAfterAbandoned) {
        out->decision = v.decision;
        out->buckets_speculated = it.n_speculated;
        out->step_after = c->prog.t;
        out->stats = c->stats;
        out->loss_scale = c->prog.loss_scale;
    }
    c->pending = false;
    c->pend_known = false;
    c->pend.reset();
    return outcome == kAfterAbandoned ? SO_ERR_TIMEOUT : SO_OK;
}

}  // namespace

namespace so {

cudaError_t launch_grad_check(const CheckArgs &a, int grad_dtype, unsigned grid, cudaStream_t stream)
{
    if (grad_dtype == SO_GRAD_BF16)
        return launch_dependent(grad_check_kernel<uint16_t>, grid, kThreads, 0, stream, a);
    if (grad_dtype == SO_GRAD_FP16)
        return launch_dependent(grad_check_kernel<half_t>, grid, kThreads, 0, stream, a);
    return launch_dependent(grad_check_kernel<float>, grid, kThreads, 0, stream, a);
}

cudaError_t grad_check_occupancy(int grad_dtype, int *blocks_per_sm)
{
    if (grad_dtype == SO_GRAD_BF16)
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, grad_check_kernel<uint16_t>,
                                                             kThreads, 0);
    if (grad_dtype == SO_GRAD_FP16)
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, grad_check_kernel<half_t>,
                                                             kThreads, 0);
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, grad_check_kernel<float>,
                                                         kThreads, 0);
}

}  // namespace so

// ============================================================================
// C ABI
// ============================================================================

// Scratch: tile sums | per-bucket records + verdict | control block | segment
// sums | slot tables | tensor table of pack / unpack.
static uint64_t round256(uint64_t x) { return (x + 255u) / 256u * 256u; }

extern "C" {

so_status so_layout_init(so_ctx **out, int32_t n_tensors, const int64_t *numel,
                         int64_t bucket_elems, int32_t grad_dtype, int32_t undo_slots,
                         so_layout_info *info)
{
    if (!out || n_tensors < 0 || (n_tensors > 0 && !numel)) return SO_ERR_INVALID_ARG;
    if (bucket_elems < 1 || bucket_elems > ((int64_t)1 << 30)) return SO_ERR_INVALID_ARG;
    if (grad_dtype != SO_GRAD_BF16 && grad_dtype != SO_GRAD_FP32 && grad_dtype != SO_GRAD_FP16)
        return SO_ERR_INVALID_ARG;
    int64_t total = 0;
    for (int32_t i = 0; i < n_tensors; ++i) {
        if (numel[i] < 0 || numel[i] > ((int64_t)1 << 46)) return SO_ERR_INVALID_ARG;
        total += numel[i];
        if (total > ((int64_t)1 << 46)) return SO_ERR_INVALID_ARG;
    }
    const int64_t nb64 = (total + bucket_elems - 1) / bucket_elems;
    if (nb64 > (1 << 24)) return SO_ERR_INVALID_ARG;
    const int32_t nb = (int32_t)nb64;
    if (undo_slots == SO_ALL) undo_slots = nb;
    if (undo_slots < 0 || undo_slots > nb) return SO_ERR_INVALID_ARG;

    so_ctx *c = new (std::nothrow) so_ctx();
    if (!c) return SO_ERR_NOMEM;
    try {
        c->numel.assign(numel, numel + n_tensors);
        c->offsets.resize(n_tensors);
        int64_t off = 0;
        for (int32_t i = 0; i < n_tensors; ++i) { c->offsets[i] = off; off += numel[i]; }
        c->total = total;
        c->bucket_elems = bucket_elems;
        c->stride = (bucket_elems + 63) / 64 * 64;
        c->n_buckets = nb;
        c->last_elems = nb == 0 ? 0 : total - (int64_t)(nb - 1) * bucket_elems;
        c->tiles_per_slot = (c->stride + kTileElems - 1) / kTileElems;
        c->undo_slots = undo_slots;
        c->n_slots = nb + undo_slots;
        c->grad_dtype = grad_dtype;
        c->slot_of.resize(nb);
        for (int32_t b = 0; b < nb; ++b) c->slot_of[b] = b;
        c->free_slot.resize(undo_slots);
        for (int32_t j = 0; j < undo_slots; ++j) c->free_slot[j] = nb + j;
        for (IterRec *it : {&c->cur, &c->pend}) {
            it->cover.assign(nb, (uint8_t)kNone);
            it->free_idx.assign(nb, -1);
        }
        c->injected.assign(nb, BucketStats{0.0, 0, 0});
    } catch (...) {
        delete c;
        return SO_ERR_NOMEM;
    }
    *out = c;
    if (info) so_layout_get_info(c, info);
    return SO_OK;
}

so_status so_layout_get_info(const so_ctx *c, so_layout_info *info)
{
    if (!c || !info) return SO_ERR_INVALID_ARG;
    std::memset(info, 0, sizeof(*info));
    info->total_elems = c->total;
    info->bucket_elems = c->bucket_elems;
    info->slot_stride_elems = c->stride;
    info->last_bucket_elems = c->last_elems;
    info->n_buckets = c->n_buckets;
    info->n_tensors = (int32_t)c->numel.size();
    info->n_state_slots = c->n_slots;
    info->undo_slots = c->undo_slots;
    info->grad_dtype = c->grad_dtype;
    info->tile_elems = kTileElems;
    info->tiles_per_slot = c->tiles_per_slot;
    const uint64_t state = (uint64_t)c->n_slots * (uint64_t)c->stride * 4u;
    info->bytes_master = info->bytes_m = info->bytes_v = state;
    info->bytes_grad = (uint64_t)c->n_buckets * (uint64_t)c->stride *
                       (c->grad_dtype == SO_GRAD_FP32 ? 4u : 2u);
    info->bytes_param_bf16 = (uint64_t)c->n_buckets * (uint64_t)c->stride * 2u;
    const uint64_t nb = (uint64_t)c->n_buckets;
    uint64_t segs = (uint64_t)((c->tiles_per_slot + kSegTiles - 1) / kSegTiles);
    if (segs < 1) segs = 1;
    info->bytes_scratch = round256(nb * (uint64_t)c->tiles_per_slot * 8u) +
                          round256(nb * sizeof(BucketStats) + sizeof(Verdict)) +
                          round256(sizeof(ControlBlock)) +
                          round256(nb * segs * sizeof(SegSum)) +
                          round256((2u * nb + (uint64_t)c->undo_slots) * 4u) +
                          round256((uint64_t)c->numel.size() * sizeof(PackTensor)) + 256u;
    return SO_OK;
}

so_status so_layout_tensor(const so_ctx *c, int32_t i, int64_t *flat_offset,
                           int32_t *first_bucket, int32_t *last_bucket)
{
    if (!c || i < 0 || i >= (int32_t)c->numel.size()) return SO_ERR_INVALID_ARG;
    const int64_t off = c->offsets[i], n = c->numel[i];
    if (flat_offset) *flat_offset = off;
    const int32_t fb = (int32_t)(off / c->bucket_elems);
    const int32_t lb = n > 0 ? (int32_t)((off + n - 1) / c->bucket_elems) : fb - 1;
    if (first_bucket) *first_bucket = fb;
    if (last_bucket) *last_bucket = lb;
    return SO_OK;
}

so_status so_layout_bind(so_ctx *c, void *master, void *m, void *v, void *grad,
                         void *param_bf16, void *scratch)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    void *ptrs[] = {master, m, v, grad, param_bf16, scratch};
    for (void *p : ptrs) {
        if (c->n_buckets > 0 && !p) return SO_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(p) & 255u) != 0) return SO_ERR_INVALID_ARG;
    }
    if (!c->dry_run) {
        cudaError_t e = cudaGetDevice(&c->device);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device);
        if (e != cudaSuccess) return cuda_fail(c, e);
        const int dt = c->grad_dtype;
        e = dt == SO_GRAD_BF16
                ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                      &c->occ_step, adamw_step_kernel<uint16_t, true, 2>, kThreads, 0)
            : dt == SO_GRAD_FP16
                ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                      &c->occ_step, adamw_step_kernel<half_t, true, 2>, kThreads, 0)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                      &c->occ_step, adamw_step_kernel<float, true, 2>, kThreads, 0);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = grad_check_occupancy(dt, &c->occ_check);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_cast, cast_params_kernel,
                                                          kThreads, 0);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = allow_smem<uint16_t, ShapeBf16>();
        if (e == cudaSuccess) e = allow_smem<half_t, ShapeBf16>();
        if (e == cudaSuccess) e = allow_smem<float, ShapeFp32>();
        // The small kernels that run between step kernels ask for the same
        // shared-memory / L1 split as those: an SM does not have to be drained
        // and reconfigured every time one follows the other.
        const auto same_split = [&](const void *kernel) {
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         cudaSharedmemCarveoutMaxShared);
        };
        same_split(reinterpret_cast<const void *>(bucket_reduce_kernel));
        same_split(reinterpret_cast<const void *>(apply_verdict_kernel));
        same_split(reinterpret_cast<const void *>(publish_to_host_kernel));
        same_split(reinterpret_cast<const void *>(cast_params_kernel));
        same_split(reinterpret_cast<const void *>(grad_check_kernel<uint16_t>));
        same_split(reinterpret_cast<const void *>(grad_check_kernel<half_t>));
        same_split(reinterpret_cast<const void *>(grad_check_kernel<float>));
        if (e != cudaSuccess) return cuda_fail(c, e);
    } else {
        c->num_sms = 148;
        c->occ_step = c->occ_check = c->occ_cast = 2;
    }
    if (!c->h_verdict) {
        if (!c->dry_run && cudaHostAlloc(reinterpret_cast<void **>(&c->h_verdict), sizeof(Verdict),
                                         cudaHostAllocMapped) == cudaSuccess) {
            c->h_verdict_pinned = true;
            std::memset(c->h_verdict, 0, sizeof(Verdict));
            void *dev_view = nullptr;
            if (cudaHostGetDevicePointer(&dev_view, c->h_verdict, 0) == cudaSuccess)
                c->h_verdict_dev = static_cast<Verdict *>(dev_view);
            else
                cudaGetLastError();                   // fall back to an explicit copy
        } else {
            if (!c->dry_run) cudaGetLastError();      // clear the failed pinned allocation
            c->h_verdict = static_cast<Verdict *>(std::calloc(1, sizeof(Verdict)));
            if (!c->h_verdict) return SO_ERR_NOMEM;
        }
    }
    c->master = static_cast<float *>(master);
    c->mom = static_cast<float *>(m);
    c->var = static_cast<float *>(v);
    c->grad = grad;
    c->param_lp = static_cast<uint16_t *>(param_bf16);
    // carve scratch up (the same arithmetic as so_layout_get_info)
    const uint64_t nb = (uint64_t)c->n_buckets;
    c->segs_per_slot = (c->tiles_per_slot + kSegTiles - 1) / kSegTiles;
    if (c->segs_per_slot < 1) c->segs_per_slot = 1;
    char *at = static_cast<char *>(scratch);
    c->d_partials = reinterpret_cast<double *>(at);
    at += round256(nb * (uint64_t)c->tiles_per_slot * 8u);
    c->d_stats = reinterpret_cast<BucketStats *>(at);
    c->d_verdict = reinterpret_cast<Verdict *>(c->d_stats + nb);
    at += round256(nb * sizeof(BucketStats) + sizeof(Verdict));
    c->d_ctrl = reinterpret_cast<ControlBlock *>(at);
    at += round256(sizeof(ControlBlock));
    c->d_seg = reinterpret_cast<SegSum *>(at);
    at += round256(nb * (uint64_t)c->segs_per_slot * sizeof(SegSum));
    c->d_slot_of = reinterpret_cast<int32_t *>(at);
    c->d_spec_idx = c->d_slot_of + nb;
    c->d_free_slot = c->d_spec_idx + nb;
    at += round256((2u * nb + (uint64_t)c->undo_slots) * 4u);
    c->d_tensors = reinterpret_cast<PackTensor *>(at);
    if (!c->dry_run && c->n_buckets > 0) {
        // the control block (status word, arrival counter) and the verdict start at zero,
        // the slot tables at the host's current map; the rest of scratch is
        // written before it is read.  (An empty model binds nothing and touches
        // no device memory.)
        cudaError_t e = cudaMemset(c->d_ctrl, 0, sizeof(ControlBlock));
        if (e == cudaSuccess) e = cudaMemset(c->d_verdict, 0, sizeof(Verdict));
        if (e == cudaSuccess) e = cudaMemset(c->d_spec_idx, 0xFF, sizeof(int32_t) * nb);
        if (e == cudaSuccess)
            e = cudaMemcpy(c->d_slot_of, c->slot_of.data(), sizeof(int32_t) * nb, cudaMemcpyHostToDevice);
        if (e == cudaSuccess && c->undo_slots > 0)
            e = cudaMemcpy(c->d_free_slot, c->free_slot.data(), sizeof(int32_t) * (size_t)c->undo_slots,
                           cudaMemcpyHostToDevice);
        if (e == cudaSuccess && !c->numel.empty()) {
            std::vector<PackTensor> table(c->numel.size());
            for (size_t i = 0; i < table.size(); ++i)
                table[i] = PackTensor{nullptr, c->offsets[i], c->numel[i]};
            e = cudaMemcpy(c->d_tensors, table.data(), sizeof(PackTensor) * table.size(),
                           cudaMemcpyHostToDevice);
        }
        if (e != cudaSuccess) return cuda_fail(c, e);
    }
    c->bound = true;
    return SO_OK;
}

so_status so_param_dtype_config(so_ctx *c, int32_t param_dtype)
{
    if (!c || (param_dtype != SO_PARAM_BF16 && param_dtype != SO_PARAM_FP16)) return SO_ERR_INVALID_ARG;
    if (c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    c->param_dtype = param_dtype;
    return SO_OK;
}

so_status so_grad_check(so_ctx *c, const so_hparams *hp, int32_t bucket, void *stream,
                        so_grad_stats *out)
{
    if (!c) return SO_ERR_INVALID_ARG;
    c->after_pipelined = false;     // the gradient arena is in use outside the host-fed pipeline
    if (!c->bound) return SO_ERR_STATE;
    if (c->cur.phase == kChecked) return SO_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bucket == SO_ALL) {
        if (c->pending) {
            // a validation has been enqueued: its statistics, as soon as they are in
            if (c->cur.phase != kIdle) return SO_ERR_STATE;
            so_status s = note_hparams(c->pend, hp);
            if (s != SO_OK) return s;
            Verdict v;
            s = pending_verdict(c, &v, /*consume_status=*/false);
            if (s != SO_OK) return s;
            if (out) {
                out->sumsq = v.sumsq;
                out->norm = v.norm;
                out->clip_coef = v.coef;
                out->nonfinite = v.nonfinite;
                out->reserved = 0;
            }
            return SO_OK;
        }
        so_status s = note_hparams(c->cur, hp);
        if (s != SO_OK) return s;
        s = scan_uncovered(c, st);
        if (s != SO_OK) return s;
        s = launch_reduce(c, hp->max_grad_norm, /*decide=*/false, st);
        if (s != SO_OK) return s;
        s = publish_to_host(c, st);
        if (s != SO_OK) return s;
        if (c->dry_run) inject_records(c, hp->max_grad_norm, false, true);
        else if ((s = wait_for_reduction(c, st)) != SO_OK) return s;
        Verdict v;
        if (c->n_buckets > 0) std::memcpy(&v, host_verdict_of(c), sizeof(v));
        else v = verdict_of(0.0, 0, 0, hp->max_grad_norm, 0);
        if (!c->cur.have_hp) { c->cur.hp = *hp; c->cur.have_hp = true; }
        if (v.status != 0) {
            // a kernel gave up waiting for one of its own copies: give the
            // iteration up (the device drops the speculative slots and derives
            // the low-precision copy of those buckets again)
            const Verdict gave_up = verdict_of(v.sumsq, v.nonfinite, v.status, hp->max_grad_norm, 0);
            s = begin_validation_known(c, *hp, gave_up, st);
            if (s != SO_OK) return s;
            return collect_validation(c, nullptr);
        }
        c->stats.sumsq = v.sumsq;
        c->stats.norm = std::sqrt(v.sumsq);
        c->stats.clip_coef = clip_coef_of(c->stats.norm, hp->max_grad_norm);
        c->stats.nonfinite = v.nonfinite;
        c->stats.reserved = 0;
        c->cur.phase = kChecked;
        if (out) *out = c->stats;
        return SO_OK;
    }
    if (bucket < 0 || bucket >= c->n_buckets) return SO_ERR_INVALID_ARG;
    if (c->cur.cover[bucket] != kNone) return SO_ERR_STATE;
    const so_status s = launch_checks(c, std::vector<int32_t>{bucket}, st);
    if (s != SO_OK) return s;
    c->cur.cover[bucket] = kCheckedOnly;
    c->cur.n_covered += 1;
    c->cur.phase = kOpen;
    return SO_OK;
}

so_status so_adam_step_speculative(so_ctx *c, const so_hparams *hp, int32_t bucket, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    c->after_pipelined = false;     // the gradient arena is in use outside the host-fed pipeline
    if (!c->bound) return SO_ERR_STATE;
    if (c->cur.phase == kChecked) return SO_ERR_STATE;
    so_status s = note_hparams(c->cur, hp);
    if (s != SO_OK) return s;
    if (bucket != SO_ALL && (bucket < 0 || bucket >= c->n_buckets)) return SO_ERR_INVALID_ARG;

    IterRec &it = c->cur;
    std::vector<BucketEntry> entries;
    int32_t next_free = it.n_speculated;
    if (bucket == SO_ALL) {
        for (int32_t b = 0; b < c->n_buckets && next_free < c->undo_slots; ++b)
            if (it.cover[b] == kNone) entries.push_back(BucketEntry{b, next_free++});
    } else {
        if (it.cover[bucket] != kNone) return SO_ERR_STATE;
        if (next_free >= c->undo_slots) return SO_ERR_UNDO_EXHAUSTED;
        entries.push_back(BucketEntry{bucket, next_free});
    }
    if (entries.empty()) return SO_OK;
    s = launch_steps(c, entries, *hp, /*speculative=*/true, static_cast<cudaStream_t>(stream));
    if (s != SO_OK) return s;
    for (const BucketEntry &e : entries) {
        it.free_idx[e.bucket] = e.free_idx;
        it.cover[e.bucket] = kSpeculated;
        c->counters.elems_stepped += elems_of(c, e.bucket);
    }
    it.n_covered += (int32_t)entries.size();
    it.n_speculated += (int32_t)entries.size();
    if (!it.have_hp) { it.hp = *hp; it.have_hp = true; }
    it.phase = kOpen;
    return SO_OK;
}

so_status so_validate_commit_or_rollback(so_ctx *c, const so_hparams *hp, void *stream,
                                         so_step_result *out)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (c->pending) {
        // a validation enqueued earlier (so_validate_begin): collect it; the
        // iteration that may have been opened since is not touched
        const so_status s = note_hparams(c->pend, hp);
        if (s != SO_OK) return s;
        return collect_validation(c, out);
    }
    so_status s = note_hparams(c->cur, hp);
    if (s != SO_OK) return s;
    if (c->cur.phase == kChecked) {
        // the check has completed on the host (possibly with global statistics)
        const Verdict v = verdict_of(c->stats.sumsq, c->stats.nonfinite, 0, hp->max_grad_norm, 0);
        s = begin_validation_known(c, *hp, v, st);
    } else {
        s = begin_validation(c, *hp, st, /*publish_now=*/true);
    }
    if (s != SO_OK) return s;
    return collect_validation(c, out);
}

so_status so_validate_begin(so_ctx *c, const so_hparams *hp, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    c->after_pipelined = false;     // the gradient arena is in use outside the host-fed pipeline
    if (!c->bound) return SO_ERR_STATE;
    if (c->pending || c->cur.phase == kChecked) return SO_ERR_STATE;
    const so_status s = note_hparams(c->cur, hp);
    if (s != SO_OK) return s;
    return begin_validation(c, *hp, static_cast<cudaStream_t>(stream), /*publish_now=*/false);
}

so_status so_abandon_iteration(so_ctx *c, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->pending) return SO_ERR_STATE;
    if (c->cur.phase == kIdle) return SO_OK;
    so_hparams hp = c->cur.hp;
    if (!c->cur.have_hp) {
        // only scans so far: any valid constants do, no step follows a give-up
        hp = so_hparams{0.0, 0.9, 0.999, 1e-8, 0.0, 0.0};
    }
    const Verdict gave_up = verdict_of(0.0, 0, 1, hp.max_grad_norm, 0);
    so_status s = begin_validation_known(c, hp, gave_up, static_cast<cudaStream_t>(stream));
    if (s != SO_OK) return s;
    s = collect_validation(c, nullptr);
    return s == SO_ERR_TIMEOUT ? SO_OK : s;
}

so_status so_set_global_grad_stats(so_ctx *c, double global_sumsq, int32_t global_nonfinite)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (c->cur.phase != kChecked) return SO_ERR_STATE;
    if (std::isnan(global_sumsq) ? false : global_sumsq < 0.0) return SO_ERR_INVALID_ARG;
    c->stats.sumsq = global_sumsq;
    c->stats.norm = std::sqrt(global_sumsq);
    c->stats.nonfinite = (global_nonfinite != 0 || !std::isfinite(global_sumsq)) ? 1 : 0;
    c->stats.clip_coef = clip_coef_of(c->stats.norm, c->cur.hp.max_grad_norm);
    return SO_OK;
}

so_status so_validate_poll(so_ctx *c, int32_t *ready)
{
    if (!c || !ready) return SO_ERR_INVALID_ARG;
    if (c->pending) {
        if (!c->pend_known && !c->pend_published && !c->dry_run) {
            const so_status s = publish_to_host(c, c->pend_stream);
            if (s != SO_OK) return s;
            c->pend_published = true;
        }
        *ready = (c->pend_known || reduction_arrived(c)) ? 1 : 0;
        return SO_OK;
    }
    if (c->cur.phase == kChecked) { *ready = 1; return SO_OK; }
    return SO_ERR_STATE;
}

so_status so_cast_params(so_ctx *c, int32_t bucket, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    if (bucket != SO_ALL && (bucket < 0 || bucket >= c->n_buckets)) return SO_ERR_INVALID_ARG;
    std::vector<int32_t> buckets;
    if (bucket == SO_ALL) {
        for (int32_t b = 0; b < c->n_buckets; ++b) buckets.push_back(b);
    } else {
        buckets.push_back(bucket);
    }
    if (buckets.empty()) return SO_OK;
    return launch_casts(c, buckets, static_cast<cudaStream_t>(stream));
}

static so_status iteration_host_body(so_ctx *c, const so_hparams *hp, const void *host_grad,
                                     void *host_param_bf16, void *stream, so_step_result *out,
                                     bool wait_at_end);

static so_status iteration_host_checked(so_ctx *c, const so_hparams *hp, const void *host_grad,
                                        void *host_param_bf16, void *stream, so_step_result *out,
                                        bool wait_at_end)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    if (!hparams_ok(hp) || (c->n_buckets > 0 && !host_grad)) return SO_ERR_INVALID_ARG;
    if (c->dry_run) return SO_ERR_UNSUPPORTED;
    const so_status s = iteration_host_body(c, hp, host_grad, host_param_bf16, stream, out, wait_at_end);
    if (s != SO_OK && c->copy_in) {
        // leave no copy in flight from or into the caller's buffers
        cudaStreamSynchronize(c->copy_in);
        cudaStreamSynchronize(c->copy_out);
        cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
        c->copies_in_flight = false;
        c->after_pipelined = false;
    }
    return s;
}

so_status so_iteration_host(so_ctx *c, const so_hparams *hp, const void *host_grad,
                            void *host_param_bf16, void *stream, so_step_result *out)
{
    return iteration_host_checked(c, hp, host_grad, host_param_bf16, stream, out, true);
}

so_status so_iteration_host_pipelined(so_ctx *c, const so_hparams *hp, const void *host_grad,
                                      void *host_param_bf16, void *stream, so_step_result *out)
{
    return iteration_host_checked(c, hp, host_grad, host_param_bf16, stream, out, false);
}

so_status so_iteration_host_wait(so_ctx *c, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->copies_in_flight && !c->after_pipelined) return SO_OK;
    cudaError_t e = c->copy_out ? cudaStreamSynchronize(c->copy_out) : cudaSuccess;
    if (e == cudaSuccess) e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    c->copies_in_flight = false;
    c->after_pipelined = false;
    return e == cudaSuccess ? SO_OK : cuda_fail(c, e);
}

static so_status iteration_host_body(so_ctx *c, const so_hparams *hp, const void *host_grad,
                                     void *host_param_bf16, void *stream, so_step_result *out,
                                     bool wait_at_end)
{
    cudaStream_t main = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (!c->copy_in) {
        e = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(c, e);
    }
    while ((int32_t)c->events.size() < 2 * c->n_buckets + 2) {
        cudaEvent_t ev;
        e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(c, e);
        c->events.push_back(ev);
    }
    const size_t gsz = c->grad_dtype == SO_GRAD_FP32 ? 4 : 2;
    const char *hg = static_cast<const char *>(host_grad);
    char *hp_out = static_cast<char *>(host_param_bf16);
    char *dgrad = static_cast<char *>(c->grad);
    cudaEvent_t start = c->events[2 * c->n_buckets];
    cudaEvent_t drained = c->events[2 * c->n_buckets + 1];

    // The incoming copies start after whatever the caller queued on `stream`
    // (which, after a pipelined call, ends with the kernels that read the
    // previous gradients).  The outgoing stream may still be sending the
    // previous call's parameters: this call's kernels overwrite the parameter
    // arena, so `stream` waits for that, while the incoming copies do not --
    // the previous parameters leave while the next gradients arrive.
    // Straight after another pipelined call the incoming copies wait for less:
    // that call returned with its verdict, so every kernel that ran before the
    // verdict is over, and a bucket whose gradient only those kernels read (a
    // speculated bucket of a committed iteration, every bucket of a skipped
    // one) can be overwritten at once; the others wait for the follow-up step
    // that still reads them, not for the whole stream.
    const bool early = c->after_pipelined;
    c->after_pipelined = false;
    e = cudaEventRecord(start, main);
    if (e != cudaSuccess) return cuda_fail(c, e);
    if (!early && (e = cudaStreamWaitEvent(c->copy_in, start, 0)) != cudaSuccess) return cuda_fail(c, e);
    if ((e = cudaStreamWaitEvent(c->copy_out, start, 0)) != cudaSuccess) return cuda_fail(c, e);
    bool waited_for_readers = !early;
    if (c->copies_in_flight) {
        if ((e = cudaEventRecord(drained, c->copy_out)) != cudaSuccess) return cuda_fail(c, e);
        if ((e = cudaStreamWaitEvent(main, drained, 0)) != cudaSuccess) return cuda_fail(c, e);
    }

    for (int32_t b = 0; b < c->n_buckets; ++b) {
        const size_t n = (size_t)elems_of(c, b);
        if (!waited_for_readers && !c->grad_done[b]) {
            if ((e = cudaStreamWaitEvent(c->copy_in, c->grads_read, 0)) != cudaSuccess) return cuda_fail(c, e);
            waited_for_readers = true;
        }
        e = cudaMemcpyAsync(dgrad + (size_t)b * (size_t)c->stride * gsz,
                            hg + (size_t)b * (size_t)c->bucket_elems * gsz, n * gsz,
                            cudaMemcpyHostToDevice, c->copy_in);
        if (e != cudaSuccess) return cuda_fail(c, e);
        if ((e = cudaEventRecord(c->events[2 * b], c->copy_in)) != cudaSuccess) return cuda_fail(c, e);
        if ((e = cudaStreamWaitEvent(main, c->events[2 * b], 0)) != cudaSuccess) return cuda_fail(c, e);
        so_status s;
        bool speculated = false;
        if (c->cur.n_speculated < c->undo_slots) {
            s = so_adam_step_speculative(c, hp, b, stream);
            speculated = true;
        } else {
            s = so_grad_check(c, hp, b, stream, nullptr);
        }
        if (s != SO_OK) return s;
        if (speculated && hp_out) {
            if ((e = cudaEventRecord(c->events[2 * b + 1], main)) != cudaSuccess) return cuda_fail(c, e);
            if ((e = cudaStreamWaitEvent(c->copy_out, c->events[2 * b + 1], 0)) != cudaSuccess) return cuda_fail(c, e);
            e = cudaMemcpyAsync(hp_out + (size_t)b * (size_t)c->bucket_elems * 2,
                                c->param_lp + (size_t)b * (size_t)c->stride, n * 2,
                                cudaMemcpyDeviceToHost, c->copy_out);
            if (e != cudaSuccess) return cuda_fail(c, e);
            c->copies_in_flight = true;
        }
    }
    std::vector<uint8_t> was_speculated(c->cur.cover.begin(), c->cur.cover.end());
    so_step_result res;
    so_status s = so_validate_commit_or_rollback(c, hp, stream, &res);
    if (s != SO_OK) return s;
    if (hp_out) {
        // whatever validation (re)wrote after the speculative copies went out
        if ((e = cudaEventRecord(start, main)) != cudaSuccess) return cuda_fail(c, e);
        if ((e = cudaStreamWaitEvent(c->copy_out, start, 0)) != cudaSuccess) return cuda_fail(c, e);
        for (int32_t b = 0; b < c->n_buckets; ++b) {
            const bool sent = was_speculated[b] == kSpeculated;
            if (sent && res.decision == SO_DECISION_COMMIT) continue;
            if (!sent && res.decision == SO_DECISION_SKIP) continue;   // never changed
            const size_t n = (size_t)elems_of(c, b);
            e = cudaMemcpyAsync(hp_out + (size_t)b * (size_t)c->bucket_elems * 2,
                                c->param_lp + (size_t)b * (size_t)c->stride, n * 2,
                                cudaMemcpyDeviceToHost, c->copy_out);
            if (e != cudaSuccess) return cuda_fail(c, e);
            c->copies_in_flight = true;
        }
    }
    if (wait_at_end) {
        e = cudaStreamSynchronize(c->copy_out);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = cudaStreamSynchronize(main);
        if (e != cudaSuccess) return cuda_fail(c, e);
        c->copies_in_flight = false;
    } else {
        // what the next pipelined call may overwrite without waiting
        if (!c->grads_read) {
            e = cudaEventCreateWithFlags(&c->grads_read, cudaEventDisableTiming);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
        if ((e = cudaEventRecord(c->grads_read, main)) != cudaSuccess) return cuda_fail(c, e);
        c->grad_done.assign((size_t)c->n_buckets, 0);
        for (int32_t b = 0; b < c->n_buckets; ++b) {
            const bool speculated = was_speculated[b] == kSpeculated;
            c->grad_done[b] = res.decision == SO_DECISION_SKIP ||
                              (res.decision == SO_DECISION_COMMIT && speculated);
        }
        c->after_pipelined = true;
    }
    if (out) *out = res;
    return SO_OK;
}

so_status so_loss_scale_config(so_ctx *c, double init_scale, double growth, double backoff,
                               int64_t interval)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    if (c->grad_dtype != SO_GRAD_FP16) return SO_ERR_UNSUPPORTED;
    if (!(init_scale > 0.0) || !std::isfinite(init_scale) || interval < 0) return SO_ERR_INVALID_ARG;
    if (interval > 0 && (!(growth >= 1.0) || !std::isfinite(growth) || !(backoff > 0.0) ||
                         !(backoff <= 1.0)))
        return SO_ERR_INVALID_ARG;
    c->prog.loss_scale = init_scale;
    c->ls_growth = growth;
    c->ls_backoff = backoff;
    c->ls_interval = interval;
    c->prog.good_steps = 0;
    return SO_OK;
}

so_status so_get_loss_scale(const so_ctx *c, double *scale)
{
    if (!c || !scale) return SO_ERR_INVALID_ARG;
    *scale = c->prog.loss_scale;
    return SO_OK;
}

}  // extern "C"

namespace {

// Copy the committed fp32 state between the slot arenas and flat arrays in
// parameter order, one asynchronous copy per bucket and array.
so_status copy_state(so_ctx *c, void *flat[3], bool to_flat, cudaStream_t stream)
{
    float *arenas[3] = {c->master, c->mom, c->var};
    for (int32_t b = 0; b < c->n_buckets; ++b) {
        const size_t n = (size_t)elems_of(c, b);
        const size_t flat_off = (size_t)b * (size_t)c->bucket_elems;
        const size_t slot_off = (size_t)c->slot_of[b] * (size_t)c->stride;
        for (int k = 0; k < 3; ++k) {
            if (!flat[k]) continue;
            float *in_arena = arenas[k] + slot_off;
            float *in_flat = static_cast<float *>(flat[k]) + flat_off;
            const cudaError_t e = cudaMemcpyAsync(to_flat ? in_flat : in_arena,
                                                  to_flat ? in_arena : in_flat, n * sizeof(float),
                                                  cudaMemcpyDefault, stream);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
    }
    return SO_OK;
}

// One launch that moves every tensor of the list between its own buffer and
// the bucket arena (see so_pack.cuh).  The pointer list goes through a pinned
// staging buffer so that the upload is asynchronous.
so_status pack_or_unpack(so_ctx *c, const void *const *tensor_ptrs, bool pack, cudaStream_t stream)
{
    const size_t nt = c->numel.size();
    if (nt == 0 || c->total == 0) return SO_OK;
    if (!tensor_ptrs) return SO_ERR_INVALID_ARG;
    const size_t esz = pack ? (c->grad_dtype == SO_GRAD_FP32 ? 4u : 2u) : 2u;
    for (size_t i = 0; i < nt; ++i) {
        if (c->numel[i] > 0 && !tensor_ptrs[i]) return SO_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(tensor_ptrs[i]) & (esz - 1)) != 0) return SO_ERR_INVALID_ARG;
    }
    cudaError_t e = cudaSuccess;
    if (!c->dry_run) {
        if (!c->h_ptr_stage) {
            e = cudaHostAlloc(reinterpret_cast<void **>(&c->h_ptr_stage), nt * sizeof(uint64_t),
                              cudaHostAllocDefault);
            if (e != cudaSuccess) {
                c->h_ptr_stage = nullptr;
                return cuda_fail(c, e);
            }
            e = cudaEventCreateWithFlags(&c->ptrs_uploaded, cudaEventDisableTiming);
            if (e != cudaSuccess) {             // all or nothing: the next call starts over
                cudaFreeHost(c->h_ptr_stage);
                c->h_ptr_stage = nullptr;
                c->ptrs_uploaded = nullptr;
                return cuda_fail(c, e);
            }
        } else {
            // the staging buffer may still feed the previous call's upload
            // (only that copy is waited for, not the stream)
            e = cudaEventSynchronize(c->ptrs_uploaded);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
        for (size_t i = 0; i < nt; ++i) c->h_ptr_stage[i] = reinterpret_cast<uint64_t>(tensor_ptrs[i]);
        // the pointer is the first member of each table entry
        e = cudaMemcpy2DAsync(c->d_tensors, sizeof(PackTensor), c->h_ptr_stage, sizeof(uint64_t),
                              sizeof(uint64_t), nt, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaEventRecord(c->ptrs_uploaded, stream);
        if (e != cudaSuccess) return cuda_fail(c, e);
        PackArgs a;
        a.tensors = c->d_tensors;
        a.n_tensors = (int32_t)nt;
        a.arena = pack ? c->grad : static_cast<void *>(c->param_lp);
        a.total = c->total;
        a.bucket_elems = c->bucket_elems;
        a.stride = c->stride;
        const int64_t tiles = (c->total + kPackTileElems - 1) / kPackTileElems;
        const int64_t per_block = (int64_t)kWarpsPerBlock * kPackRunsPerWarp;
        const unsigned grid = (unsigned)((tiles + per_block - 1) / per_block);
        if (esz == 4) {
            if (pack) e = launch_dependent(pack_kernel<uint32_t, true>, grid, kThreads, 0, stream, a);
            else e = launch_dependent(pack_kernel<uint32_t, false>, grid, kThreads, 0, stream, a);
        } else {
            if (pack) e = launch_dependent(pack_kernel<uint16_t, true>, grid, kThreads, 0, stream, a);
            else e = launch_dependent(pack_kernel<uint16_t, false>, grid, kThreads, 0, stream, a);
        }
    }
    return after_launch(c, e);
}

}  // namespace

extern "C" {

so_status so_layout_pack_grads(so_ctx *c, const void *const *tensor_grads, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    if (c->cur.phase != kIdle) return SO_ERR_STATE;         // its gradients are in use
    c->after_pipelined = false;
    return pack_or_unpack(c, tensor_grads, /*pack=*/true, static_cast<cudaStream_t>(stream));
}

so_status so_layout_unpack_params(so_ctx *c, void *const *tensor_params, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    return pack_or_unpack(c, tensor_params, /*pack=*/false, static_cast<cudaStream_t>(stream));
}

so_status so_state_export(so_ctx *c, void *master, void *m, void *v, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    if (c->dry_run) return SO_ERR_UNSUPPORTED;
    void *flat[3] = {master, m, v};
    return copy_state(c, flat, /*to_flat=*/true, static_cast<cudaStream_t>(stream));
}

so_status so_state_import(so_ctx *c, const void *master, const void *m, const void *v,
                          void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    if (c->dry_run) return SO_ERR_UNSUPPORTED;
    void *flat[3] = {const_cast<void *>(master), const_cast<void *>(m), const_cast<void *>(v)};
    return copy_state(c, flat, /*to_flat=*/false, static_cast<cudaStream_t>(stream));
}

so_status so_bucket_slot(const so_ctx *c, int32_t bucket, int32_t *slot)
{
    if (!c || !slot || bucket < 0 || bucket >= c->n_buckets) return SO_ERR_INVALID_ARG;
    *slot = c->slot_of[bucket];
    return SO_OK;
}

so_status so_get_step(const so_ctx *c, int64_t *t)
{
    if (!c || !t) return SO_ERR_INVALID_ARG;
    *t = c->prog.t;
    return SO_OK;
}

so_status so_set_step(so_ctx *c, int64_t t)
{
    if (!c || t < 0) return SO_ERR_INVALID_ARG;
    if (c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    c->prog.t = t;
    return SO_OK;
}

so_status so_pending_buckets(const so_ctx *c, int32_t *n)
{
    if (!c || !n) return SO_ERR_INVALID_ARG;
    *n = c->n_buckets - c->cur.n_covered;
    return SO_OK;
}

so_status so_get_counters(const so_ctx *c, so_counters *out)
{
    if (!c || !out) return SO_ERR_INVALID_ARG;
    *out = c->counters;
    return SO_OK;
}

int32_t so_last_cuda_error(const so_ctx *c) { return c ? c->last_cuda_error : 0; }

const char *so_strerror(so_status s)
{
    switch (s) {
        case SO_OK: return "ok";
        case SO_ERR_INVALID_ARG: return "invalid argument";
        case SO_ERR_STATE: return "call not allowed in the current phase of the iteration";
        case SO_ERR_CUDA: return "CUDA error (see so_last_cuda_error)";
        case SO_ERR_UNDO_EXHAUSTED: return "no free slot for another speculative step";
        case SO_ERR_NOMEM: return "host allocation failed";
        case SO_ERR_UNSUPPORTED: return "unsupported";
        case SO_ERR_TIMEOUT: return "a kernel gave up waiting for one of its own copies";
        case SO_ERR_TOO_LARGE: return "input exceeds the fixed built-in capacity of this entry point";
        default: return "unknown status";
    }
}

void so_destroy(so_ctx *c)
{
    if (!c) return;
    for (cudaEvent_t ev : c->events) cudaEventDestroy(ev);
    if (c->reduce_done) cudaEventDestroy(c->reduce_done);
    if (c->grads_read) cudaEventDestroy(c->grads_read);
    if (c->ptrs_uploaded) cudaEventDestroy(c->ptrs_uploaded);
    if (c->copy_in) cudaStreamDestroy(c->copy_in);
    if (c->copy_out) cudaStreamDestroy(c->copy_out);
    if (c->h_ptr_stage) cudaFreeHost(c->h_ptr_stage);
    if (c->h_verdict) {
        if (c->h_verdict_pinned) cudaFreeHost(c->h_verdict);
        else std::free(c->h_verdict);
    }
    delete c;
}

so_status so_debug_set_dry_run(so_ctx *c, int32_t on)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (c->bound) return SO_ERR_STATE;
    c->dry_run = on != 0;
    return SO_OK;
}

so_status so_debug_set_step_variant(so_ctx *c, int32_t variant)
{
    if (!c || variant < 0 || variant > 2) return SO_ERR_INVALID_ARG;
    if (c->cur.phase != kIdle || c->pending) return SO_ERR_STATE;
    c->step_variant = variant;
    return SO_OK;
}

so_status so_debug_set_spin_limit(so_ctx *c, int64_t polls)
{
    if (!c || polls < 0 || polls > (int64_t)kSpinLimit) return SO_ERR_INVALID_ARG;
    c->spin_limit = (uint32_t)polls;
    return SO_OK;
}

so_status so_debug_set_bucket_stats(so_ctx *c, int32_t bucket, double sumsq, int32_t nonfinite)
{
    if (c && bucket == SO_ALL) {          // the device status word of the next check
        c->injected_status = nonfinite;
        return SO_OK;
    }
    if (!c || bucket < 0 || bucket >= c->n_buckets) return SO_ERR_INVALID_ARG;
    c->injected[bucket] = BucketStats{sumsq, nonfinite, 0};
    return SO_OK;
}

}  // extern "C"
