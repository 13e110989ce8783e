// Host side of the bucketized speculative AdamW library: layout arithmetic,
// the slot map, the per-iteration state machine, and the kernel launches.
// The C ABI is documented in include/superoffload.h.
#include "superoffload.h"

#include <cmath>
#include <cstdlib>
#include <chrono>
#include <cstring>
#include <atomic>
#include <new>
#include <vector>

#include "so_kernels.cuh"
#include "so_step_tma.cuh"

using namespace so;

namespace {

enum Phase { kIdle = 0, kOpen = 1, kReducing = 2, kChecked = 3 };
enum Cover : uint8_t { kNone = 0, kCheckedOnly = 1, kSpeculated = 2 };

}  // namespace

struct so_ctx {
    // ---- layout (immutable after init) ----
    std::vector<int64_t> numel, offsets;
    int64_t total = 0, bucket_elems = 0, stride = 0, last_elems = 0, tiles_per_slot = 0;
    int32_t n_buckets = 0, undo_slots = 0, n_slots = 0, grad_dtype = SO_GRAD_BF16;
    // ---- binding ----
    bool bound = false;
    int device = -1, num_sms = 0;
    float *master = nullptr, *mom = nullptr, *var = nullptr;
    void *grad = nullptr;
    uint16_t *param_bf16 = nullptr;
    double *d_partials = nullptr;
    BucketStats *d_stats = nullptr;     // n_buckets results, then one record whose first
                                        // word is the device status (0 = fine)
    ControlBlock *d_ctrl = nullptr;     // status word + tile counters, right after d_stats
    uint32_t launch_seq = 0;            // picks the counter pair of each pipeline launch
    int step_variant = 0;               // 0: bulk-copy pipeline, 1: register path
    BucketStats *h_stats = nullptr;
    BucketStats *h_stats_dev = nullptr; // device view of h_stats when it is mapped pinned memory
    bool h_stats_pinned = false;
    SegSum *d_seg = nullptr;            // per-bucket segment sums of the reduction
    uint32_t *d_arrivals = nullptr;     // per-bucket arrival counters of the reduction
    int64_t segs_per_slot = 1;
    int32_t reduce_seq = 0;             // stamp of the latest reduction (never 0)
    cudaStream_t reduce_stream = nullptr;   // stream the reduction in flight was launched on
    cudaEvent_t reduce_done = nullptr;  // completion of the copy-back when h_stats is not mapped
    int occ_step = 0, occ_check = 0, occ_cast = 0;
    // ---- slot map ----
    std::vector<int32_t> slot_of;       // committed slot of each bucket
    std::vector<int32_t> spec_slot;     // slot holding the speculative result, or -1
    std::vector<int32_t> free_slots;
    // ---- iteration state ----
    int phase = kIdle;
    std::vector<uint8_t> cover;
    int32_t n_covered = 0, n_speculated = 0;
    bool have_hp = false;
    so_hparams hp_iter{};
    so_grad_stats stats{};
    int64_t t = 0;
    // ---- loss scaling (fp16 gradients) ----
    double loss_scale = 1.0;            // stored gradient = loss_scale * gradient
    double ls_growth = 2.0, ls_backoff = 0.5;
    int64_t ls_interval = 0;            // clean iterations before growth; 0 = static scale
    int64_t ls_good_steps = 0;
    double iter_unscale = 1.0;          // 1 / loss_scale, fixed for the iteration in flight
    // ---- bookkeeping ----
    so_counters counters{};
    int32_t last_cuda_error = 0;
    bool dry_run = false;
    std::vector<BucketStats> injected;
    int32_t injected_status = 0;
    // ---- host-fed iteration: copy streams and ordering events (lazy) ----
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    std::vector<cudaEvent_t> events;
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

AdamScalars scalars_for(const so_hparams &hp, int64_t step_index, double scale, double unscale)
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
    k.scale = scale;
    k.unscale = unscale;
    return k;
}

double clip_coef_of(double norm, double max_norm)
{
    if (!(max_norm > 0.0)) return 1.0;
    const double c = max_norm / (norm + 1e-6);
    return c < 1.0 ? c : 1.0;
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

so_status after_launch(so_ctx *c)
{
    c->counters.kernel_launches += 1;
    if (c->dry_run) return SO_OK;
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SO_OK : cuda_fail(c, e);
}

// ---- launches --------------------------------------------------------------

// Shapes of the bulk-copy pipeline: rows per chunk, warps per block (one block
// per SM), input stages, output stages.  The defaults came out of a sweep on
// B200: 512-element chunks halve the per-chunk bookkeeping, two input stages of
// 7 KB per warp keep ~140 KB of loads in flight per SM, and ten warps are the
// most that fit in shared memory (nine with fp32 gradients).  The alternates
// stay selectable for measurements (so_debug_set_step_variant 10 / 11).
using ShapeBf16 = PipeShape<4, 10, 2, 1>;
using ShapeFp32 = PipeShape<4, 9, 2, 1>;
using ShapeAlt16 = PipeShape<2, 16, 3, 1>;      // bf16 gradients only
using ShapeAlt12 = PipeShape<2, 12, 3, 1>;

template <typename GradT, typename S>
void launch_tma(so_ctx *c, const StepArgs &a, int n, bool speculative, cudaStream_t stream)
{
    int64_t blocks = ((int64_t)n * a.geo.tiles_per_slot + S::kWarps - 1) / S::kWarps;
    if (blocks > c->num_sms) blocks = c->num_sms;
    const unsigned grid = (unsigned)(blocks < 1 ? 1 : blocks);
    // launches that may overlap in time (other streams) must not share a tile counter
    const int pair = (int)(c->launch_seq++ % kCounterPairs);
    const size_t sm = TmaLayout<GradT, S>::kSmemBytes;
    if (speculative)
        adamw_step_tma_kernel<GradT, true, S><<<grid, S::kThreads, sm, stream>>>(a, c->d_ctrl, pair);
    else
        adamw_step_tma_kernel<GradT, false, S><<<grid, S::kThreads, sm, stream>>>(a, c->d_ctrl, pair);
}

void launch_tma_variant(so_ctx *c, const StepArgs &a, int n, bool speculative, cudaStream_t stream)
{
    const int dt = c->grad_dtype;
    if (c->step_variant == 10 && dt == SO_GRAD_BF16) {
        launch_tma<uint16_t, ShapeAlt16>(c, a, n, speculative, stream);
    } else if (c->step_variant == 11 && dt != SO_GRAD_FP16) {
        if (dt == SO_GRAD_BF16) launch_tma<uint16_t, ShapeAlt12>(c, a, n, speculative, stream);
        else launch_tma<float, ShapeAlt12>(c, a, n, speculative, stream);
    } else {
        if (dt == SO_GRAD_BF16) launch_tma<uint16_t, ShapeBf16>(c, a, n, speculative, stream);
        else if (dt == SO_GRAD_FP16) launch_tma<half_t, ShapeBf16>(c, a, n, speculative, stream);
        else launch_tma<float, ShapeFp32>(c, a, n, speculative, stream);
    }
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

// Step the listed buckets (src slot -> dst slot).  speculative: scale 1 and
// tile sums written; otherwise the given scale and no sums.
so_status launch_steps(so_ctx *c, const std::vector<BucketEntry> &entries, const so_hparams &hp,
                       bool speculative, double scale, cudaStream_t stream)
{
    const Geometry geo = geometry_of(c);
    for (size_t first = 0; first < entries.size(); first += kMaxBatch) {
        const int n = (int)std::min<size_t>(kMaxBatch, entries.size() - first);
        StepArgs a;
        a.grad = c->grad;
        a.master = c->master;
        a.mom = c->mom;
        a.var = c->var;
        a.param_bf16 = c->param_bf16;
        a.partials = c->d_partials;
        a.geo = geo;
        a.k = scalars_for(hp, c->t + 1, scale, c->iter_unscale);
        a.n_entries = n;
        for (int i = 0; i < n; ++i) {
            a.e[i] = entries[first + i];
            c->counters.elems_stepped += elems_of(c, a.e[i].bucket);
        }
        for (int i = n; i < kMaxBatch; ++i) a.e[i] = BucketEntry{0, 0, 0};
        if (!c->dry_run) {
            const int dt = c->grad_dtype;
            const unsigned grid = grid_for(c, (int64_t)n * geo.tiles_per_slot, c->occ_step);
            if (c->step_variant != 1) {
                launch_tma_variant(c, a, n, speculative, stream);
            } else if (speculative) {
                if (dt == SO_GRAD_BF16) adamw_step_kernel<uint16_t, true, 2><<<grid, kThreads, 0, stream>>>(a);
                else if (dt == SO_GRAD_FP16) adamw_step_kernel<half_t, true, 2><<<grid, kThreads, 0, stream>>>(a);
                else adamw_step_kernel<float, true, 2><<<grid, kThreads, 0, stream>>>(a);
            } else {
                if (dt == SO_GRAD_BF16) adamw_step_kernel<uint16_t, false, 2><<<grid, kThreads, 0, stream>>>(a);
                else if (dt == SO_GRAD_FP16) adamw_step_kernel<half_t, false, 2><<<grid, kThreads, 0, stream>>>(a);
                else adamw_step_kernel<float, false, 2><<<grid, kThreads, 0, stream>>>(a);
            }
        }
        const so_status s = after_launch(c);
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
        a.unscale = c->iter_unscale;
        int exponent = 0;
        a.unscale_is_pow2 = std::frexp(a.unscale, &exponent) == 0.5 ? 1 : 0;
        a.geo = geo;
        a.n_entries = n;
        for (int i = 0; i < n; ++i) {
            a.bucket[i] = buckets[first + i];
            c->counters.elems_checked += elems_of(c, a.bucket[i]);
        }
        for (int i = n; i < kMaxBatch; ++i) a.bucket[i] = 0;
        if (!c->dry_run) {
            const unsigned grid = grid_for(c, (int64_t)n * geo.tiles_per_slot, c->occ_check);
            if (c->grad_dtype == SO_GRAD_BF16)
                grad_check_kernel<uint16_t><<<grid, kThreads, 0, stream>>>(a);
            else if (c->grad_dtype == SO_GRAD_FP16)
                grad_check_kernel<half_t><<<grid, kThreads, 0, stream>>>(a);
            else
                grad_check_kernel<float><<<grid, kThreads, 0, stream>>>(a);
        }
        const so_status s = after_launch(c);
        if (s != SO_OK) return s;
    }
    return SO_OK;
}

so_status launch_casts(so_ctx *c, const std::vector<BucketEntry> &entries, cudaStream_t stream)
{
    const Geometry geo = geometry_of(c);
    for (size_t first = 0; first < entries.size(); first += kMaxBatch) {
        const int n = (int)std::min<size_t>(kMaxBatch, entries.size() - first);
        CastArgs a;
        a.master = c->master;
        a.param_bf16 = c->param_bf16;
        a.geo = geo;
        a.n_entries = n;
        for (int i = 0; i < n; ++i) {
            a.e[i] = entries[first + i];
            c->counters.elems_cast += elems_of(c, a.e[i].bucket);
        }
        for (int i = n; i < kMaxBatch; ++i) a.e[i] = BucketEntry{0, 0, 0};
        if (!c->dry_run) {
            const unsigned grid = grid_for(c, (int64_t)n * geo.tiles_per_slot, c->occ_cast);
            cast_params_kernel<<<grid, kThreads, 0, stream>>>(a);
        }
        const so_status s = after_launch(c);
        if (s != SO_OK) return s;
    }
    return SO_OK;
}

// First half of finishing the gradient check: scan what is still uncovered and
// launch the per-bucket reduction, whose records travel to the host on their
// own.  Nothing here waits.
so_status begin_check(so_ctx *c, cudaStream_t stream)
{
    std::vector<int32_t> todo;
    for (int32_t b = 0; b < c->n_buckets; ++b)
        if (c->cover[b] == kNone) todo.push_back(b);
    if (!todo.empty()) {
        const so_status s = launch_checks(c, todo, stream);
        if (s != SO_OK) return s;
        for (int32_t b : todo) c->cover[b] = kCheckedOnly;
        c->n_covered = c->n_buckets;
    }
    c->reduce_stream = stream;
    if (c->n_buckets > 0) {
        if (!c->dry_run) {
            ReduceArgs r;
            r.partials = c->d_partials;
            r.seg = c->d_seg;
            r.arrivals = c->d_arrivals;
            r.stats = c->d_stats;
            r.host_stats = c->h_stats_dev;     // records land in host memory directly
            r.status = &c->d_ctrl->status;
            r.buckets_done = &c->d_ctrl->buckets_done;
            c->reduce_seq = c->reduce_seq == 0x7FFFFFFF ? 1 : c->reduce_seq + 1;
            r.seq = c->reduce_seq;
            r.geo = geometry_of(c);
            r.segs_per_slot = (uint32_t)c->segs_per_slot;
            r.n_buckets = c->n_buckets;
            const int64_t blocks = (int64_t)c->n_buckets * c->segs_per_slot;
            // Programmatic dependent launch: the reduction's blocks may be set up
            // while the step (or scan) kernel before it in the stream drains; they
            // wait for its completion and memory flush before reading anything.
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)blocks);
            cfg.blockDim = dim3(kReduceThreads);
            cfg.dynamicSmemBytes = 0;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            cudaLaunchKernelEx(&cfg, bucket_reduce_kernel, r);
        }
        const so_status s = after_launch(c);
        if (s != SO_OK) return s;
        if (!c->dry_run && !c->h_stats_dev) {
            cudaError_t e = cudaMemcpyAsync(c->h_stats, c->d_stats,
                                            sizeof(BucketStats) * (size_t)(c->n_buckets + 1),
                                            cudaMemcpyDeviceToHost, stream);
            if (e == cudaSuccess && !c->reduce_done)
                e = cudaEventCreateWithFlags(&c->reduce_done, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventRecord(c->reduce_done, stream);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
    }
    c->phase = kReducing;
    return SO_OK;
}

// Have the records of the reduction in flight reached the host?  Never blocks.
bool check_arrived(so_ctx *c)
{
    if (c->dry_run || c->n_buckets == 0) return true;
    if (c->h_stats_dev) {
        const volatile int32_t *stamp = &c->h_stats[c->n_buckets].pad;
        return *stamp == c->reduce_seq;
    }
    return cudaEventQuery(c->reduce_done) == cudaSuccess;
}

void end_iteration(so_ctx *c);

// A kernel of this iteration gave up waiting for one of its own copies: give
// the iteration up.  Speculative slots go back to the free list (the committed
// slots were never written), the bf16 copy of the speculated buckets - partly
// overwritten - is derived again from the committed master, and the context is
// idle again with step count and loss scale as they were.
so_status abandon_iteration(so_ctx *c)
{
    std::vector<BucketEntry> recast;
    for (int32_t b = 0; b < c->n_buckets; ++b)
        if (c->cover[b] == kSpeculated) {
            recast.push_back(BucketEntry{b, c->slot_of[b], 0});
            c->free_slots.push_back(c->spec_slot[b]);
        }
    if (!recast.empty()) launch_casts(c, recast, c->reduce_stream);   // best effort
    c->counters.timeouts += 1;
    end_iteration(c);
    return SO_ERR_TIMEOUT;
}

// Second half: wait for the per-bucket records to reach the host, fold over
// buckets in index order, derive norm and clip coefficient.
so_status finish_check(so_ctx *c, const so_hparams &hp)
{
    if (c->n_buckets > 0) {
        if (!c->dry_run) {
            cudaError_t e = cudaSuccess;
            if (c->h_stats_dev) {
                // The records arrive in mapped host memory; watching for the
                // stamp that follows them is several microseconds quicker than
                // waiting for the stream's completion to be signalled.  Bounded:
                // after two seconds fall back to a stream synchronisation, which
                // also surfaces any launch or execution error.
                const auto t0 = std::chrono::steady_clock::now();
                bool arrived = false;
                for (uint32_t spins = 0;; ++spins) {
                    if (check_arrived(c)) { arrived = true; break; }
                    if ((spins & 0xFFFu) == 0xFFFu &&
                        std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2))
                        break;
                }
                std::atomic_thread_fence(std::memory_order_acquire);
                if (!arrived) {
                    e = cudaStreamSynchronize(c->reduce_stream);
                    if (e != cudaSuccess) return cuda_fail(c, e);
                    if (!check_arrived(c)) return cuda_fail(c, cudaErrorUnknown);
                }
            } else {
                e = cudaStreamSynchronize(c->reduce_stream);
                if (e != cudaSuccess) return cuda_fail(c, e);
            }
            int32_t device_status = c->h_stats[c->n_buckets].nonfinite;
            if (!c->h_stats_dev)
                std::memcpy(&device_status, &c->h_stats[c->n_buckets], sizeof(device_status));
            if (device_status != 0) {
                // a kernel gave up waiting for one of its own copies; its tile
                // counters may be left mid-way, so re-arm the whole control block
                cudaMemsetAsync(c->d_ctrl, 0, sizeof(ControlBlock), c->reduce_stream);
                if (c->h_stats_dev) std::memset(&c->h_stats[c->n_buckets], 0, sizeof(BucketStats));
                return abandon_iteration(c);
            }
        } else {
            for (int32_t b = 0; b < c->n_buckets; ++b) c->h_stats[b] = c->injected[b];
            if (c->injected_status != 0) {
                c->injected_status = 0;
                return abandon_iteration(c);
            }
        }
    }
    double sumsq = 0.0;
    int32_t nonfinite = 0;
    for (int32_t b = 0; b < c->n_buckets; ++b) {
        sumsq += c->h_stats[b].sumsq;
        nonfinite |= (c->h_stats[b].nonfinite != 0);
    }
    c->stats.sumsq = sumsq;
    c->stats.norm = std::sqrt(sumsq);
    c->stats.clip_coef = clip_coef_of(c->stats.norm, hp.max_grad_norm);
    c->stats.nonfinite = nonfinite;
    c->stats.reserved = 0;
    c->phase = kChecked;
    return SO_OK;
}

so_status finalize_check(so_ctx *c, const so_hparams &hp, cudaStream_t stream)
{
    if (c->phase != kReducing) {
        const so_status s = begin_check(c, stream);
        if (s != SO_OK) return s;
    }
    return finish_check(c, hp);
}

void end_iteration(so_ctx *c)
{
    c->iter_unscale = 1.0 / c->loss_scale;
    std::fill(c->cover.begin(), c->cover.end(), (uint8_t)kNone);
    std::fill(c->spec_slot.begin(), c->spec_slot.end(), -1);
    c->n_covered = 0;
    c->n_speculated = 0;
    c->have_hp = false;
    c->phase = kIdle;
}

so_status note_hparams(so_ctx *c, const so_hparams *hp)
{
    if (!hparams_ok(hp)) return SO_ERR_INVALID_ARG;
    if (c->have_hp && !hparams_equal(c->hp_iter, *hp)) return SO_ERR_INVALID_ARG;
    return SO_OK;
}

}  // namespace

// ============================================================================
// C ABI
// ============================================================================

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
        c->spec_slot.assign(nb, -1);
        for (int32_t s = c->n_slots - 1; s >= nb; --s) c->free_slots.push_back(s);
        c->cover.assign(nb, (uint8_t)kNone);
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
    const uint64_t partial_bytes = (uint64_t)c->n_buckets * (uint64_t)c->tiles_per_slot * 8u;
    const uint64_t stats_bytes = (uint64_t)c->n_buckets * sizeof(BucketStats) + sizeof(ControlBlock);
    const uint64_t segs = (uint64_t)((c->tiles_per_slot + kSegTiles - 1) / kSegTiles);
    const uint64_t reduce_bytes = (uint64_t)c->n_buckets * (segs * sizeof(SegSum) + 4u);
    info->bytes_scratch = (partial_bytes + 255u) / 256u * 256u + stats_bytes + reduce_bytes + 512u;
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
    if (c->phase != kIdle) return SO_ERR_STATE;
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
        e = dt == SO_GRAD_BF16
                ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                      &c->occ_check, grad_check_kernel<uint16_t>, kThreads, 0)
            : dt == SO_GRAD_FP16
                ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                      &c->occ_check, grad_check_kernel<half_t>, kThreads, 0)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                      &c->occ_check, grad_check_kernel<float>, kThreads, 0);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c->occ_cast, cast_params_kernel,
                                                          kThreads, 0);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = allow_smem<uint16_t, ShapeBf16>();
        if (e == cudaSuccess) e = allow_smem<half_t, ShapeBf16>();
        if (e == cudaSuccess) e = allow_smem<float, ShapeFp32>();
        if (e == cudaSuccess) e = allow_smem<uint16_t, ShapeAlt16>();
        if (e == cudaSuccess) e = allow_smem<uint16_t, ShapeAlt12>();
        if (e == cudaSuccess) e = allow_smem<float, ShapeAlt12>();
        if (e != cudaSuccess) return cuda_fail(c, e);
    } else {
        c->num_sms = 148;
        c->occ_step = c->occ_check = c->occ_cast = 2;
    }
    if (!c->h_stats) {
        const size_t bytes = sizeof(BucketStats) * (size_t)(c->n_buckets + 1);
        if (!c->dry_run && cudaHostAlloc(reinterpret_cast<void **>(&c->h_stats), bytes,
                                         cudaHostAllocMapped) == cudaSuccess) {
            c->h_stats_pinned = true;
            std::memset(c->h_stats, 0, bytes);
            void *dev_view = nullptr;
            if (cudaHostGetDevicePointer(&dev_view, c->h_stats, 0) == cudaSuccess)
                c->h_stats_dev = static_cast<BucketStats *>(dev_view);
            else
                cudaGetLastError();                   // fall back to an explicit copy
        } else {
            if (!c->dry_run) cudaGetLastError();      // clear the failed pinned allocation
            c->h_stats = static_cast<BucketStats *>(std::malloc(bytes));
            if (!c->h_stats) return SO_ERR_NOMEM;
        }
    }
    c->master = static_cast<float *>(master);
    c->mom = static_cast<float *>(m);
    c->var = static_cast<float *>(v);
    c->grad = grad;
    c->param_bf16 = static_cast<uint16_t *>(param_bf16);
    c->d_partials = static_cast<double *>(scratch);
    const uint64_t partial_bytes = (uint64_t)c->n_buckets * (uint64_t)c->tiles_per_slot * 8u;
    c->d_stats = reinterpret_cast<BucketStats *>(static_cast<char *>(scratch) +
                                                 (partial_bytes + 255u) / 256u * 256u);
    c->d_ctrl = reinterpret_cast<ControlBlock *>(c->d_stats + c->n_buckets);
    c->segs_per_slot = (c->tiles_per_slot + kSegTiles - 1) / kSegTiles;
    if (c->segs_per_slot < 1) c->segs_per_slot = 1;
    c->d_seg = reinterpret_cast<SegSum *>(c->d_ctrl + 1);
    c->d_arrivals = reinterpret_cast<uint32_t *>(c->d_seg + (int64_t)c->n_buckets * c->segs_per_slot);
    if (!c->dry_run) {
        // the control block and the arrival counters must start at zero; the
        // rest of scratch is written before it is read
        cudaError_t e = cudaMemset(c->d_ctrl, 0, sizeof(ControlBlock));
        if (e == cudaSuccess && c->n_buckets > 0)
            e = cudaMemset(c->d_arrivals, 0, sizeof(uint32_t) * (size_t)c->n_buckets);
        if (e != cudaSuccess) return cuda_fail(c, e);
    }
    c->bound = true;
    return SO_OK;
}

so_status so_grad_check(so_ctx *c, const so_hparams *hp, int32_t bucket, void *stream,
                        so_grad_stats *out)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    if (c->phase == kChecked) return SO_ERR_STATE;
    if (c->phase == kReducing && bucket != SO_ALL) return SO_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (bucket == SO_ALL) {
        so_status s = note_hparams(c, hp);
        if (s != SO_OK) return s;
        s = finalize_check(c, *hp, st);
        if (s != SO_OK) return s;
        if (!c->have_hp) { c->hp_iter = *hp; c->have_hp = true; }
        if (out) *out = c->stats;
        return SO_OK;
    }
    if (bucket < 0 || bucket >= c->n_buckets) return SO_ERR_INVALID_ARG;
    if (c->cover[bucket] != kNone) return SO_ERR_STATE;
    const so_status s = launch_checks(c, std::vector<int32_t>{bucket}, st);
    if (s != SO_OK) return s;
    c->cover[bucket] = kCheckedOnly;
    c->n_covered += 1;
    c->phase = kOpen;
    return SO_OK;
}

so_status so_adam_step_speculative(so_ctx *c, const so_hparams *hp, int32_t bucket, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    if (c->phase == kChecked || c->phase == kReducing) return SO_ERR_STATE;
    so_status s = note_hparams(c, hp);
    if (s != SO_OK) return s;
    if (bucket != SO_ALL && (bucket < 0 || bucket >= c->n_buckets)) return SO_ERR_INVALID_ARG;

    std::vector<BucketEntry> entries;
    if (bucket == SO_ALL) {
        size_t free_left = c->free_slots.size();
        for (int32_t b = 0; b < c->n_buckets && free_left > 0; ++b)
            if (c->cover[b] == kNone) {
                entries.push_back(BucketEntry{b, c->slot_of[b], c->free_slots[free_left - 1]});
                --free_left;
            }
    } else {
        if (c->cover[bucket] != kNone) return SO_ERR_STATE;
        if (c->free_slots.empty()) return SO_ERR_UNDO_EXHAUSTED;
        entries.push_back(BucketEntry{bucket, c->slot_of[bucket], c->free_slots.back()});
    }
    if (entries.empty()) return SO_OK;
    s = launch_steps(c, entries, *hp, /*speculative=*/true, 1.0, static_cast<cudaStream_t>(stream));
    if (s != SO_OK) return s;
    for (const BucketEntry &e : entries) {
        c->free_slots.pop_back();
        c->spec_slot[e.bucket] = e.dst_slot;
        c->cover[e.bucket] = kSpeculated;
    }
    c->n_covered += (int32_t)entries.size();
    c->n_speculated += (int32_t)entries.size();
    if (!c->have_hp) { c->hp_iter = *hp; c->have_hp = true; }
    c->phase = kOpen;
    return SO_OK;
}

so_status so_validate_commit_or_rollback(so_ctx *c, const so_hparams *hp, void *stream,
                                         so_step_result *out)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    so_status s = note_hparams(c, hp);
    if (s != SO_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (c->phase != kChecked) {
        s = finalize_check(c, *hp, st);
        if (s != SO_OK) return s;
    }
    // the coefficient always follows the hyper-parameters given here
    c->stats.clip_coef = clip_coef_of(c->stats.norm, hp->max_grad_norm);

    int32_t decision;
    if (c->stats.nonfinite) decision = SO_DECISION_SKIP;
    else if (c->stats.clip_coef < 1.0) decision = SO_DECISION_CLIP_RESTEP;
    else decision = SO_DECISION_COMMIT;

    const int32_t n_spec = c->n_speculated;
    if (decision == SO_DECISION_SKIP) {
        // drop the speculative slots; the bf16 copy of those buckets was
        // overwritten by the speculative step and is re-derived from the old master
        std::vector<BucketEntry> recast;
        for (int32_t b = 0; b < c->n_buckets; ++b)
            if (c->cover[b] == kSpeculated) recast.push_back(BucketEntry{b, c->slot_of[b], 0});
        if (!recast.empty()) {
            s = launch_casts(c, recast, st);
            if (s != SO_OK) return s;
        }
        for (int32_t b = 0; b < c->n_buckets; ++b)
            if (c->cover[b] == kSpeculated) c->free_slots.push_back(c->spec_slot[b]);
        c->counters.skips += 1;
    } else {
        const bool clip = decision == SO_DECISION_CLIP_RESTEP;
        // buckets to (re-)step with the validated scale: all of them after a
        // clip, only the never-speculated ones after a commit
        std::vector<BucketEntry> work;
        for (int32_t b = 0; b < c->n_buckets; ++b) {
            if (c->cover[b] == kSpeculated) {
                if (clip) work.push_back(BucketEntry{b, c->slot_of[b], c->spec_slot[b]});
            } else {
                work.push_back(BucketEntry{b, c->slot_of[b], c->slot_of[b]});
            }
        }
        if (!work.empty()) {
            s = launch_steps(c, work, *hp, /*speculative=*/false,
                             clip ? c->stats.clip_coef : 1.0, st);
            if (s != SO_OK) return s;
        }
        for (int32_t b = 0; b < c->n_buckets; ++b)
            if (c->cover[b] == kSpeculated) {
                c->free_slots.push_back(c->slot_of[b]);
                c->slot_of[b] = c->spec_slot[b];
            }
        c->t += 1;
        if (clip) c->counters.clip_resteps += 1; else c->counters.commits += 1;
    }
    // dynamic loss scaling: back off after an overflow, grow after a run of
    // clean iterations (takes effect from the next iteration on)
    if (c->ls_interval > 0) {
        if (decision == SO_DECISION_SKIP) {
            c->loss_scale *= c->ls_backoff;
            c->ls_good_steps = 0;
        } else if (++c->ls_good_steps == c->ls_interval) {
            c->loss_scale *= c->ls_growth;
            c->ls_good_steps = 0;
        }
    }
    if (out) {
        out->decision = decision;
        out->buckets_speculated = n_spec;
        out->step_after = c->t;
        out->stats = c->stats;
        out->loss_scale = c->loss_scale;
    }
    end_iteration(c);
    return SO_OK;
}

so_status so_validate_begin(so_ctx *c, const so_hparams *hp, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound) return SO_ERR_STATE;
    if (c->phase == kChecked || c->phase == kReducing) return SO_ERR_STATE;
    so_status s = note_hparams(c, hp);
    if (s != SO_OK) return s;
    s = begin_check(c, static_cast<cudaStream_t>(stream));
    if (s != SO_OK) return s;
    if (!c->have_hp) { c->hp_iter = *hp; c->have_hp = true; }
    return SO_OK;
}

so_status so_set_global_grad_stats(so_ctx *c, double global_sumsq, int32_t global_nonfinite)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (c->phase != kChecked) return SO_ERR_STATE;
    if (std::isnan(global_sumsq) ? false : global_sumsq < 0.0) return SO_ERR_INVALID_ARG;
    c->stats.sumsq = global_sumsq;
    c->stats.norm = std::sqrt(global_sumsq);
    c->stats.nonfinite = (global_nonfinite != 0 || !std::isfinite(global_sumsq)) ? 1 : 0;
    c->stats.clip_coef = clip_coef_of(c->stats.norm, c->hp_iter.max_grad_norm);
    return SO_OK;
}

so_status so_validate_poll(so_ctx *c, int32_t *ready)
{
    if (!c || !ready) return SO_ERR_INVALID_ARG;
    if (c->phase == kChecked) { *ready = 1; return SO_OK; }
    if (c->phase != kReducing) return SO_ERR_STATE;
    *ready = check_arrived(c) ? 1 : 0;
    return SO_OK;
}

so_status so_cast_params(so_ctx *c, int32_t bucket, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->phase != kIdle) return SO_ERR_STATE;
    if (bucket != SO_ALL && (bucket < 0 || bucket >= c->n_buckets)) return SO_ERR_INVALID_ARG;
    std::vector<BucketEntry> entries;
    if (bucket == SO_ALL) {
        for (int32_t b = 0; b < c->n_buckets; ++b)
            entries.push_back(BucketEntry{b, c->slot_of[b], 0});
    } else {
        entries.push_back(BucketEntry{bucket, c->slot_of[bucket], 0});
    }
    if (entries.empty()) return SO_OK;
    return launch_casts(c, entries, static_cast<cudaStream_t>(stream));
}

static so_status iteration_host_body(so_ctx *c, const so_hparams *hp, const void *host_grad,
                                     void *host_param_bf16, void *stream, so_step_result *out);

so_status so_iteration_host(so_ctx *c, const so_hparams *hp, const void *host_grad,
                            void *host_param_bf16, void *stream, so_step_result *out)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->phase != kIdle) return SO_ERR_STATE;
    if (!hparams_ok(hp) || (c->n_buckets > 0 && !host_grad)) return SO_ERR_INVALID_ARG;
    if (c->dry_run) return SO_ERR_UNSUPPORTED;
    const so_status s = iteration_host_body(c, hp, host_grad, host_param_bf16, stream, out);
    if (s != SO_OK && c->copy_in) {
        // leave no copy in flight from or into the caller's buffers
        cudaStreamSynchronize(c->copy_in);
        cudaStreamSynchronize(c->copy_out);
        cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    }
    return s;
}

static so_status iteration_host_body(so_ctx *c, const so_hparams *hp, const void *host_grad,
                                     void *host_param_bf16, void *stream, so_step_result *out)
{
    cudaStream_t main = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (!c->copy_in) {
        e = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(c, e);
        e = cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(c, e);
    }
    while ((int32_t)c->events.size() < 2 * c->n_buckets + 1) {
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

    // the copy streams start after whatever the caller queued on `stream`
    e = cudaEventRecord(start, main);
    if (e != cudaSuccess) return cuda_fail(c, e);
    if ((e = cudaStreamWaitEvent(c->copy_in, start, 0)) != cudaSuccess) return cuda_fail(c, e);
    if ((e = cudaStreamWaitEvent(c->copy_out, start, 0)) != cudaSuccess) return cuda_fail(c, e);

    for (int32_t b = 0; b < c->n_buckets; ++b) {
        const size_t n = (size_t)elems_of(c, b);
        e = cudaMemcpyAsync(dgrad + (size_t)b * (size_t)c->stride * gsz,
                            hg + (size_t)b * (size_t)c->bucket_elems * gsz, n * gsz,
                            cudaMemcpyHostToDevice, c->copy_in);
        if (e != cudaSuccess) return cuda_fail(c, e);
        if ((e = cudaEventRecord(c->events[2 * b], c->copy_in)) != cudaSuccess) return cuda_fail(c, e);
        if ((e = cudaStreamWaitEvent(main, c->events[2 * b], 0)) != cudaSuccess) return cuda_fail(c, e);
        so_status s;
        bool speculated = false;
        if (!c->free_slots.empty()) {
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
                                c->param_bf16 + (size_t)b * (size_t)c->stride, n * 2,
                                cudaMemcpyDeviceToHost, c->copy_out);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
    }
    std::vector<uint8_t> was_speculated(c->cover.begin(), c->cover.end());
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
                                c->param_bf16 + (size_t)b * (size_t)c->stride, n * 2,
                                cudaMemcpyDeviceToHost, c->copy_out);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
    }
    e = cudaStreamSynchronize(c->copy_out);
    if (e != cudaSuccess) return cuda_fail(c, e);
    e = cudaStreamSynchronize(main);
    if (e != cudaSuccess) return cuda_fail(c, e);
    if (out) *out = res;
    return SO_OK;
}

so_status so_loss_scale_config(so_ctx *c, double init_scale, double growth, double backoff,
                               int64_t interval)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (c->phase != kIdle) return SO_ERR_STATE;
    if (c->grad_dtype != SO_GRAD_FP16) return SO_ERR_UNSUPPORTED;
    if (!(init_scale > 0.0) || !std::isfinite(init_scale) || interval < 0) return SO_ERR_INVALID_ARG;
    if (interval > 0 && (!(growth >= 1.0) || !std::isfinite(growth) || !(backoff > 0.0) ||
                         !(backoff <= 1.0)))
        return SO_ERR_INVALID_ARG;
    c->loss_scale = init_scale;
    c->ls_growth = growth;
    c->ls_backoff = backoff;
    c->ls_interval = interval;
    c->ls_good_steps = 0;
    c->iter_unscale = 1.0 / init_scale;
    return SO_OK;
}

so_status so_get_loss_scale(const so_ctx *c, double *scale)
{
    if (!c || !scale) return SO_ERR_INVALID_ARG;
    *scale = c->loss_scale;
    return SO_OK;
}

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

}  // namespace

so_status so_state_export(so_ctx *c, void *master, void *m, void *v, void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->phase != kIdle) return SO_ERR_STATE;
    if (c->dry_run) return SO_ERR_UNSUPPORTED;
    void *flat[3] = {master, m, v};
    return copy_state(c, flat, /*to_flat=*/true, static_cast<cudaStream_t>(stream));
}

so_status so_state_import(so_ctx *c, const void *master, const void *m, const void *v,
                          void *stream)
{
    if (!c) return SO_ERR_INVALID_ARG;
    if (!c->bound || c->phase != kIdle) return SO_ERR_STATE;
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
    *t = c->t;
    return SO_OK;
}

so_status so_set_step(so_ctx *c, int64_t t)
{
    if (!c || t < 0) return SO_ERR_INVALID_ARG;
    if (c->phase != kIdle) return SO_ERR_STATE;
    c->t = t;
    return SO_OK;
}

so_status so_pending_buckets(const so_ctx *c, int32_t *n)
{
    if (!c || !n) return SO_ERR_INVALID_ARG;
    *n = c->n_buckets - c->n_covered;
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
    if (c->copy_in) cudaStreamDestroy(c->copy_in);
    if (c->copy_out) cudaStreamDestroy(c->copy_out);
    if (c->h_stats) {
        if (c->h_stats_pinned) cudaFreeHost(c->h_stats);
        else std::free(c->h_stats);
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
    if (!c || (variant != 0 && variant != 1 && variant != 10 && variant != 11)) return SO_ERR_INVALID_ARG;
    if (c->phase != kIdle) return SO_ERR_STATE;
    c->step_variant = variant;
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
