/*
 * superoffload.h -- C ABI of the B200 bucketized speculative AdamW library.
 *
 * The library implements the optimizer hot path of SuperOffload (arXiv
 * 2509.21271) on one GPU: model states flattened into fixed-size buckets
 * (Section 4.3), a mixed-precision AdamW step that runs per bucket *before*
 * the global gradient check has finished (speculation-then-validation,
 * Section 4.4), the check itself (global L2 gradient norm + NaN/Inf flag),
 * commit or bit-exact rollback (Section 4.4, "in-place rollback" and its two
 * scenarios), and the fp32 -> bf16 parameter cast (Section 4.5).
 *
 * General conventions
 *   - Every function returns an so_status (0 = SO_OK, negative = error) and
 *     never throws, aborts or prints.  Argument and state errors are detected
 *     before anything is launched and leave the context untouched.
 *   - All DEVICE memory is allocated and owned by the caller, in the sizes
 *     so_layout_init reports; the library keeps host-side metadata only and
 *     so_destroy frees only that.  Device pointers must be 256-byte aligned.
 *   - `stream` arguments are cudaStream_t values passed as void* (NULL = the
 *     legacy default stream).  Calls that launch work enqueue it and return;
 *     only calls that fill a host struct from device results wait for the
 *     device (stated per function).  The library adds no dependencies
 *     between streams: when the per-bucket calls of an iteration go to several
 *     streams, the stream given to so_grad_check(SO_ALL) / so_validate_* must
 *     have been made to wait for the others (an event per stream), and the
 *     others must wait for it before the next iteration touches the buckets.
 *   - The device that is current when so_layout_bind is called must be current
 *     for every later call on that context.  A context is not thread-safe;
 *     separate contexts are independent.
 *   - Hyper-parameters are doubles so that host and device see one constant.
 *
 * Memory layout (what the caller allocates)
 *   The flat parameter space [0, N) is the concatenation of the tensors in the
 *   order given.  Bucket b covers flat [b*B, min((b+1)*B, N)).  Arenas are
 *   arrays of fixed-size *slots* of `slot_stride_elems` elements (B rounded up
 *   to a multiple of 64, so every slot starts 256-byte aligned); flat element
 *   i sits at position (i / B) * slot_stride_elems + (i % B) of the gradient
 *   and bf16-parameter arenas (identity when B is a multiple of 64).
 *   The fp32 state arenas (master, m, v) hold n_buckets + undo_slots slots:
 *   bucket b's committed state lives in slot so_bucket_slot(b) (initially b).
 *   A speculative step writes the new state of a bucket into a free slot and
 *   leaves the old one untouched; commit re-points the bucket at the new slot,
 *   rollback simply drops it.  Nothing is ever copied to undo a step.
 */
#ifndef SUPEROFFLOAD_H
#define SUPEROFFLOAD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct so_ctx so_ctx;          /* opaque, host-side, library-owned */
typedef int32_t so_status;

enum {
    SO_OK = 0,
    SO_ERR_INVALID_ARG = -1,           /* bad pointer, size, dtype, hyper-parameter  */
    SO_ERR_STATE = -2,                 /* call not allowed in the current step phase */
    SO_ERR_CUDA = -3,                  /* a CUDA call failed; see so_last_cuda_error */
    SO_ERR_UNDO_EXHAUSTED = -4,        /* no free slot for another speculative step  */
    SO_ERR_NOMEM = -5,                 /* host allocation failed                     */
    SO_ERR_UNSUPPORTED = -6,
    SO_ERR_TIMEOUT = -7,               /* a kernel's bounded wait on its own copies ran out */
    SO_ERR_TOO_LARGE = -8              /* input exceeds a fixed built-in capacity           */
};

enum { SO_GRAD_BF16 = 0, SO_GRAD_FP32 = 1, SO_GRAD_FP16 = 2 };
enum { SO_PARAM_BF16 = 0, SO_PARAM_FP16 = 1 };   /* dtype of the low-precision parameter copy */
enum { SO_DECISION_COMMIT = 0, SO_DECISION_SKIP = 1, SO_DECISION_CLIP_RESTEP = 2 };
#define SO_ALL (-1)

/* AdamW hyper-parameters.  max_grad_norm <= 0 disables clipping. */
typedef struct {
    double lr, beta1, beta2, eps, weight_decay, max_grad_norm;
} so_hparams;

typedef struct {
    int64_t total_elems;               /* N                                          */
    int64_t bucket_elems;              /* B                                          */
    int64_t slot_stride_elems;         /* B rounded up to a multiple of 64           */
    int64_t last_bucket_elems;         /* elements in the last bucket (0 if N == 0)  */
    int32_t n_buckets;                 /* ceil(N / B)                                */
    int32_t n_tensors;
    int32_t n_state_slots;             /* n_buckets + undo_slots                     */
    int32_t undo_slots;
    int32_t grad_dtype;
    int32_t tile_elems;                /* elements per reduction tile (1024)         */
    int64_t tiles_per_slot;
    uint64_t bytes_master, bytes_m, bytes_v;   /* n_state_slots * stride * 4 each    */
    uint64_t bytes_grad;               /* n_buckets * stride * (2 or 4)              */
    uint64_t bytes_param_bf16;         /* n_buckets * stride * 2                     */
    uint64_t bytes_scratch;            /* tile partial sums + per-bucket results     */
} so_layout_info;

typedef struct {
    double sumsq;                      /* sum over all gradients of g^2              */
    double norm;                       /* sqrt(sumsq)                                */
    double clip_coef;                  /* min(1, max_grad_norm / (norm + 1e-6))      */
    int32_t nonfinite;                 /* 1 if any gradient is NaN or +-Inf          */
    int32_t reserved;
} so_grad_stats;

typedef struct {
    int32_t decision;                  /* SO_DECISION_*                              */
    int32_t buckets_speculated;        /* buckets that had been stepped speculatively*/
    int64_t step_after;                /* committed step count after this call       */
    so_grad_stats stats;
    double loss_scale;                 /* loss scale in effect for the next iteration */
} so_step_result;

typedef struct {
    int64_t commits, skips, clip_resteps;      /* validated iterations by outcome    */
    int64_t kernel_launches;                   /* kernels this context has launched  */
    int64_t elems_stepped, elems_checked, elems_cast;  /* work done by those kernels; what a
                                                  verdict's follow-up launches did is added
                                                  when the host collects that verdict        */
    int64_t timeouts;                          /* iterations given up (SO_ERR_TIMEOUT, so_abandon_iteration) */
} so_counters;

/*
 * so_layout_init -- flatten a tensor list into fixed-size buckets
 * (Section 4.3: model states are divided into buckets, the unit of transfer,
 * of the optimizer step and of rollback).  Host-only integer arithmetic.
 *   out          receives a new context (caller frees it with so_destroy)
 *   n_tensors    number of tensors (>= 0); numel[i] >= 0 elements each (host)
 *   bucket_elems B, 1 <= B <= 2^30
 *   grad_dtype   SO_GRAD_BF16, SO_GRAD_FP32 or SO_GRAD_FP16 (dtype of the gradient arena)
 *   undo_slots   how many buckets may be stepped speculatively per iteration:
 *                0..n_buckets, or SO_ALL for n_buckets
 *   info         optional (host): filled with the sizes to allocate
 * Errors: SO_ERR_INVALID_ARG, SO_ERR_NOMEM.
 */
so_status so_layout_init(so_ctx **out, int32_t n_tensors, const int64_t *numel,
                         int64_t bucket_elems, int32_t grad_dtype, int32_t undo_slots,
                         so_layout_info *info);

/* Copy of the layout description.  Host-only. */
so_status so_layout_get_info(const so_ctx *ctx, so_layout_info *info);

/* Where tensor i lives: its flat offset and the first/last bucket it touches
 * (first > last for an empty tensor).  Host-only. */
so_status so_layout_tensor(const so_ctx *ctx, int32_t i, int64_t *flat_offset,
                           int32_t *first_bucket, int32_t *last_bucket);

/*
 * so_layout_bind -- hand the caller-owned DEVICE arenas to the context.
 * Sizes as reported by so_layout_init; pointers 256-byte aligned; master, m, v
 * are fp32, grad is bf16, fp16 or fp32 per grad_dtype, param_bf16 is the 2-byte
 * low-precision parameter copy (bf16, or binary16 after so_param_dtype_config).  The
 * caller fills master/m/v slot b with bucket b's initial state (m = v = 0 for
 * a fresh optimizer) and normally calls so_cast_params(SO_ALL) once.  Scratch
 * needs no initialisation by the caller (bind zeroes a small control block and
 * the reduction counters and uploads the slot tables, synchronously; with an
 * empty tensor list it touches no device memory and all pointers may be NULL).
 * Records the current device.
 */
so_status so_layout_bind(so_ctx *ctx, void *master, void *m, void *v, void *grad,
                         void *param_bf16, void *scratch);

/*
 * so_param_dtype_config -- dtype of the low-precision parameter copy (Section
 * 4.5 casts FP32 <-> FP16: the paper's runs keep FP16 parameters; bf16 is the
 * default here).  With SO_PARAM_FP16 the fused step and so_cast_params write
 * IEEE binary16, round to nearest even (values beyond 65504 + half an ulp
 * become infinities, subnormals are kept).  Only between iterations; call
 * so_cast_params(SO_ALL) afterwards to re-derive the copy.  Host-only.
 */
so_status so_param_dtype_config(so_ctx *ctx, int32_t param_dtype);

/*
 * so_layout_pack_grads / so_layout_unpack_params -- the device part of the
 * flattening (Section 4.3: model states are flattened into buckets).  One
 * kernel launch copies every tensor's gradient from its own buffer into the
 * gradient arena (pack), or every tensor's low-precision parameters from the
 * parameter arena back into its own buffer (unpack).
 *   tensor_grads / tensor_params   HOST array of n_tensors DEVICE pointers in
 *                the order given to so_layout_init, each to numel[i] elements
 *                of the gradient dtype (pack) or of 2 bytes (unpack), aligned
 *                to its element size; an empty tensor's pointer may be NULL.
 *                The array is read before the call returns.
 * Tensors may start at any element alignment and straddle buckets; interior
 * runs move as 128-bit accesses, ragged heads and tails element by element.
 * Pack only between iterations (SO_ERR_STATE once a bucket is covered); unpack
 * at any time, ordered on `stream` like any other work.  Enqueues only (the
 * pointer list is staged in one pinned buffer and one device table: a second
 * call on the same context first waits for the previous call's upload of the
 * list, a few microseconds of copy, and calls that go to different streams
 * must be ordered by the caller).
 */
so_status so_layout_pack_grads(so_ctx *ctx, const void *const *tensor_grads, void *stream);
so_status so_layout_unpack_params(so_ctx *ctx, void *const *tensor_params, void *stream);

/*
 * so_grad_check -- the global gradient check (Section 4.4: the global
 * gradient norm needed for clipping and the global NaN/Inf check).
 *   bucket >= 0 : enqueue the sum of squares + non-finite scan of that bucket's
 *                 gradients (a bucket that was stepped speculatively already
 *                 has them: SO_ERR_STATE).  `hp` and `out` are ignored.
 *   bucket == SO_ALL : scan every bucket not yet covered this iteration, reduce
 *                 per bucket and over buckets, and fill `out` (host, may be
 *                 NULL) with sumsq, norm, clip coefficient for
 *                 hp->max_grad_norm, and the flag.  Blocks until the reduction's
 *                 results have reached the host (everything enqueued on
 *                 `stream` before this call has completed by then).
 * The reduction order is fixed (independent of grid size and of whether the
 * scan ran inside the fused step), so results repeat bit for bit.
 */
so_status so_grad_check(so_ctx *ctx, const so_hparams *hp, int32_t bucket, void *stream,
                        so_grad_stats *out);

/*
 * so_adam_step_speculative -- step a bucket before validation has finished
 * (Section 4.4: the optimizer starts with the gradients available, assuming
 * finite values and no clipping).  One fused kernel reads bf16/fp32 gradients
 * and the fp32 master/m/v of the bucket, writes the new fp32 state into a free
 * slot and the bf16 parameter copy in the same pass, and leaves the tile sums
 * of g^2 in scratch as a by-product; the old state stays where it is, which is
 * everything an undo needs.  AdamW with bias correction for step t+1, gradient
 * scale 1.
 *   bucket >= 0 : that bucket.  SO_ERR_STATE if already covered this iteration,
 *                 SO_ERR_UNDO_EXHAUSTED if no slot is free (check it with
 *                 so_grad_check instead; validation then steps it in place).
 *   bucket == SO_ALL : every uncovered bucket, in index order, for as long as
 *                 slots are free (batched launches); never UNDO_EXHAUSTED.
 * All speculative steps of one iteration must use equal hyper-parameters.
 * Enqueues only; no synchronisation.  Calls for different buckets may go to
 * different streams and their kernels may overlap; at most 4096 step launches
 * of one context may be outstanding (enqueued and unfinished) at any time.
 * While a validation begun with so_validate_begin is pending, the call opens
 * the NEXT iteration: its kernels take the step index and the loss scale that
 * follow from the pending verdict, read on the device (the first such launch
 * also carries that verdict to the host).
 */
so_status so_adam_step_speculative(so_ctx *ctx, const so_hparams *hp, int32_t bucket,
                                   void *stream);

/*
 * so_validate_commit_or_rollback -- end the iteration (Section 4.4: after
 * validation, either keep the speculative update, skip the iteration when a
 * NaN/Inf was found, or revert it and re-execute with clipped gradients).
 * If a validation begun with so_validate_begin is pending, this call collects
 * it.  Otherwise it enqueues the end of the open iteration -- the scan of
 * uncovered buckets, the reduction with the verdict formed on the device (or,
 * after so_grad_check(SO_ALL), a one-block kernel that applies the statistics
 * the host holds), and the follow-up launch -- and then waits for the verdict
 * to reach the host; the follow-up kernels run meanwhile.  On the device
 *   nonfinite          -> SKIP: speculative slots are dropped, the low-precision
 *                         copy of those buckets is re-derived from the untouched
 *                         master, the step count does not advance;
 *   else clip_coef < 1 -> CLIP_RESTEP: every bucket is stepped from its
 *                         untouched prior state with gradients scaled by
 *                         clip_coef (same step index), then committed;
 *   else               -> COMMIT: speculated buckets are re-pointed at their new
 *                         slot (the follow-up launch returns at once); buckets
 *                         that were only checked are stepped in place, scale 1.
 * `hp` must equal the hyper-parameters of this iteration's speculative steps.
 * `out` (host, may be NULL) receives the decision, statistics and step count.
 * Follow-up kernels are enqueued on `stream`; the call does not wait for them.
 * SO_ERR_TIMEOUT (also from so_grad_check(SO_ALL)): a kernel gave up a bounded
 * wait for one of its own copies, so tiles are missing.  The iteration is given
 * up: speculative slots are released, the bf16 copy of the speculated buckets is
 * derived again from the committed master, step count and loss scale stay, and
 * the context is idle (the iteration may be repeated).  The committed fp32
 * state is untouched if the kernel was one of this iteration's (speculative
 * steps, scans).  Kernels that validation itself enqueues (in-place steps,
 * re-steps) report one iteration late, through the same status; if one of
 * those can have been the cause, restore the state with so_state_import.
 */
so_status so_validate_commit_or_rollback(so_ctx *ctx, const so_hparams *hp, void *stream,
                                         so_step_result *out);

/*
 * so_validate_begin / so_validate_poll -- validation off the critical path
 * (Section 4.4: validation runs while the GPU executes the next forward pass,
 * and the result is consulted after it).  so_validate_begin enqueues the whole
 * end of the iteration and returns at once: the scan of whatever is still
 * uncovered, the reduction, whose last block forms the verdict ON THE DEVICE
 * (norm, clip coefficient, decision) and re-points the speculated buckets if
 * the iteration is kept, and one follow-up launch that reads that verdict and
 * does what it entails (see so_validate_commit_or_rollback).  No host round
 * trip separates these kernels.  The verdict also travels to mapped host
 * memory; so_validate_poll tells without blocking whether it has arrived
 * (*ready = 1), and so_validate_commit_or_rollback, called later, collects it
 * for the host's bookkeeping (step count, loss scale, counters, slot map).
 * Until it has been collected:
 *   - the NEXT iteration may already be assembled: so_adam_step_speculative and
 *     so_grad_check(bucket) are accepted and enqueue kernels that carry the
 *     constants (step index, loss scale) for each way the pending iteration can
 *     end and choose among them on the device;
 *   - so_grad_check(SO_ALL) waits for the pending verdict and reports its
 *     statistics without collecting it (only while no new iteration is open);
 *   - so_validate_begin, so_cast_params, so_layout_bind, so_set_step, state
 *     export / import and the loss-scale / dtype setters return SO_ERR_STATE;
 *   - so_validate_commit_or_rollback collects the pending verdict and leaves
 *     the newly opened iteration alone.
 * All of one context's kernels must be ordered by the caller's streams as
 * before: the next iteration's steps after the follow-up launch of this one.
 */
so_status so_validate_begin(so_ctx *ctx, const so_hparams *hp, void *stream);
so_status so_validate_poll(so_ctx *ctx, int32_t *ready);

/*
 * so_set_global_grad_stats -- the hook for sharded optimizer states (Section
 * 4.7: with ZeRO-style partitioning each process updates only its own subset
 * of the parameters).  The norm and the NaN/Inf check are global quantities:
 * a process that holds a shard calls so_grad_check(SO_ALL) to get its LOCAL
 * sum of squares and flag, combines them with the other shards' (one small
 * all-reduce: sum of the sums, sum of the flags), hands the result back here,
 * and then calls so_validate_commit_or_rollback, which decides and acts on the
 * global values.  Only after so_grad_check(SO_ALL) and before validation
 * (SO_ERR_STATE otherwise).  Host-only.
 */
so_status so_set_global_grad_stats(so_ctx *ctx, double global_sumsq, int32_t global_nonfinite);

/*
 * so_abandon_iteration -- give the open iteration up (the caller's side of what
 * SO_ERR_TIMEOUT does by itself; Section 4.7: with sharded states every process
 * must end an iteration the same way, so a process told that another one failed
 * drops its own).  Speculative slots are released, the low-precision copy of the
 * speculated buckets is derived again from the committed master (one predicated
 * launch on `stream`), step count and loss scale stay, so_counters.timeouts
 * counts it, and the context is idle.  Allowed while buckets are covered or
 * after so_grad_check(SO_ALL); SO_ERR_STATE while a begun validation is
 * pending; a no-op on an idle context.
 */
so_status so_abandon_iteration(so_ctx *ctx, void *stream);

/*
 * so_cast_params -- fp32 master -> low-precision parameter copy (bf16, or
 * binary16 after so_param_dtype_config), round to nearest even (Section 4.5:
 * the cast runs on the GPU).  bucket >= 0 or SO_ALL.  Only between iterations
 * (SO_ERR_STATE while buckets are covered or a verdict is pending).  Enqueues only.
 */
so_status so_cast_params(so_ctx *ctx, int32_t bucket, void *stream);

/*
 * so_iteration_host -- one whole iteration fed from and drained to HOST memory,
 * pipelined per bucket the way Section 4.3 overlaps bucket transfers with
 * compute: the gradient bucket b is copied host -> device while bucket b-1 is
 * being stepped speculatively and the bf16 parameters of bucket b-2 travel
 * device -> host (Section 4.5: only low-precision data crosses the link, the
 * casts run on the GPU).  Then validation as in
 * so_validate_commit_or_rollback; after a SKIP or CLIP_RESTEP the bf16
 * parameters are sent again.
 *   host_grad        flat gradient of N elements in grad_dtype, parameter order
 *                    (pinned host memory for asynchronous copies)
 *   host_param_bf16  flat bf16 output of N elements, or NULL for none
 * Buckets beyond the undo capacity are scanned instead of stepped and receive
 * their step inside validation.  Uses two internal copy streams created on
 * first use.  Returns after all copies have completed (synchronises); on an
 * error too, so that no copy is left in flight from or into the host buffers.
 */
so_status so_iteration_host(so_ctx *ctx, const so_hparams *hp, const void *host_grad,
                            void *host_param_bf16, void *stream, so_step_result *out);

/*
 * so_iteration_host_pipelined / so_iteration_host_wait -- the same iteration
 * without the wait at its end, so that consecutive iterations overlap on the
 * link (Section 4.3's point, carried across the iteration boundary: the link is
 * full duplex, and the parameters that can only leave after the verdict -- those
 * of the buckets beyond the undo window, or all of them after a clip -- travel
 * while the next iteration's gradients arrive).  The call returns once the
 * verdict is known (it fills `out`) and every copy is enqueued; the next call's
 * kernels wait on the device for the previous call's outgoing copies before they
 * overwrite the parameter arena, its incoming copies do not.  Directly after
 * another pipelined call those incoming copies wait only for the library's own
 * kernels that still read the gradient bucket they overwrite (none for a bucket
 * that was speculated in a committed iteration: its last reader ran before the
 * verdict), not for other work the caller put on `stream` in between -- such
 * work must leave the gradient arena alone.
 * Until so_iteration_host_wait (or the next blocking call) has returned:
 *   - host_param_bf16 of the previous call is still being written;
 *   - host_grad of this call has been read completely only after this call's
 *     own return (all its incoming copies precede its verdict), so a gradient
 *     buffer may be refilled as soon as the call that was given it returns;
 *   - any other work of the context must go to `stream` (it is ordered behind
 *     the iteration's kernels there).
 * so_iteration_host_wait waits for the outgoing copies and for `stream`.
 */
so_status so_iteration_host_pipelined(so_ctx *ctx, const so_hparams *hp, const void *host_grad,
                                      void *host_param_bf16, void *stream, so_step_result *out);
so_status so_iteration_host_wait(so_ctx *ctx, void *stream);

/*
 * so_grad_check_static -- the gradient check for callers that cannot allocate.
 * (The paper has no counterpart: this is a packaging variant of so_grad_check,
 * not a step of its method.)
 *
 * so_grad_check needs a scratch arena that somebody allocated with cudaMalloc
 * or a framework allocator.  Some callers have neither: code running inside a
 * memory pool that is already fully handed out, start-up or diagnostic paths
 * where a device-synchronising allocation is not acceptable, plug-ins that are
 * given raw pointers and nothing else.  This entry point needs no context and
 * no scratch from the caller: its tile sums live in a fixed array inside the
 * library image (SO_STATIC_CHECK_MAX_ELEMS / 1024 doubles = 512 KB of device
 * memory on every GPU that uses the library, held until the process exits).
 * It calls no cudaMalloc / cudaFree and nothing else that allocates.
 *   grad          DEVICE, flat gradient of n_elems values in grad_dtype,
 *                 16-byte aligned (input; not modified)
 *   grad_dtype    SO_GRAD_BF16 or SO_GRAD_FP32 only: binary16 gradients need a
 *                 loss scale, which lives in a context, and are refused here
 *                 with SO_ERR_INVALID_ARG
 *   n_elems       0 .. SO_STATIC_CHECK_MAX_ELEMS; larger -> SO_ERR_TOO_LARGE
 *   max_grad_norm clip threshold for the coefficient (<= 0: coefficient 1)
 *   out_device    DEVICE, 8-byte aligned so_grad_stats written by the call
 *                 (sumsq, norm, clip_coef, nonfinite); caller-owned output
 * Enqueues two kernels on `stream` and returns; no synchronisation, no host
 * copy.  Sums fold in a fixed order; the result is bit-identical to
 * so_grad_check over one bucket of n_elems up to 4 Mi elements and equal to
 * rounding beyond that.
 * The first call on each device looks up the device address of the built-in
 * array (cudaGetSymbolAddress, with that device current) and caches it; make
 * that first call outside any stream capture.  All calls on a device share the
 * one array: it keeps whatever the previous call left, which is harmless
 * because each call overwrites every entry it later reads (nothing has to
 * start at zero), but two calls whose kernels overlap on the GPU (different
 * streams, or different threads/processes' streams of one process) race on it
 * -- serialise them.
 */
#define SO_STATIC_CHECK_MAX_ELEMS (1 << 26)
so_status so_grad_check_static(const void *grad, int64_t n_elems, int32_t grad_dtype,
                               double max_grad_norm, void *stream, so_grad_stats *out_device);

/*
 * so_loss_scale_config -- loss scaling for fp16 gradients (the paper trains in
 * FP16 mixed precision, Section 4.5; the NaN/Inf check of Section 4.4 is the
 * overflow test of this scheme).  The gradient arena then holds
 * loss_scale * gradient; the check and the step multiply every stored value by
 * 1 / loss_scale first, so norm, clipping and the update see the true gradient.
 * interval > 0 enables the dynamic schedule: after an iteration that was
 * skipped for a non-finite gradient the scale is multiplied by `backoff`
 * (0 < backoff <= 1), after `interval` consecutive kept iterations by `growth`
 * (>= 1); interval = 0 keeps the scale fixed.  The scale used by an iteration
 * is the one in effect when the iteration starts; so_step_result.loss_scale
 * tells the producer of the next gradients which scale to apply.
 * Only for SO_GRAD_FP16 contexts (SO_ERR_UNSUPPORTED otherwise), only between
 * iterations.  Host-only.
 */
so_status so_loss_scale_config(so_ctx *ctx, double init_scale, double growth, double backoff,
                               int64_t interval);
so_status so_get_loss_scale(const so_ctx *ctx, double *scale);

/*
 * so_state_export / so_state_import -- checkpoint and resume.  Copy the
 * committed fp32 state (master weights, first and second moments) between the
 * slot arenas and flat arrays of N floats in parameter order; each of master,
 * m, v may be NULL to skip it, and may point to device or host memory (pinned
 * for truly asynchronous copies).  One cudaMemcpyAsync per bucket and array on
 * `stream`; no synchronisation.  Together with so_get_step / so_set_step (and,
 * for fp16, the loss scale) this is the whole optimizer state.  After an
 * import call so_cast_params(SO_ALL) to re-derive the bf16 copy.  Only between
 * iterations.
 */
so_status so_state_export(so_ctx *ctx, void *master, void *m, void *v, void *stream);
so_status so_state_import(so_ctx *ctx, const void *master, const void *m, const void *v,
                          void *stream);

/* Slot of the state arenas that holds bucket b's committed master/m/v. */
so_status so_bucket_slot(const so_ctx *ctx, int32_t bucket, int32_t *slot);

/* Committed step count t (starts at 0); so_set_step restores it on resume
 * (only between iterations). */
so_status so_get_step(const so_ctx *ctx, int64_t *t);
so_status so_set_step(so_ctx *ctx, int64_t t);

/* Number of buckets not yet covered (stepped or checked) this iteration. */
so_status so_pending_buckets(const so_ctx *ctx, int32_t *n);

so_status so_get_counters(const so_ctx *ctx, so_counters *out);

/* Raw cudaError_t of the last failing CUDA call on this context (0 if none). */
int32_t so_last_cuda_error(const so_ctx *ctx);

const char *so_strerror(so_status s);

/* Frees the host-side context.  Never touches device memory. */
void so_destroy(so_ctx *ctx);

/*
 * Host-logic test hooks.  In dry-run mode no CUDA call is made: launches are
 * only counted, and the per-bucket check results come from
 * so_debug_set_bucket_stats instead of the device (with bucket == SO_ALL it
 * sets, from `nonfinite`, the device status word the next check will read, which
 * is how the SO_ERR_TIMEOUT handling is tested).  This lets the slot map and
 * the per-iteration state machine be exercised on a machine without a GPU.
 */
so_status so_debug_set_dry_run(so_ctx *ctx, int32_t on);
so_status so_debug_set_bucket_stats(so_ctx *ctx, int32_t bucket, double sumsq,
                                    int32_t nonfinite);

/* Which implementation of the fused step runs.  There are two kernels with the
 * same results bit for bit: one stages bulk copies through shared memory (the
 * fast one on anything large), one keeps everything in registers (lower fixed
 * cost per launch).  0 (default): by launch size -- the register kernel for
 * launches of at most 3 Mi elements, the pipeline otherwise; 1: always the
 * register kernel; 2: always the pipeline.  1 and 2 exist for measurements and
 * for testing the two against each other. */
so_status so_debug_set_step_variant(so_ctx *ctx, int32_t variant);

/* How many times the bulk-copy step kernel polls for a chunk's loads before it
 * gives the launch up (0 .. 2^20, the default).  The waits that drain copies in
 * flight before a block exits always use the full limit, so a small value makes
 * the kernel raise its status word (SO_ERR_TIMEOUT at the next check) without
 * leaving anything in flight: this is how the give-up path is tested.  Applies
 * to launches made after the call. */
so_status so_debug_set_spin_limit(so_ctx *ctx, int64_t polls);

#ifdef __cplusplus
}
#endif
#endif /* SUPEROFFLOAD_H */
