/*
 * Walks the host side of the library (layout arithmetic, slot map, the
 * per-iteration state machine, argument checks) in dry-run mode -- no GPU, no
 * CUDA call -- so that a build of the library with -fsanitize=address,undefined
 * can catch out-of-bounds accesses, leaks and undefined arithmetic in it.
 * Prints "sanitized ok" when it gets to the end.
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include "superoffload.h"

static uint32_t rng_state = 2463534242u;
static uint32_t rng(void) { rng_state ^= rng_state << 13; rng_state ^= rng_state >> 17; rng_state ^= rng_state << 5; return rng_state; }

#define CHECK(cond) do { if (!(cond)) { printf("line %d: %s\n", __LINE__, #cond); exit(2); } } while (0)

static so_ctx *make(int n_tensors, const int64_t *numel, int64_t bucket, int dtype, int undo,
                    so_layout_info *info)
{
    so_ctx *ctx = NULL;
    CHECK(so_layout_init(&ctx, n_tensors, numel, bucket, dtype, undo, info) == SO_OK);
    CHECK(so_debug_set_dry_run(ctx, 1) == SO_OK);
    char *base = (char *)0x10000000;
    CHECK(so_layout_bind(ctx, base, base + 0x1000000, base + 0x2000000, base + 0x3000000,
                         base + 0x4000000, base + 0x5000000) == SO_OK);
    return ctx;
}

static void walk(int64_t total, int64_t bucket, int dtype, int undo, int iterations)
{
    so_layout_info info;
    int64_t numel[4];
    numel[0] = total / 3; numel[1] = 0; numel[2] = total / 5; numel[3] = total - numel[0] - numel[2];
    so_ctx *ctx = make(4, numel, bucket, dtype, undo, &info);
    const int nb = info.n_buckets;
    so_hparams hp = {1e-3, 0.9, 0.999, 1e-8, 0.01, 1.0};
    if (dtype == SO_GRAD_FP16) CHECK(so_loss_scale_config(ctx, 65536.0, 2.0, 0.5, 3) == SO_OK);
    for (int it = 0; it < iterations; ++it) {
        for (int b = 0; b < nb; ++b)
            so_debug_set_bucket_stats(ctx, b, (rng() % 3) ? 0.01 / (nb + 1) : 5.0, rng() % 11 == 0);
        if (rng() % 9 == 0) so_debug_set_bucket_stats(ctx, SO_ALL, 0.0, 1);      /* a kernel gives up */
        const int calls = (int)(rng() % (2 * (unsigned)nb + 3));
        for (int k = 0; k < calls && nb > 0; ++k) {
            const int b = (int)(rng() % (unsigned)(nb + 1)) - (rng() % 13 == 0);  /* sometimes out of range */
            switch (rng() % 5) {
                case 0: case 1: (void)so_adam_step_speculative(ctx, &hp, b, NULL); break;
                case 2: (void)so_grad_check(ctx, NULL, b, NULL, NULL); break;
                case 3: (void)so_adam_step_speculative(ctx, &hp, SO_ALL, NULL); break;
                default: (void)so_cast_params(ctx, b, NULL); break;
            }
        }
        so_step_result r;
        so_grad_stats st;
        int32_t ready = 0, pending = 0, slot = 0;
        so_status s;
        switch (rng() % 4) {
            case 0:
                s = so_validate_commit_or_rollback(ctx, &hp, NULL, &r);
                CHECK(s == SO_OK || s == SO_ERR_TIMEOUT);
                break;
            case 1:
                s = so_grad_check(ctx, &hp, SO_ALL, NULL, &st);
                CHECK(s == SO_OK || s == SO_ERR_TIMEOUT);
                if (s == SO_OK && rng() % 2) (void)so_set_global_grad_stats(ctx, st.sumsq * 2.0, st.nonfinite);
                if (s == SO_OK && rng() % 5 == 0) { CHECK(so_abandon_iteration(ctx, NULL) == SO_OK); break; }
                s = so_validate_commit_or_rollback(ctx, &hp, NULL, &r);
                CHECK(s == SO_OK);
                break;
            case 2:
                CHECK(so_validate_begin(ctx, &hp, NULL) == SO_OK);
                CHECK(so_validate_poll(ctx, &ready) == SO_OK && ready == 1);
                (void)so_adam_step_speculative(ctx, &hp, SO_ALL, NULL);           /* the next iteration */
                CHECK(so_validate_begin(ctx, &hp, NULL) == SO_ERR_STATE);
                s = so_validate_commit_or_rollback(ctx, &hp, NULL, &r);           /* collects the first */
                CHECK(s == SO_OK || s == SO_ERR_TIMEOUT);
                s = so_validate_commit_or_rollback(ctx, &hp, NULL, &r);           /* validates the second */
                CHECK(s == SO_OK || s == SO_ERR_TIMEOUT);
                break;
            default:
                CHECK(so_abandon_iteration(ctx, NULL) == SO_OK);
                break;
        }
        CHECK(so_pending_buckets(ctx, &pending) == SO_OK && pending == nb);
        for (int b = 0; b < nb; ++b) CHECK(so_bucket_slot(ctx, b, &slot) == SO_OK && slot >= 0 && slot < info.n_state_slots);
    }
    so_counters c;
    int64_t t = 0, off = 0;
    int32_t fb = 0, lb = 0;
    CHECK(so_get_counters(ctx, &c) == SO_OK && so_get_step(ctx, &t) == SO_OK);
    CHECK(t == c.commits + c.clip_resteps);
    for (int i = 0; i < 4; ++i) CHECK(so_layout_tensor(ctx, i, &off, &fb, &lb) == SO_OK);
    CHECK(so_layout_tensor(ctx, 4, &off, &fb, &lb) == SO_ERR_INVALID_ARG);
    const void *ptrs[4] = {(void *)0x100, NULL, (void *)0x200, (void *)0x300};
    (void)so_layout_pack_grads(ctx, ptrs, NULL);
    (void)so_layout_unpack_params(ctx, (void *const *)ptrs, NULL);
    CHECK(so_layout_pack_grads(ctx, NULL, NULL) == (total ? SO_ERR_INVALID_ARG : SO_OK));
    CHECK(so_param_dtype_config(ctx, SO_PARAM_FP16) == SO_OK && so_param_dtype_config(ctx, 7) == SO_ERR_INVALID_ARG);
    CHECK(so_set_step(ctx, 12) == SO_OK && so_set_step(ctx, -1) == SO_ERR_INVALID_ARG);
    CHECK(so_debug_set_spin_limit(ctx, 0) == SO_OK && so_debug_set_spin_limit(ctx, -5) == SO_ERR_INVALID_ARG);
    so_destroy(ctx);
}

int main(void)
{
    so_ctx *bad = NULL;
    int64_t one = 5, neg = -1;
    CHECK(so_layout_init(&bad, 1, &one, 0, SO_GRAD_BF16, 0, NULL) == SO_ERR_INVALID_ARG);
    CHECK(so_layout_init(&bad, 1, &neg, 4, SO_GRAD_BF16, 0, NULL) == SO_ERR_INVALID_ARG);
    CHECK(so_layout_init(&bad, 1, &one, 4, 9, 0, NULL) == SO_ERR_INVALID_ARG);
    CHECK(so_layout_init(&bad, 1, &one, 4, SO_GRAD_BF16, 3, NULL) == SO_ERR_INVALID_ARG);
    CHECK(so_layout_init(NULL, 1, &one, 4, SO_GRAD_BF16, 0, NULL) == SO_ERR_INVALID_ARG);
    walk(0, 64, SO_GRAD_BF16, 0, 5);
    walk(1, 1, SO_GRAD_BF16, SO_ALL, 20);
    walk(1537, 256, SO_GRAD_BF16, SO_ALL, 60);
    walk(1537, 256, SO_GRAD_FP32, 3, 60);
    walk(1537, 256, SO_GRAD_FP16, 2, 60);
    walk(300 * 64 + 5, 64, SO_GRAD_BF16, 150, 25);       /* more than 128 buckets: several launches */
    walk(1000, 7, SO_GRAD_BF16, 0, 10);
    for (int s = -9; s <= 1; ++s) CHECK(so_strerror(s) != NULL);
    CHECK(so_last_cuda_error(NULL) == 0);
    so_destroy(NULL);
    printf("sanitized ok\n");
    return 0;
}
