/*
 * Drives every function of the CPU oracle on small and degenerate inputs so
 * that a build with -fsanitize=address,undefined can catch out-of-bounds
 * accesses, leaks, misaligned or overflowing arithmetic.  Allocations are
 * exactly as large as the ranges handed in: one element too far is a fault.
 * Prints "sanitized ok" when it gets to the end.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

float orc_bf16_to_f32(uint16_t b);
void orc_widen_bf16(const uint16_t *b, float *out, int64_t n);
float orc_fp16_to_f32(uint16_t h);
void orc_widen_fp16(const uint16_t *h, float *out, int64_t n);
uint16_t orc_bf16_rne(float x);
void orc_cast_params(const float *p, uint16_t *pb, int64_t n);
uint16_t orc_fp16_rne(float x);
void orc_cast_params_fp16(const float *p, uint16_t *ph, int64_t n);
int orc_grad_check_range(const void *g, int grad_dtype, int64_t begin, int64_t end, double unscale,
                         double *sumsq_out);
int orc_global_grad_check(const void *g, int grad_dtype, int64_t n, int64_t bucket_elems,
                          double unscale, double *sumsq_out, double *norm_out);
double orc_clip_coef(double norm, double max_norm);
int orc_decision(int nonfinite, double coef);
void orc_adamw_step_range(float *p, float *m, float *v, const void *g, int grad_dtype, int64_t begin,
                          int64_t end, double unscale, double scale, int64_t tt, double lr,
                          double beta1, double beta2, double eps, double wd);
int orc_iteration_ste(float *p, float *m, float *v, uint16_t *pb, const void *g, int grad_dtype,
                      int64_t n, int64_t bucket_elems, int64_t *t, double lr, double beta1,
                      double beta2, double eps, double wd, double max_norm, double unscale,
                      double *sumsq_out, double *norm_out, double *coef_out, int *nonfinite_out);
int orc_iteration_stv(float *p, float *m, float *v, uint16_t *pb, const void *g, int grad_dtype,
                      int64_t n, int64_t bucket_elems, int64_t *t, double lr, double beta1,
                      double beta2, double eps, double wd, double max_norm, double unscale,
                      double forced_coef, double *sumsq_out, double *norm_out, double *coef_out,
                      int *nonfinite_out);
void orc_loss_scale_update(double *scale, int64_t *good_steps, int nonfinite, double growth,
                           double backoff, int64_t interval);
int64_t orc_layout_offsets(const int64_t *numel, int32_t n_tensors, int64_t *offsets);
int64_t orc_num_buckets(int64_t total, int64_t bucket_elems);
int64_t orc_resident_bytes(int64_t total);

static uint32_t rng_state = 12345u;
static uint32_t rng(void) { rng_state = rng_state * 1664525u + 1013904223u; return rng_state; }
static float small_float(void) { return ((int)(rng() >> 8) - (1 << 23)) * (1.0f / (1 << 30)); }

static void iterations(int grad_dtype, int64_t n, int64_t bucket)
{
    size_t count = (size_t)(n ? n : 1);
    float *p = malloc(count * 4), *m = malloc(count * 4), *v = malloc(count * 4);
    uint16_t *pb = malloc(count * 2);
    size_t gsz = grad_dtype == 1 ? 4 : 2;
    void *g = malloc(count * gsz);
    for (int64_t i = 0; i < n; ++i) {
        p[i] = small_float();
        m[i] = 0.0f;
        v[i] = 0.0f;
        float gi = small_float() * (i % 7 == 0 ? 64.0f : 1.0f);
        if (grad_dtype == 1) ((float *)g)[i] = gi;
        else if (grad_dtype == 0) ((uint16_t *)g)[i] = orc_bf16_rne(gi);
        else ((uint16_t *)g)[i] = orc_fp16_rne(gi * 256.0f);
    }
    orc_cast_params(p, pb, n);
    int64_t t = 0;
    double s, nrm, coef;
    int flag;
    double unscale = grad_dtype == 2 ? 1.0 / 256.0 : 1.0;
    for (int step = 0; step < 4; ++step) {
        double max_norm = step % 2 ? 1e-3 : 0.0;               /* clip on odd steps */
        orc_iteration_ste(p, m, v, pb, g, grad_dtype, n, bucket, &t, 1e-3, 0.9, 0.999, 1e-8, 0.01,
                          max_norm, unscale, &s, &nrm, &coef, &flag);
        orc_iteration_stv(p, m, v, pb, g, grad_dtype, n, bucket, &t, 1e-3, 0.9, 0.999, 1e-8, 0.01,
                          max_norm, unscale, step == 3 ? 0.5 : 0.0, &s, &nrm, &coef, &flag);
    }
    if (n > 0) {                                               /* a non-finite gradient: skip */
        if (grad_dtype == 1) ((float *)g)[n - 1] = INFINITY;
        else ((uint16_t *)g)[n - 1] = grad_dtype == 0 ? 0x7FC0 : 0x7C00;
        int64_t before = t;
        orc_iteration_stv(p, m, v, pb, g, grad_dtype, n, bucket, &t, 1e-3, 0.9, 0.999, 1e-8, 0.01,
                          1.0, unscale, 0.0, &s, &nrm, &coef, &flag);
        if (!flag || t != before) { printf("skip not taken\n"); exit(2); }
    }
    free(p); free(m); free(v); free(pb); free(g);
}

int main(void)
{
    /* casts and widenings over every 16-bit pattern and a spread of fp32 patterns */
    uint16_t *h = malloc(65536 * 2);
    float *w = malloc(65536 * 4);
    for (int i = 0; i < 65536; ++i) h[i] = (uint16_t)i;
    orc_widen_bf16(h, w, 65536);
    orc_widen_fp16(h, w, 65536);
    orc_widen_bf16(h, w, 0);
    uint16_t *c = malloc(65536 * 2);
    for (int rep = 0; rep < 64; ++rep) {
        for (int i = 0; i < 65536; ++i) {
            uint32_t bits = ((uint32_t)i << 16) | (rng() & 0xFFFFu);
            memcpy(&w[i], &bits, 4);
        }
        orc_cast_params(w, c, 65536);
        orc_cast_params_fp16(w, c, 65536);
    }
    (void)orc_bf16_to_f32(0x7F80); (void)orc_fp16_to_f32(0xFC00);
    (void)orc_bf16_rne(NAN); (void)orc_fp16_rne(-NAN); (void)orc_fp16_rne(65520.0f);
    free(h); free(w); free(c);

    /* check, step and whole iterations on empty, single, ragged and multi-bucket inputs */
    const int64_t sizes[][2] = {{0, 8}, {1, 1}, {1, 64}, {7, 3}, {64, 64}, {65, 64}, {1000, 256},
                                {4097, 1024}};
    for (int dt = 0; dt < 3; ++dt)
        for (size_t k = 0; k < sizeof(sizes) / sizeof(sizes[0]); ++k)
            iterations(dt, sizes[k][0], sizes[k][1]);

    /* ranges inside a larger array, scalars, schedule, layout */
    float g[10] = {3, 4, 0, 0, 1e30f, -1e30f, 1e-30f, 0, 0, 0};
    double s, nrm;
    orc_grad_check_range(g, 1, 0, 2, 1.0, &s);
    if (s != 25.0) { printf("sum wrong\n"); return 2; }
    orc_grad_check_range(g, 1, 9, 9, 1.0, &s);
    orc_global_grad_check(g, 1, 10, 3, 1.0, &s, &nrm);
    (void)orc_clip_coef(nrm, 1.0); (void)orc_clip_coef(0.0, 0.0); (void)orc_clip_coef(INFINITY, 1.0);
    (void)orc_decision(0, 1.0); (void)orc_decision(1, 0.5); (void)orc_decision(0, 0.5);
    float p3[3] = {1, 2, 3}, m3[3] = {0}, v3[3] = {0};
    orc_adamw_step_range(p3, m3, v3, g, 1, 1, 2, 1.0, 1.0, 1, 1e-3, 0.9, 0.999, 1e-8, 0.0);
    double scale = 65536.0;
    int64_t good = 0;
    for (int i = 0; i < 12; ++i) orc_loss_scale_update(&scale, &good, i % 5 == 4, 2.0, 0.5, 3);
    int64_t numel[5] = {3, 0, 1000, 1, (int64_t)1 << 40}, off[5];
    if (orc_layout_offsets(numel, 5, off) != 1004 + ((int64_t)1 << 40)) { printf("layout wrong\n"); return 2; }
    (void)orc_layout_offsets(numel, 0, off);
    (void)orc_num_buckets(0, 5); (void)orc_num_buckets(((int64_t)1 << 46), 1); (void)orc_resident_bytes((int64_t)1 << 40);
    printf("sanitized ok\n");
    return 0;
}
