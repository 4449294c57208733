/*
 * Minimal C user of the C-ABI: fits a small planted problem from host buffers and prints loss and accuracy.
 *
 *   gcc -std=c99 -O2 -I include paper_2308_10037_b200/examples/fit_host.c \
 *       -L paper_2308_10037_b200 -llrgd -Wl,-rpath,$PWD/paper_2308_10037_b200 -lm -o fit_host && ./fit_host
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "lrgd.h"

static uint32_t rng_state = 12345u;
static float uniform01(void) {                      /* xorshift32: only to make some data */
    rng_state ^= rng_state << 13; rng_state ^= rng_state >> 17; rng_state ^= rng_state << 5;
    return (float)(rng_state >> 8) * (1.0f / 16777216.0f);
}

int main(void) {
    const int64_t m = 200000;
    const int32_t n = 32, iters = 200;
    float* X = (float*)malloc(sizeof(float) * (size_t)m * n);
    float* y = (float*)malloc(sizeof(float) * (size_t)m);
    float* w = (float*)calloc((size_t)n, sizeof(float));
    float* hist = (float*)malloc(sizeof(float) * iters);
    uint8_t* labels = (uint8_t*)malloc((size_t)m);
    float wstar[32], b = 0.0f;
    if (!X || !y || !w || !hist || !labels) return 1;
    for (int j = 0; j < n; ++j) wstar[j] = 2.0f * uniform01() - 1.0f;
    for (int64_t i = 0; i < m; ++i) {
        float z = 0.3f;
        for (int j = 0; j < n; ++j) { X[i * n + j] = 2.0f * uniform01() - 1.0f; z += X[i * n + j] * wstar[j]; }
        y[i] = uniform01() < 1.0f / (1.0f + expf(-z)) ? 1.0f : 0.0f;
    }
    lr_ctx* ctx = NULL;
    int rc = lr_create(&ctx, 0, n);
    if (rc != LR_OK) { fprintf(stderr, "lr_create: %s\n", lr_status_string(rc)); return 1; }
    rc = lr_fit_host(ctx, X, y, m, n, 1.0f, iters, w, &b, hist);
    if (rc != LR_OK) { fprintf(stderr, "lr_fit_host: %s (cuda %d)\n", lr_status_string(rc), lr_last_cuda_error(ctx)); return 1; }
    rc = lr_predict_host(ctx, X, m, n, w, &b, 0.5f, labels);
    if (rc != LR_OK) { fprintf(stderr, "lr_predict_host: %s\n", lr_status_string(rc)); return 1; }
    int64_t agree = 0;
    for (int64_t i = 0; i < m; ++i) agree += (labels[i] != 0) == (y[i] > 0.5f);
    int32_t status = 0;
    lr_last_device_status(ctx, &status);
    printf("loss %.6f -> %.6f after %d iterations, training accuracy %.4f, device status %d\n", hist[0], hist[iters - 1], iters,
           (double)agree / (double)m, status);
    const int ok = status == 0 && hist[iters - 1] < hist[0];
    lr_destroy(ctx);
    free(X); free(y); free(w); free(hist); free(labels);
    return ok ? 0 : 1;
}
