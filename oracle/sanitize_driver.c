/*
 * Driver that runs every entry point of the CPU oracle (qesgd_oracle.c) on small and ragged
 * sizes with exactly sized heap buffers, meant to be built with
 *   gcc -fsanitize=address,undefined -fno-sanitize-recover=all
 * so that an out-of-bounds access, a signed overflow or a bad shift inside the oracle ends the
 * run with a non-zero status.  TEST INFRASTRUCTURE ONLY, like the oracle itself.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

int qesgd_ref_encode(const float *, const float *, uint64_t, uint64_t, uint32_t, uint32_t, uint32_t, uint32_t,
                     float, uint64_t, uint32_t, uint32_t, uint32_t *, float *, uint32_t *);
int qesgd_ref_decode(const uint32_t *, const float *, uint64_t, uint32_t, uint32_t, uint32_t, float *);
int qesgd_ref_decode_average_apply(float *, uint64_t, uint32_t, const uint32_t *, uint64_t, const float *,
                                   uint64_t, uint32_t, uint32_t, uint32_t);
int qesgd_ref_decode_average_axpy(float *, uint64_t, uint32_t, const uint32_t *, uint64_t, const float *,
                                  uint64_t, uint32_t, uint32_t, uint32_t, float);
int qesgd_ref_requantize(float *, const float *, uint64_t, uint64_t, uint32_t, uint32_t, uint32_t, uint32_t,
                         float, uint64_t, uint32_t, uint32_t, float *, uint32_t *, float *, uint32_t *);
double qesgd_ref_lr_loss(const float *, const float *, uint64_t, uint64_t, const float *);
int qesgd_ref_lr_sgd_step(const float *, const float *, uint32_t, uint64_t, float, float *);
int qesgd_ref_lr_local_epoch(const float *, const float *, uint64_t, uint64_t, uint32_t, float, float *);
int qesgd_ref_lr_gradient(const float *, const float *, uint32_t, uint64_t, const float *, float *);
uint32_t qesgd_ref_draw16(uint64_t, uint32_t, uint32_t, uint64_t);

static uint64_t lcg = 88172645463325252ull;
static float rnd(void)
{
    lcg ^= lcg << 13; lcg ^= lcg >> 7; lcg ^= lcg << 17;
    return (float)((double)(lcg >> 11) / 9007199254740992.0 - 0.5) * 2e-3f;
}

static void fail(const char *what) { fprintf(stderr, "sanitize_driver: %s\n", what); exit(2); }

int main(void)
{
    const uint64_t sizes[] = {1, 7, 63, 64, 65, 511, 513, 1000, 4097};
    const uint32_t buckets[] = {64, 512, 8192};
    const uint32_t bits_s[][2] = {{2, 1}, {4, 7}, {8, 127}, {8, 100}};
    unsigned long checksum = 0;
    for (size_t a = 0; a < sizeof(sizes) / sizeof(sizes[0]); ++a)
        for (size_t b = 0; b < 3; ++b)
            for (size_t c = 0; c < 4; ++c)
                for (uint32_t mode = 0; mode < 3; ++mode) {
                    const uint64_t n = sizes[a];
                    const uint32_t B = buckets[b], bits = bits_s[c][0], s = bits_s[c][1], K = 3;
                    const uint64_t nb = (n + B - 1) / B, words = nb * B * bits / 32;
                    float *local = malloc(sizeof(float) * n), *anchor = malloc(sizeof(float) * n);
                    float *out = malloc(sizeof(float) * n), *zsum = malloc(sizeof(float) * n);
                    uint32_t *codes = malloc(sizeof(uint32_t) * words * K);
                    float *scales = malloc(sizeof(float) * nb * K);
                    uint32_t status = 0;
                    if (!local || !anchor || !out || !zsum || !codes || !scales) fail("malloc");
                    for (uint64_t i = 0; i < n; ++i) { anchor[i] = 50.0f * rnd(); local[i] = anchor[i] + rnd(); zsum[i] = rnd(); }
                    if (n > 5) { local[3] = 0.0f; anchor[3] = 0.0f; local[5] = -anchor[5]; }
                    for (uint32_t k = 0; k < K; ++k)
                        if (qesgd_ref_encode(local, k == 1 ? NULL : anchor, n, 0, B, s, bits, mode, 1e-4f, 77, k, 5,
                                             codes + k * words, scales + k * nb, &status)) fail("encode");
                    if (qesgd_ref_decode(codes, scales, n, B, s, bits, out)) fail("decode");
                    if (qesgd_ref_decode_average_apply(anchor, n, K, codes, words * 4, scales, nb, B, s, bits)) fail("apply");
                    if (qesgd_ref_decode_average_axpy(anchor, n, K, codes, words * 4, scales, nb, B, s, bits, -0.1f)) fail("axpy");
                    if (qesgd_ref_requantize(local, anchor, n, 0, B, s, bits, mode, 1e-4f, 9, 1, 2, zsum, codes, scales, &status)) fail("requantize");
                    checksum += codes[0] + (unsigned long)(fabsf(out[n - 1]) * 1e6f) + status;
                    free(local); free(anchor); free(out); free(zsum); free(codes); free(scales);
                }
    /* a slice with a global offset, and non-finite input */
    {
        const uint64_t n = 200; const uint32_t B = 64;
        float *z = malloc(sizeof(float) * n); uint32_t *codes = malloc(sizeof(uint32_t) * 4 * B * 4 / 32); float *sc = malloc(sizeof(float) * 4);
        uint32_t status = 0;
        for (uint64_t i = 0; i < n; ++i) z[i] = rnd();
        z[10] = INFINITY; z[70] = NAN; z[150] = -INFINITY;
        for (uint32_t mode = 0; mode < 3; ++mode)
            if (qesgd_ref_encode(z, NULL, n, (uint64_t)B << 32, B, 7, 4, mode, 1e-4f, 1, 0, 0, codes, sc, &status)) fail("encode nonfinite");
        checksum += status + qesgd_ref_draw16(~0ull, ~0u, ~0u, ~0ull);
        free(z); free(codes); free(sc);
    }
    /* logistic regression */
    {
        const uint32_t m = 37; const uint64_t d = 101, rows = 3 * m + 5;
        float *X = malloc(sizeof(float) * rows * d), *y = malloc(sizeof(float) * rows), *u = calloc(d, sizeof(float)), *g = malloc(sizeof(float) * d);
        for (uint64_t i = 0; i < rows * d; ++i) X[i] = 100.0f * rnd();
        for (uint64_t j = 0; j < rows; ++j) y[j] = rnd() > 0 ? 1.0f : -1.0f;
        if (qesgd_ref_lr_sgd_step(X, y, m, d, 0.1f, u)) fail("step");
        if (qesgd_ref_lr_local_epoch(X, y, rows, d, m, 0.1f, u)) fail("epoch");
        if (qesgd_ref_lr_gradient(X, y, m, d, u, g)) fail("gradient");
        checksum += (unsigned long)(qesgd_ref_lr_loss(X, y, rows, d, u) * 1e6);
        free(X); free(y); free(u); free(g);
    }
    printf("sanitize_driver ok %lu\n", checksum);
    return 0;
}
