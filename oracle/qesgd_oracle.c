/*
 * QESGD hot path -- plain CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, obviously-correct statement of what the quantised
 * epoch-SGD data path computes.  It exists so that tests and the benchmark's
 * CPU leg have something to compare the CUDA library with.  It shares no code,
 * header, table or constant generator with the CUDA library, and the product
 * never calls it.
 *
 * Every floating-point operation below is one IEEE-754 round-to-nearest-even
 * operation in the precision written (compile with -ffp-contract=off, no
 * fast-math, no flush-to-zero).  There is no blocking, fusion or reordering
 * beyond what each cited passage states.
 *
 * Parity pins: every function here is pinned by tests that do not go through
 * this file's own arithmetic (published Philox known-answer vectors, exact
 * rational sums, the closed-form rounding probabilities and variance of the
 * paper's Lemma 1, grid fixed points, brute-force enumeration on d <= 8,
 * finite differences of the logistic loss).  What cannot be pinned here --
 * the paper's accuracy tables and training curves -- is "parity unpinned":
 * it needs the paper's data sets and networks.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define QREF_OK 0
#define QREF_EINVAL (-1)
#define QREF_ENOMEM (-2)

#define QREF_SCALE_NORM 0u   /* scale = L2 norm of the bucket            */
#define QREF_SCALE_MAX 1u    /* scale = largest magnitude in the bucket  */
#define QREF_SCALE_FIXED 2u  /* scale = s * delta, delta given by caller */

#define QREF_STATUS_NONFINITE 1u

/* ------------------------------------------------------------------------ */
/* Counter-based random numbers: Philox4x32 with 10 rounds, as published by  */
/* Salmon, Moraes, Dror and Shaw (SC'11).  The paper only says "with         */
/* probability" (Eq. 4) and that coordinates are rounded independently       */
/* (Sec. 2.1); a counter-based generator makes every draw a pure function of */
/* (seed, worker, epoch, element).                                           */
/* ------------------------------------------------------------------------ */
void qesgd_ref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { /* the key is bumped between rounds, not before the first */
            k0 += W0;
            k1 += W1;
        }
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 16-bit uniform draw h in [0, 65536) of element i (Eq. 4's "with
 * probability"; Sec. 2.1: each coordinate independently).  One Philox block
 * serves the 8 elements that share i >> 3: counter = (i>>3 low, i>>3 high,
 * worker, epoch), key = (seed low, seed high); element i takes half-word
 * (i & 1) of 32-bit word (i >> 1) & 3. */
uint32_t qesgd_ref_draw16(uint64_t seed, uint32_t worker, uint32_t epoch, uint64_t i)
{
    uint64_t block = i >> 3;
    uint32_t ctr[4] = {(uint32_t)block, (uint32_t)(block >> 32), worker, epoch};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t x[4];
    qesgd_ref_philox4x32_10(ctr, key, x);
    uint32_t word = x[(i >> 1) & 3];
    return (i & 1) ? (word >> 16) : (word & 0xFFFFu);
}

/* ------------------------------------------------------------------------ */
/* Bucket scale.  The paper's experiments use delta = ||g|| for a quantised  */
/* vector (Sec. 5, CNN paragraph) and note that vectors may be split into    */
/* buckets that are compressed one by one (Sec. 3).  ||.|| is the L2 norm    */
/* (Sec. 2).  Lemma 2 only needs every coordinate to lie inside the grid's   */
/* range, which the largest magnitude also guarantees (second mode).         */
/* ------------------------------------------------------------------------ */

/* Sum of n = 2^m doubles over the balanced binary tree on index order:
 * T(x[0..n)) = x[0] if n == 1, else fl64(T(left half) + T(right half)). */
static double tree_sum(const double *x, size_t n)
{
    if (n == 1) return x[0];
    return tree_sum(x, n / 2) + tree_sum(x + n / 2, n / 2);
}

/* The fp64 sum of squares of one zero-padded bucket, before the square root (exposed so
 * that tests can check the summation tree in fp64, where its shape is visible). */
double qesgd_ref_bucket_sumsq(const float *z, uint32_t B, double *scratch)
{
    for (uint32_t j = 0; j < B; ++j)
        scratch[j] = (double)z[j] * (double)z[j]; /* exact: 24-bit x 24-bit */
    return tree_sum(scratch, B);
}

/* z holds one zero-padded bucket of B = 2^m fp32 values. */
float qesgd_ref_bucket_scale(const float *z, uint32_t B, uint32_t scale_mode, double *scratch)
{
    if (scale_mode == QREF_SCALE_NORM) {
        double S = qesgd_ref_bucket_sumsq(z, B, scratch);
        return (float)sqrt(S); /* fl32(fl64(sqrt(S))) */
    }
    float m = 0.0f;
    for (uint32_t j = 0; j < B; ++j) {
        float a = fabsf(z[j]);
        if (a > m) m = a;
    }
    return m;
}

/* ------------------------------------------------------------------------ */
/* Stochastic rounding of one magnitude (Eq. 4 with delta = scale / s and    */
/* the grid taken symmetric, |k| <= s): r = a / delta computed as a * inv    */
/* with inv = fl32(s / scale); values at or above the top of the range stay  */
/* at s (first branch of Eq. 4); inside the range the result is floor(r)     */
/* with probability ceil - r and floor(r) + 1 with probability r - floor     */
/* (second and third branch).  The draw h decides: up iff (h + 1/2)/2^16 < p.*/
/* ------------------------------------------------------------------------ */
uint32_t qesgd_ref_level(float a, float inv, uint32_t s, uint32_t h)
{
    float r = a * inv;
    if (r > (float)s) r = (float)s;
    float f = floorf(r);
    float p = r - f;                                /* exact in fp32 */
    int up = (float)(2u * h + 1u) < p * 131072.0f;  /* both sides exact */
    return (uint32_t)f + (uint32_t)up;
}

/* inv = fl32(s / scale): one correctly rounded fp32 division per bucket.  Rounded to
 * nearest it can exceed the exact quotient by half an ulp, so the product |z| * inv of the
 * bucket's largest coordinate can land one ulp above s; the min() in qesgd_ref_level is
 * Eq. 4's first branch and takes that back to s. */
float qesgd_ref_inv(uint32_t s, float scale)
{
    return (float)s / scale;
}

static int valid_bits(uint32_t bits) { return bits == 2 || bits == 4 || bits == 8; }
static int valid_bucket(uint32_t B) { return B >= 64 && B <= 8192 && (B & (B - 1)) == 0; }

uint64_t qesgd_ref_num_buckets(uint64_t d, uint32_t bucket) { return (d + bucket - 1) / bucket; }
uint64_t qesgd_ref_code_bytes(uint64_t d, uint32_t bucket, uint32_t bits)
{
    return qesgd_ref_num_buckets(d, bucket) * bucket / 8 * bits;
}

/* ------------------------------------------------------------------------ */
/* Worker side: delta against the anchor (Sec. 2.2: compress z = u - w_t),   */
/* per-bucket scale (Sec. 3, bucket remark), stochastic rounding (Eq. 4),    */
/* sign + level packing (the grid of Eq. 3 has 2^b points).                  */
/*                                                                           */
/* local/anchor point at n elements whose first has GLOBAL index i0 (a       */
/* multiple of bucket); the last bucket is padded with +0.  anchor == NULL   */
/* means local already is z.  codes_out receives ceil(n/B)*B codes, element  */
/* e of the slice in bits [(e mod (32/bits))*bits, +bits) of little-endian   */
/* 32-bit word e / (32/bits); scales_out receives ceil(n/B) floats.          */
/* For QREF_SCALE_FIXED, fixed_delta is the grid spacing and nothing is      */
/* reduced: scale = fl32(s * delta) for every bucket.                        */
/* ------------------------------------------------------------------------ */
int qesgd_ref_encode(const float *local, const float *anchor, uint64_t n, uint64_t i0,
                     uint32_t bucket, uint32_t s, uint32_t bits, uint32_t scale_mode,
                     float fixed_delta, uint64_t seed, uint32_t worker, uint32_t epoch,
                     uint32_t *codes_out, float *scales_out, uint32_t *status)
{
    if (!valid_bits(bits) || !valid_bucket(bucket)) return QREF_EINVAL;
    if (s < 1 || s > (1u << (bits - 1)) - 1u) return QREF_EINVAL;
    if (n == 0) return QREF_OK; /* empty vector: nothing to write */
    if (!local || !codes_out || !scales_out) return QREF_EINVAL;
    if (scale_mode > QREF_SCALE_FIXED || (i0 % bucket) != 0) return QREF_EINVAL;
    if (scale_mode == QREF_SCALE_FIXED && !(fixed_delta > 0.0f && isfinite(fixed_delta)))
        return QREF_EINVAL;

    const uint32_t B = bucket;
    const uint32_t per_word = 32u / bits;
    const uint64_t nb = (n + B - 1) / B;
    float *z = (float *)malloc(sizeof(float) * B);
    double *scratch = (double *)malloc(sizeof(double) * B);
    if (!z || !scratch) { free(z); free(scratch); return QREF_ENOMEM; }
    memset(codes_out, 0, (size_t)(nb * B / per_word) * sizeof(uint32_t));

    for (uint64_t j = 0; j < nb; ++j) {
        const uint64_t lo = j * B;
        int finite = 1;
        for (uint32_t e = 0; e < B; ++e) {
            uint64_t idx = lo + e;
            float v = 0.0f;
            if (idx < n) v = anchor ? local[idx] - anchor[idx] : local[idx];
            if (scale_mode == QREF_SCALE_FIXED) {
                /* Nothing couples the elements of a bucket here.  +-Inf lies beyond
                 * the range and clips like any large value (first and last branch of
                 * Eq. 4); NaN has no place on the grid: flagged, encoded as 0. */
                if (isnan(v)) {
                    if (status) *status |= QREF_STATUS_NONFINITE;
                    v = 0.0f;
                }
            } else if (!isfinite(v)) {
                finite = 0;
            }
            z[e] = v;
        }
        float scale;
        if (scale_mode == QREF_SCALE_FIXED)
            scale = (float)s * fixed_delta;
        else
            scale = finite ? qesgd_ref_bucket_scale(z, B, scale_mode, scratch) : 0.0f;
        if (!finite || !isfinite(scale)) {
            if (status) *status |= QREF_STATUS_NONFINITE;
            scales_out[j] = 0.0f;
            continue; /* codes stay 0 */
        }
        if (scale < 0x1p-100f) { /* all-zero or vanishing bucket */
            scales_out[j] = 0.0f;
            continue;
        }
        scales_out[j] = scale;
        const float inv = qesgd_ref_inv(s, scale);
        for (uint32_t e = 0; e < B; ++e) {
            uint64_t idx = lo + e; /* index inside the slice */
            uint32_t h = qesgd_ref_draw16(seed, worker, epoch, i0 + idx);
            uint32_t level = qesgd_ref_level(fabsf(z[e]), inv, s, h);
            uint32_t sign = (z[e] < 0.0f && level > 0) ? 1u : 0u; /* no "-0" code */
            uint32_t code = (sign << (bits - 1)) | level;
            codes_out[idx / per_word] |= code << ((idx % per_word) * bits);
        }
    }
    free(z);
    free(scratch);
    return QREF_OK;
}

/* Value of one code: +-level * delta with delta = fl32(scale / s) (Eq. 3:
 * the quantised value is a grid point delta * k). */
static float code_value(uint32_t code, float step, uint32_t bits)
{
    uint32_t level = code & ((1u << (bits - 1)) - 1u);
    float v = (float)level * step;
    return (code >> (bits - 1)) & 1u ? -v : v;
}

static uint32_t code_at(const uint32_t *codes, uint64_t e, uint32_t bits)
{
    uint32_t per_word = 32u / bits;
    return (codes[e / per_word] >> ((e % per_word) * bits)) & ((1u << bits) - 1u);
}

/* Server side, decoding alone: out[e] = value of code e, e < n. */
int qesgd_ref_decode(const uint32_t *codes, const float *scales, uint64_t n, uint32_t bucket,
                     uint32_t s, uint32_t bits, float *out)
{
    if (!valid_bits(bits) || !valid_bucket(bucket)) return QREF_EINVAL;
    if (s < 1 || s > (1u << (bits - 1)) - 1u) return QREF_EINVAL;
    if (n == 0) return QREF_OK;
    if (!codes || !scales || !out) return QREF_EINVAL;
    for (uint64_t e = 0; e < n; ++e) {
        float step = scales[e / bucket] / (float)s;
        out[e] = code_value(code_at(codes, e, bits), step, bits);
    }
    return QREF_OK;
}

/* Server side: w <- w + (1/K) sum_k z_k (last line of the server task in
 * Algorithm 3; same average as the last line of Algorithms 1 and 2), the sum
 * taken in fp64 over k ascending and rounded once to fp32.  Worker k's codes
 * start code_stride BYTES after worker k-1's, its scales scale_stride floats. */
int qesgd_ref_decode_average_apply(float *param, uint64_t n, uint32_t K, const uint32_t *codes,
                                   uint64_t code_stride, const float *scales,
                                   uint64_t scale_stride, uint32_t bucket, uint32_t s,
                                   uint32_t bits)
{
    if (!valid_bits(bits) || !valid_bucket(bucket) || K == 0) return QREF_EINVAL;
    if (s < 1 || s > (1u << (bits - 1)) - 1u) return QREF_EINVAL;
    if (n == 0) return QREF_OK;
    if (!param || !codes || !scales) return QREF_EINVAL;
    for (uint64_t e = 0; e < n; ++e) {
        double sum = 0.0;
        for (uint32_t k = 0; k < K; ++k) {
            const uint32_t *ck = (const uint32_t *)((const char *)codes + (size_t)k * code_stride);
            const float *sk = scales + (size_t)k * scale_stride;
            float step = sk[e / bucket] / (float)s;
            sum += (double)code_value(code_at(ck, e, bits), step, bits);
        }
        param[e] = (float)((double)param[e] + sum / (double)K);
    }
    return QREF_OK;
}

/* One inner step of QESGD after the gradient update (Algorithm 2: z_{t,k+1} =
 * Q(z^_{t,k+1}), u_{t,k+1} = w_t + z_{t,k+1}; server task of Algorithm 3: z <- Q(z), send z):
 * on entry u holds w_t + z^ (the parameter after the SGD step); it is quantised against the
 * anchor w_t exactly as qesgd_ref_encode does (the inner step index plays the role of the
 * epoch in the draw counter), then u <- fl32(w_t + Q(z^)) and, if zsum is given,
 * zsum <- fl32(zsum + Q(z^)) (the running sum of the epoch average, last line of
 * Algorithms 2 and 3).  Q(z^) is the decoded value fl32(level * fl32(scale/s)) with its sign.
 * codes_out / scales_out receive the stream that would be sent to the workers. */
int qesgd_ref_requantize(float *u, const float *anchor, uint64_t n, uint64_t i0, uint32_t bucket,
                         uint32_t s, uint32_t bits, uint32_t scale_mode, float fixed_delta,
                         uint64_t seed, uint32_t worker, uint32_t step, float *zsum,
                         uint32_t *codes_out, float *scales_out, uint32_t *status)
{
    if (!anchor) return QREF_EINVAL;
    int rc = qesgd_ref_encode(u, anchor, n, i0, bucket, s, bits, scale_mode, fixed_delta, seed,
                              worker, step, codes_out, scales_out, status);
    if (rc != QREF_OK) return rc;
    for (uint64_t e = 0; e < n; ++e) {
        float delta = scales_out[e / bucket] / (float)s;
        float v = code_value(code_at(codes_out, e, bits), delta, bits);
        u[e] = anchor[e] + v;
        if (zsum) zsum[e] = zsum[e] + v;
    }
    return QREF_OK;
}

/* Gradient compression on the push side (Sec. 3, remark after Algorithm 3; the QSGD
 * baseline of Sec. 5 quantises gradients): the K streams hold quantised gradients and the
 * server takes w <- w + alpha * (1/K) sum_k g_k with alpha = -learning rate (Eq. 2 with the
 * minibatch mean replaced by the mean of the decoded workers).  alpha = 1 is the averaging
 * line of Algorithm 3.  fp64 sum over k ascending, one rounding to fp32. */
int qesgd_ref_decode_average_axpy(float *param, uint64_t n, uint32_t K, const uint32_t *codes,
                                  uint64_t code_stride, const float *scales,
                                  uint64_t scale_stride, uint32_t bucket, uint32_t s,
                                  uint32_t bits, float alpha)
{
    if (!valid_bits(bits) || !valid_bucket(bucket) || K == 0) return QREF_EINVAL;
    if (s < 1 || s > (1u << (bits - 1)) - 1u) return QREF_EINVAL;
    if (n == 0) return QREF_OK;
    if (!param || !codes || !scales) return QREF_EINVAL;
    for (uint64_t e = 0; e < n; ++e) {
        double sum = 0.0;
        for (uint32_t k = 0; k < K; ++k) {
            const uint32_t *ck = (const uint32_t *)((const char *)codes + (size_t)k * code_stride);
            const float *sk = scales + (size_t)k * scale_stride;
            float step = sk[e / bucket] / (float)s;
            sum += (double)code_value(code_at(ck, e, bits), step, bits);
        }
        param[e] = (float)((double)param[e] + (double)alpha * (sum / (double)K));
    }
    return QREF_OK;
}

/* ------------------------------------------------------------------------ */
/* Logistic regression (Sec. 1: f_i(w) = log(1 + exp(-y_i x_i^T w))) and the */
/* minibatch SGD update of Eq. 2.  fp64 accumulation, u rounded to fp32 once */
/* per step.                                                                 */
/* ------------------------------------------------------------------------ */

/* Mean loss over m rows of X (row-major, m x d). */
double qesgd_ref_lr_loss(const float *X, const float *y, uint64_t m, uint64_t d, const float *w)
{
    double total = 0.0;
    for (uint64_t j = 0; j < m; ++j) {
        double dot = 0.0;
        for (uint64_t i = 0; i < d; ++i) dot += (double)X[j * d + i] * (double)w[i];
        double t = -(double)y[j] * dot;
        /* log(1 + e^t) without overflow */
        total += t > 0.0 ? t + log1p(exp(-t)) : log1p(exp(t));
    }
    return total / (double)m;
}

/* One step of Eq. 2 on the m rows of Xb: u <- u - (lr/m) sum_j grad f_j(u),
 * grad f_j(u) = c_j x_j with c_j = -y_j / (1 + exp(y_j x_j^T u)). */
int qesgd_ref_lr_sgd_step(const float *Xb, const float *yb, uint32_t m, uint64_t d, float lr,
                          float *u)
{
    if (!Xb || !yb || !u || m == 0 || d == 0) return QREF_EINVAL;
    double *c = (double *)malloc(sizeof(double) * m);
    if (!c) return QREF_ENOMEM;
    for (uint32_t j = 0; j < m; ++j) {
        double dot = 0.0;
        for (uint64_t i = 0; i < d; ++i) dot += (double)Xb[(uint64_t)j * d + i] * (double)u[i];
        c[j] = -(double)yb[j] / (1.0 + exp((double)yb[j] * dot));
    }
    const double rate = (double)lr / (double)m;
    for (uint64_t i = 0; i < d; ++i) {
        double g = 0.0;
        for (uint32_t j = 0; j < m; ++j) g += c[j] * (double)Xb[(uint64_t)j * d + i];
        u[i] = (float)((double)u[i] - rate * g);
    }
    free(c);
    return QREF_OK;
}

/* A worker's local epoch (worker task of Algorithm 3 with the minibatches
 * taken in row order): rows [0, n_local) in consecutive batches of `batch`
 * rows; a last partial batch uses its own size in Eq. 2. */
int qesgd_ref_lr_local_epoch(const float *X, const float *y, uint64_t n_local, uint64_t d,
                             uint32_t batch, float lr, float *u)
{
    if (!X || !y || !u || n_local == 0 || d == 0 || batch == 0) return QREF_EINVAL;
    for (uint64_t r = 0; r < n_local; r += batch) {
        uint32_t m = (uint32_t)((n_local - r < batch) ? (n_local - r) : batch);
        int rc = qesgd_ref_lr_sgd_step(X + r * d, y + r, m, d, lr, u);
        if (rc != QREF_OK) return rc;
    }
    return QREF_OK;
}

/* Minibatch mean gradient of the logistic loss at w (the summand of Eq. 2):
 * g = (1/m) sum_j c_j x_j, c_j = -y_j / (1 + exp(y_j x_j^T w)); fp64, rounded once. */
int qesgd_ref_lr_gradient(const float *Xb, const float *yb, uint32_t m, uint64_t d, const float *w,
                          float *g)
{
    if (!Xb || !yb || !w || !g || m == 0 || d == 0) return QREF_EINVAL;
    double *c = (double *)malloc(sizeof(double) * m);
    if (!c) return QREF_ENOMEM;
    for (uint32_t j = 0; j < m; ++j) {
        double dot = 0.0;
        for (uint64_t i = 0; i < d; ++i) dot += (double)Xb[(uint64_t)j * d + i] * (double)w[i];
        c[j] = -(double)yb[j] / (1.0 + exp((double)yb[j] * dot));
    }
    for (uint64_t i = 0; i < d; ++i) {
        double acc = 0.0;
        for (uint32_t j = 0; j < m; ++j) acc += c[j] * (double)Xb[(uint64_t)j * d + i];
        g[i] = (float)(acc / (double)m);
    }
    free(c);
    return QREF_OK;
}
