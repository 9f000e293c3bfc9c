// C ABI of libqesgd.so: context management, argument validation, dispatch.
// Contracts are stated in include/qesgd.h.
#include <new>

#include "qesgd_internal.h"

namespace {

inline bool aligned(const void *p, uintptr_t a) { return ((uintptr_t)p % a) == 0; }

inline int log2_exact(uint32_t v)
{
    int l = 0;
    while ((1u << l) < v) ++l;
    return l;
}

inline bool valid_bucket(uint32_t b)
{
    return b >= QESGD_MIN_BUCKET && b <= QESGD_MAX_BUCKET && (b & (b - 1u)) == 0u;
}

inline bool valid_codec(uint32_t bucket, uint32_t s, uint32_t bits)
{
    if (!(bits == 2 || bits == 4 || bits == 8)) return false;
    if (!valid_bucket(bucket)) return false;
    return s >= 1u && s <= (1u << (bits - 1)) - 1u;
}

// Binds the context's device for the duration of a call and restores the caller's.
struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int device)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == device) || cudaSetDevice(device) == cudaSuccess;
        if (prev == device) prev = -1;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

int cuda_fail(qesgd_ctx *ctx, int err)
{
    ctx->last_cuda_error = err;
    return QESGD_ECUDA;
}

}  // namespace

extern "C" {

int qesgd_create(qesgd_ctx **out, int device, void *cuda_stream)
{
    if (!out) return QESGD_EINVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) return QESGD_ECUDA;
    if (device < 0 || device >= count) return QESGD_EINVAL;
    qesgd_ctx *ctx = new (std::nothrow) qesgd_ctx();
    if (!ctx) return QESGD_ENOMEM;
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->launches = 0;
    ctx->last_cuda_error = 0;
    ctx->d_status = nullptr;
    ctx->d_lr_work = nullptr;
    ctx->lr_work_floats = QESGD_LR_WORK_FLOATS;
    ctx->wait_ns = QESGD_DEFAULT_WAIT_NS;
    ctx->drop_cta = 0xFFFFFFFFu;
    DeviceGuard guard(device);
    if (!guard.ok) { delete ctx; return QESGD_ECUDA; }
    cudaError_t e = cudaMalloc((void **)&ctx->d_status, 256);
    if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->d_lr_work, ctx->lr_work_floats * sizeof(float));
    // the head of the workspace holds arrival counters that the kernels leave at zero
    if (e == cudaSuccess) e = cudaMemset(ctx->d_lr_work, 0, 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 256);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) {
        cudaFree(ctx->d_status);
        cudaFree(ctx->d_lr_work);
        delete ctx;
        return e == cudaErrorMemoryAllocation ? QESGD_ENOMEM : QESGD_ECUDA;
    }
    *out = ctx;
    return QESGD_OK;
}

int qesgd_destroy(qesgd_ctx *ctx)
{
    if (!ctx) return QESGD_EINVAL;
    DeviceGuard guard(ctx->device);
    if (guard.ok) {
        cudaStreamSynchronize(ctx->stream);
        cudaFree(ctx->d_status);
        cudaFree(ctx->d_lr_work);
    }
    delete ctx;
    return guard.ok ? QESGD_OK : QESGD_ECUDA;
}

int qesgd_set_stream(qesgd_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return QESGD_EINVAL;
    ctx->stream = (cudaStream_t)cuda_stream;
    return QESGD_OK;
}

int qesgd_set_wait_limit(qesgd_ctx *ctx, uint64_t nanoseconds)
{
    if (!ctx || nanoseconds > QESGD_MAX_WAIT_NS) return QESGD_EINVAL;
    ctx->wait_ns = nanoseconds == 0 ? QESGD_DEFAULT_WAIT_NS : nanoseconds;
    return QESGD_OK;
}

int qesgd_debug_drop_signal(qesgd_ctx *ctx, int64_t cta)
{
    if (!ctx || cta < -1 || cta > 0x7FFFFFFF) return QESGD_EINVAL;
    ctx->drop_cta = cta < 0 ? 0xFFFFFFFFu : (uint32_t)cta;
    return QESGD_OK;
}

uint64_t qesgd_num_buckets(uint64_t d, uint32_t bucket)
{
    if (!valid_bucket(bucket)) return 0;
    return (d + bucket - 1) / bucket;
}

uint64_t qesgd_code_bytes(uint64_t d, uint32_t bucket, uint32_t bits)
{
    if (!valid_bucket(bucket) || !(bits == 2 || bits == 4 || bits == 8)) return 0;
    return qesgd_num_buckets(d, bucket) * (bucket / 8u) * bits;
}

static int encode_impl(qesgd_ctx *ctx, const float *local, uint64_t local_stride,
                       const float *anchor, uint64_t d, uint32_t K, uint32_t bucket, uint32_t s,
                       uint32_t bits, uint32_t scale_mode, float fixed_delta, uint64_t seed,
                       uint32_t worker0, uint32_t epoch, uint32_t *codes_out,
                       uint64_t code_stride, float *scales_out, uint64_t scale_stride,
                       float *u_out, float *zsum)
{
    if (!ctx) return QESGD_EINVAL;
    if (!valid_codec(bucket, s, bits) || scale_mode > QESGD_SCALE_FIXED) return QESGD_EINVAL;
    if (K < 1 || K > QESGD_MAX_WORKERS) return QESGD_EINVAL;
    if (scale_mode == QESGD_SCALE_FIXED && !(fixed_delta > 0.0f && fixed_delta <= 3.402823466e38f))
        return QESGD_EINVAL;
    if (d == 0) return QESGD_OK;
    if (!local || !codes_out || !scales_out) return QESGD_EINVAL;
    if (!aligned(local, 4) || !aligned(anchor, 4)) return QESGD_EINVAL;
    if (!aligned(codes_out, 16) || !aligned(scales_out, 16)) return QESGD_EINVAL;
    const uint64_t nb = qesgd_num_buckets(d, bucket);
    const uint64_t cbytes = qesgd_code_bytes(d, bucket, bits);
    if (K > 1) {
        if (local_stride < d || code_stride < cbytes || scale_stride < nb) return QESGD_EINVAL;
        if (code_stride % 16 != 0 || (scale_stride * 4) % 16 != 0) return QESGD_EINVAL;
    }
    EncodeArgs a;
    a.local = local;
    a.local_stride = K > 1 ? local_stride : 0;
    a.anchor = anchor;
    a.d = d;
    a.padded = nb * bucket;
    a.log2_bucket = (uint32_t)log2_exact(bucket);
    a.s = s;
    a.fixed_scale = scale_mode == QESGD_SCALE_FIXED ? (float)s * fixed_delta : 0.0f;
    for (uint32_t r = 0; r < 10; ++r) {   // Philox4x32 key schedule (Weyl sequence)
        a.round_key[r][0] = (uint32_t)seed + r * 0x9E3779B9u;
        a.round_key[r][1] = (uint32_t)(seed >> 32) + r * 0xBB67AE85u;
    }
    a.worker0 = worker0;
    a.epoch = epoch;
    a.K = K;
    a.codes = codes_out;
    a.code_stride = K > 1 ? code_stride : 0;
    a.scales = scales_out;
    a.scale_stride = K > 1 ? scale_stride : 0;
    a.status = ctx->d_status;
    a.u_out = u_out;
    a.zsum = zsum;
    const bool vec = aligned(local, 32) && aligned(anchor, 32) && (a.local_stride % 8 == 0);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    const int e = qesgd_launch_encode(a, K, bits, scale_mode, vec, ctx->sm_count, ctx->stream);
    if (e != 0) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return QESGD_OK;
}

int qesgd_encode_batch(qesgd_ctx *ctx, const float *local, uint64_t local_stride,
                       const float *anchor, uint64_t d, uint32_t K, uint32_t bucket, uint32_t s,
                       uint32_t bits, uint32_t scale_mode, float fixed_delta, uint64_t seed,
                       uint32_t worker0, uint32_t epoch, uint32_t *codes_out,
                       uint64_t code_stride, float *scales_out, uint64_t scale_stride)
{
    return encode_impl(ctx, local, local_stride, anchor, d, K, bucket, s, bits, scale_mode,
                       fixed_delta, seed, worker0, epoch, codes_out, code_stride, scales_out,
                       scale_stride, nullptr, nullptr);
}

int qesgd_requantize(qesgd_ctx *ctx, float *u, const float *anchor, uint64_t d, uint32_t bucket,
                     uint32_t s, uint32_t bits, uint32_t scale_mode, float fixed_delta,
                     uint64_t seed, uint32_t worker, uint32_t step, float *zsum,
                     uint32_t *codes_out, float *scales_out)
{
    if (!anchor || !u) return QESGD_EINVAL;
    if (zsum && !aligned(zsum, 4)) return QESGD_EINVAL;
    if (zsum && (aligned(u, 32) != aligned(zsum, 32))) return QESGD_EINVAL;  // one load path for both
    return encode_impl(ctx, u, 0, anchor, d, 1, bucket, s, bits, scale_mode, fixed_delta, seed,
                       worker, step, codes_out, 0, scales_out, 0, u, zsum);
}

int qesgd_lr_qesgd_step(qesgd_ctx *ctx, const float *Xb, const float *yb, uint32_t m, uint64_t d,
                        float lr, float *u, const float *anchor, uint32_t bucket, uint32_t s,
                        uint32_t bits, uint32_t scale_mode, float fixed_delta, uint64_t seed,
                        uint32_t worker, uint32_t step, float *zsum, uint32_t *codes_out,
                        float *scales_out)
{
    if (!ctx) return QESGD_EINVAL;
    if (m < 1 || m > QESGD_MAX_LR_BATCH) return QESGD_EINVAL;
    if (!valid_codec(bucket, s, bits) || scale_mode > QESGD_SCALE_FIXED) return QESGD_EINVAL;
    if (scale_mode == QESGD_SCALE_FIXED && !(fixed_delta > 0.0f && fixed_delta <= 3.402823466e38f))
        return QESGD_EINVAL;
    if (d == 0) return QESGD_OK;
    if (!Xb || !yb || !u || !anchor || !codes_out || !scales_out) return QESGD_EINVAL;
    if (!aligned(Xb, 4) || !aligned(yb, 4) || !aligned(u, 4) || !aligned(anchor, 4)) return QESGD_EINVAL;
    if (zsum && !aligned(zsum, 4)) return QESGD_EINVAL;
    if (zsum && (aligned(u, 32) != aligned(zsum, 32))) return QESGD_EINVAL;
    if (!aligned(codes_out, 16) || !aligned(scales_out, 16)) return QESGD_EINVAL;
    const bool fused = bucket <= 1024u && d % 4 == 0 && aligned(Xb, 16) && aligned(u, 16) &&
                       (uint64_t)m <= ctx->lr_work_floats;
    if (!fused) {   // the same two steps as separate calls
        const int rc = qesgd_lr_local_epoch_batch(ctx, Xb, yb, m, d, 1, m, lr, u, 0);
        if (rc != QESGD_OK) return rc;
        return qesgd_requantize(ctx, u, anchor, d, bucket, s, bits, scale_mode, fixed_delta, seed, worker,
                                step, zsum, codes_out, scales_out);
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    QstepArgs q;
    const float *margins = nullptr;
    int e = qesgd_launch_lr_margins(Xb, yb, m, d, u, ctx->d_lr_work, ctx->lr_work_floats, ctx->stream, &margins);
    if (e != 0) return cuda_fail(ctx, e);
    ctx->launches += 1;
    EncodeArgs &a = q.e;
    const uint64_t nb = qesgd_num_buckets(d, bucket);
    a.local = u;
    a.local_stride = 0;
    a.anchor = anchor;
    a.d = d;
    a.padded = nb * bucket;
    a.log2_bucket = (uint32_t)log2_exact(bucket);
    a.s = s;
    a.fixed_scale = scale_mode == QESGD_SCALE_FIXED ? (float)s * fixed_delta : 0.0f;
    for (uint32_t r = 0; r < 10; ++r) {
        a.round_key[r][0] = (uint32_t)seed + r * 0x9E3779B9u;
        a.round_key[r][1] = (uint32_t)(seed >> 32) + r * 0xBB67AE85u;
    }
    a.worker0 = worker;
    a.epoch = step;
    a.K = 1;
    a.codes = codes_out;
    a.code_stride = 0;
    a.scales = scales_out;
    a.scale_stride = 0;
    a.status = ctx->d_status;
    a.u_out = u;
    a.zsum = zsum;
    q.X = Xb;
    q.y = yb;
    q.m = m;
    q.rate = lr / (float)m;
    q.margins = margins;
    switch (bits) {
        case 2: e = qesgd_launch_lr_qstep_2(q, scale_mode, ctx->stream); break;
        case 4: e = qesgd_launch_lr_qstep_4(q, scale_mode, ctx->stream); break;
        default: e = qesgd_launch_lr_qstep_8(q, scale_mode, ctx->stream); break;
    }
    if (e != 0) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return QESGD_OK;
}

int qesgd_encode(qesgd_ctx *ctx, const float *local, const float *anchor, uint64_t d,
                 uint32_t bucket, uint32_t s, uint32_t bits, uint32_t scale_mode,
                 float fixed_delta, uint64_t seed, uint32_t worker, uint32_t epoch,
                 uint32_t *codes_out, float *scales_out)
{
    return qesgd_encode_batch(ctx, local, 0, anchor, d, 1, bucket, s, bits, scale_mode,
                              fixed_delta, seed, worker, epoch, codes_out, 0, scales_out, 0);
}

int qesgd_decode_average_axpy(qesgd_ctx *ctx, float *param, uint64_t d, uint32_t K,
                              const uint32_t *codes, uint64_t code_stride, const float *scales,
                              uint64_t scale_stride, uint32_t bucket, uint32_t s, uint32_t bits,
                              float alpha)
{
    if (!ctx) return QESGD_EINVAL;
    if (!valid_codec(bucket, s, bits)) return QESGD_EINVAL;
    if (K < 1 || K > QESGD_MAX_WORKERS) return QESGD_EINVAL;
    if (!(alpha >= -3.402823466e38f && alpha <= 3.402823466e38f)) return QESGD_EINVAL;
    if (d == 0) return QESGD_OK;
    if (!param || !codes || !scales) return QESGD_EINVAL;
    if (!aligned(param, 4) || !aligned(codes, 16) || !aligned(scales, 16)) return QESGD_EINVAL;
    const uint64_t nb = qesgd_num_buckets(d, bucket);
    if (K > 1) {
        if (code_stride < qesgd_code_bytes(d, bucket, bits) || scale_stride < nb) return QESGD_EINVAL;
        if (code_stride % 16 != 0 || (scale_stride * 4) % 16 != 0) return QESGD_EINVAL;
    }
    DecodeArgs a;
    a.param = param;
    a.d = d;
    a.nb = nb;
    a.K = K;
    a.avg_scale = alpha / (float)K;
    a.log2_bucket = (uint32_t)log2_exact(bucket);
    a.s = s;
    a.codes = codes;
    a.code_stride = K > 1 ? code_stride : 0;
    a.scales = scales;
    a.scale_stride = K > 1 ? scale_stride : 0;
    a.status = ctx->d_status;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    const int e = qesgd_launch_decode_average_apply(a, bits, aligned(param, 32), ctx->stream);
    if (e != 0) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return QESGD_OK;
}

int qesgd_decode_average_apply(qesgd_ctx *ctx, float *param, uint64_t d, uint32_t K,
                               const uint32_t *codes, uint64_t code_stride, const float *scales,
                               uint64_t scale_stride, uint32_t bucket, uint32_t s, uint32_t bits)
{
    return qesgd_decode_average_axpy(ctx, param, d, K, codes, code_stride, scales, scale_stride,
                                     bucket, s, bits, 1.0f);
}

int qesgd_decode(qesgd_ctx *ctx, const uint32_t *codes, const float *scales, uint64_t d,
                 uint32_t bucket, uint32_t s, uint32_t bits, float *out)
{
    if (!ctx) return QESGD_EINVAL;
    if (!valid_codec(bucket, s, bits)) return QESGD_EINVAL;
    if (d == 0) return QESGD_OK;
    if (!out || !codes || !scales) return QESGD_EINVAL;
    if (!aligned(out, 4) || !aligned(codes, 16) || !aligned(scales, 16)) return QESGD_EINVAL;
    DecodeArgs a;
    a.param = out;
    a.d = d;
    a.nb = qesgd_num_buckets(d, bucket);
    a.K = 1;
    a.avg_scale = 1.0f;
    a.log2_bucket = (uint32_t)log2_exact(bucket);
    a.s = s;
    a.codes = codes;
    a.code_stride = 0;
    a.scales = scales;
    a.scale_stride = 0;
    a.status = ctx->d_status;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    const int e = qesgd_launch_decode(a, bits, aligned(out, 32), ctx->stream);
    if (e != 0) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return QESGD_OK;
}

int qesgd_lr_local_epoch_batch(qesgd_ctx *ctx, const float *X, const float *y, uint64_t n_local,
                               uint64_t d, uint32_t K, uint32_t batch, float lr, float *u,
                               uint64_t u_stride)
{
    if (!ctx) return QESGD_EINVAL;
    if (K < 1 || K > QESGD_MAX_WORKERS) return QESGD_EINVAL;
    if (batch < 1 || batch > QESGD_MAX_LR_BATCH) return QESGD_EINVAL;
    if (n_local == 0 || d == 0) return QESGD_OK;
    if (!X || !y || !u) return QESGD_EINVAL;
    if (!aligned(X, 4) || !aligned(y, 4) || !aligned(u, 4)) return QESGD_EINVAL;
    if (K > 1 && u_stride < d) return QESGD_EINVAL;
    const uint32_t m_max = (uint32_t)(n_local < batch ? n_local : batch);
    if ((uint64_t)K * m_max > ctx->lr_work_floats) return QESGD_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    {   // the whole epoch in one persistent kernel where its shape allows
        int launched = 0;
        const int e = qesgd_launch_lr_epoch_fused(X, y, n_local, d, K, batch, lr, u, K > 1 ? u_stride : 0,
                                                  ctx->d_lr_work, ctx->lr_work_floats, ctx->d_status,
                                                  ctx->device, ctx->sm_count, ctx->wait_ns, ctx->drop_cta,
                                                  ctx->stream, &launched);
        ctx->launches += (uint64_t)launched;
        if (e > 0) return cuda_fail(ctx, e);
        if (e == 0) return QESGD_OK;
    }
    for (uint64_t r = 0; r < n_local; r += batch) {
        const uint32_t m = (uint32_t)(n_local - r < batch ? n_local - r : batch);
        int launched = 0;
        const int e = qesgd_launch_lr_step(X + r * d, n_local * d, y + r, n_local, m, d, K, lr, u,
                                           K > 1 ? u_stride : 0, ctx->d_lr_work,
                                           ctx->lr_work_floats, ctx->stream, &launched);
        ctx->launches += (uint64_t)launched;
        if (e != 0) return cuda_fail(ctx, e);
    }
    return QESGD_OK;
}

int qesgd_lr_local_epoch(qesgd_ctx *ctx, const float *X, const float *y, uint64_t n_local,
                         uint64_t d, uint32_t batch, float lr, float *u)
{
    return qesgd_lr_local_epoch_batch(ctx, X, y, n_local, d, 1, batch, lr, u, 0);
}

int qesgd_lr_sgd_step(qesgd_ctx *ctx, const float *Xb, const float *yb, uint32_t m, uint64_t d,
                      float lr, float *u)
{
    if (m < 1 || m > QESGD_MAX_LR_BATCH) return QESGD_EINVAL;
    return qesgd_lr_local_epoch_batch(ctx, Xb, yb, m, d, 1, m, lr, u, 0);
}

int qesgd_lr_gradient(qesgd_ctx *ctx, const float *Xb, const float *yb, uint32_t m, uint64_t d,
                      const float *w, float *g_out)
{
    if (!ctx) return QESGD_EINVAL;
    if (m < 1 || m > QESGD_MAX_LR_BATCH) return QESGD_EINVAL;
    if (d == 0) return QESGD_OK;
    if (!Xb || !yb || !w || !g_out || w == g_out) return QESGD_EINVAL;
    if (!aligned(Xb, 4) || !aligned(yb, 4) || !aligned(w, 4) || !aligned(g_out, 4)) return QESGD_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    int launched = 0;
    const int e = qesgd_launch_lr_gradient(Xb, yb, m, d, w, g_out, ctx->d_lr_work,
                                           ctx->lr_work_floats, ctx->stream, &launched);
    ctx->launches += (uint64_t)launched;
    if (e != 0) return cuda_fail(ctx, e);
    return QESGD_OK;
}

int qesgd_status(qesgd_ctx *ctx, uint32_t *flags_out)
{
    if (!ctx || !flags_out) return QESGD_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    cudaError_t e = cudaMemcpyAsync(flags_out, ctx->d_status, sizeof(uint32_t),
                                    cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(uint32_t), ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
    return QESGD_OK;
}

int qesgd_debug_build(void)
{
#ifdef QESGD_DEBUG
    return 1;
#else
    return 0;
#endif
}

int qesgd_debug_range_selftest(qesgd_ctx *ctx)
{
    if (!ctx) return QESGD_EINVAL;
#ifdef QESGD_DEBUG
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, (int)cudaErrorInvalidDevice);
    const int e = qesgd_launch_range_selftest(ctx->d_status, ctx->stream);
    if (e != 0) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return QESGD_OK;
#else
    return QESGD_EINVAL;
#endif
}

uint64_t qesgd_launch_count(const qesgd_ctx *ctx) { return ctx ? ctx->launches : 0; }

int qesgd_last_cuda_error(const qesgd_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

const char *qesgd_strerror(int code)
{
    switch (code) {
        case QESGD_OK: return "ok";
        case QESGD_EINVAL: return "invalid argument";
        case QESGD_ECUDA: return "CUDA error (see qesgd_last_cuda_error)";
        case QESGD_ENOMEM: return "out of memory";
        case QESGD_ELIMIT: return "size exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown error";
    }
}

}  // extern "C"
