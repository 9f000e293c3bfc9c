/*
 * qesgd.h -- C ABI of the B200 (sm_100a) QESGD hot path.
 *
 * Quantized Epoch-SGD (Zhao, Gao, Li, arXiv 1901.03040) compresses the epoch
 * delta z = u - w_t of a parameter vector against the server's anchor w_t
 * with a uniform stochastic quantiser and averages the quantised deltas on the
 * server.  This library is that data path on one GPU:
 *
 *   worker side   qesgd_encode[_batch]         delta, per-bucket scale, stochastic
 *                                              rounding to s levels, sign+level packing
 *   server side   qesgd_decode_average_apply   decode K streams, average, add to w_t
 *                 qesgd_decode                 decode one stream to fp32
 *   local epoch   qesgd_lr_sgd_step / qesgd_lr_local_epoch[_batch]
 *                                              logistic-regression minibatch SGD
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller and valid on
 *     the context's device, unless marked "host".  The library never frees or
 *     reallocates caller memory.  Vectors (local, anchor, param, out, X, u) need
 *     4-byte alignment; 32-byte alignment of the base pointers and of the
 *     per-worker strides selects the fast 256-bit load path.  Code and scale
 *     buffers must be 16-byte aligned and their per-worker strides multiples of
 *     16 bytes.
 *   - Calls enqueue work on the context's stream and return without waiting;
 *     only qesgd_status and qesgd_destroy synchronise.  The codec calls (encode,
 *     encode_batch, requantize, decode, decode_average_apply/_axpy) do nothing but
 *     launch kernels on that stream, so they may be recorded by CUDA stream capture
 *     and replayed as a graph (worth it when a launch is as short as a host call).
 *   - Return value: QESGD_OK or a negative error code.  Nothing is enqueued
 *     when an error is returned.  No call aborts or throws.
 *   - Data problems (a non-finite value in a bucket) never fail a call: the
 *     bucket is encoded as scale 0 / codes 0 and QESGD_STATUS_NONFINITE is set
 *     in the context's status word, read with qesgd_status.
 *   - Element counts d are 64-bit; d == 0 is a valid no-op.
 *
 * Stream format (shared by encode and decode)
 *   bucket j covers elements [j*bucket, (j+1)*bucket); the last bucket is padded
 *   with zeros; nb = ceil(d/bucket).  A worker's stream is nb*bucket codes of
 *   `bits` bits (bits in {2,4,8}; top bit = sign, low bits-1 bits = level in
 *   [0, s]); element e occupies bits [(e mod (32/bits))*bits, +bits) of the
 *   little-endian 32-bit word e/(32/bits).  Padding codes are 0.  Its scales are
 *   nb floats; a decoded value is +-level * fl32(scale/s).
 */
#ifndef QESGD_H
#define QESGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QESGD_OK 0
#define QESGD_EINVAL (-1) /* NULL / misaligned pointer, unsupported bits, bucket, s, K, mode */
#define QESGD_ECUDA (-2)  /* CUDA runtime or launch error; see qesgd_last_cuda_error      */
#define QESGD_ENOMEM (-3) /* host or device allocation failed (qesgd_create only)          */
#define QESGD_ELIMIT (-4) /* size beyond the fixed scratch of a no-allocation entry point   */

#define QESGD_SCALE_NORM 0u  /* scale = L2 norm of the bucket's delta              */
#define QESGD_SCALE_MAX 1u   /* scale = largest magnitude of the bucket's delta    */
#define QESGD_SCALE_FIXED 2u /* scale = s*delta with the grid spacing delta given  */

#define QESGD_STATUS_NONFINITE 1u /* a bucket held NaN/Inf or its norm overflowed fp32 */
#define QESGD_STATUS_TIMEOUT 2u   /* a bounded wait inside the local-epoch kernel ran out   */
#define QESGD_STATUS_RANGE 4u     /* debug build only: a codec kernel computed an index outside
                                     its buffer; the access was skipped                       */

#define QESGD_MAX_WORKERS 64u
#define QESGD_MIN_BUCKET 64u
#define QESGD_MAX_BUCKET 8192u
#define QESGD_MAX_LR_BATCH 1024u
#define QESGD_NOALLOC_MAX_LR_BATCH 256u /* rows per step of qesgd_lr_sgd_step_noalloc */

typedef struct qesgd_ctx qesgd_ctx;

/* Create a context bound to `device` and to `cuda_stream` (a cudaStream_t passed
 * as void*; NULL = the legacy default stream).  Allocates 256 bytes (status word) and
 * 4 MiB (logistic-regression workspace) of device memory that qesgd_destroy frees.
 * This is the only call that allocates. */
int qesgd_create(qesgd_ctx **out, int device, void *cuda_stream);
int qesgd_destroy(qesgd_ctx *ctx);
/* Rebind the context to another stream of the same device. */
int qesgd_set_stream(qesgd_ctx *ctx, void *cuda_stream);

/* ceil(d / bucket); 0 for an invalid bucket. */
uint64_t qesgd_num_buckets(uint64_t d, uint32_t bucket);
/* Bytes of one worker's code stream: nb * bucket * bits / 8 (a multiple of 16). */
uint64_t qesgd_code_bytes(uint64_t d, uint32_t bucket, uint32_t bits);

/*
 * Worker side (paper Sec. 2.2: compress z = u - w_t; Sec. 3: bucket remark;
 * Eq. 4: stochastic rounding; Eq. 3: b-bit grid).
 *
 *   z_i   = fl32(local_i - anchor_i), or local_i when anchor == NULL
 *   scale = fl32(sqrt(sum z_i^2))  (NORM; fp64 sum over the balanced binary tree on
 *           index order)  |  max |z_i|  (MAX)  |  fl32(s*fixed_delta)  (FIXED)
 *   r_i   = min(fl32(|z_i| * fl32(s/scale)), s);  level_i = floor(r_i) + [u_i < frac(r_i)]
 *   u_i   = (h_i + 1/2) / 2^16 with h_i the 16-bit draw of element i from
 *           Philox4x32-10, counter (i>>3 low, i>>3 high, worker, epoch), key = seed,
 *           32-bit word (i>>1)&3, half (i&1)
 *   code  = sign<<(bits-1) | level, sign = (z_i < 0 and level > 0)
 * A bucket with scale < 2^-100 or non-finite content is written as scale 0, codes 0.
 *
 * local, anchor: float[d] (anchor may be NULL).  codes_out: qesgd_code_bytes()
 * bytes.  scales_out: float[nb].  All nb*bucket codes and nb scales are written.
 * s in [1, 2^(bits-1)-1]; bucket a power of two in [64, 8192]; fixed_delta is
 * read only for QESGD_SCALE_FIXED and must then be finite and > 0.
 */
int qesgd_encode(qesgd_ctx *ctx, const float *local, const float *anchor, uint64_t d,
                 uint32_t bucket, uint32_t s, uint32_t bits, uint32_t scale_mode,
                 float fixed_delta, uint64_t seed, uint32_t worker, uint32_t epoch,
                 uint32_t *codes_out, float *scales_out);

/* K workers in one launch (K simulated workers of Algorithm 3 on one device):
 * worker k reads local + k*local_stride (elements) against the shared anchor,
 * draws with worker id worker0 + k, writes codes_out + k*code_stride (BYTES) and
 * scales_out + k*scale_stride (elements).  1 <= K <= 64. */
int qesgd_encode_batch(qesgd_ctx *ctx, const float *local, uint64_t local_stride,
                       const float *anchor, uint64_t d, uint32_t K, uint32_t bucket, uint32_t s,
                       uint32_t bits, uint32_t scale_mode, float fixed_delta, uint64_t seed,
                       uint32_t worker0, uint32_t epoch, uint32_t *codes_out,
                       uint64_t code_stride, float *scales_out, uint64_t scale_stride);

/*
 * Server side (last line of the server task of Algorithm 3, same average as the
 * last line of Algorithms 1 and 2):
 *   param_i <- param_i + (1/K) * sum_k (+-level_{k,i} * fl32(scale_{k,bucket(i)} / s))
 * param: float[d], updated in place: every element receives exactly one add,
 * fl32(param_i + fl32(sum_i * (1/K))), carried out by the memory system (a reduction,
 * not a load and a store of the kernel), so the line is read and written once and the
 * result does not depend on any order.  Stream k starts at codes + k*code_stride
 * (BYTES) and scales + k*scale_stride (elements).  fp32 accumulation over k
 * ascending; result within 1e-6 * max(|param_i|, max_k scale) of the exactly
 * rounded value.  1 <= K <= 64.
 */
int qesgd_decode_average_apply(qesgd_ctx *ctx, float *param, uint64_t d, uint32_t K,
                               const uint32_t *codes, uint64_t code_stride, const float *scales,
                               uint64_t scale_stride, uint32_t bucket, uint32_t s, uint32_t bits);

/*
 * Per-step QESGD (Algorithm 2: z_{t,k+1} = Q(z^_{t,k+1}), u_{t,k+1} = w_t + z_{t,k+1};
 * server task of Algorithm 3: z <- Q(z), send z to all workers).  On entry u (float[d])
 * holds w_t + z^, the parameter after the gradient step.  In one pass the delta against
 * `anchor` (= w_t, required) is quantised exactly as by qesgd_encode (`step`, the inner
 * iteration index, takes the place of the epoch in the draw counter; the stream that would
 * be sent goes to codes_out / scales_out), u is overwritten with fl32(anchor + Q(z^)), and,
 * if zsum != NULL, zsum_i <- fl32(zsum_i + Q(z^)_i): the running sum of the epoch average
 * w_{t+1} = w_t + (1/K_t) sum_k z_{t,k} (last line of Algorithms 2 and 3; apply it with any
 * axpy).  Q(z^)_i = +-level_i * fl32(scale/s).  Everything is bit-exact against the oracle.
 * u and zsum (float[d]) must both or neither be 32-byte aligned; other arguments as for
 * qesgd_encode.
 */
int qesgd_requantize(qesgd_ctx *ctx, float *u, const float *anchor, uint64_t d, uint32_t bucket,
                     uint32_t s, uint32_t bits, uint32_t scale_mode, float fixed_delta,
                     uint64_t seed, uint32_t worker, uint32_t step, float *zsum,
                     uint32_t *codes_out, float *scales_out);

/*
 * The whole inner iteration of Algorithm 2 on logistic regression (its three lines: z^ = z -
 * eta * grad f(u), z = Q(z^), u = w_t + z; Eq. 2 for the gradient step on the m rows of Xb):
 * qesgd_lr_sgd_step followed by qesgd_requantize, without the updated parameter ever being
 * written before it is quantised.  Two launches: the margin pass, then one kernel in which a
 * CTA forms u^ = u - (lr/m) sum_j c_j x_j for a tile of 1024 columns in shared memory and
 * requantises it there (u, zsum, codes_out, scales_out as for qesgd_requantize).  The update
 * takes the arithmetic of qesgd_lr_sgd_step's two-pass form, so the result equals that call
 * followed by qesgd_requantize bit for bit.  Shapes the fused kernel does not take (bucket
 * above 1024, d not a multiple of 4, X or u not 16-byte aligned) run as those two calls.
 * 1 <= m <= QESGD_MAX_LR_BATCH; other arguments as for qesgd_requantize.
 */
int qesgd_lr_qesgd_step(qesgd_ctx *ctx, const float *Xb, const float *yb, uint32_t m, uint64_t d,
                        float lr, float *u, const float *anchor, uint32_t bucket, uint32_t s,
                        uint32_t bits, uint32_t scale_mode, float fixed_delta, uint64_t seed,
                        uint32_t worker, uint32_t step, float *zsum, uint32_t *codes_out,
                        float *scales_out);

/*
 * Gradient compression on the push side (Sec. 3, remark after Algorithm 3; the QSGD
 * baseline of Sec. 5 quantises gradients with delta = ||g||): the K streams hold quantised
 * gradients, encoded with anchor == NULL, and the server takes
 *   param_i <- param_i + alpha * (1/K) * sum_k (+-level_{k,i} * fl32(scale_{k,bucket(i)} / s))
 * with alpha = -learning rate (Eq. 2 on the mean of the decoded workers).  alpha = 1 is
 * qesgd_decode_average_apply.  Same layout, limits and accuracy (1e-6 * max(|param_i|,
 * |alpha| * max_k scale)); alpha must be finite.
 */
int qesgd_decode_average_axpy(qesgd_ctx *ctx, float *param, uint64_t d, uint32_t K,
                              const uint32_t *codes, uint64_t code_stride, const float *scales,
                              uint64_t scale_stride, uint32_t bucket, uint32_t s, uint32_t bits,
                              float alpha);

/* Decoding alone (the grid points delta*k of Eq. 3): out_i = +-level_i *
 * fl32(scale/s), i < d, bit-exact.  out: float[d]. */
int qesgd_decode(qesgd_ctx *ctx, const uint32_t *codes, const float *scales, uint64_t d,
                 uint32_t bucket, uint32_t s, uint32_t bits, float *out);

/*
 * Local epoch on logistic regression (Sec. 1: f_i(w) = log(1 + exp(-y_i x_i^T w));
 * Eq. 2: u <- u - (lr/m) * sum_j grad f_j(u); worker task of Algorithm 3).
 * One step on the m rows of Xb (row-major float[m][d]) with labels yb (float[m],
 * +-1): u (float[d]) is updated in place.  fp32 arithmetic, fp32 accumulation.
 * 1 <= m <= QESGD_MAX_LR_BATCH.
 */
int qesgd_lr_sgd_step(qesgd_ctx *ctx, const float *Xb, const float *yb, uint32_t m, uint64_t d,
                      float lr, float *u);
/* The summand of Eq. 2 alone: g_out = (1/m) * sum_j grad f_j(w) on the m rows of Xb, for
 * workers that push (quantised) gradients instead of parameters.  w and g_out are float[d]
 * and must not overlap.  One margin pass and one pass that writes the gradient; fp32
 * arithmetic and accumulation as for qesgd_lr_sgd_step. */
int qesgd_lr_gradient(qesgd_ctx *ctx, const float *Xb, const float *yb, uint32_t m, uint64_t d,
                      const float *w, float *g_out);
/* Rows [0, n_local) of X in consecutive minibatches of `batch` rows, in row
 * order; a last partial batch uses its own size in Eq. 2. */
int qesgd_lr_local_epoch(qesgd_ctx *ctx, const float *X, const float *y, uint64_t n_local,
                         uint64_t d, uint32_t batch, float lr, float *u);
/* K workers side by side: worker k owns rows [k*n_local, (k+1)*n_local) of X and
 * y and updates u + k*u_stride (elements).
 * Where the shape allows (d a multiple of 4 and at most 512 columns per SM, minibatches
 * of at most 256 rows, X and u 16-byte aligned, u_stride a multiple of 4) the whole epoch
 * of all K workers is ONE persistent kernel, launched cooperatively with one CTA per SM,
 * that stages every minibatch in shared memory by TMA and reads X from HBM once; its
 * CTAs exchange partial margins through the context's workspace, which the call clears
 * first.  The partial margins of a row are summed across the CTAs as fixed-point integers
 * (units of 2^-28 below 2^17 in magnitude, units of 2^-6 from there to 2^49), so the sum
 * does not depend on the order in which the CTAs arrive; a NaN partial makes the row's
 * margin NaN, an infinite one (or one of 2^49 or more, far beyond where the step
 * coefficient saturates) makes it that infinity, and both then spread through u as they
 * would in floating point.  Every wait the kernel loops on (for another CTA, another warp group, a copy) is
 * bounded by the context's wait limit (one second unless qesgd_set_wait_limit changed it):
 * should one run out, the kernel returns, u is left partly updated and
 * QESGD_STATUS_TIMEOUT is set in the status word; the context stays usable and the next call
 * starts clean.  One wait has no bound of its own: at its start the kernel allocates the
 * SM's tensor memory, and that allocation blocks while another kernel resident on the same
 * SM (another stream or process) holds tensor memory, until that kernel ends.  The kernel
 * needs all its CTAs resident at once, so do not run it next to other kernels that occupy
 * the device for long.  Other shapes run one margin pass and one
 * update pass per minibatch, step t of every worker in the same launches.  Results are
 * deterministic (order-free integer sums or a fixed summation order) on either path. */
int qesgd_lr_local_epoch_batch(qesgd_ctx *ctx, const float *X, const float *y, uint64_t n_local,
                               uint64_t d, uint32_t K, uint32_t batch, float lr, float *u,
                               uint64_t u_stride);

/* Limit, in nanoseconds, of each wait inside the persistent local-epoch kernel (its CTAs
 * wait for one another's partial margins and for their own TMA copies).  0 restores the
 * default of one second; at most 10 seconds.  A limit below one microsecond means "look once
 * more, then give up" (the device timer is not finer than that).  Takes effect with the next
 * qesgd_lr_local_epoch[_batch] / qesgd_lr_sgd_step call of this context. */
int qesgd_set_wait_limit(qesgd_ctx *ctx, uint64_t nanoseconds);
/* Test hook for the give-up path of that kernel (no counterpart in the paper): CTA number
 * `cta` does not announce its partial margins of the first minibatch, so every CTA's wait
 * for them runs out after the wait limit, the kernel returns and QESGD_STATUS_TIMEOUT is
 * set.  Nothing faults or hangs.  cta = -1 (the default) switches the hook off. */
int qesgd_debug_drop_signal(qesgd_ctx *ctx, int64_t cta);

/*
 * The paper has no counterpart for this entry point; it exists for callers that are
 * not allowed to allocate device memory at the moment they need a step: code running
 * inside a memory-pool or allocator callback, a real-time loop that must not touch
 * the driver's allocator, or a host that was handed a fixed memory budget and may
 * not create a qesgd_ctx (qesgd_create allocates).  It is qesgd_lr_sgd_step without
 * a context, always in the two-pass form (one margin pass, one update pass).  The context
 * entry point may run the step in its persistent kernel instead, whose sums run in another
 * order: the two agree to rounding (1e-5 relative), not bit for bit.
 *
 * The partial margins the two passes exchange live in a fixed array inside the
 * library image (64 KB of device memory on every GPU that loads the library, held
 * until the process exits) instead of a context's workspace.  Consequences:
 *   - m must not exceed QESGD_NOALLOC_MAX_LR_BATCH; larger batches return
 *     QESGD_ELIMIT and enqueue nothing.  d is unlimited.
 *   - the call works on the CURRENT device and enqueues on cuda_stream (NULL = legacy
 *     default stream); Xb, yb, u are device pointers as for qesgd_lr_sgd_step.
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine.  The first
 *     call on each device looks up the array's device address; with lazy module loading
 *     that query may be the moment the driver loads this library's device image (and
 *     places the array).  So make one warm-up call per device OUTSIDE the region in which
 *     allocation is forbidden, and before starting any stream capture; later calls only
 *     launch two kernels.
 *   - every call shares the one array, which keeps the previous call's contents.
 *     The first pass overwrites every slot the second pass reads; only the arrival
 *     counter at the head of the array (by which the last CTA of the first pass knows
 *     that it is the last) has to be zero between calls: it starts at zero with the
 *     library image and the kernel that uses it sets it back.  Two calls that overlap
 *     on the GPU (different streams, or different host threads) race on the array:
 *     serialise them on one stream.
 */
int qesgd_lr_sgd_step_noalloc(void *cuda_stream, const float *Xb, const float *yb, uint32_t m,
                              uint64_t d, float lr, float *u);

/* Waits for the stream, copies the status word to *flags_out (host) and clears it. */
int qesgd_status(qesgd_ctx *ctx, uint32_t *flags_out);
/* 1 if the library was built with QESGD_DEBUG (the codec kernels then check every store index,
 * and the indices of their code and scale loads, against the extent of the buffer, skip an
 * access that falls outside and set QESGD_STATUS_RANGE instead of faulting), else 0. */
int qesgd_debug_build(void);
/* Debug build only: runs the range check on an index that is out of range by construction (no
 * memory access is made), so that QESGD_STATUS_RANGE appears in the status word; in a release
 * build it returns QESGD_EINVAL and enqueues nothing. */
int qesgd_debug_range_selftest(qesgd_ctx *ctx);
/* Number of kernels this context has launched since creation. */
uint64_t qesgd_launch_count(const qesgd_ctx *ctx);
/* Last cudaError_t seen by this context (0 if none). */
int qesgd_last_cuda_error(const qesgd_ctx *ctx);
/* Static text for a return code. */
const char *qesgd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* QESGD_H */
