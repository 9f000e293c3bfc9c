// Internal declarations shared by the translation units of libqesgd.so.
// Nothing here is part of the public ABI (that is include/qesgd.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "qesgd.h"

// Debug build: an index is checked against its limit; outside it the status word receives
// QESGD_STATUS_RANGE and the caller skips the access.  Release build: always true, no code.
#ifdef QESGD_DEBUG
#define QESGD_IN_RANGE(status, cond) ((cond) ? true : (atomicOr((status), QESGD_STATUS_RANGE), false))
#else
#define QESGD_IN_RANGE(status, cond) true
#endif

struct qesgd_ctx {
    int device;
    cudaStream_t stream;
    uint32_t *d_status;     // device status word (bit set by kernels)
    float *d_lr_work;       // logistic-regression partial margins
    uint64_t lr_work_floats;
    uint64_t launches;
    int last_cuda_error;
    int sm_count;
    uint64_t wait_ns;       // limit of each wait inside the local-epoch kernel
    uint32_t drop_cta;      // give-up-path test hook of the local-epoch kernel (none: ~0)
};
static const uint64_t QESGD_DEFAULT_WAIT_NS = 1000000000ull;
static const uint64_t QESGD_MAX_WAIT_NS = 10000000000ull;

// Workspace for partial margins: K * P * m floats must fit.
static const uint64_t QESGD_LR_WORK_FLOATS = 1ull << 20;

struct EncodeArgs {
    const float *local;
    uint64_t local_stride;  // elements between workers
    const float *anchor;    // may be null
    uint64_t d;             // elements per worker
    uint64_t padded;        // nb * bucket
    uint32_t log2_bucket;
    uint32_t s;
    float fixed_scale;      // fl32(s * delta), FIXED mode only
    uint32_t round_key[10][2];  // Philox round keys: seed + r * Weyl constants
    uint32_t worker0, epoch;
    uint32_t K;             // workers in this launch
    uint32_t *codes;
    uint64_t code_stride;   // bytes between workers
    float *scales;
    uint64_t scale_stride;  // elements between workers
    uint32_t *status;
    float *u_out;           // per-step QESGD: receives anchor + Q(z) (same layout as local); else null
    float *zsum;            // per-step QESGD: running sum of Q(z), may be null
};

// One inner step of QESGD on logistic regression in two launches: the margin pass of the
// plain step, then one kernel that forms the updated parameter of a tile in shared memory
// and requantises it there.
struct QstepArgs {
    EncodeArgs e;           // the requantisation of u (K = 1, u_out = local = u)
    const float *X, *y;     // the minibatch, m rows of d columns
    uint32_t m;
    float rate;             // lr / m
    const float *margins;   // the m margins, as the margin pass left them
};

struct DecodeArgs {
    float *param;           // decode-average-apply: in/out; decode: out
    uint64_t d;
    uint64_t nb;
    uint32_t K;
    float avg_scale;        // alpha / K applied to the sum over workers (1/K for the plain average)
    uint32_t log2_bucket;
    uint32_t s;
    const uint32_t *codes;
    uint64_t code_stride;   // bytes
    const float *scales;
    uint64_t scale_stride;  // elements
    uint32_t *status;
};
int qesgd_launch_range_selftest(uint32_t *status, cudaStream_t stream);

// Launchers.  Return a cudaError_t as int.  qesgd_codec.cu is compiled once per code width
// and defines the *_2, *_4, *_8 functions; the width-dispatching wrappers are inline here.
#define QESGD_DECLARE_WIDTH(B)                                                                  \
    int qesgd_launch_encode_##B(const EncodeArgs &a, uint32_t K, uint32_t scale_mode, bool vec, \
                                int sm_count, cudaStream_t stream);                             \
    int qesgd_launch_decode_##B(const DecodeArgs &a, bool vec, cudaStream_t stream);            \
    int qesgd_launch_decode_average_apply_##B(const DecodeArgs &a, bool vec, cudaStream_t stream);
int qesgd_launch_lr_qstep_2(const QstepArgs &a, uint32_t scale_mode, cudaStream_t stream);
int qesgd_launch_lr_qstep_4(const QstepArgs &a, uint32_t scale_mode, cudaStream_t stream);
int qesgd_launch_lr_qstep_8(const QstepArgs &a, uint32_t scale_mode, cudaStream_t stream);
QESGD_DECLARE_WIDTH(2)
QESGD_DECLARE_WIDTH(4)
QESGD_DECLARE_WIDTH(8)
#undef QESGD_DECLARE_WIDTH

inline int qesgd_launch_encode(const EncodeArgs &a, uint32_t K, uint32_t bits, uint32_t scale_mode,
                               bool vec, int sm_count, cudaStream_t stream)
{
    switch (bits) {
        case 2: return qesgd_launch_encode_2(a, K, scale_mode, vec, sm_count, stream);
        case 4: return qesgd_launch_encode_4(a, K, scale_mode, vec, sm_count, stream);
        default: return qesgd_launch_encode_8(a, K, scale_mode, vec, sm_count, stream);
    }
}
inline int qesgd_launch_decode(const DecodeArgs &a, uint32_t bits, bool vec, cudaStream_t stream)
{
    switch (bits) {
        case 2: return qesgd_launch_decode_2(a, vec, stream);
        case 4: return qesgd_launch_decode_4(a, vec, stream);
        default: return qesgd_launch_decode_8(a, vec, stream);
    }
}
inline int qesgd_launch_decode_average_apply(const DecodeArgs &a, uint32_t bits, bool vec,
                                             cudaStream_t stream)
{
    switch (bits) {
        case 2: return qesgd_launch_decode_average_apply_2(a, vec, stream);
        case 4: return qesgd_launch_decode_average_apply_4(a, vec, stream);
        default: return qesgd_launch_decode_average_apply_8(a, vec, stream);
    }
}
// One minibatch step for K workers; returns the number of kernels launched in *launched.
int qesgd_launch_lr_step(const float *Xb, uint64_t x_worker_stride, const float *yb,
                         uint64_t y_worker_stride, uint32_t m, uint64_t d, uint32_t K, float lr,
                         float *u, uint64_t u_stride, float *work, uint64_t work_floats,
                         cudaStream_t stream, int *launched);
// The margin pass alone (pass 1 of a step) for one worker; *parts_out receives the number of
// partial margins per row that the pass leaves in `work` ([parts][m]).
int qesgd_launch_lr_margins(const float *Xb, const float *yb, uint32_t m, uint64_t d, const float *u,
                            float *work, uint64_t work_floats, cudaStream_t stream, const float **margins_out);
// Minibatch mean gradient at w into g (same two passes; the second writes instead of updating).
int qesgd_launch_lr_gradient(const float *Xb, const float *yb, uint32_t m, uint64_t d,
                             const float *w, float *g, float *work, uint64_t work_floats,
                             cudaStream_t stream, int *launched);
// A whole local epoch of K workers as one persistent kernel that keeps each minibatch in
// shared memory between its two uses.  Returns 0 = launched (one memset + one kernel),
// -1 = shape not covered (the caller falls back to qesgd_launch_lr_step per minibatch),
// > 0 = cudaError_t.  `work` is zeroed and used for the inter-CTA counters and partial margins.
int qesgd_launch_lr_epoch_fused(const float *X, const float *y, uint64_t n_local, uint64_t d,
                                uint32_t K, uint32_t batch, float lr, float *u, uint64_t u_stride,
                                float *work, uint64_t work_floats, uint32_t *status, int device,
                                int sm_count, uint64_t wait_ns, uint32_t drop_cta, cudaStream_t stream,
                                int *launched);
