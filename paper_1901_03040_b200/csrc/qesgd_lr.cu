// Logistic-regression minibatch SGD step for sm_100a (paper Sec. 1: f_i(w) =
// log(1 + exp(-y_i x_i^T w)); Eq. 2: u <- u - (lr/m) sum_j grad f_j(u)).
//
// Two streaming passes over the minibatch X_B (m rows, d columns, row-major):
//   pass 1  partial margins: CTA p owns column segments p, p+P, ... of 1024 columns,
//           keeps its slice of u in registers and writes sum_{cols} x_jc u_c for every
//           row j to work[(k*P + p)*m + j]   (no atomics, fixed summation order)
//   pass 2  every CTA sums the P partials of each row, forms the step coefficients
//           (lr/m) * y_j / (1 + exp(y_j m_j)) in shared memory and updates 256 columns
//           of u with sum_j coef_j x_jc, the rows split over four thread groups.  X_B is normally still in L2 for this pass.
// No tensor cores: with m = 64 rows the work is 64 dot products, bound by memory.
#include <mutex>

#include "qesgd_internal.h"

namespace {

constexpr int SEG = 1024;        // columns per segment in pass 1 (32 lanes x 8 float4)
#ifndef QESGD_LR_MAX_PARTS
#define QESGD_LR_MAX_PARTS 296
#endif
constexpr int MAX_PARTS = QESGD_LR_MAX_PARTS;   // CTAs of the margin pass per worker: two per SM of a B200
constexpr int DONE_WORDS = 64;   // one arrival counter per worker at the head of the workspace
constexpr int UPD_COLS = 256;      // pass 2: columns per CTA (64 groups of 4)
constexpr int UPD_ROWGROUPS = 4;   // pass 2: row groups per CTA
constexpr int UPD_THREADS = (UPD_COLS / 4) * UPD_ROWGROUPS;

struct LrArgs {
    const float *X;
    uint64_t x_stride;   // elements between workers
    const float *y;
    uint64_t y_stride;
    uint32_t m;
    uint64_t d;
    float rate;          // lr / m
    const float *u;      // point the margins are taken at
    float *dst;          // accumulate != 0: dst += step (dst == u); else dst = gradient
    uint32_t accumulate;
    uint64_t u_stride;
    float *work;         // partial margins [K][P][m]
    float *margins;      // the margins themselves [K][m], written by the last CTA of each worker
    uint32_t *done;      // arrival counters [K], zero between launches
    uint32_t parts;      // P
    uint32_t nseg;
};

template <bool VEC>
__global__ void __launch_bounds__(256) qesgd_lr_margin_kernel(const LrArgs a)
{
    __shared__ float s_part[QESGD_MAX_LR_BATCH];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t k = blockIdx.y, p = blockIdx.x;
    const float *__restrict__ X = a.X + (uint64_t)k * a.x_stride;
    const float *__restrict__ u = a.u + (uint64_t)k * a.u_stride;
    for (uint32_t j = threadIdx.x; j < a.m; j += blockDim.x) s_part[j] = 0.0f;
    __syncthreads();

    for (uint32_t seg = p; seg < a.nseg; seg += a.parts) {
        const uint64_t c0 = (uint64_t)seg * SEG;
        float4 uu[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint64_t c = c0 + (uint64_t)i * 128 + lane * 4u;
            if (VEC && c + 4 <= a.d) {
                uu[i] = *reinterpret_cast<const float4 *>(u + c);
            } else {
                uu[i].x = c + 0 < a.d ? u[c + 0] : 0.0f;
                uu[i].y = c + 1 < a.d ? u[c + 1] : 0.0f;
                uu[i].z = c + 2 < a.d ? u[c + 2] : 0.0f;
                uu[i].w = c + 3 < a.d ? u[c + 3] : 0.0f;
            }
        }
        // each row belongs to one warp; two rows at a time so that 16 loads are in flight
        // per lane and the two shuffle reductions interleave
        for (uint32_t j = warp; j < a.m; j += 16) {
            const uint32_t j2 = j + 8;
            const bool two = j2 < a.m;
            const float *__restrict__ row0 = X + (uint64_t)j * a.d;
            const float *__restrict__ row1 = X + (uint64_t)(two ? j2 : j) * a.d;
            float4 xa[8], xb[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint64_t c = c0 + (uint64_t)i * 128 + lane * 4u;
                if (VEC && c + 4 <= a.d) {
                    xa[i] = __ldg(reinterpret_cast<const float4 *>(row0 + c));
                    xb[i] = __ldg(reinterpret_cast<const float4 *>(row1 + c));
                } else {
                    xa[i].x = c + 0 < a.d ? __ldg(row0 + c + 0) : 0.0f;
                    xa[i].y = c + 1 < a.d ? __ldg(row0 + c + 1) : 0.0f;
                    xa[i].z = c + 2 < a.d ? __ldg(row0 + c + 2) : 0.0f;
                    xa[i].w = c + 3 < a.d ? __ldg(row0 + c + 3) : 0.0f;
                    xb[i].x = c + 0 < a.d ? __ldg(row1 + c + 0) : 0.0f;
                    xb[i].y = c + 1 < a.d ? __ldg(row1 + c + 1) : 0.0f;
                    xb[i].z = c + 2 < a.d ? __ldg(row1 + c + 2) : 0.0f;
                    xb[i].w = c + 3 < a.d ? __ldg(row1 + c + 3) : 0.0f;
                }
            }
            float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                acc0 = fmaf(xa[i].x, uu[i].x, acc0);
                acc0 = fmaf(xa[i].y, uu[i].y, acc0);
                acc0 = fmaf(xa[i].z, uu[i].z, acc0);
                acc0 = fmaf(xa[i].w, uu[i].w, acc0);
                acc1 = fmaf(xb[i].x, uu[i].x, acc1);
                acc1 = fmaf(xb[i].y, uu[i].y, acc1);
                acc1 = fmaf(xb[i].z, uu[i].z, acc1);
                acc1 = fmaf(xb[i].w, uu[i].w, acc1);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                acc0 += __shfl_xor_sync(0xFFFFFFFFu, acc0, off);
                acc1 += __shfl_xor_sync(0xFFFFFFFFu, acc1, off);
            }
            if (lane == 0) {
                s_part[j] += acc0;
                if (two) s_part[j2] += acc1;
            }
        }
    }
    __syncthreads();
    float *__restrict__ out = a.work + ((uint64_t)k * a.parts + p) * a.m;
    for (uint32_t j = threadIdx.x; j < a.m; j += blockDim.x) out[j] = s_part[j];
    // The CTA that arrives last sums the partial margins of its worker, once, in an order that
    // does not depend on which CTA that is: a row's P partials in four consecutive runs (one
    // thread each, in index order), the four run sums added in run order.
    __shared__ uint32_t s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(a.done + k, 1u) == a.parts - 1u ? 1u : 0u;
    __syncthreads();
    if (s_last == 0u) return;
    __threadfence();
    const float *__restrict__ w = a.work + (uint64_t)k * a.parts * a.m;
    const uint32_t run = (a.parts + 3u) / 4u;
    for (uint32_t j0 = 0; j0 < a.m; j0 += blockDim.x / 4u) {
        const uint32_t j = j0 + (threadIdx.x >> 2), r = threadIdx.x & 3u;
        float sum = 0.0f;
        if (j < a.m) {
            const uint32_t p0 = r * run, p1 = min(p0 + run, a.parts);
#pragma unroll 8
            for (uint32_t q = p0; q < p1; ++q) sum += __ldcg(w + (uint64_t)q * a.m + j);
        }
        // lanes 4i .. 4i+3 hold the runs of one row
        const float s1 = __shfl_down_sync(0xFFFFFFFFu, sum, 1);
        const float s2 = __shfl_down_sync(0xFFFFFFFFu, sum, 2);
        const float s3 = __shfl_down_sync(0xFFFFFFFFu, sum, 3);
        if (r == 0u && j < a.m) a.margins[(uint64_t)k * a.m + j] = ((sum + s1) + s2) + s3;
    }
    if (threadIdx.x == 0) a.done[k] = 0u;   // ready for the next launch
}

// Pass 2.  A CTA updates UPD_COLS consecutive columns: 64 column groups of 4 columns
// times UPD_ROWGROUPS row groups; row group g sums rows g, g + G, g + 2G, ... (coalesced
// 1 KB per row), the G partial sums meet in shared memory in fixed order.
template <bool VEC>
__global__ void __launch_bounds__(UPD_THREADS) qesgd_lr_update_kernel(const LrArgs a)
{
    __shared__ float s_coef[QESGD_MAX_LR_BATCH];
    __shared__ float4 s_sum[UPD_ROWGROUPS][UPD_COLS / 4];
    const uint32_t k = blockIdx.y;
    const float *__restrict__ X = a.X + (uint64_t)k * a.x_stride;
    const float *__restrict__ y = a.y + (uint64_t)k * a.y_stride;
    float *__restrict__ u = a.dst + (uint64_t)k * a.u_stride;
    const float *__restrict__ margins = a.margins + (uint64_t)k * a.m;
    for (uint32_t j = threadIdx.x; j < a.m; j += blockDim.x) {
        const float margin = margins[j];
        const float yj = __ldg(y + j);
        // -(lr/m) * c_j with c_j = -y_j / (1 + exp(y_j m_j))
        s_coef[j] = a.rate * yj / (1.0f + expf(yj * margin));
    }
    __syncthreads();

    const uint32_t cg = threadIdx.x % (UPD_COLS / 4);     // column group inside the CTA
    const uint32_t rg = threadIdx.x / (UPD_COLS / 4);     // row group
    const uint64_t c = (uint64_t)blockIdx.x * UPD_COLS + cg * 4u;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (VEC && c + 4 <= a.d) {
        const float *__restrict__ col = X + c;
#pragma unroll 8
        for (uint32_t j = rg; j < a.m; j += UPD_ROWGROUPS) {
            const float4 x = __ldg(reinterpret_cast<const float4 *>(col + (uint64_t)j * a.d));
            const float cj = s_coef[j];
            acc.x = fmaf(cj, x.x, acc.x);
            acc.y = fmaf(cj, x.y, acc.y);
            acc.z = fmaf(cj, x.z, acc.z);
            acc.w = fmaf(cj, x.w, acc.w);
        }
    } else if (c < a.d) {
        for (uint32_t j = rg; j < a.m; j += UPD_ROWGROUPS) {
            const float cj = s_coef[j];
            const float *__restrict__ row = X + (uint64_t)j * a.d + c;
            acc.x = fmaf(cj, __ldg(row), acc.x);
            if (c + 1 < a.d) acc.y = fmaf(cj, __ldg(row + 1), acc.y);
            if (c + 2 < a.d) acc.z = fmaf(cj, __ldg(row + 2), acc.z);
            if (c + 3 < a.d) acc.w = fmaf(cj, __ldg(row + 3), acc.w);
        }
    }
    s_sum[rg][cg] = acc;
    __syncthreads();
    if (rg == 0 && c < a.d) {
        float4 t = s_sum[0][cg];
#pragma unroll
        for (int g = 1; g < UPD_ROWGROUPS; ++g) {
            const float4 v = s_sum[g][cg];
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        if (VEC && c + 4 <= a.d) {
            float4 uu = make_float4(0.f, 0.f, 0.f, 0.f);
            if (a.accumulate) uu = *reinterpret_cast<float4 *>(u + c);
            uu.x += t.x; uu.y += t.y; uu.z += t.z; uu.w += t.w;
            *reinterpret_cast<float4 *>(u + c) = uu;
        } else {
            const bool acc_mode = a.accumulate != 0u;
            u[c] = (acc_mode ? u[c] : 0.0f) + t.x;
            if (c + 1 < a.d) u[c + 1] = (acc_mode ? u[c + 1] : 0.0f) + t.y;
            if (c + 2 < a.d) u[c + 2] = (acc_mode ? u[c + 2] : 0.0f) + t.z;
            if (c + 3 < a.d) u[c + 3] = (acc_mode ? u[c + 3] : 0.0f) + t.w;
        }
    }
}

}  // namespace

namespace {

// Workspace: arrival counters | margins [K][m] | partial margins [K][P][m].  P = as many CTAs
// per worker as the workspace, the segment count and MAX_PARTS allow; 0 if nothing fits.
uint64_t lay_out_work(LrArgs &a, float *work, uint64_t work_floats, uint32_t K, uint32_t m, uint64_t nseg)
{
    const uint64_t head = (uint64_t)DONE_WORDS + (uint64_t)K * m;
    if (K > (uint32_t)DONE_WORDS || work_floats <= head) return 0;
    uint64_t parts = (work_floats - head) / ((uint64_t)K * m);
    if (parts > (uint64_t)MAX_PARTS) parts = MAX_PARTS;
    if (parts > nseg) parts = nseg;
    a.done = reinterpret_cast<uint32_t *>(work);
    a.margins = work + DONE_WORDS;
    a.work = work + head;
    a.parts = (uint32_t)parts;
    return parts;
}

// Both passes for K workers.  rate multiplies y_j / (1 + exp(y_j m_j)): lr/m for the SGD
// step (dst = u, accumulated), -1/m for the mean gradient (dst = g, overwritten).
int launch_lr_passes(const float *Xb, uint64_t x_worker_stride, const float *yb,
                     uint64_t y_worker_stride, uint32_t m, uint64_t d, uint32_t K, float rate,
                     const float *u, float *dst, bool accumulate, uint64_t u_stride, float *work,
                     uint64_t work_floats, cudaStream_t stream, int *launched)
{
    *launched = 0;
    LrArgs a;
    a.X = Xb; a.x_stride = x_worker_stride;
    a.y = yb; a.y_stride = y_worker_stride;
    a.m = m; a.d = d;
    a.rate = rate;
    a.u = u; a.dst = dst; a.accumulate = accumulate ? 1u : 0u; a.u_stride = u_stride;
    const uint64_t nseg = (d + SEG - 1) / SEG;
    const uint64_t parts = lay_out_work(a, work, work_floats, K, m, nseg);
    if (parts == 0 || nseg > 0xFFFFFFFFull) return (int)cudaErrorInvalidValue;
    a.nseg = (uint32_t)nseg;
    const bool vec = (d % 4 == 0) && (x_worker_stride % 4 == 0) && (u_stride % 4 == 0) &&
                     (((uintptr_t)Xb | (uintptr_t)u | (uintptr_t)dst) % 16 == 0);
    dim3 g1((unsigned)parts, K), b1(256);
    if (vec) qesgd_lr_margin_kernel<true><<<g1, b1, 0, stream>>>(a);
    else qesgd_lr_margin_kernel<false><<<g1, b1, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    *launched = 1;
    const uint64_t ublocks = (d + UPD_COLS - 1) / UPD_COLS;
    if (ublocks > 0x7FFFFFFFull) return (int)cudaErrorInvalidValue;
    dim3 g2((unsigned)ublocks, K), b2(UPD_THREADS);
    if (vec) qesgd_lr_update_kernel<true><<<g2, b2, 0, stream>>>(a);
    else qesgd_lr_update_kernel<false><<<g2, b2, 0, stream>>>(a);
    e = cudaGetLastError();
    if (e == cudaSuccess) *launched = 2;
    return (int)e;
}

}  // namespace

int qesgd_launch_lr_margins(const float *Xb, const float *yb, uint32_t m, uint64_t d, const float *u,
                            float *work, uint64_t work_floats, cudaStream_t stream, const float **margins_out)
{
    LrArgs a;
    a.X = Xb; a.x_stride = 0;
    a.y = yb; a.y_stride = 0;
    a.m = m; a.d = d;
    a.rate = 0.0f;
    a.u = u; a.dst = nullptr; a.accumulate = 0u; a.u_stride = 0;
    const uint64_t nseg = (d + SEG - 1) / SEG;
    const uint64_t parts = lay_out_work(a, work, work_floats, 1u, m, nseg);
    if (parts == 0 || nseg > 0xFFFFFFFFull) return (int)cudaErrorInvalidValue;
    a.nseg = (uint32_t)nseg;
    const bool vec = (d % 4 == 0) && (((uintptr_t)Xb | (uintptr_t)u) % 16 == 0);
    dim3 g1((unsigned)parts, 1), b1(256);
    if (vec) qesgd_lr_margin_kernel<true><<<g1, b1, 0, stream>>>(a);
    else qesgd_lr_margin_kernel<false><<<g1, b1, 0, stream>>>(a);
    *margins_out = a.margins;
    return (int)cudaGetLastError();
}

int qesgd_launch_lr_step(const float *Xb, uint64_t x_worker_stride, const float *yb,
                         uint64_t y_worker_stride, uint32_t m, uint64_t d, uint32_t K, float lr,
                         float *u, uint64_t u_stride, float *work, uint64_t work_floats,
                         cudaStream_t stream, int *launched)
{
    return launch_lr_passes(Xb, x_worker_stride, yb, y_worker_stride, m, d, K, lr / (float)m, u, u,
                            true, u_stride, work, work_floats, stream, launched);
}

int qesgd_launch_lr_gradient(const float *Xb, const float *yb, uint32_t m, uint64_t d,
                             const float *w, float *g, float *work, uint64_t work_floats,
                             cudaStream_t stream, int *launched)
{
    return launch_lr_passes(Xb, 0, yb, 0, m, d, 1, -1.0f / (float)m, w, g, false, 0, work,
                            work_floats, stream, launched);
}

// ---------------------------------------------------------------------------
// Entry point that allocates nothing: the partial margins go to a fixed array in
// the library image.  In host code the array's name is only a handle; the device
// address is looked up once per device with cudaGetSymbolAddress and cached.
// ---------------------------------------------------------------------------
namespace {

constexpr uint32_t NOALLOC_FLOATS = 64 * QESGD_NOALLOC_MAX_LR_BATCH;   // 64 KB: counters, margins, up to 62 parts of 256 rows
static __device__ __align__(256) float g_noalloc_lr_scratch[NOALLOC_FLOATS];

constexpr int MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
float *g_noalloc_ptr[MAX_DEVICES] = {nullptr};

// Device address of the scratch array on the current device; looked up on first use.
cudaError_t noalloc_scratch(float **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_lr_scratch);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = static_cast<float *>(p);
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int qesgd_lr_sgd_step_noalloc(void *cuda_stream, const float *Xb, const float *yb,
                                         uint32_t m, uint64_t d, float lr, float *u)
{
    if (m < 1) return QESGD_EINVAL;
    if (m > QESGD_NOALLOC_MAX_LR_BATCH) return QESGD_ELIMIT;
    if (d == 0) return QESGD_OK;
    if (!Xb || !yb || !u) return QESGD_EINVAL;
    if (((uintptr_t)Xb | (uintptr_t)yb | (uintptr_t)u) % 4 != 0) return QESGD_EINVAL;
    float *scratch = nullptr;
    if (noalloc_scratch(&scratch) != cudaSuccess) return QESGD_ECUDA;
    int launched = 0;
    const int e = qesgd_launch_lr_step(Xb, 0, yb, 0, m, d, 1, lr, u, 0, scratch, NOALLOC_FLOATS,
                                       (cudaStream_t)cuda_stream, &launched);
    return e == 0 ? QESGD_OK : QESGD_ECUDA;
}
