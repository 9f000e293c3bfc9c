// Local epoch of logistic-regression minibatch SGD as ONE persistent kernel for sm_100a
// (paper Sec. 1: f_i(w) = log(1 + exp(-y_i x_i^T w)); Eq. 2: u <- u - (lr/m) sum_j grad f_j(u);
// worker task of Algorithm 3: consecutive minibatches of the worker's shard).
//
// A step needs the minibatch twice -- once for the margins x_j . u, once for the update
// sum_j c_j x_j -- with a reduction over all columns in between.  Here every CTA owns a
// slice of `cols` columns for the whole epoch and keeps its slice of each minibatch in
// shared memory between the two uses, so X is read from HBM exactly once:
//
//   tile (t, k)  = minibatch t of worker k; tiles are processed t-major, k-minor, and
//                  alternate between two shared-memory buffers
//   sub-tile     = SUB rows of a tile's column slice, fetched by TMA (one or two 2-D boxes,
//                  cp.async.bulk.tensor global -> shared, completion on an mbarrier per
//                  sub-tile); a producer warp issues the copies of tile i+2 as soon as the
//                  consumer warps have released the buffer of tile i
//   M(i)  margins of tile i over the CTA's columns; each row's partial margin is added, as a
//         fixed-point integer, to the row's accumulator acc[i % RING][row] by one 64-bit
//         reduction that also counts the contribution in the word's top bits
//   W(i)  wait until every row's count equals the number of CTAs, margins from the sums,
//         coefficients (lr/m) y_j / (1 + exp(y_j m_j)) into shared memory
//   U(i)  u[cols] += sum_j coef_j x_j from the tile
//
// The exchange of the margins is what the epoch waits for, so it is one step: integer addition
// is exact and commutes, so the sum over the CTAs needs no order, no second pass over 148
// partials and -- the count travelling in the same word as the sum -- no fence between data and
// signal; the result is the same in every run.  A word is count << 55 | sum, every contribution
// adds 1 << 55 plus 2^45 + round(partial * 2^28) (the 2^45 keeps it positive; |partial| < 2^17;
// up to 511 CTAs fit below the count).  A larger finite partial goes, in units of 2^-6 (the
// spacing of fp32 at 2^17), into the second word of the row; a NaN is counted in the third word
// and makes the margin NaN; an infinite partial, or one of 2^49 or more, is counted by sign in
// the fourth and makes the margin that infinity (NaN if both signs occur), which the step
// coefficient saturates on as it would on the number itself.  These rare kinds fence before they
// count themselves in the first word.  The slot that tile i + RING/2 will use is cleared by one CTA
// during M(i): every CTA has read it by then (it has taken part in tile i-2, hence finished
// tile i-4) and none adds to it before it has seen that CTA's contributions to tile i+2.
//
// Where the minibatch has at most 64 rows the tile does not wait in shared memory between M
// and U: right after M every thread moves its share of it into tensor memory (tcgen05.st;
// the SM's 256 KB of it hold one tile per consumer group and are otherwise unused here) and
// the shared-memory slots go back to the producer, so the next tile's copies run while this
// one waits for the other CTAs; U reads the tile back with tcgen05.ld.  Larger minibatches
// stay in shared memory and release their slots during U.
//
// Each tile's M, W, U is a chain of dependent round trips to global memory (reductions out,
// sums back) that lasts longer than the tile's own transfer from HBM.  The eight
// consumer warps therefore form two groups of four; group g owns buffer g and the tiles
// g, g+2, g+4, ... and runs M(i), W(i), U(i) for them, so one group computes while the other
// waits, and the copies of the tile after next are in flight meanwhile.  A worker's
// consecutive minibatches are K tiles apart: with an even K they stay in one group, with an
// odd K a group waits for the other group's update before it takes the margins.
//
// The CTAs wait on one another, so the kernel is launched cooperatively (all CTAs are
// resident by construction: at most one per SM).  Every wait the kernel itself loops on is
// bounded by the context's wait limit: a wait that runs out sets QESGD_STATUS_TIMEOUT and an
// abort word that the other CTAs poll, and the CTA's consumer warps leave.  The producer warp
// is the last to go on every path: it waits (on a bound of its own) for each copy it has
// requested and nobody has consumed, so no CTA ends with a copy still writing its shared
// memory.  The one wait without a bound is the tensor-memory allocation at the start, which
// blocks while another kernel resident on the same SM holds tensor memory (until that kernel
// ends).
#include <cuda.h>

#include <mutex>

#include "qesgd_internal.h"

namespace {

constexpr int EP_CONSUMERS = 256;                 // 8 consumer warps
constexpr int EP_GROUP = EP_CONSUMERS / 2;        // two groups of 4 warps, one per tile buffer
constexpr int EP_THREADS = EP_CONSUMERS + 32;     // + 1 producer warp
constexpr int SUB = 8;               // rows per sub-tile
constexpr int EP_RING = 8;           // accumulator slots; a slot is cleared RING/2 tiles before its use
constexpr int EP_MAX_COLS = 512;     // columns per CTA: 128 groups of 4
constexpr int EP_BOX_COLS = 256;     // widest TMA box
constexpr int EP_MAX_M = 256;        // rows per minibatch the fused path takes
constexpr int EP_MAX_NSUB = EP_MAX_M / SUB;
constexpr uint64_t DRAIN_LIMIT_NS = 2000000000ull;   // the producer's last wait for its own copies
constexpr uint64_t COARSE_TIMER_NS = 1024ull;        // limits below this mean "one look, then give up"
constexpr uint32_t EP_HEADER_WORDS = 64;             // word 0 = abort flag
constexpr uint32_t EP_ROW_WORDS = 4;                 // 64-bit words per accumulator row (one 32-byte sector)
constexpr float FX_SCALE = 268435456.0f;             // 2^28: unit of the first word
constexpr float FX_LIMIT = 131072.0f;                // 2^17: partials below go to the first word
constexpr float FX_WIDE_SCALE = 64.0f;               // 2^6: unit of the second word
constexpr float FX_WIDE_LIMIT = 562949953421312.0f;  // 2^49: partials below go to the second word
constexpr unsigned long long FX_BIAS = 1ull << 45;   // makes every contribution to the first word positive
constexpr unsigned long long FX_ONE = 1ull << 55;    // one contribution counted

struct EpochArgs {
    const float *y;
    uint64_t y_stride;
    uint64_t n_local;       // rows per worker
    uint64_t d;
    uint32_t K, batch, nsteps;
    uint32_t m_last;        // rows of the last minibatch
    uint32_t nsub_max, nsub_last;
    uint32_t cols;          // columns per CTA, multiple of 4
    float lr;
    float *u;
    uint64_t u_stride;
    uint32_t *header;       // [0] abort flag
    unsigned long long *acc;   // [EP_RING][batch][EP_ROW_WORDS] margin accumulators, zero at launch
    uint32_t *status;
    uint64_t wait_ns;       // limit of every wait on another CTA, warp group or copy
    uint32_t poll_mask;     // the clock is read every (poll_mask + 1) looks at a counter
    uint32_t drop_cta;      // test hook: this CTA does not count itself for tile 0 (none: ~0)
};

// ------------------------------------------------------------- primitives ----
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint64_t now_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0u;
}
// Has a wait that began at t0 used up `limit`?  The global timer may tick as coarsely as a
// microsecond, so a smaller limit is read as "give up after one round of looks".
__device__ __forceinline__ bool expired(uint64_t t0, uint64_t limit)
{
    return limit < COARSE_TIMER_NS || now_ns() - t0 > limit;
}
// Bounded wait for phase `parity` of a barrier; gives up early when `*stop` is set.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, const volatile uint32_t *stop,
                                          uint64_t limit)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = now_ns();
    for (;;) {
        for (int n = 0; n < 32; ++n)
            if (mbar_try_wait(bar, parity)) return true;
        if (*stop != 0u || expired(t0, limit)) return false;
    }
}
// One 2-D box of the row-major matrix X: columns [x, x + box width), rows [y, y + SUB).
// x * 4 bytes is a multiple of 16; dst is 128-byte aligned.  The copy goes to this CTA alone.
__device__ __forceinline__ void tma_load_box(float *dst, const CUtensorMap *map, uint32_t x, uint32_t y,
                                             uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
            "r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ ulonglong2 ld_relaxed_v2(const unsigned long long *p)
{
    ulonglong2 v;
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
    return v;
}

// Barrier `id` of `count` threads that also answers one question the same way for all of them:
// has any of them seen `flag` set?  (Each thread reads the flag for itself; a plain barrier
// followed by separate reads could send the threads different ways while another warp sets it,
// and the ones that stay would then wait at the next barrier for the ones that left.)
__device__ __forceinline__ bool sync_any(uint32_t id, uint32_t count, uint32_t flag)
{
    uint32_t r;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 q, %1, 0;\n"
        "bar.red.or.pred p, %2, %3, q;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}"
        : "=r"(r)
        : "r"(flag), "r"(id), "r"(count)
        : "memory");
    return r != 0u;
}

// ---- tensor memory as a stash for a tile between its two uses --------------------------
// The SM's 256 KB of tensor memory (128 lanes x 512 columns of 32 bits) is not needed for
// any matrix product here, so it holds a consumer group's tile while the group waits for the
// other CTAs: thread t of a warp owns lane 32 * (warp % 4) + t and reads back exactly what it
// stored, so no ordering between threads is involved.  One access moves 32 registers of
// every thread of the warp (the 8 rows x 4 columns a thread takes of a sub-tile).
__device__ __forceinline__ void tmem_alloc_all(uint32_t *smem_result)   // one whole warp
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(smem_result))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free_all(uint32_t taddr)           // the same warp
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float4 (&v)[8])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, "
        "%14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "f"(v[0].x), "f"(v[0].y), "f"(v[0].z), "f"(v[0].w), "f"(v[1].x), "f"(v[1].y), "f"(v[1].z), "f"(v[1].w),
        "f"(v[2].x), "f"(v[2].y), "f"(v[2].z), "f"(v[2].w), "f"(v[3].x), "f"(v[3].y), "f"(v[3].z), "f"(v[3].w),
        "f"(v[4].x), "f"(v[4].y), "f"(v[4].z), "f"(v[4].w), "f"(v[5].x), "f"(v[5].y), "f"(v[5].z), "f"(v[5].w),
        "f"(v[6].x), "f"(v[6].y), "f"(v[6].z), "f"(v[6].w), "f"(v[7].x), "f"(v[7].y), "f"(v[7].z), "f"(v[7].w)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float4 (&v)[8])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
        "%15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=f"(v[0].x), "=f"(v[0].y), "=f"(v[0].z), "=f"(v[0].w), "=f"(v[1].x), "=f"(v[1].y), "=f"(v[1].z),
          "=f"(v[1].w), "=f"(v[2].x), "=f"(v[2].y), "=f"(v[2].z), "=f"(v[2].w), "=f"(v[3].x), "=f"(v[3].y),
          "=f"(v[3].z), "=f"(v[3].w), "=f"(v[4].x), "=f"(v[4].y), "=f"(v[4].z), "=f"(v[4].w), "=f"(v[5].x),
          "=f"(v[5].y), "=f"(v[5].z), "=f"(v[5].w), "=f"(v[6].x), "=f"(v[6].y), "=f"(v[6].z), "=f"(v[6].w),
          "=f"(v[7].x), "=f"(v[7].y), "=f"(v[7].z), "=f"(v[7].w)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Sum over the 32 lanes of 8 per-lane values at once: three halving exchanges leave one
// value per lane, two plain butterflies finish.  Lane L ends with the total of value
// 4*bit4(L) + 2*bit3(L) + bit2(L); the order of the additions is fixed.
__device__ __forceinline__ float reduce8(float (&v)[8], uint32_t lane)
{
    const bool h4 = lane & 16u, h3 = lane & 8u, h2 = lane & 4u;
    float a[4], b[2];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const float keep = h4 ? v[r + 4] : v[r], send = h4 ? v[r] : v[r + 4];
        a[r] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const float keep = h3 ? a[r + 2] : a[r], send = h3 ? a[r] : a[r + 2];
        b[r] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
    }
    const float keep = h2 ? b[1] : b[0], send = h2 ? b[0] : b[1];
    float c = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
    c += __shfl_xor_sync(0xFFFFFFFFu, c, 2);
    c += __shfl_xor_sync(0xFFFFFFFFu, c, 1);
    return c;
}
__device__ __forceinline__ uint32_t reduce8_row(uint32_t lane)
{
    return ((lane >> 4) & 1u) * 4u + ((lane >> 3) & 1u) * 2u + ((lane >> 2) & 1u);
}

struct Tile {
    uint32_t t, k, m, nsub;
};
__device__ __forceinline__ Tile tile_of(const EpochArgs &a, uint32_t i)
{
    Tile r;
    r.t = i / a.K;
    r.k = i - r.t * a.K;
    const bool last = r.t == a.nsteps - 1u;
    r.m = last ? a.m_last : a.batch;
    r.nsub = last ? a.nsub_last : a.nsub_max;
    return r;
}

extern __shared__ __align__(1024) unsigned char ep_smem[];

// Shared memory: two tile buffers of nsub_max slots of SUB x cols floats (a slot holds
// the box of the first 256 columns, then the box of the rest), the step coefficients of
// the two consumer groups, the barriers, a few flag words.
__global__ void __launch_bounds__(EP_THREADS, 1)
    qesgd_lr_epoch_kernel(const EpochArgs a, const __grid_constant__ CUtensorMap map_a,
                          const __grid_constant__ CUtensorMap map_b)
{
    const uint32_t slot_floats = SUB * a.cols;
    float *const tile = reinterpret_cast<float *>(ep_smem);
    float *const s_coef = tile + (size_t)2u * a.nsub_max * slot_floats;
    uint64_t *const full = reinterpret_cast<uint64_t *>(s_coef + 2 * EP_MAX_M);
    uint64_t *const consumed = full + 2 * EP_MAX_NSUB;
    // [0] a wait ran out in this CTA, [3] always zero, [4], [5] tiles completed by consumer
    // group 0, 1, [8] base address of the tensor memory
    volatile uint32_t *const s_flag = reinterpret_cast<volatile uint32_t *>(consumed + 2 * EP_MAX_NSUB);

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t cta = blockIdx.x, ncta = gridDim.x;
    const uint32_t c0 = cta * a.cols;
    const uint32_t cols_a = min(a.cols, (uint32_t)EP_BOX_COLS), cols_b = a.cols - cols_a;
    const uint32_t ntiles = a.nsteps * a.K;

    if (tid == 0) {
        for (uint32_t s = 0; s < 2u * a.nsub_max; ++s) mbar_init(&full[s], 1u);
        for (uint32_t s = 0; s < 2u * a.nsub_max; ++s) mbar_init(&consumed[s], EP_GROUP / 32);
        for (int f = 0; f < 16; ++f) s_flag[f] = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Minibatches of at most 64 rows (8 sub-tiles x 32 registers x 2 groups = all 512 columns)
    // are stashed in tensor memory between their two uses; larger ones stay in shared memory.
    const bool stash = a.nsub_max <= 8u;
    if (stash && warp == 0) tmem_alloc_all(const_cast<uint32_t *>(&s_flag[8]));
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = s_flag[8];

    // ------------------------------------------------------------ producer ----
    if (warp == EP_CONSUMERS / 32) {
        // Lane L remembers, for slots L and L + 32 of the 2 * nsub_max slots, the tile whose copy
        // was requested into the slot last (none: ~0).
        uint32_t last_tile[2] = {0xFFFFFFFFu, 0xFFFFFFFFu};
        for (uint32_t i = 0; i < ntiles; ++i) {
            const uint32_t b = i & 1u;
            const Tile T = tile_of(a, i);
            const uint32_t row0 = (uint32_t)((uint64_t)T.k * a.n_local + (uint64_t)T.t * a.batch);
            bool ok = true;
            for (uint32_t s = 0; s < T.nsub && ok; ++s) {
                // a slot is free once the update of tile i-2 has read sub-tile s
                if (i >= 2u)
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(&consumed[b * a.nsub_max + s], ((i - 2u) >> 1) & 1u,
                                                           &s_flag[0], a.wait_ns)) != 0;
                if (ok) {
                    const uint32_t q = b * a.nsub_max + s;
                    if (q == lane) last_tile[0] = i;
                    if (q == lane + 32u) last_tile[1] = i;
                }
                if (ok && lane == 0) {
                    uint64_t *const bar = &full[b * a.nsub_max + s];
                    float *const dst = tile + (size_t)(b * a.nsub_max + s) * slot_floats;
                    mbar_arrive_expect_tx(bar, slot_floats * 4u);
                    tma_load_box(dst, &map_a, c0, row0 + s * SUB, bar);
                    if (cols_b) tma_load_box(dst + SUB * cols_a, &map_b, c0 + cols_a, row0 + s * SUB, bar);
                }
            }
            if (!ok) {
                if (lane == 0) {
                    s_flag[0] = 1u;
                    atomicOr(a.status, QESGD_STATUS_TIMEOUT);
                    atomicExch(a.header, 1u);
                }
                break;
            }
        }
        // Last out, on every path: each slot's latest copy has been consumed (then it has
        // landed) or is waited for here, so that the CTA does not end -- and its shared memory
        // is not handed to another CTA -- while a copy is still writing it.  After a normal
        // epoch these waits end with the consumers' last tiles.
        __syncwarp();
#pragma unroll
        for (int h = 0; h < 2; ++h)
            if (last_tile[h] != 0xFFFFFFFFu)
                mbar_wait(&full[lane + 32u * h], (last_tile[h] >> 1) & 1u, &s_flag[3], DRAIN_LIMIT_NS);
        return;
    }

    // ----------------------------------------------------------- consumers ----
    // Two groups of four warps; group g owns buffer g and the tiles i = g, g+2, g+4, ...
    // Each runs M(i), W(i), U(i) for its own tiles, so that one group computes while the
    // other waits for the other CTAs.
    const uint32_t g = warp >> 2, wg = warp & 3u, tg = tid & (EP_GROUP - 1u);
    float *const coef = s_coef + g * EP_MAX_M;
    auto group_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(1u + g), "n"(EP_GROUP) : "memory"); };

    // this lane's columns of worker k's u (columns lane*4 + 128*it), zeros past the slice
    auto load_u = [&](uint32_t k, float4 (&uu)[EP_MAX_COLS / 128]) {
        const float *__restrict__ ug = a.u + (uint64_t)k * a.u_stride + c0;
#pragma unroll
        for (int it = 0; it < EP_MAX_COLS / 128; ++it) {
            const uint32_t c = lane * 4u + it * 128u;
            uu[it] = (c < a.cols && (uint64_t)c0 + c < a.d) ? *reinterpret_cast<const float4 *>(ug + c)
                                                           : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    // With an even K >= 4 the group's next tile belongs to a worker whose previous minibatch
    // this group finished an iteration ago: its slice of u is requested a tile early.
    const bool early_u = (a.K & 1u) == 0u && a.K >= 4u;
    float4 un[EP_MAX_COLS / 128];
    if (early_u && g < ntiles) load_u(g % a.K, un);

    // the update's (and the stash's) share of a tile: four columns, all rows
    const uint32_t col = tg * 4u;
    const bool colok = col < a.cols && (uint64_t)c0 + col < a.d;
    const bool first = col < (uint32_t)EP_BOX_COLS;
    const uint32_t off = first ? col : SUB * cols_a + (col - EP_BOX_COLS);
    const uint32_t pitch = first ? cols_a : cols_b;
    const uint32_t taddr = tmem_base + ((32u * wg) << 16) + 256u * g;   // this thread's lane, this group's columns

    for (uint32_t i = g; i < ntiles; i += 2u) {
        const Tile T = tile_of(a, i);
        const uint32_t parity = (i >> 1) & 1u;
        uint64_t *const bars = full + g * a.nsub_max;
        const float *const buf = tile + (size_t)g * a.nsub_max * slot_floats;

        // The worker's previous minibatch is tile i-K.  With an odd K it belonged to the other
        // group: wait until that group has stored its update.
        if (i >= a.K && ((i - a.K) & 1u) != g) {
            const uint32_t need = ((i - a.K) >> 1) + 1u;
            if (tg == 0) {
                const uint64_t t0 = now_ns();
                while (s_flag[4u + (g ^ 1u)] < need) {
                    if (s_flag[0] != 0u || expired(t0, a.wait_ns)) {
                        s_flag[0] = 1u;
                        break;
                    }
                }
                __threadfence_block();
            }
            if (sync_any(1u + g, EP_GROUP, s_flag[0])) break;
        }

        // ---- M(i): margins over this CTA's columns, then the signal to the other CTAs ----
        {
            float4 uu[EP_MAX_COLS / 128];
            if (early_u) {
#pragma unroll
                for (int it = 0; it < EP_MAX_COLS / 128; ++it) uu[it] = un[it];
                if (i + 2u < ntiles) load_u((i + 2u) % a.K, un);
            } else {
                load_u(T.k, uu);
            }
            unsigned long long *const arow = a.acc + (uint64_t)(i % EP_RING) * a.batch * EP_ROW_WORDS;
            if (cta == i % ncta) {   // this CTA clears the slot that tile i + RING/2 will add into
                ulonglong2 *z = reinterpret_cast<ulonglong2 *>(
                    a.acc + (uint64_t)((i + EP_RING / 2) % EP_RING) * a.batch * EP_ROW_WORDS);
                for (uint32_t j = tg; j < 2u * a.batch; j += EP_GROUP) z[j] = make_ulonglong2(0ull, 0ull);
                __threadfence();     // cleared for every CTA before this thread goes on
            }
            const bool signal = i != 0u || cta != a.drop_cta;
            bool ok = true;
            for (uint32_t s = wg; s < T.nsub; s += EP_GROUP / 32) {   // a warp per sub-tile
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars[s], parity, &s_flag[0], a.wait_ns)) != 0;
                if (!ok) break;
                const float *__restrict__ xs = buf + (size_t)s * slot_floats;
                float acc[SUB];
#pragma unroll
                for (int r = 0; r < SUB; ++r) acc[r] = 0.0f;
#pragma unroll
                for (int it = 0; it < EP_MAX_COLS / 128; ++it) {
                    const uint32_t c = lane * 4u + it * 128u;
                    if (c < a.cols) {
                        const bool first = it < EP_BOX_COLS / 128;
                        const float *__restrict__ base = first ? xs + c : xs + SUB * cols_a + (c - EP_BOX_COLS);
                        const uint32_t pitch = first ? cols_a : cols_b;
#pragma unroll
                        for (int r = 0; r < SUB; ++r) {
                            const float4 x = *reinterpret_cast<const float4 *>(base + r * pitch);
                            acc[r] = fmaf(x.x, uu[it].x, acc[r]);
                            acc[r] = fmaf(x.y, uu[it].y, acc[r]);
                            acc[r] = fmaf(x.z, uu[it].z, acc[r]);
                            acc[r] = fmaf(x.w, uu[it].w, acc[r]);
                        }
                    }
                }
                const float tot = reduce8(acc, lane);
                const uint32_t jj = s * SUB + reduce8_row(lane);
                if ((lane & 3u) == 0u && jj < T.m && signal) {
                    unsigned long long *const r = arow + (uint64_t)jj * EP_ROW_WORDS;
                    if (fabsf(tot) < FX_LIMIT) {
                        atomicAdd(r, FX_ONE + FX_BIAS + (unsigned long long)__float2ll_rn(tot * FX_SCALE));
                    } else {
                        // rare: the wide word or the not-a-number count first, visible before the count
                        if (fabsf(tot) < FX_WIDE_LIMIT)
                            atomicAdd(r + 1, (unsigned long long)__float2ll_rn(tot * FX_WIDE_SCALE));
                        else if (tot != tot)
                            atomicAdd(r + 2, 1ull);                               // NaN
                        else
                            atomicAdd(r + 3, tot > 0.0f ? (1ull << 32) : 1ull);   // +-Inf, or beyond the wide word
                        __threadfence();
                        atomicAdd(r, FX_ONE + FX_BIAS);
                    }
                }
            }
            if (!ok) s_flag[0] = 1u;
            if (sync_any(1u + g, EP_GROUP, s_flag[0])) break;
        }

        // ---- stash: the tile moves from shared to tensor memory and its slots go back to the
        // producer now, so that the copies of the group's next tile run during the exchange ----
        if (stash) {
            // every warp observes the arrival of every sub-tile itself (lane s looks at sub-tile s)
            for (uint32_t s = lane; s < T.nsub; s += 32u) mbar_wait(&bars[s], parity, &s_flag[0], a.wait_ns);
            __syncwarp();
            for (uint32_t s = 0; s < T.nsub; ++s) {
                const float *__restrict__ base = buf + (size_t)s * slot_floats + off;
                float4 x[SUB];
#pragma unroll
                for (uint32_t r = 0; r < (uint32_t)SUB; ++r)
                    x[r] = colok ? *reinterpret_cast<const float4 *>(base + (size_t)r * pitch)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
                tmem_st32(taddr + 32u * s, x);
                __syncwarp();
                if (lane == 0) mbar_arrive(&consumed[g * a.nsub_max + s]);
            }
            tmem_wait_st();
        }

        // ---- W(i): all CTAs' partial margins -> step coefficients in shared memory ----
        {
            // the labels of the rows this lane will finish, requested before the wait
            const float *__restrict__ yt = a.y + (uint64_t)T.k * a.y_stride + (uint64_t)T.t * a.batch;
            const unsigned long long *const ain = a.acc + (uint64_t)(i % EP_RING) * a.batch * EP_ROW_WORDS;
            if (tg == 0) {   // one thread waits for the row that every CTA adds to last
                const unsigned long long *const last = ain + (uint64_t)(T.m - 1u) * EP_ROW_WORDS;
                const uint64_t t0 = now_ns();
                uint32_t n = 0u;
                while ((ld_relaxed_v2(last).x >> 55) < ncta) {
                    if ((++n & a.poll_mask) == 0u) {
                        if (s_flag[0] != 0u || ld_acquire(a.header) != 0u || expired(t0, a.wait_ns)) {
                            s_flag[0] = 1u;
                            break;
                        }
                        __nanosleep(64);
                    }
                }
            }
            if (sync_any(1u + g, EP_GROUP, s_flag[0])) break;
            // a thread per row: the other rows are complete by now or within a few looks
            for (uint32_t j = tg; j < T.m; j += EP_GROUP) {
                const unsigned long long *const r = ain + (uint64_t)j * EP_ROW_WORDS;
                const float yj = __ldg(yt + j);
                ulonglong2 v = ld_relaxed_v2(r);
                if ((v.x >> 55) < ncta) {
                    const uint64_t t0 = now_ns();
                    uint32_t n = 0u;
                    while (((v = ld_relaxed_v2(r)).x >> 55) < ncta) {
                        if ((++n & a.poll_mask) == 0u &&
                            (s_flag[0] != 0u || ld_acquire(a.header) != 0u || expired(t0, a.wait_ns))) {
                            s_flag[0] = 1u;
                            break;
                        }
                    }
                }
                const ulonglong2 special = ld_relaxed_v2(r + 2);   // NaN count | +Inf count << 32 + -Inf count
                const long long fine = (long long)((v.x & (FX_ONE - 1ull)) - (unsigned long long)ncta * FX_BIAS);
                float margin = (float)((double)fine * (1.0 / (double)FX_SCALE) +
                                       (double)(long long)v.y * (1.0 / (double)FX_WIDE_SCALE));
                if (special.y != 0ull) {
                    const bool pos = (special.y >> 32) != 0ull, neg = (special.y & 0xFFFFFFFFull) != 0ull;
                    margin = pos && neg ? __int_as_float(0x7FC00000)
                                        : __int_as_float(pos ? 0x7F800000 : (int)0xFF800000);
                }
                if (special.x != 0ull) margin = __int_as_float(0x7FC00000);
                // -(lr/m) * c_j with c_j = -y_j / (1 + exp(y_j m_j))
                coef[j] = (a.lr / (float)T.m) * yj / (1.0f + expf(yj * margin));
            }
            if (sync_any(1u + g, EP_GROUP, s_flag[0])) break;
        }

        // ---- U(i): update this CTA's columns of u from the buffer, release the buffer ----
        {
            float4 *const up = reinterpret_cast<float4 *>(a.u + (uint64_t)T.k * a.u_stride + c0 + col);
            float4 uold = make_float4(0.f, 0.f, 0.f, 0.f);
            if (colok) uold = *up;                       // requested now, needed after the loop
            // Every warp observes the arrival of every sub-tile itself before it reads what TMA
            // wrote: lane s looks at sub-tile s (a look costs about 0.1 us, so the lanes look in
            // parallel), and the warp follows its lanes through __syncwarp.  All of them have
            // landed: the warps that took the margins waited for them.
            if (!stash)
                for (uint32_t s = lane; s < T.nsub; s += 32u) mbar_wait(&bars[s], parity, &s_flag[0], a.wait_ns);
            __syncwarp();
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t s = 0; stash && s < T.nsub; ++s) {
                float4 x[SUB];
                tmem_ld32(taddr + 32u * s, x);
                tmem_wait_ld();
#pragma unroll
                for (uint32_t r = 0; r < (uint32_t)SUB; ++r) {
                    const uint32_t jj = s * SUB + r;
                    if (colok && jj < T.m) {
                        const float cj = coef[jj];
                        acc.x = fmaf(cj, x[r].x, acc.x);
                        acc.y = fmaf(cj, x[r].y, acc.y);
                        acc.z = fmaf(cj, x[r].z, acc.z);
                        acc.w = fmaf(cj, x[r].w, acc.w);
                    }
                }
            }
            for (uint32_t s = 0; !stash && s < T.nsub; ++s) {
                if (colok) {
                    const float *__restrict__ base = buf + (size_t)s * slot_floats + off;
#pragma unroll
                    for (uint32_t r = 0; r < (uint32_t)SUB; ++r) {
                        const uint32_t jj = s * SUB + r;
                        if (jj < T.m) {
                            const float4 x = *reinterpret_cast<const float4 *>(base + (size_t)r * pitch);
                            const float cj = coef[jj];
                            acc.x = fmaf(cj, x.x, acc.x);
                            acc.y = fmaf(cj, x.y, acc.y);
                            acc.z = fmaf(cj, x.z, acc.z);
                            acc.w = fmaf(cj, x.w, acc.w);
                        }
                    }
                }
                // the warp is through with this slot: one arrival per warp hands it back to the
                // producer, which refills it while the update goes on
                __syncwarp();
                if (lane == 0) mbar_arrive(&consumed[g * a.nsub_max + s]);
            }
            if (colok) {
                uold.x += acc.x;
                uold.y += acc.y;
                uold.z += acc.z;
                uold.w += acc.w;
                *up = uold;
            }
            group_sync();                                 // u stored by the whole group
            if (tg == 0) {
                __threadfence_block();
                s_flag[4u + g] = (i >> 1) + 1u;           // this group's tiles completed
            }
        }
    }

    // Both groups meet here, whether they finished or gave up.
    asm volatile("bar.sync 3, %0;" ::"n"(EP_CONSUMERS) : "memory");
    if (stash && warp == 0) tmem_free_all(tmem_base);   // on every path out of the kernel
    // A wait ran out: tell the host and the other CTAs.  The copies still in flight are the
    // producer warp's to wait for.
    if (s_flag[0] != 0u && tid == 0) {
        atomicOr(a.status, QESGD_STATUS_TIMEOUT);
        atomicExch(a.header, 1u);
    }
}

// ------------------------------------------------------------------ host ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// Per-device set-up: shared-memory limit of the kernel, the driver's tensor-map encoder.
constexpr int MAX_DEVICES = 64;
std::mutex g_epoch_mutex;
int g_epoch_smem_limit[MAX_DEVICES] = {0};   // 0 = not queried, -1 = unsupported
EncodeTiledFn g_encode_tiled = nullptr;

int epoch_smem_limit(int device)
{
    if (device < 0 || device >= MAX_DEVICES) return -1;
    std::lock_guard<std::mutex> lock(g_epoch_mutex);
    if (g_epoch_smem_limit[device] == 0) {
        int coop = 0, optin = 0;
        cudaError_t e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device);
        if (e == cudaSuccess)
            e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
        if (e == cudaSuccess && coop && optin > 0)
            e = cudaFuncSetAttribute(qesgd_lr_epoch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     optin);
        if (e == cudaSuccess && !g_encode_tiled) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
            e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
            if (e == cudaSuccess && q == cudaDriverEntryPointSuccess) g_encode_tiled = (EncodeTiledFn)fn;
        }
        g_epoch_smem_limit[device] =
            (e == cudaSuccess && coop && optin > 0 && g_encode_tiled) ? optin : -1;
        if (e != cudaSuccess) cudaGetLastError();
    }
    return g_epoch_smem_limit[device];
}

// Row-major float matrix [rows][d] seen as a 2-D tensor; a box is SUB rows of box_cols columns.
// Elements outside the matrix read as zero.
bool make_map(CUtensorMap *map, const float *X, uint64_t rows, uint64_t d, uint32_t box_cols)
{
    const cuuint64_t dims[2] = {d, rows};
    const cuuint64_t strides[1] = {d * sizeof(float)};
    const cuuint32_t box[2] = {box_cols, (cuuint32_t)SUB};
    const cuuint32_t elem[2] = {1u, 1u};
    return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2u, const_cast<float *>(X), dims, strides, box,
                          elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Returns 0 = launched, -1 = shape not covered by the fused kernel (caller uses the
// two-pass steps), > 0 = cudaError_t.
int qesgd_launch_lr_epoch_fused(const float *X, const float *y, uint64_t n_local, uint64_t d,
                                uint32_t K, uint32_t batch, float lr, float *u, uint64_t u_stride,
                                float *work, uint64_t work_floats, uint32_t *status, int device,
                                int sm_count, uint64_t wait_ns, uint32_t drop_cta, cudaStream_t stream,
                                int *launched)
{
    *launched = 0;
    const uint32_t m_full = (uint32_t)(n_local < batch ? n_local : batch);
    if (m_full > (uint32_t)EP_MAX_M) return -1;
    const uint64_t nsteps64 = (n_local + m_full - 1) / m_full;
    if (nsteps64 * K > (1u << 20)) return -1;
    if ((uint64_t)K * n_local + EP_MAX_M >= (1ull << 31)) return -1;   // TMA row coordinates
    if (d % 4 != 0 || u_stride % 4 != 0 || ((uintptr_t)X | (uintptr_t)u) % 16 != 0) return -1;
    if (sm_count < 1) return -1;
    uint64_t cols = (d + (uint64_t)sm_count - 1) / (uint64_t)sm_count;
    cols = (cols + 3) / 4 * 4;
    if (cols > (uint64_t)EP_MAX_COLS) return -1;
    const uint32_t ncta = (uint32_t)((d + cols - 1) / cols);
    if (ncta > 256u) return -1;   // the accumulator word counts up to 511 contributions
    const int limit = epoch_smem_limit(device);
    if (limit <= 0) return -1;

    EpochArgs a;
    a.y = y; a.y_stride = n_local; a.n_local = n_local;
    a.d = d; a.K = K; a.batch = m_full; a.nsteps = (uint32_t)nsteps64;
    a.m_last = (uint32_t)(n_local - (nsteps64 - 1) * m_full);
    a.nsub_max = (m_full + SUB - 1) / SUB;
    a.nsub_last = (a.m_last + SUB - 1) / SUB;
    a.cols = (uint32_t)cols;
    a.lr = lr;
    a.u = u; a.u_stride = u_stride;
    a.status = status;
    a.wait_ns = wait_ns;
    a.poll_mask = wait_ns < COARSE_TIMER_NS ? 0u : 31u;
    a.drop_cta = drop_cta;

    // shared memory: two tile buffers | coefficients of both groups | barriers | flags
    const size_t smem = (size_t)2 * a.nsub_max * SUB * cols * sizeof(float) + 2 * EP_MAX_M * sizeof(float) +
                        (4 * EP_MAX_NSUB) * sizeof(uint64_t) + 64;
    if (smem > (size_t)limit) return -1;

    // workspace: header | margin accumulators (the workspace is 256-byte aligned)
    const uint64_t words = EP_HEADER_WORDS + (uint64_t)EP_RING * m_full * EP_ROW_WORDS * 2u;
    if (words > work_floats) return -1;
    a.header = reinterpret_cast<uint32_t *>(work);
    a.acc = reinterpret_cast<unsigned long long *>(work + EP_HEADER_WORDS);

    CUtensorMap map_a, map_b;
    const uint32_t cols_a = cols < (uint64_t)EP_BOX_COLS ? (uint32_t)cols : (uint32_t)EP_BOX_COLS;
    const uint32_t cols_b = (uint32_t)cols - cols_a;
    if (!make_map(&map_a, X, (uint64_t)K * n_local, d, cols_a)) return -1;
    if (!make_map(&map_b, X, (uint64_t)K * n_local, d, cols_b ? cols_b : cols_a)) return -1;

    cudaError_t e = cudaMemsetAsync(work, 0, words * sizeof(float), stream);
    if (e != cudaSuccess) return (int)e;
    void *params[] = {(void *)&a, (void *)&map_a, (void *)&map_b};
    e = cudaLaunchCooperativeKernel((const void *)qesgd_lr_epoch_kernel, dim3(ncta), dim3(EP_THREADS), params,
                                    smem, stream);
    if (e == cudaErrorCooperativeLaunchTooLarge || e == cudaErrorLaunchOutOfResources ||
        e == cudaErrorInvalidConfiguration || e == cudaErrorNotSupported) {
        cudaGetLastError();   // the device cannot hold all CTAs at once as configured: two-pass steps
        return -1;
    }
    if (e != cudaSuccess) return (int)e;
    *launched = 1;
    return 0;
}
