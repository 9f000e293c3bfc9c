// QESGD codec kernels for sm_100a: fused encode (delta, bucket scale, stochastic
// rounding, packing), decode, and fused decode-average-apply.
//
// This file must be compiled with -fmad=false: the rounding chain is a sequence
// of single IEEE operations and must not be contracted into FMAs.  Where an FMA
// is wanted it is written explicitly.
//
// Work unit: an "octet" of 8 consecutive elements per lane -- one 256-bit load,
// one Philox4x32-10 block (8 draws of 16 bits), and 8 codes that form 2 / 4 / 8
// whole bytes of the output stream, so no cross-lane transposition is needed.
// A warp instruction covers a "chunk" of 256 consecutive elements (1 KB).
#include "qesgd_internal.h"

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr int CHUNK = 256;  // elements covered by one warp-wide 256-bit load
#ifndef QESGD_ENCODE_CHUNKS
#define QESGD_ENCODE_CHUNKS 4  // chunks per warp in the encode kernel (2 or 4)
#endif
#ifndef QESGD_DAA_THREADS
#define QESGD_DAA_THREADS 32    // threads per CTA of the decode-average-apply kernel
#endif
#ifndef QESGD_DAA_BATCH
#define QESGD_DAA_BATCH 4       // workers whose code words are fetched together
#endif
// chunks (64-bit code words per worker) a lane of that kernel owns, by code width
#ifndef QESGD_DAA_WORDS_2BIT
#define QESGD_DAA_WORDS_2BIT 1
#endif
#ifndef QESGD_DAA_WORDS_WIDE
#define QESGD_DAA_WORDS_WIDE 2
#endif
#ifndef QESGD_DECODE_OCTETS
#define QESGD_DECODE_OCTETS 4   // octets per thread of the plain decode kernel
#endif
#ifndef QESGD_DAA_MIN_CTAS
#define QESGD_DAA_MIN_CTAS 24   // resident CTAs per SM its register budget is set for
#endif
#ifndef QESGD_ENCODE_MIN_WARPS
#define QESGD_ENCODE_MIN_WARPS 24  // resident warps per SM the register budget is set for
#endif
#ifndef QESGD_ENCODE_WARPS
#define QESGD_ENCODE_WARPS 1   // warps per CTA unless a bucket needs more
#endif

// ---------------------------------------------------------------- memory ----
__device__ __forceinline__ void ld256(const float *p, float (&v)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]),
                   "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}

// Read-modify-write data (the parameter) goes through the coherent path.
__device__ __forceinline__ void ld256_rw(const float *p, float (&v)[8])
{
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]),
                   "=f"(v[6]), "=f"(v[7])
                 : "l"(p)
                 : "memory");
}

__device__ __forceinline__ void st256(float *p, const float (&v)[8])
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]),
                 "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
}

// 8 elements starting at element index eb of a vector of d elements; zeros past d.
// RW = the buffer is also written by this kernel: no read-only (non-coherent) loads.
template <bool VEC, bool RW = false>
__device__ __forceinline__ void load_octet(const float *p, uint64_t eb, uint64_t d, float (&v)[8])
{
    if (VEC && eb + 8 <= d) {
        if (RW) ld256_rw(p + eb, v);
        else ld256(p + eb, v);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (eb + j < d) ? (RW ? p[eb + j] : __ldg(p + eb + j)) : 0.0f;
    }
}

// ---------------------------------------------------------------- Philox ----
// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11), written from the
// published round function: two 32x32->64 multiplies, the high halves xor'ed with
// the other counter words and the round key; the key grows by the Weyl constants.
// Two independent blocks advanced round by round: four multiply chains in flight instead
// of two (measured 2 % faster than one block at a time; four at a time costs registers).
// rk[r] = key + r * (0x9E3779B9, 0xBB67AE85): the ten round keys, prepared on the host so
// that they reach the xor as kernel-parameter operands instead of per-thread additions.
__device__ __forceinline__ void philox4x32_10_x2(uint32_t (&c)[2][4], const uint32_t (&rk)[10][2])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            const uint64_t p0 = (uint64_t)0xD2511F53u * c[n][0];
            const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[n][2];
            const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[n][1] ^ rk[r][0];
            const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[n][3] ^ rk[r][1];
            c[n][1] = (uint32_t)p1;
            c[n][3] = (uint32_t)p0;
            c[n][0] = n0;
            c[n][2] = n2;
        }
    }
}

// ------------------------------------------------- packed fp32 pairs --------
// sm_100 adds add / sub / mul / fma on two floats held in a 64-bit register pair.
__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi)
{
    uint64_t p;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "r"(lo), "r"(hi));
    return p;
}
__device__ __forceinline__ uint64_t pack2f(float lo, float hi)
{
    uint64_t p;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "f"(lo), "f"(hi));
    return p;
}
__device__ __forceinline__ void unpack2(uint64_t p, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t fma2_ru(uint64_t a, uint64_t b, uint64_t c)   // toward +inf
{
    uint64_t d;
    asm("fma.rp.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// ------------------------------------------------------- rounding (Eq. 4) ----
// level = floor(r) + [h + 1/2 < frac(r) * 2^16] for r = min(|z|*inv, s), 0 <= r <= 127.
//
// With U = ceil(r * 2^16 - 1/2) the level is (U + 65535 - h) >> 16: writing U =
// floor(r) * 2^16 + T, T = ceil(frac(r) * 2^16 - 1/2) in [0, 2^16], the draw rounds
// up iff h < T.  U comes from ONE fused multiply-add rounded toward +infinity:
// r * 2^16 + (2^23 - 1/2) lies in [2^23, 2^24) where floats are the integers, so
// the bit pattern of the result is 0x4B000000 + U.  r is kept >= 2^-30 so that
// r = 0 (where the sum would be 2^23 - 1/2 exactly, below the integer binade)
// gives U = 0 like every r with r * 2^16 <= 1/2; the same clamp turns the NaN of
// an invalid bucket (inv = 0) into level 0.
// Two neighbouring elements at a time: the multiply and the fused multiply-add run on
// packed pairs, the clamp stays scalar (it takes |.| for free).  x0, x1 receive the level
// in bits 16..22 (what is below is of no interest).
// CLIP: only a caller-given spacing needs the upper clamp min(r, s).  With a scale taken
// from the bucket itself |z| <= scale, and inv = fl32(s/scale) is at most (s/scale) *
// (1 + 2^-24), so the exact product is below s + ulp(s) and its fp32 rounding is s or
// s + ulp(s).  (Where s/scale is subnormal -- scale > s * 2^126, so s < 4 -- inv is off by
// at most 2^-150 and the product by at most 2^128 * 2^-150 = 2^-22.)  Either way r - s <=
// 2^-17 for s <= 127, i.e. at most 1/2 after the scaling by 2^16, and ceil(s * 2^16 + 1/2
// - 1/2) is still s * 2^16: the overshoot never reaches a level, so the clamp would change
// nothing.
template <bool CLIP>
__device__ __forceinline__ void level_pair(float z0, float z1, uint64_t inv2, float sf,
                                           uint32_t h0, uint32_t h1, uint32_t &x0, uint32_t &x1)
{
    float t0, t1;
    unpack2(mul2(pack2f(z0, z1), inv2), t0, t1);           // sign rides along, removed by |.|
    float r0 = fmaxf(fabsf(t0), 0x1p-30f);
    float r1 = fmaxf(fabsf(t1), 0x1p-30f);
    if (CLIP) {
        r0 = fminf(r0, sf);
        r1 = fminf(r1, sf);
    }
    float u0, u1;
    unpack2(fma2_ru(pack2f(r0, r1), pack2f(65536.0f, 65536.0f), pack2f(8388607.5f, 8388607.5f)),
            u0, u1);
    x0 = __float_as_uint(u0) - h0 + (65535u - 0x4B000000u);
    x1 = __float_as_uint(u1) - h1 + (65535u - 0x4B000000u);
}

// (a & b) | c and (a & b) ^ c as one three-input logic operation each
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t and_xor(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// Packing.  X[j] holds the level of element j in byte 2 (bits 16..22) and Z[j] the
// sign of z_j in bit 31.  Bytes are gathered with PRMT, fields merged with
// multiply-adds; the sign is kept only where the level is not zero, which is
// tested on whole words (a field plus its largest level never carries).
// X[j] = U + 65535 - h lies in [0, 2^23), so its byte 3 is always zero and serves as the
// source of zero bytes.  PRMT's replicate mode (selector nibble 8 + n) turns the top bit of
// byte n into a whole byte of ones or zeros, so a sign lands on any bit of its byte by a
// mask alone, without a shift.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t bytes2(uint32_t a, uint32_t b)   // [a.b2, b.b2, 0, 0]
{
    return prmt(a, b, 0x3362u);
}
__device__ __forceinline__ uint32_t bytes3(uint32_t a, uint32_t b)   // [a.b3, b.b3, ., .]
{
    return __byte_perm(a, b, 0x0073);
}
__device__ __forceinline__ uint32_t signs2(uint32_t a, uint32_t b)   // [a<0 ? FF : 00, b<0 ? FF : 00, ., .]
{
    return prmt(a, b, 0x00FBu);
}

template <int BITS>
__device__ __forceinline__ void pack_octet(const uint32_t (&X)[8], const uint32_t (&Z)[8],
                                           uint32_t (&out)[2])
{
    if (BITS == 8) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e = 4 * h;
            const uint32_t lv = __byte_perm(__byte_perm(X[e], X[e + 1], 0x0062),
                                            __byte_perm(X[e + 2], X[e + 3], 0x0062), 0x5410);
            const uint32_t sg = __byte_perm(bytes3(Z[e], Z[e + 1]), bytes3(Z[e + 2], Z[e + 3]), 0x5410);
            out[h] = lv | (sg & (lv + 0x7F7F7F7Fu) & 0x80808080u);
        }
    } else if (BITS == 4) {
        // even elements fill the low nibbles, odd elements the high nibbles
        const uint32_t le = __byte_perm(__byte_perm(X[0], X[2], 0x0062), __byte_perm(X[4], X[6], 0x0062), 0x5410);
        const uint32_t lo = __byte_perm(__byte_perm(X[1], X[3], 0x0062), __byte_perm(X[5], X[7], 0x0062), 0x5410);
        const uint32_t lv = le + lo * 16u;
        const uint32_t se = __byte_perm(signs2(Z[0], Z[2]), signs2(Z[4], Z[6]), 0x5410);
        const uint32_t so = __byte_perm(signs2(Z[1], Z[3]), signs2(Z[5], Z[7]), 0x5410);
        const uint32_t sg = and_or(se, 0x08080808u, so & 0x80808080u);
        out[0] = lv | (sg & (lv + 0x77777777u));
        out[1] = 0u;
    } else {
        // element j sits at bits 2j, 2j+1: byte 0 holds elements 0..3, byte 1 elements 4..7
        const uint32_t g0 = bytes2(X[0], X[4]), g1 = bytes2(X[1], X[5]);
        const uint32_t g2 = bytes2(X[2], X[6]), g3 = bytes2(X[3], X[7]);
        const uint32_t lv = (g0 + g1 * 4u) + (g2 * 16u + g3 * 64u);
        const uint32_t h0 = signs2(Z[0], Z[4]), h1 = signs2(Z[1], Z[5]);
        const uint32_t h2 = signs2(Z[2], Z[6]), h3 = signs2(Z[3], Z[7]);
        const uint32_t sg = and_or(h3, 0x8080u, and_or(h2, 0x2020u, and_or(h1, 0x0808u, h0 & 0x0202u)));
        out[0] = lv | (sg & (lv << 1));
        out[1] = 0u;
    }
}

// ----------------------------------------------------- bucket reductions ----
struct SumF64 {
    typedef double T;
    static __device__ __forceinline__ double op(double x, double y) { return __dadd_rn(x, y); }
};
struct MaxU32 {
    typedef uint32_t T;
    static __device__ __forceinline__ uint32_t op(uint32_t x, uint32_t y) { return max(x, y); }
};

// Reduces the V per-chunk partials of every lane over the lanes (and chunks) of a
// bucket, in the order of the balanced binary tree on element index: lanes xor 1, 2,
// 4, (8), (16), then chunk pairs, then chunk quads.  The first step(s) hand each lane
// ONE chunk to carry on with (V = 4: even/odd lanes split chunks {0,1}/{2,3}, then
// bit 1 of the lane splits the pair; V = 2: even lanes take chunk 0, odd lanes chunk
// 1), so the rest of the tree costs one value per step instead of V.  On return lane
// L holds the bucket total of chunk chunk_of_lane<V>(L) of its own lane group (once a
// bucket spans several chunks, all of them hold its total).
template <int V>
__device__ __forceinline__ uint32_t chunk_of_lane(uint32_t lane)
{
    return V == 4 ? 2u * (lane & 1u) + ((lane >> 1) & 1u) : (lane & 1u);
}
template <int V>
__device__ __forceinline__ uint32_t lane_of_chunk(uint32_t lane, int c)
{
    return V == 4 ? ((lane & 28u) | ((c >> 1) & 1) | ((c & 1) << 1)) : ((lane & 30u) | (c & 1));
}

template <typename R>
__device__ __forceinline__ typename R::T reduce_chunks(const typename R::T (&t)[4], uint32_t lane,
                                                       uint32_t lb)
{
    typedef typename R::T T;
    const bool b0 = lane & 1u, b1 = lane & 2u;
    T k0 = b0 ? t[2] : t[0], k1 = b0 ? t[3] : t[1];
    const T s0 = b0 ? t[0] : t[2], s1 = b0 ? t[1] : t[3];
    k0 = R::op(k0, __shfl_xor_sync(FULL, s0, 1));
    k1 = R::op(k1, __shfl_xor_sync(FULL, s1, 1));
    T k = b1 ? k1 : k0;
    const T s = b1 ? k0 : k1;
    k = R::op(k, __shfl_xor_sync(FULL, s, 2));
    k = R::op(k, __shfl_xor_sync(FULL, k, 4));
    if (lb >= 7) k = R::op(k, __shfl_xor_sync(FULL, k, 8));
    if (lb >= 8) k = R::op(k, __shfl_xor_sync(FULL, k, 16));
    if (lb >= 9) k = R::op(k, __shfl_xor_sync(FULL, k, 2));    // chunks (0,1) and (2,3)
    if (lb >= 10) k = R::op(k, __shfl_xor_sync(FULL, k, 1));   // all four chunks
    return k;
}

template <typename R>
__device__ __forceinline__ typename R::T reduce_chunks(const typename R::T (&t)[2], uint32_t lane,
                                                       uint32_t lb)
{
    typedef typename R::T T;
    const bool b0 = lane & 1u;
    T k = b0 ? t[1] : t[0];
    const T s = b0 ? t[0] : t[1];
    k = R::op(k, __shfl_xor_sync(FULL, s, 1));
    k = R::op(k, __shfl_xor_sync(FULL, k, 2));
    k = R::op(k, __shfl_xor_sync(FULL, k, 4));
    if (lb >= 7) k = R::op(k, __shfl_xor_sync(FULL, k, 8));
    if (lb >= 8) k = R::op(k, __shfl_xor_sync(FULL, k, 16));
    if (lb >= 9) k = R::op(k, __shfl_xor_sync(FULL, k, 1));    // both chunks
    return k;
}

// Buckets wider than a warp's V*256 elements: combine the totals of the wpb consecutive
// warps that share a bucket (wpb a power of two <= 16), adjacent pairs first.
template <typename R>
__device__ __forceinline__ typename R::T reduce_warps(typename R::T k, typename R::T *smem,
                                                      uint32_t lane, uint32_t warp, uint32_t wpb)
{
    typedef typename R::T T;
    if (lane == 0) smem[warp] = k;
    __syncthreads();
    // lanes 0..wpb-1 (and every further group of wpb lanes) pick up the warps' totals; the
    // xor butterfly over them is the balanced tree on warp order
    T v = smem[(warp & ~(wpb - 1u)) + (lane & (wpb - 1u))];
#pragma unroll
    for (int off = 1; off < 16; off <<= 1)
        if ((uint32_t)off < wpb) v = R::op(v, __shfl_xor_sync(FULL, v, off));
    return v;
}

// ------------------------------------------------------------- encode -------
// MODE: 0 = L2 norm, 1 = max magnitude, 2 = caller-given spacing.
// A warp owns V chunks = V*256 consecutive elements, a CTA of W warps W*V*256.
// Buckets are powers of two in [64, 8192]:
//   bucket <= 256     : bucket/8 lanes of one chunk
//   bucket <= 256*V   : bucket/256 chunks of one warp
//   bucket  > 256*V   : bucket/(256*V) consecutive warps of the CTA (shared memory)
struct EncodeShared {
    double part[2][16];     // cross-warp partial sums, double-buffered by iteration
    uint32_t maxv[2][16];
};

// Everything after the deltas z of one warp tile are in registers: bucket scale,
// Philox draws, stochastic rounding, packing, stores.  `iter` selects the half of the
// cross-warp scratch (callers alternate it between consecutive tiles of one CTA).
// FULL = the whole warp tile lies inside the vector: no store needs a bounds check.
// REQ = per-step QESGD (Algorithm 2: z = Q(z^), u = w_t + z): besides the stream, the
// quantised delta is decoded on the spot, written back as u = fl32(anchor + Q(z)) and
// added to the running sum of the epoch average.
template <int BITS, int MODE, int V, bool FULL, bool REQ>
__device__ __forceinline__ void encode_warp_tile(const EncodeArgs &a, float (&z)[V][8],
                                                 uint64_t warp_base, uint32_t k, uint32_t lane,
                                                 uint32_t warp, EncodeShared &sh, uint32_t iter)
{
    constexpr uint32_t LOG2_WARP_ELEMS = V == 4 ? 10 : 9;
    const uint32_t lb = a.log2_bucket;
    const float sf = (float)a.s;
    float my_scale, my_inv, my_delta = 0.0f;
    bool flag = false;
    // All addresses of the tile derive from three values computed once; inside the
    // chunk loop only small compile-time offsets are added.  warp_base is a multiple of
    // V*256, so the Philox block index (warp_base/8 + lane + 32c) never carries into
    // its high word when c advances.
    const uint32_t loff = lane * 8u;
    uint8_t *const cbase = reinterpret_cast<uint8_t *>(a.codes) + (uint64_t)k * a.code_stride +
                           ((warp_base + loff) >> 3) * (uint64_t)BITS;
    float *const sbase = a.scales + (uint64_t)k * a.scale_stride + (warp_base >> lb);
    const uint64_t blk0 = (warp_base >> 3) + lane;
    const uint32_t blk_lo = (uint32_t)blk0, blk_hi = (uint32_t)(blk0 >> 32);
    const uint32_t bucket_mask = (1u << lb) - 1u;
    const bool wide = lb > LOG2_WARP_ELEMS;                     // bucket spans several warps
    const bool wide_first = ((uint32_t)warp_base & bucket_mask) == 0u;   // this warp starts it
    const uint32_t wid = a.worker0 + k;
    uint32_t xx[2][4];

    // The draws of the first two chunks are computed before the scale: they depend on nothing
    // loaded, so they fill the time the reduction's shuffles and the square root wait.
#pragma unroll
    for (int n = 0; n < 2; ++n) {
        xx[n][0] = blk_lo + 32u * n;
        xx[n][1] = blk_hi;
        xx[n][2] = wid;
        xx[n][3] = a.epoch;
    }
    philox4x32_10_x2(xx, a.round_key);

    // ---- per-bucket scale: one value per lane, then handed back per chunk ------
    if (MODE == 0) {
        // fp64 sum of squares over the balanced binary tree on index order.  The product
        // of two fp32 values is exact in fp64, so fma(z1,z1,z0*z0) is fl64(q0+q1).
        double t[V];
#pragma unroll
        for (int c = 0; c < V; ++c) {
            double q[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const double e0 = (double)z[c][2 * j], e1 = (double)z[c][2 * j + 1];
                q[j] = __fma_rn(e1, e1, __dmul_rn(e0, e0));
            }
            t[c] = __dadd_rn(__dadd_rn(q[0], q[1]), __dadd_rn(q[2], q[3]));
        }
        double tot = reduce_chunks<SumF64>(t, lane, lb);
        if (lb > LOG2_WARP_ELEMS)
            tot = reduce_warps<SumF64>(tot, sh.part[iter & 1u], lane, warp, 1u << (lb - LOG2_WARP_ELEMS));
        my_scale = __double2float_rn(__dsqrt_rn(tot));
    } else if (MODE == 1) {
        // Largest magnitude: bit patterns of |z| order like unsigned integers, and
        // Inf/NaN patterns compare above every finite value.
        uint32_t m[V];
#pragma unroll
        for (int c = 0; c < V; ++c) {
            m[c] = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) m[c] = max(m[c], __float_as_uint(z[c][j]) & 0x7FFFFFFFu);
        }
        uint32_t mm = reduce_chunks<MaxU32>(m, lane, lb);
        if (lb > LOG2_WARP_ELEMS)
            mm = reduce_warps<MaxU32>(mm, sh.maxv[iter & 1u], lane, warp, 1u << (lb - LOG2_WARP_ELEMS));
        my_scale = __uint_as_float(mm);
    } else {
        my_scale = a.fixed_scale;
    }
    {
        const bool nonfinite = !(my_scale <= 3.402823466e38f);   // Inf or NaN (scales are >= 0)
        const bool ok = !nonfinite && my_scale >= 0x1p-100f;
        my_inv = ok ? __fdiv_rn(sf, my_scale) : 0.0f;
        my_scale = ok ? my_scale : 0.0f;
        if (REQ) my_delta = __fdiv_rn(my_scale, sf);   // grid spacing of the decoder
        // Lanes past the padded length hold zeros, so a set flag always belongs to real data.
        flag = nonfinite;
    }

    // ---- rounding, packing, stores ---------------------------------------------
#pragma unroll
    for (int c = 0; c < V; ++c) {
        const uint32_t off = (uint32_t)c * CHUNK + loff;        // element offset inside the tile
        const bool inside = FULL || warp_base + off < a.padded;
        float scale = my_scale, inv = my_inv, delta = my_delta;
        if (MODE != 2) {   // fetch chunk c's bucket scale from the neighbour lane that carried it
            const int src = (int)lane_of_chunk<V>(lane, c);
            scale = __shfl_sync(FULL, my_scale, src);
            inv = __shfl_sync(FULL, my_inv, src);
            if (REQ) delta = __shfl_sync(FULL, my_delta, src);
        }
        if (inside) {      // the first lane of every bucket writes its scale
            if (!wide) {
                if ((off & bucket_mask) == 0u &&
                    QESGD_IN_RANGE(a.status, ((warp_base + off) >> lb) < (a.padded >> lb)))
                    sbase[off >> lb] = scale;
            } else if (off == 0u && wide_first && QESGD_IN_RANGE(a.status, (warp_base >> lb) < (a.padded >> lb))) {
                sbase[0] = scale;
            }
        }

        if ((c & 1) == 0 && c > 0) {   // draws for this chunk and the next, interleaved
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                xx[n][0] = blk_lo + 32u * (c + n);
                xx[n][1] = blk_hi;
                xx[n][2] = wid;
                xx[n][3] = a.epoch;
            }
            philox4x32_10_x2(xx, a.round_key);
        }
        const uint32_t (&x)[4] = xx[c & 1];

        uint32_t X[8], Z[8];
        const uint64_t inv2 = pack2f(inv, inv);
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            Z[j] = __float_as_uint(z[c][j]);
            Z[j + 1] = __float_as_uint(z[c][j + 1]);
            if (MODE == 2)   // NaN has no place on the grid: flagged (and encoded as 0 by the clamp)
                flag |= (Z[j] & 0x7FFFFFFFu) > 0x7F800000u || (Z[j + 1] & 0x7FFFFFFFu) > 0x7F800000u;
            level_pair<MODE == 2>(z[c][j], z[c][j + 1], inv2, sf, x[j >> 1] & 0xFFFFu, x[j >> 1] >> 16,
                       X[j], X[j + 1]);
        }
        if (REQ) {
            // decode what was just quantised: +-level * delta, the sign only where level > 0
            float v[8], w[8];
            const uint64_t e0 = warp_base + off;
            const uint64_t go = (uint64_t)k * a.local_stride + e0;
            if (FULL) ld256(a.anchor + e0, w);
            else load_octet<false>(a.anchor, e0, a.d, w);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t lv = X[j] >> 16;
                const float lf = __fsub_rn(__uint_as_float(0x4B000000u | lv), 8388608.0f);
                const uint32_t sign31 = Z[j] & (lv + 0x7FFFFFFFu) & 0x80000000u;
                v[j] = __uint_as_float(__float_as_uint(__fmul_rn(lf, delta)) | sign31);
                w[j] = __fadd_rn(w[j], v[j]);
            }
            if (FULL) {
                if (QESGD_IN_RANGE(a.status, e0 + 8 <= a.d)) st256(a.u_out + go, w);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (e0 + j < a.d) a.u_out[go + j] = w[j];
            }
            if (a.zsum) {
                float zs[8];
                if (FULL) ld256_rw(a.zsum + go, zs);
                else load_octet<false, true>(a.zsum, go, (uint64_t)k * a.local_stride + a.d, zs);
#pragma unroll
                for (int j = 0; j < 8; ++j) zs[j] = __fadd_rn(zs[j], v[j]);
                if (FULL) {
                    if (QESGD_IN_RANGE(a.status, e0 + 8 <= a.d)) st256(a.zsum + go, zs);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (e0 + j < a.d) a.zsum[go + j] = zs[j];
                }
            }
        }
        uint32_t out[2];
        pack_octet<BITS>(X, Z, out);
        if (inside && QESGD_IN_RANGE(a.status, warp_base + off + 8 <= a.padded)) {
            uint8_t *const q = cbase + c * (CHUNK * BITS / 8);
            if (BITS == 8) {
                *reinterpret_cast<uint2 *>(q) = make_uint2(out[0], out[1]);
            } else if (BITS == 4) {
                *reinterpret_cast<uint32_t *>(q) = out[0];
            } else {
                *reinterpret_cast<uint16_t *>(q) = (uint16_t)out[0];
            }
        }
    }
    if (flag) atomicOr(a.status, QESGD_STATUS_NONFINITE);
}

// One CTA per (tile, worker); every lane requests all of its 256-bit loads before it
// uses any of them, and several CTAs per SM overlap one another's load and arithmetic
// phases.  VEC = false (pointers not 32-byte aligned) falls back to scalar loads.
template <int BITS, int MODE, bool ANCHOR, bool VEC, int V, int WARPS, bool REQ>
__global__ void __launch_bounds__(WARPS * 32, QESGD_ENCODE_MIN_WARPS / WARPS)
    qesgd_encode_kernel(const EncodeArgs a)
{
    __shared__ EncodeShared sh;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    // Workers vary fastest over the grid: the K CTAs that share a tile of the anchor run
    // close together in time, so the anchor comes from HBM once and from L2 K-1 times.
    const uint32_t k = blockIdx.x % a.K;
    const uint32_t tile = blockIdx.x / a.K;
    const float *__restrict__ local = a.local + (uint64_t)k * a.local_stride;
    const uint64_t warp_base = ((uint64_t)tile * WARPS + warp) * (uint64_t)(V * CHUNK);

    float z[V][8];
    if (VEC && warp_base + V * CHUNK <= a.d) {   // the whole warp tile is inside the vector
        const float *__restrict__ p = local + warp_base + lane * 8u;
#pragma unroll
        for (int c = 0; c < V; ++c) {
            if (REQ) ld256_rw(p + c * CHUNK, z[c]);   // u is written back below
            else ld256(p + c * CHUNK, z[c]);
        }
        if (ANCHOR) {
            const float *__restrict__ q = a.anchor + warp_base + lane * 8u;
            float w[V][8];
#pragma unroll
            for (int c = 0; c < V; ++c) ld256(q + c * CHUNK, w[c]);
#pragma unroll
            for (int c = 0; c < V; ++c)
#pragma unroll
                for (int j = 0; j < 8; j += 2)
                    unpack2(sub2(pack2f(z[c][j], z[c][j + 1]), pack2f(w[c][j], w[c][j + 1])),
                            z[c][j], z[c][j + 1]);
        }
        encode_warp_tile<BITS, MODE, V, true, REQ>(a, z, warp_base, k, lane, warp, sh, 0u);
        return;
    }
#pragma unroll
    for (int c = 0; c < V; ++c)
        load_octet<VEC, REQ>(local, warp_base + (uint64_t)c * CHUNK + lane * 8u, a.d, z[c]);
    if (ANCHOR) {
#pragma unroll
        for (int c = 0; c < V; ++c) {
            float w[8];
            load_octet<VEC>(a.anchor, warp_base + (uint64_t)c * CHUNK + lane * 8u, a.d, w);
#pragma unroll
            for (int j = 0; j < 8; ++j) z[c][j] = __fsub_rn(z[c][j], w[j]);
        }
    }
    encode_warp_tile<BITS, MODE, V, false, REQ>(a, z, warp_base, k, lane, warp, sh, 0u);
}

// ---------------------------------- update + requantise (Algorithm 2 inner step) ----
// One inner iteration of QESGD on logistic regression after the margin pass: a CTA owns a
// tile of 1024 columns, forms u^ = u - (lr/m) sum_j c_j x_j for them in shared memory (the
// arithmetic of the plain update pass, in its order: rows split over four groups, group sums
// added in group order), and its first warp then quantises u^ - w_t, writes u = w_t + Q(z^),
// the running sum and the stream exactly as qesgd_requantize would.  The updated parameter
// never travels to global memory before it is quantised.  Buckets of at most 1024 elements,
// d a multiple of 4, 16-byte aligned X and u.  The register budget is set for three CTAs per SM
// (the requantising warp needs its 80 registers, the update loop needs the occupancy: with two
// CTAs per SM the call was 13 % slower than the two separate calls, with three it equals them).
constexpr int QS_COLS = 256;                   // columns per sub-tile: 64 groups of 4
constexpr int QS_ROWGROUPS = 4;
constexpr int QS_THREADS = (QS_COLS / 4) * QS_ROWGROUPS;
constexpr int QS_TILE = 4 * CHUNK;             // columns per CTA

template <int BITS, int MODE>
__global__ void __launch_bounds__(QS_THREADS, 3) qesgd_lr_qstep_kernel(const QstepArgs q)
{
    __shared__ float s_coef[QESGD_MAX_LR_BATCH];
    __shared__ float4 s_sum[QS_ROWGROUPS][QS_COLS / 4];
    __shared__ __align__(32) float s_u[QS_TILE];
    __shared__ EncodeShared sh;
    const EncodeArgs &a = q.e;
    for (uint32_t j = threadIdx.x; j < q.m; j += blockDim.x) {
        const float margin = q.margins[j];
        const float yj = __ldg(q.y + j);
        // -(lr/m) * c_j with c_j = -y_j / (1 + exp(y_j m_j))
        s_coef[j] = q.rate * yj / (1.0f + expf(yj * margin));
    }
    __syncthreads();
    const uint32_t cg = threadIdx.x % (QS_COLS / 4), rg = threadIdx.x / (QS_COLS / 4);
    const uint64_t tile0 = (uint64_t)blockIdx.x * QS_TILE;
#pragma unroll 1
    for (int sub = 0; sub < QS_TILE / QS_COLS; ++sub) {
        const uint64_t c = tile0 + (uint64_t)sub * QS_COLS + cg * 4u;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c + 4 <= a.d) {
            const float *__restrict__ col = q.X + c;
#pragma unroll 8
            for (uint32_t j = rg; j < q.m; j += QS_ROWGROUPS) {
                const float4 x = __ldg(reinterpret_cast<const float4 *>(col + (uint64_t)j * a.d));
                const float cj = s_coef[j];
                acc.x = fmaf(cj, x.x, acc.x);
                acc.y = fmaf(cj, x.y, acc.y);
                acc.z = fmaf(cj, x.z, acc.z);
                acc.w = fmaf(cj, x.w, acc.w);
            }
        }
        s_sum[rg][cg] = acc;
        __syncthreads();
        if (rg == 0) {
            float4 uu = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c + 4 <= a.d) {
                float4 t = s_sum[0][cg];
#pragma unroll
                for (int g = 1; g < QS_ROWGROUPS; ++g) {
                    const float4 v = s_sum[g][cg];
                    t.x = __fadd_rn(t.x, v.x); t.y = __fadd_rn(t.y, v.y);
                    t.z = __fadd_rn(t.z, v.z); t.w = __fadd_rn(t.w, v.w);
                }
                uu = *reinterpret_cast<const float4 *>(a.local + c);
                uu.x = __fadd_rn(uu.x, t.x); uu.y = __fadd_rn(uu.y, t.y);
                uu.z = __fadd_rn(uu.z, t.z); uu.w = __fadd_rn(uu.w, t.w);
            }
            *reinterpret_cast<float4 *>(s_u + sub * QS_COLS + cg * 4u) = uu;
        }
        __syncthreads();
    }
    if (threadIdx.x >= 32) return;
    // the first warp requantises the tile: z = u^ - w_t, zeros past d
    const uint32_t lane = threadIdx.x;
    float z[4][8];
    const bool full = tile0 + QS_TILE <= a.d &&
                      ((reinterpret_cast<uintptr_t>(a.anchor) | reinterpret_cast<uintptr_t>(a.u_out) |
                        reinterpret_cast<uintptr_t>(a.zsum)) & 31u) == 0u;
    if (full) {   // interior tile, aligned vectors: 256-bit loads and stores throughout
        float w[4][8];
#pragma unroll
        for (int c = 0; c < 4; ++c) ld256(a.anchor + tile0 + (uint64_t)c * CHUNK + lane * 8u, w[c]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float4 u0 = *reinterpret_cast<const float4 *>(s_u + c * CHUNK + lane * 8u);
            const float4 u1 = *reinterpret_cast<const float4 *>(s_u + c * CHUNK + lane * 8u + 4u);
            const float uj[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) z[c][j] = __fsub_rn(uj[j], w[c][j]);
        }
        encode_warp_tile<BITS, MODE, 4, true, true>(a, z, tile0, 0u, lane, 0u, sh, 0u);
        return;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint64_t e0 = tile0 + (uint64_t)c * CHUNK + lane * 8u;
        float w[8];
        load_octet<false>(a.anchor, e0, a.d, w);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float uj = s_u[c * CHUNK + lane * 8u + j];
            z[c][j] = (e0 + j < a.d) ? __fsub_rn(uj, w[j]) : 0.0f;
        }
    }
    encode_warp_tile<BITS, MODE, 4, false, true>(a, z, tile0, 0u, lane, 0u, sh, 0u);
}

// ------------------------------------------------------------- decode -------
// Signed value of slot j of a packed word: +-level * step.  The level is spliced
// into the mantissa of 2^23 (exact integer -> float without the conversion pipe).
template <int BITS>
__device__ __forceinline__ float code_value(uint32_t word, int slot, float step)
{
    constexpr uint32_t LEVEL_MASK = (1u << (BITS - 1)) - 1u;
    const uint32_t lv = (word >> (slot * BITS)) & LEVEL_MASK;
    const float lf = __fsub_rn(__uint_as_float(0x4B000000u | lv), 8388608.0f);
    const uint32_t sign31 = (word << (31 - (slot * BITS + BITS - 1))) & 0x80000000u;
    return __uint_as_float(__float_as_uint(__fmul_rn(lf, step)) ^ sign31);
}

// The packed codes of the octet starting at element eb: 8*BITS bits.
template <int BITS>
__device__ __forceinline__ void load_codes(const uint8_t *__restrict__ codes, uint64_t eb,
                                           uint32_t (&w)[2])
{
    if (BITS == 8) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(codes + eb));
        w[0] = v.x;
        w[1] = v.y;
    } else if (BITS == 4) {
        w[0] = __ldg(reinterpret_cast<const uint32_t *>(codes + (eb >> 1)));
        w[1] = 0u;
    } else {
        w[0] = __ldg(reinterpret_cast<const uint16_t *>(codes + (eb >> 2)));
        w[1] = 0u;
    }
}

// A thread decodes QESGD_DECODE_OCTETS octets that lie a whole grid apart (so every load and
// store instruction of a warp stays contiguous); all its code and scale loads are requested
// before the first is used.  Measured against one octet per thread: 5-14 % faster (four
// octets; eight are slower again).
template <int BITS, bool VEC>
__global__ void __launch_bounds__(256) qesgd_decode_kernel(const DecodeArgs a)
{
    constexpr int OPT = QESGD_DECODE_OCTETS;
    const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
    const uint64_t t0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint8_t *__restrict__ codes = reinterpret_cast<const uint8_t *>(a.codes);
    uint32_t w[OPT][2];
    float sc[OPT];
    uint64_t ebs[OPT];
#pragma unroll
    for (int i = 0; i < OPT; ++i) {
        ebs[i] = (t0 + (uint64_t)i * nthreads) * 8u;
        w[i][0] = w[i][1] = 0u;
        sc[i] = 0.0f;
        if (ebs[i] < a.d && QESGD_IN_RANGE(a.status, ebs[i] + 8 <= (a.nb << a.log2_bucket))) {
            load_codes<BITS>(codes, ebs[i], w[i]);
            sc[i] = __ldg(a.scales + (ebs[i] >> a.log2_bucket));
        }
    }
#pragma unroll
    for (int i = 0; i < OPT; ++i) {
        const uint64_t eb = ebs[i];
        if (eb >= a.d) continue;
        const float step = __fdiv_rn(sc[i], (float)a.s);
        float v[8];
        constexpr int PER_WORD = 32 / BITS;
        if (BITS == 2) {
            // A two-bit code moved to bits 31 and 30 IS the float +-2.0 (level 1) or +-0.0 (level 0);
            // times step/2 (exact: s = 1, so step is the scale, far above the subnormal range or 0)
            // that is +-step or +-0 bit for bit, the value fl32(level * step) with the code's sign.
            const float hs = __fmul_rn(step, 0.5f);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                v[j] = __fmul_rn(__uint_as_float((w[i][0] << (30 - 2 * j)) & 0xC0000000u), hs);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = code_value<BITS>(w[i][j / PER_WORD], j % PER_WORD, step);
        }
        if (VEC && eb + 8 <= a.d) {
            st256(a.param + eb, v);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (eb + j < a.d) a.param[eb + j] = v[j];
        }
    }
}

// -------------------------------------------- decode + average + apply ------

// acc += +-level * step for the 8 codes of one octet, two elements per arithmetic
// instruction (acc[p] holds elements 2p, 2p+1).  One rounding per product-sum: the sign
// is folded into the multiplier.  `cw` is the 64-bit code word of the lane and `o` the
// octet inside it (8/BITS octets per word).
template <int BITS>
__device__ __forceinline__ void accumulate_octet(const uint32_t (&cw)[2], int o, float step,
                                                 uint64_t (&acc)[4])
{
    if (BITS == 2) {
        // Two-bit codes are (sign, level) with level in {0, 1}.  Moved to bits 31 and 30
        // they ARE the floats +-2.0 (level 1) and +-0.0 (level 0): bit 31 is the sign and
        // bit 30 the top exponent bit.  So a shift and a mask decode a code, and multiplying
        // by step/2 (exact: steps are far above the subnormal range) gives +-step or 0.
        const uint32_t hs = __float_as_uint(__fmul_rn(step, 0.5f));
        const uint64_t hs2 = pack2(hs, hs);
        const uint32_t word = cw[o >> 1];
        const int base = 16 * (o & 1);           // bit offset of the octet inside the word
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const int s0 = 30 - base - 4 * p, s1 = 28 - base - 4 * p;   // left shifts; < 0 = right
            const uint32_t f0 = (s0 >= 0 ? word << (s0 >= 0 ? s0 : 0) : word >> (s0 < 0 ? -s0 : 0));
            const uint32_t f1 = (s1 >= 0 ? word << (s1 >= 0 ? s1 : 0) : word >> (s1 < 0 ? -s1 : 0));
            acc[p] = fma2(pack2(f0 & 0xC0000000u, f1 & 0xC0000000u), hs2, acc[p]);
        }
        return;
    }
    // Levels are spliced into the mantissa of 2^23 and the 2^23 is subtracted again, which
    // converts them to float exactly.
    const uint32_t sb = __float_as_uint(step);
    const uint64_t neg_magic = pack2(0xCB000000u, 0xCB000000u);   // (-2^23, -2^23)
    uint32_t m[8], sg[8];
    if (BITS == 8) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t lv = cw[h] & 0x7F7F7F7Fu;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // byte j of lv under the upper three bytes of 2^23
                m[4 * h + j] = __byte_perm(lv, 0x4B000000u, 0x7650 + j);
                sg[4 * h + j] = and_xor(j == 3 ? cw[h] : (cw[h] << (24 - 8 * j)), 0x80000000u, sb);
            }
        }
    } else {
        const uint32_t word = cw[o];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            m[j] = and_or(word >> (j * 4), 7u, 0x4B000000u);
            sg[j] = and_xor(word << (28 - j * 4), 0x80000000u, sb);
        }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p)
        acc[p] = fma2(add2(pack2(m[2 * p], m[2 * p + 1]), neg_magic),
                      pack2(sg[2 * p], sg[2 * p + 1]), acc[p]);
}

// A warp works on a tile of W chunks of 256 * 8/BITS consecutive elements.  In every
// chunk a lane owns 8/BITS consecutive octets -- exactly one 64-bit code word per worker --
// so a warp's loads of code words are contiguous.  The grid spacings fl32(scale/s) a warp
// needs are computed once per warp (one division per lane) and handed out by shuffle;
// code words are fetched several workers at a time so that independent loads are in
// flight before the first is used.
// KS > 0: the number of workers is that compile-time constant and the worker loop is unrolled
// completely (no loop counter, no predicates on the worker index).  Measured: 14 % faster for
// 8-bit, 4 % for 4-bit and 4 % for 2-bit codes at K = 8, but slower for 2-bit codes at K = 4
// (1 %) and at K = 16 (3-9 %: 16 workers x 32 codes per lane no longer fit the instruction
// cache), where unrolling half the loop gives 2-3 %; the launcher picks accordingly.
// Register budget: 24 resident CTAs per SM, 28 for 4-bit codes (measured 4-5 % faster there,
// slower for the other widths).
template <int BITS, bool VEC, int W, int KS = 0>
__global__ void __launch_bounds__(QESGD_DAA_THREADS, BITS == 4 ? QESGD_DAA_MIN_CTAS + 4 : QESGD_DAA_MIN_CTAS)
    qesgd_decode_average_apply_kernel(const DecodeArgs a)
{
    const uint32_t K = KS ? (uint32_t)KS : a.K;
    constexpr int OPL = 8 / BITS;                 // octets per lane and chunk: 4, 2, 1
    constexpr int LANE_ELEMS = 8 * OPL;
    constexpr uint32_t WCHUNK = 32 * LANE_ELEMS;  // elements per chunk: 1024, 512, 256
    constexpr uint32_t TILE = W * WCHUNK;         // elements per warp
    constexpr uint32_t LOG2_TILE = (BITS == 2 ? 10 : (BITS == 4 ? 9 : 8)) + (W == 4 ? 2 : (W == 2 ? 1 : 0));
    constexpr int BATCH = QESGD_DAA_BATCH / W > 0 ? QESGD_DAA_BATCH / W : 1;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp_eb =
        (((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * (uint64_t)TILE;
    if (warp_eb >= a.d) return;  // whole warp out of range
    const uint32_t lb = a.log2_bucket;
    const uint32_t nbw = lb >= LOG2_TILE ? 1u : TILE >> lb;              // buckets per warp: 1..16
    const uint64_t bucket0 = warp_eb >> lb;
    const uint32_t per_pass = 32u / nbw;                                 // workers per pass
    const float sf = (float)a.s;

    uint64_t eb[W];      // first element of the lane in chunk c
    uint32_t sub[W];     // its bucket, counted from the warp's first bucket
    const uint8_t *__restrict__ cp[W];
    uint64_t acc[W][OPL][4];
#pragma unroll
    for (int c = 0; c < W; ++c) {
        const uint32_t off = (uint32_t)c * WCHUNK + lane * (uint32_t)LANE_ELEMS;
        eb[c] = warp_eb + off;
        sub[c] = lb >= LOG2_TILE ? 0u : off >> lb;
        // Lanes past the padded length of the streams read the warp's first word instead
        // (their result is never stored), so no load needs a predicate.  The padded length
        // is a multiple of 64, so a lane's 8, 16 or 32 elements are inside it or outside it.
        const uint64_t safe_eb = eb[c] < (a.nb << lb) ? eb[c] : warp_eb;
        cp[c] = reinterpret_cast<const uint8_t *>(a.codes) + (safe_eb >> 3) * (uint64_t)BITS;
#ifdef QESGD_DEBUG
        if (!QESGD_IN_RANGE(a.status, safe_eb + LANE_ELEMS <= (a.nb << lb))) cp[c] = reinterpret_cast<const uint8_t *>(a.codes);
#endif
#pragma unroll
        for (int o = 0; o < OPL; ++o)
#pragma unroll
            for (int p = 0; p < 4; ++p) acc[c][o][p] = 0ull;   // pairs of +0.0f
    }

    // Four-bit codes with buckets of at least 256 elements: a half-warp (16 lanes x 16
    // elements) lies inside one bucket, so the 16 possible code values +-level * step of a
    // worker fit one per lane and decoding becomes a 16-wide shuffle.  signed_level is the
    // level of code (lane & 15) with its sign: 0..7, -0..-7.
    const bool lut = BITS == 4 && lb >= 8;
    const float signed_level = (lane & 8u) ? -(float)(lane & 7u) : (float)(lane & 7u);

    // Code words of BATCH workers are requested one batch ahead of the batch being decoded.
    auto fetch = [&](uint32_t kfirst, uint32_t (&dst)[BATCH][W][2]) {
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
#pragma unroll
            for (int c = 0; c < W; ++c) {
                dst[i][c][0] = dst[i][c][1] = 0u;
                if (kfirst + i < K) {
                    const uint2 v = __ldg(reinterpret_cast<const uint2 *>(
                        cp[c] + (uint64_t)(kfirst + i) * a.code_stride));
                    dst[i][c][0] = v.x;
                    dst[i][c][1] = v.y;
                }
            }
        }
    };
    // One scale per lane and pass: lane L serves worker (first of the pass) + L / nbw, bucket
    // bucket0 + L % nbw.  The scales of a pass are requested one pass ahead.
    auto fetch_scale = [&](uint32_t kfirst) {
        const uint32_t kk = kfirst + lane / nbw;
        const uint64_t bb = bucket0 + (lane % nbw);
        return (kk < K && bb < a.nb && QESGD_IN_RANGE(a.status, bb < a.nb))
                   ? __ldg(a.scales + (uint64_t)kk * a.scale_stride + bb)
                   : 0.0f;
    };
    uint32_t cw[BATCH][W][2], nx[BATCH][W][2];
    fetch(0u, cw);
    float sc_next = fetch_scale(0u);
    float st = 0.0f;
    // 2-bit codes of 16 workers: two batches per loop iteration (the whole loop would not fit
    // the instruction cache); every other compile-time worker count: the whole loop
    constexpr int OUTER_UNROLL = KS == 0 ? 1 : ((BITS == 2 && KS > 8) ? 2 : 64);
#pragma unroll OUTER_UNROLL
    for (uint32_t kb = 0; kb < (KS ? (uint32_t)KS : a.K); kb += BATCH) {
        fetch(kb + BATCH, nx);
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            const uint32_t k = kb + i;
            if (k < K) {   // uniform across the warp
                // position of worker k inside its pass (per_pass is a power of two)
                const uint32_t kp = KS ? (k & (per_pass - 1u)) : k % per_pass;
                if (kp == 0u) {   // a new pass: every lane computes one spacing
                    st = __fdiv_rn(sc_next, sf);
                    sc_next = fetch_scale(k + per_pass);
                }
#pragma unroll
                for (int c = 0; c < W; ++c) {
                    const float step = __shfl_sync(FULL, st, kp * nbw + sub[c]);
                    if (BITS == 4 && lut) {
                        // every lane holds the value of code (lane & 15) for this worker; a
                        // code is decoded by fetching its value from that lane of the same
                        // half-warp
                        const float tab = __fmul_rn(signed_level, step);
#pragma unroll
                        for (int o = 0; o < OPL; ++o) {
                            const uint32_t word = cw[i][c][o];
#pragma unroll
                            for (int p = 0; p < 4; ++p) {
                                const float v0 = __shfl_sync(FULL, tab, (int)(word >> (8 * p)), 16);
                                const float v1 = __shfl_sync(FULL, tab, (int)(word >> (8 * p + 4)), 16);
                                acc[c][o][p] = add2(acc[c][o][p], pack2f(v0, v1));
                            }
                        }
                    } else {
#pragma unroll
                        for (int o = 0; o < OPL; ++o)
                            accumulate_octet<BITS>(cw[i][c], o, step, acc[c][o]);
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < BATCH; ++i)
#pragma unroll
            for (int c = 0; c < W; ++c) {
                cw[i][c][0] = nx[i][c][0];
                cw[i][c][1] = nx[i][c][1];
            }
    }
    // Apply: param += (alpha / K) * sum.  The warp never loads the parameter: every element
    // gets exactly one add, done by the memory system (a vector reduction of four floats), so a
    // warp's life ends with its last code word instead of a further round trip to memory, and the
    // result, fl32(param + fl32(sum * alpha / K)), does not depend on any order.  A lane's
    // elements are LANE_ELEMS consecutive floats, 32 to 128 bytes apart from the next lane's;
    // the increments go through shared memory once so that every reduction instruction covers
    // 512 consecutive bytes (32 lanes x 16 bytes).  Pieces of 16 bytes are stored at index
    // P ^ ((P >> 3) & 7), which keeps both the lane-major writes and the piece-major reads free
    // of bank conflicts for 2, 4 or 8 pieces per lane.
    const float inv_k = a.avg_scale;   // alpha / K
    constexpr int NCH = LANE_ELEMS / 4;           // 16-byte pieces per lane and chunk: 8, 4, 2
    __shared__ float4 s_inc[(QESGD_DAA_THREADS / 32) * W * 32 * NCH];
    float4 *wt = s_inc + (threadIdx.x >> 5) * (W * 32 * NCH);
#pragma unroll
    for (int c = 0; c < W; ++c) {
#pragma unroll
        for (int o = 0; o < OPL; ++o) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float f0, f1, f2, f3;
                unpack2(acc[c][o][2 * h], f0, f1);
                unpack2(acc[c][o][2 * h + 1], f2, f3);
                const uint32_t P = lane * NCH + 2 * o + h;
                wt[c * 32 * NCH + (P ^ ((P >> 3) & 7u))] =
                    make_float4(__fmul_rn(f0, inv_k), __fmul_rn(f1, inv_k), __fmul_rn(f2, inv_k),
                                __fmul_rn(f3, inv_k));
            }
        }
    }
    __syncwarp();
#pragma unroll
    for (int c = 0; c < W; ++c) {
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const uint32_t g = i * 32 + lane;     // piece g of the chunk: elements 4g .. 4g+3
            const float4 v = wt[c * 32 * NCH + (g ^ ((g >> 3) & 7u))];
            const uint64_t e = warp_eb + (uint64_t)c * WCHUNK + 4u * g;
            float *q = a.param + e;
            if (VEC && e + 4 <= a.d) {
                if (QESGD_IN_RANGE(a.status, e + 4 <= a.d))
                    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                                 :: "l"(q), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
            } else {
                if (e < a.d) atomicAdd(q, v.x);
                if (e + 1 < a.d) atomicAdd(q + 1, v.y);
                if (e + 2 < a.d) atomicAdd(q + 2, v.z);
                if (e + 3 < a.d) atomicAdd(q + 3, v.w);
            }
        }
    }
}

// ------------------------------------------------------------ dispatch ------
template <int BITS, int MODE, bool ANCHOR, bool VEC, int WARPS>
cudaError_t launch_encode_w(const EncodeArgs &a, uint32_t K, cudaStream_t stream)
{
    constexpr int V = QESGD_ENCODE_CHUNKS;
    const uint64_t tile = (uint64_t)WARPS * V * CHUNK;
    const uint64_t tiles = (a.padded + tile - 1) / tile;
    if (tiles == 0 || tiles * K > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    dim3 grid((unsigned)(tiles * K), 1, 1), block(WARPS * 32u, 1, 1);
    if (ANCHOR && a.u_out)   // per-step QESGD: write back u = anchor + Q(z)
        qesgd_encode_kernel<BITS, MODE, ANCHOR, VEC, V, WARPS, ANCHOR><<<grid, block, 0, stream>>>(a);
    else
        qesgd_encode_kernel<BITS, MODE, ANCHOR, VEC, V, WARPS, false><<<grid, block, 0, stream>>>(a);
    return cudaGetLastError();
}

template <int BITS, int MODE, bool ANCHOR, bool VEC>
cudaError_t launch_encode_v(const EncodeArgs &a, uint32_t K, int sm_count, cudaStream_t stream)
{
    (void)sm_count;
    constexpr int V = QESGD_ENCODE_CHUNKS;
    constexpr uint32_t SMALL = QESGD_ENCODE_WARPS;        // warps of the usual CTA
    // a bucket never leaves its CTA: as many warps as the bucket spans, no more
    const uint32_t need = (1u << a.log2_bucket) / (uint32_t)(V * CHUNK);
    if (need <= SMALL) return launch_encode_w<BITS, MODE, ANCHOR, VEC, SMALL>(a, K, stream);
    if (need <= 2u) return launch_encode_w<BITS, MODE, ANCHOR, VEC, (SMALL > 2 ? SMALL : 2)>(a, K, stream);
    if (need <= 4u) return launch_encode_w<BITS, MODE, ANCHOR, VEC, (SMALL > 4 ? SMALL : 4)>(a, K, stream);
    constexpr uint32_t LARGE = QESGD_MAX_BUCKET / (V * CHUNK);   // enough for the widest bucket
    return launch_encode_w<BITS, MODE, ANCHOR, VEC, (LARGE > SMALL ? LARGE : SMALL)>(a, K, stream);
}

template <int BITS, int MODE>
cudaError_t launch_encode_m(const EncodeArgs &a, uint32_t K, bool vec, int sm_count,
                            cudaStream_t stream)
{
    if (a.anchor)
        return vec ? launch_encode_v<BITS, MODE, true, true>(a, K, sm_count, stream)
                   : launch_encode_v<BITS, MODE, true, false>(a, K, sm_count, stream);
    return vec ? launch_encode_v<BITS, MODE, false, true>(a, K, sm_count, stream)
               : launch_encode_v<BITS, MODE, false, false>(a, K, sm_count, stream);
}

template <int BITS>
cudaError_t launch_encode_b(const EncodeArgs &a, uint32_t K, uint32_t mode, bool vec,
                            int sm_count, cudaStream_t stream)
{
    switch (mode) {
        case QESGD_SCALE_NORM: return launch_encode_m<BITS, 0>(a, K, vec, sm_count, stream);
        case QESGD_SCALE_MAX: return launch_encode_m<BITS, 1>(a, K, vec, sm_count, stream);
        default: return launch_encode_m<BITS, 2>(a, K, vec, sm_count, stream);
    }
}

#if defined(QESGD_DEBUG) && QESGD_BITS == 2
__global__ void qesgd_range_selftest_kernel(uint32_t *status, uint64_t index, uint64_t limit)
{
    if (QESGD_IN_RANGE(status, index < limit)) status[1] = 1u;   // never: the index is outside
}
#endif

}  // namespace

#if defined(QESGD_DEBUG) && QESGD_BITS == 2
int qesgd_launch_range_selftest(uint32_t *status, cudaStream_t stream)
{
    qesgd_range_selftest_kernel<<<1, 1, 0, stream>>>(status, 7u, 7u);
    return (int)cudaGetLastError();
}
#endif

// This file is compiled once per code width (-DQESGD_BITS=2, 4, 8) so that the three sets
// of kernel instantiations build in parallel; qesgd_api.cu picks the set at run time.
#ifndef QESGD_BITS
#error "compile with -DQESGD_BITS=2, 4 or 8"
#endif
#define QESGD_CAT2(a, b) a##b
#define QESGD_CAT(a, b) QESGD_CAT2(a, b)

int QESGD_CAT(qesgd_launch_encode_, QESGD_BITS)(const EncodeArgs &a, uint32_t K, uint32_t scale_mode,
                                                bool vec, int sm_count, cudaStream_t stream)
{
    return (int)launch_encode_b<QESGD_BITS>(a, K, scale_mode, vec, sm_count, stream);
}

int QESGD_CAT(qesgd_launch_lr_qstep_, QESGD_BITS)(const QstepArgs &a, uint32_t scale_mode, cudaStream_t stream)
{
    const uint64_t tiles = (a.e.padded + QS_TILE - 1) / QS_TILE;
    if (tiles == 0 || tiles > 0x7FFFFFFFull) return (int)cudaErrorInvalidValue;
    dim3 grid((unsigned)tiles), block(QS_THREADS);
    switch (scale_mode) {
        case QESGD_SCALE_NORM: qesgd_lr_qstep_kernel<QESGD_BITS, 0><<<grid, block, 0, stream>>>(a); break;
        case QESGD_SCALE_MAX: qesgd_lr_qstep_kernel<QESGD_BITS, 1><<<grid, block, 0, stream>>>(a); break;
        default: qesgd_lr_qstep_kernel<QESGD_BITS, 2><<<grid, block, 0, stream>>>(a); break;
    }
    return (int)cudaGetLastError();
}

int QESGD_CAT(qesgd_launch_decode_, QESGD_BITS)(const DecodeArgs &a, bool vec, cudaStream_t stream)
{
    const uint64_t octets = (a.d + 7) / 8;
    const uint64_t blocks = (octets + 256 * QESGD_DECODE_OCTETS - 1) / (256 * QESGD_DECODE_OCTETS);
    if (blocks == 0 || blocks > 0x7FFFFFFFull) return (int)cudaErrorInvalidValue;
    dim3 grid((unsigned)blocks), block(256);
    if (vec) qesgd_decode_kernel<QESGD_BITS, true><<<grid, block, 0, stream>>>(a);
    else qesgd_decode_kernel<QESGD_BITS, false><<<grid, block, 0, stream>>>(a);
    return (int)cudaGetLastError();
}

int QESGD_CAT(qesgd_launch_decode_average_apply_, QESGD_BITS)(const DecodeArgs &a, bool vec,
                                                              cudaStream_t stream)
{
    constexpr int W = QESGD_BITS == 2 ? QESGD_DAA_WORDS_2BIT : QESGD_DAA_WORDS_WIDE;
    const uint64_t warp_elems = 256ull * (8u / QESGD_BITS) * W;   // one tile per warp (see the kernel)
    const uint64_t warps = (a.d + warp_elems - 1) / warp_elems;
    const uint64_t wpc = QESGD_DAA_THREADS / 32;
    const uint64_t blocks = (warps + wpc - 1) / wpc;
    if (blocks == 0 || blocks > 0x7FFFFFFFull) return (int)cudaErrorInvalidValue;
    dim3 grid((unsigned)blocks), block(QESGD_DAA_THREADS);
    if (vec && a.K == 8)
        qesgd_decode_average_apply_kernel<QESGD_BITS, true, W, 8><<<grid, block, 0, stream>>>(a);
    else if (vec && QESGD_BITS != 2 && a.K == 4)
        qesgd_decode_average_apply_kernel<QESGD_BITS, true, W, (QESGD_BITS != 2 ? 4 : 0)><<<grid, block, 0, stream>>>(a);
    else if (vec && QESGD_BITS != 4 && a.K == 16)
        qesgd_decode_average_apply_kernel<QESGD_BITS, true, W, (QESGD_BITS != 4 ? 16 : 0)><<<grid, block, 0, stream>>>(a);
    else if (vec) qesgd_decode_average_apply_kernel<QESGD_BITS, true, W><<<grid, block, 0, stream>>>(a);
    else qesgd_decode_average_apply_kernel<QESGD_BITS, false, W><<<grid, block, 0, stream>>>(a);
    return (int)cudaGetLastError();
}
