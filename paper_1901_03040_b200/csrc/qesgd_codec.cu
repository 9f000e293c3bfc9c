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
template <bool VEC>
__device__ __forceinline__ void load_octet(const float *__restrict__ p, uint64_t eb, uint64_t d,
                                           float (&v)[8])
{
    if (VEC && eb + 8 <= d) {
        ld256(p + eb, v);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (eb + j < d) ? __ldg(p + eb + j) : 0.0f;
    }
}

// ---------------------------------------------------------------- Philox ----
// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11), written from the
// published round function: two 32x32->64 multiplies, the high halves xor'ed with
// the other counter words and the round key; the key grows by the Weyl constants.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&x)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    x[0] = c0; x[1] = c1; x[2] = c2; x[3] = c3;
}

// ------------------------------------------------------- rounding (Eq. 4) ----
// level = floor(r) + [h + 1/2 < frac(r) * 2^16] for r = min(|z|*inv, s), 0 <= r <= 127.
// Adding 2^23 with round-toward-zero leaves 2^23 + floor(r) in the mantissa, which
// gives floor(r) both as a float (one exact subtract) and as the low byte of the bit
// pattern; (2^23 + h) - (2^23 - 1/2) is h + 1/2 exactly.  All full-rate fp32/int ops.
__device__ __forceinline__ uint32_t stochastic_level(float a, float inv, float sf, uint32_t h)
{
    const float r = fminf(__fmul_rn(a, inv), sf);
    const float t = __fadd_rz(r, 8388608.0f);
    const float f = __fsub_rn(t, 8388608.0f);
    const float p = __fsub_rn(r, f);
    const float hh = __fsub_rn(__uint_as_float(0x4B000000u | h), 8388607.5f);
    const uint32_t up = hh < __fmul_rn(p, 65536.0f) ? 1u : 0u;
    return (__float_as_uint(t) & 0xFFu) + up;
}

// code = sign << (BITS-1) | level with no "-0" code; returned already shifted to slot j.
template <int BITS>
__device__ __forceinline__ uint32_t place_code(uint32_t level, uint32_t zbits, int slot)
{
    // bit 31 of (level + 0x7FFFFFFF) is set iff level > 0
    const uint32_t sign31 = zbits & (level + 0x7FFFFFFFu) & 0x80000000u;
    const int top = slot * BITS + BITS - 1;
    return (level << (slot * BITS)) | (sign31 >> (31 - top));
}

// ------------------------------------------------------------- encode -------
// MODE: 0 = L2 norm, 1 = max magnitude, 2 = caller-given spacing.
// V = chunks per warp; a warp owns V*256 consecutive elements, a CTA of W warps
// owns W*V*256.  Buckets are powers of two in [64, 8192]:
//   bucket <= 256      : bucket/8 lanes of one chunk
//   bucket <= 256*V    : bucket/256 chunks of one warp
//   bucket  > 256*V    : bucket/(256*V) consecutive warps of the CTA (shared memory)
template <int BITS, int MODE, bool ANCHOR, bool VEC, int V>
__global__ void __launch_bounds__(256) qesgd_encode_kernel(const EncodeArgs a)
{
    __shared__ double s_part[8];
    __shared__ uint32_t s_max[8];

    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t warps = blockDim.x >> 5;
    // Workers vary fastest over the grid: the K CTAs that share a tile of the anchor run
    // close together in time, so the anchor comes from HBM once and from L2 K-1 times.
    const uint32_t k = blockIdx.x % a.K;
    const uint32_t tile = blockIdx.x / a.K;
    const uint32_t lb = a.log2_bucket;
    const float *__restrict__ local = a.local + (uint64_t)k * a.local_stride;
    const uint64_t warp_base = ((uint64_t)tile * warps + warp) * (uint64_t)(V * CHUNK);

    // ---- loads: everything this lane needs is requested before any use -------
    float z[V][8];
#pragma unroll
    for (int c = 0; c < V; ++c)
        load_octet<VEC>(local, warp_base + (uint64_t)c * CHUNK + lane * 8u, a.d, z[c]);
    if (ANCHOR) {
        float w[V][8];
#pragma unroll
        for (int c = 0; c < V; ++c)
            load_octet<VEC>(a.anchor, warp_base + (uint64_t)c * CHUNK + lane * 8u, a.d, w[c]);
#pragma unroll
        for (int c = 0; c < V; ++c)
#pragma unroll
            for (int j = 0; j < 8; ++j) z[c][j] = __fsub_rn(z[c][j], w[c][j]);
    }

    // ---- per-bucket scale ------------------------------------------------------
    float scale[V];
    bool nonfinite[V];
    if (MODE == 0) {
        // fp64 sum of squares over the balanced binary tree on index order: 8 in the
        // lane, then lanes (xor 1,2,4,8,16), then chunks, then warps.  The product of
        // two fp32 values is exact in fp64, so fma(z1,z1,z0*z0) is fl64(q0+q1).
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
#pragma unroll
        for (int off = 1; off <= 16; off <<= 1) {
            if ((uint32_t)(off * 8) < (1u << lb)) {  // partner lane is in the same bucket
#pragma unroll
                for (int c = 0; c < V; ++c)
                    t[c] = __dadd_rn(t[c], __shfl_xor_sync(FULL, t[c], off));
            }
        }
        if (lb >= 9) {
#pragma unroll
            for (int c = 0; c < V; c += 2) t[c] = t[c + 1] = __dadd_rn(t[c], t[c + 1]);
        }
        if (V == 4 && lb >= 10) t[0] = t[1] = t[2] = t[3] = __dadd_rn(t[0], t[2]);
        if ((1u << lb) > (uint32_t)(V * CHUNK)) {
            const uint32_t wpb = (1u << lb) / (uint32_t)(V * CHUNK);  // warps per bucket
            if (lane == 0) s_part[warp] = t[0];
            __syncthreads();
            const uint32_t g0 = warp & ~(wpb - 1u);
            double acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = (i < (int)wpb) ? s_part[g0 + i] : 0.0;
#pragma unroll
            for (int w2 = 1; w2 < 8; w2 <<= 1) {
                if ((uint32_t)w2 < wpb) {
#pragma unroll
                    for (int i = 0; i < 8; i += 2 * w2) acc[i] = __dadd_rn(acc[i], acc[i + w2]);
                }
            }
#pragma unroll
            for (int c = 0; c < V; ++c) t[c] = acc[0];
        }
#pragma unroll
        for (int c = 0; c < V; ++c) {
            scale[c] = __double2float_rn(__dsqrt_rn(t[c]));
            nonfinite[c] = !(fabsf(scale[c]) <= 3.402823466e38f);  // Inf or NaN
        }
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
#pragma unroll
        for (int off = 1; off <= 16; off <<= 1) {
            if ((uint32_t)(off * 8) < (1u << lb)) {
#pragma unroll
                for (int c = 0; c < V; ++c) m[c] = max(m[c], __shfl_xor_sync(FULL, m[c], off));
            }
        }
        if (lb >= 9) {
#pragma unroll
            for (int c = 0; c < V; c += 2) m[c] = m[c + 1] = max(m[c], m[c + 1]);
        }
        if (V == 4 && lb >= 10) m[0] = m[1] = m[2] = m[3] = max(m[0], m[2]);
        if ((1u << lb) > (uint32_t)(V * CHUNK)) {
            const uint32_t wpb = (1u << lb) / (uint32_t)(V * CHUNK);
            if (lane == 0) s_max[warp] = m[0];
            __syncthreads();
            const uint32_t g0 = warp & ~(wpb - 1u);
            uint32_t mm = 0u;
            for (uint32_t i = 0; i < wpb; ++i) mm = max(mm, s_max[g0 + i]);
#pragma unroll
            for (int c = 0; c < V; ++c) m[c] = mm;
        }
#pragma unroll
        for (int c = 0; c < V; ++c) {
            nonfinite[c] = m[c] >= 0x7F800000u;
            scale[c] = __uint_as_float(m[c]);
        }
    } else {
#pragma unroll
        for (int c = 0; c < V; ++c) {
            scale[c] = a.fixed_scale;
            nonfinite[c] = !(fabsf(scale[c]) <= 3.402823466e38f);
        }
    }

    // ---- rounding, packing, stores ---------------------------------------------
    const float sf = (float)a.s;
    uint8_t *__restrict__ codes = reinterpret_cast<uint8_t *>(a.codes) + (uint64_t)k * a.code_stride;
    float *__restrict__ scales = a.scales + (uint64_t)k * a.scale_stride;
    const uint32_t bucket_mask = (1u << lb) - 1u;
    bool flag = false;

#pragma unroll
    for (int c = 0; c < V; ++c) {
        const uint64_t eb = warp_base + (uint64_t)c * CHUNK + lane * 8u;
        const bool ok = !nonfinite[c] && scale[c] >= 0x1p-100f;
        const float inv = ok ? __fdiv_rn(sf, scale[c]) : 0.0f;
        if (eb < a.padded && ((uint32_t)eb & bucket_mask) == 0u) {
            scales[eb >> lb] = ok ? scale[c] : 0.0f;
            flag |= nonfinite[c];
        }
        uint32_t x[4];
        const uint64_t blk = eb >> 3;
        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.worker0 + k, a.epoch, a.key0, a.key1, x);

        uint32_t word[(8 * BITS) / 32 > 0 ? (8 * BITS) / 32 : 1];
#pragma unroll
        for (int i = 0; i < (int)(sizeof(word) / 4); ++i) word[i] = 0u;
        bool nan_seen = false;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t h = (j & 1) ? (x[j >> 1] >> 16) : (x[j >> 1] & 0xFFFFu);
            const uint32_t zb = __float_as_uint(z[c][j]);
            float av = fabsf(z[c][j]);
            if (MODE == 2) {  // per element: NaN is flagged and encoded as 0, Inf clips
                const bool isn = (zb & 0x7FFFFFFFu) > 0x7F800000u;
                nan_seen |= isn;
                av = isn ? 0.0f : av;
            }
            const uint32_t level = stochastic_level(av, inv, sf, h);
            constexpr int PER_WORD = 32 / BITS;
            word[j / PER_WORD] |= place_code<BITS>(level, zb, j % PER_WORD);
        }
        if (MODE == 2) flag |= nan_seen;
        if (eb < a.padded) {
            const uint32_t keep = ok ? FULL : 0u;
            if (BITS == 8) {
                uint2 o = make_uint2(word[0] & keep, word[(8 * BITS) / 32 > 1 ? 1 : 0] & keep);
                *reinterpret_cast<uint2 *>(codes + eb) = o;
            } else if (BITS == 4) {
                *reinterpret_cast<uint32_t *>(codes + (eb >> 1)) = word[0] & keep;
            } else {
                *reinterpret_cast<uint16_t *>(codes + (eb >> 2)) = (uint16_t)(word[0] & keep);
            }
        }
    }
    if (flag) atomicOr(a.status, QESGD_STATUS_NONFINITE);
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

// acc += +-level * step with one rounding (the sign is folded into the multiplier).
template <int BITS>
__device__ __forceinline__ void accumulate_code(uint32_t word, int slot, float step, float &acc)
{
    constexpr uint32_t LEVEL_MASK = (1u << (BITS - 1)) - 1u;
    const uint32_t lv = (word >> (slot * BITS)) & LEVEL_MASK;
    const float lf = __fsub_rn(__uint_as_float(0x4B000000u | lv), 8388608.0f);
    const uint32_t sign31 = (word << (31 - (slot * BITS + BITS - 1))) & 0x80000000u;
    acc = __fmaf_rn(lf, __uint_as_float(__float_as_uint(step) ^ sign31), acc);
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

template <int BITS, bool VEC>
__global__ void __launch_bounds__(256) qesgd_decode_kernel(const DecodeArgs a)
{
    const uint64_t eb = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8u;
    if (eb >= a.d) return;
    const uint8_t *__restrict__ codes = reinterpret_cast<const uint8_t *>(a.codes);
    uint32_t w[2];
    load_codes<BITS>(codes, eb, w);
    const float step = __fdiv_rn(__ldg(a.scales + (eb >> a.log2_bucket)), (float)a.s);
    float v[8];
    constexpr int PER_WORD = 32 / BITS;
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = code_value<BITS>(w[j / PER_WORD], j % PER_WORD, step);
    if (VEC && eb + 8 <= a.d) {
        st256(a.param + eb, v);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (eb + j < a.d) a.param[eb + j] = v[j];
    }
}

// -------------------------------------------- decode + average + apply ------
// One octet per lane, one chunk of 256 elements per warp.  The K grid spacings
// fl32(scale/s) a chunk needs are computed once per warp (one division per lane)
// and handed out by shuffle, so the inner loop per code is shift/mask/fma work.
template <int BITS, bool VEC>
__global__ void __launch_bounds__(256) qesgd_decode_average_apply_kernel(const DecodeArgs a)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp_eb =
        (((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * (uint64_t)CHUNK;
    if (warp_eb >= a.d) return;  // whole warp out of range
    const uint64_t eb = warp_eb + lane * 8u;
    const uint32_t lb = a.log2_bucket;
    const uint32_t nbw = lb >= 8 ? 1u : (uint32_t)CHUNK >> lb;  // buckets per chunk: 1, 2, 4
    const uint32_t sub = lb >= 8 ? 0u : (lane * 8u) >> lb;      // this lane's bucket in the chunk
    const uint64_t bucket0 = warp_eb >> lb;
    const uint32_t per_pass = 32u / nbw;                        // workers per pass
    const float sf = (float)a.s;
    const bool live = eb < a.d;

    float w[8];
    if (VEC && eb + 8 <= a.d) {
        ld256_rw(a.param + eb, w);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) w[j] = (eb + j < a.d) ? a.param[eb + j] : 0.0f;
    }
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.0f;

    const uint8_t *__restrict__ codes = reinterpret_cast<const uint8_t *>(a.codes);
    constexpr int PER_WORD = 32 / BITS;
    for (uint32_t k0 = 0; k0 < a.K; k0 += per_pass) {
        const uint32_t kk = k0 + lane / nbw;
        const uint64_t bb = bucket0 + (lane % nbw);
        float st = 0.0f;
        if (kk < a.K && bb < a.nb)
            st = __fdiv_rn(__ldg(a.scales + (uint64_t)kk * a.scale_stride + bb), sf);
        const uint32_t count = min(per_pass, a.K - k0);
#pragma unroll 4
        for (uint32_t i = 0; i < count; ++i) {
            const float step = __shfl_sync(FULL, st, i * nbw + sub);
            uint32_t cw[2] = {0u, 0u};
            if (live) load_codes<BITS>(codes + (uint64_t)(k0 + i) * a.code_stride, eb, cw);
#pragma unroll
            for (int j = 0; j < 8; ++j) accumulate_code<BITS>(cw[j / PER_WORD], j % PER_WORD, step, acc[j]);
        }
    }
    const float inv_k = __fdiv_rn(1.0f, (float)a.K);
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = __fmaf_rn(acc[j], inv_k, w[j]);
    if (VEC && eb + 8 <= a.d) {
        st256(a.param + eb, w);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (eb + j < a.d) a.param[eb + j] = w[j];
    }
}

// ------------------------------------------------------------ dispatch ------
template <int BITS, int MODE, bool ANCHOR, bool VEC>
cudaError_t launch_encode_v(const EncodeArgs &a, uint32_t K, cudaStream_t stream)
{
    constexpr int V = 4;
    constexpr uint32_t warps = 8;  // 8 warps * V * 256 = 8192 elements: the largest bucket fits
    static_assert(warps * V * CHUNK >= QESGD_MAX_BUCKET, "a bucket never leaves its CTA");
    const uint64_t tile = (uint64_t)warps * V * CHUNK;
    const uint64_t tiles = (a.padded + tile - 1) / tile;
    if (tiles == 0 || tiles * K > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    dim3 grid((unsigned)(tiles * K), 1, 1), block(warps * 32u, 1, 1);
    qesgd_encode_kernel<BITS, MODE, ANCHOR, VEC, V><<<grid, block, 0, stream>>>(a);
    return cudaGetLastError();
}

template <int BITS, int MODE>
cudaError_t launch_encode_m(const EncodeArgs &a, uint32_t K, bool vec, cudaStream_t stream)
{
    if (a.anchor)
        return vec ? launch_encode_v<BITS, MODE, true, true>(a, K, stream)
                   : launch_encode_v<BITS, MODE, true, false>(a, K, stream);
    return vec ? launch_encode_v<BITS, MODE, false, true>(a, K, stream)
               : launch_encode_v<BITS, MODE, false, false>(a, K, stream);
}

template <int BITS>
cudaError_t launch_encode_b(const EncodeArgs &a, uint32_t K, uint32_t mode, bool vec,
                            cudaStream_t stream)
{
    switch (mode) {
        case QESGD_SCALE_NORM: return launch_encode_m<BITS, 0>(a, K, vec, stream);
        case QESGD_SCALE_MAX: return launch_encode_m<BITS, 1>(a, K, vec, stream);
        default: return launch_encode_m<BITS, 2>(a, K, vec, stream);
    }
}

}  // namespace

int qesgd_launch_encode(const EncodeArgs &a, uint32_t K, uint32_t bits, uint32_t scale_mode,
                        bool vec, cudaStream_t stream)
{
    switch (bits) {
        case 2: return (int)launch_encode_b<2>(a, K, scale_mode, vec, stream);
        case 4: return (int)launch_encode_b<4>(a, K, scale_mode, vec, stream);
        default: return (int)launch_encode_b<8>(a, K, scale_mode, vec, stream);
    }
}

int qesgd_launch_decode(const DecodeArgs &a, uint32_t bits, bool vec, cudaStream_t stream)
{
    const uint64_t octets = (a.d + 7) / 8;
    const uint64_t blocks = (octets + 255) / 256;
    if (blocks == 0 || blocks > 0x7FFFFFFFull) return (int)cudaErrorInvalidValue;
    dim3 grid((unsigned)blocks), block(256);
#define QESGD_DEC(B)                                                                 \
    if (vec) qesgd_decode_kernel<B, true><<<grid, block, 0, stream>>>(a);            \
    else qesgd_decode_kernel<B, false><<<grid, block, 0, stream>>>(a)
    if (bits == 2) { QESGD_DEC(2); }
    else if (bits == 4) { QESGD_DEC(4); }
    else { QESGD_DEC(8); }
#undef QESGD_DEC
    return (int)cudaGetLastError();
}

int qesgd_launch_decode_average_apply(const DecodeArgs &a, uint32_t bits, bool vec,
                                      cudaStream_t stream)
{
    const uint64_t chunks = (a.d + CHUNK - 1) / CHUNK;  // one warp each
    const uint64_t blocks = (chunks + 7) / 8;
    if (blocks == 0 || blocks > 0x7FFFFFFFull) return (int)cudaErrorInvalidValue;
    dim3 grid((unsigned)blocks), block(256);
#define QESGD_DAA(B)                                                                          \
    if (vec) qesgd_decode_average_apply_kernel<B, true><<<grid, block, 0, stream>>>(a);       \
    else qesgd_decode_average_apply_kernel<B, false><<<grid, block, 0, stream>>>(a)
    if (bits == 2) { QESGD_DAA(2); }
    else if (bits == 4) { QESGD_DAA(4); }
    else { QESGD_DAA(8); }
#undef QESGD_DAA
    return (int)cudaGetLastError();
}
