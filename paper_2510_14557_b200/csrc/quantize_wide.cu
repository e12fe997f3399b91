// MXFP6 / MXFP6+ (E2M3 elements) and MXFP8 / MXFP8+ (E4M3 elements): block quantization and
// decode (Table "Concrete MX-compliant formats"; Sec. 4.1: the BM keeps its sign bit and spends
// every other bit on mantissa, E0M5 = 4 + m/8 resp. E0M7 = 256 + 2 m, its exponent being emax
// by construction; Sec. 4.2: one index byte per block).  Same scheme as MXFP4+ with
// emax = 2 (E2M3) or 8 (E4M3): shared_exp = floor(log2 BM) - emax (Eq. 1), blocks with
// floor(log2 BM) <= -127 + emax are flushed (scale byte 0, all codes 0).
//
// Storage: 8-bit codes one per byte; 6-bit codes packed, code i of a row in bits 6i..6i+5 of the
// little-endian bit stream (24 bytes per block).  HBM-bound kernels, one thread per block of 32:
// a thread reads its 64 (bf16) or 128 (fp32) bytes with 128-bit loads (neighbouring lanes' loads
// fall into the same lines, which L1 serves) and writes 24 or 32 contiguous bytes.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace mxp {
namespace {

constexpr int kThreads = 256;

// Two scaled values -> two codes in the low bytes of the result (a in byte 0), round to nearest
// even, saturating at the largest finite magnitude, sign of zero kept.
template <int kFmt>
__device__ __forceinline__ uint32_t cvt_pair(float a, float b)
{
    uint16_t r;
    if (kFmt == 8)
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %2, %1;" : "=h"(r) : "f"(a), "f"(b));
    else
        asm("cvt.rn.satfinite.e2m3x2.f32 %0, %2, %1;" : "=h"(r) : "f"(a), "f"(b));
    return r;
}

// Two codes (low bytes of c) -> two floats, exact.
template <int kFmt>
__device__ __forceinline__ float2 decode_pair(uint32_t c)
{
    uint32_t h;
    const uint16_t c16 = (uint16_t)c;
    if (kFmt == 8)
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"(c16));
    else
        asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h) : "h"(c16));
    return __half22float2(*reinterpret_cast<const __half2*>(&h));
}

template <typename T>
__device__ __forceinline__ void load_block(const T* p, float (&v)[32])
{
    if (sizeof(T) == 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 w = __ldg(reinterpret_cast<const uint4*>(p) + i);
            const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[8 * i + 2 * j] = __uint_as_float(x[j] << 16);
                v[8 * i + 2 * j + 1] = __uint_as_float(x[j] & 0xFFFF0000u);
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 w = __ldg(reinterpret_cast<const float4*>(p) + i);
            v[4 * i] = w.x; v[4 * i + 1] = w.y; v[4 * i + 2] = w.z; v[4 * i + 3] = w.w;
        }
    }
}

// kFmt: 6 (E2M3) or 8 (E4M3).
template <typename T, int kFmt, bool kPlus>
__global__ void __launch_bounds__(kThreads)
quantize_wide_kernel(const T* __restrict__ src, int64_t ld_src, int nbk, int64_t total_blocks,
                     uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                     uint8_t* __restrict__ bm_index)
{
    constexpr uint32_t kEmax = kFmt == 8 ? 8u : 2u;
    constexpr int kMb = kFmt - 1;  // BM mantissa bits
    const int64_t blk = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (blk >= total_blocks) return;
    const int64_t row = blk / nbk;
    const int b = (int)(blk - row * nbk);
    float v[32];
    load_block(src + row * ld_src + (int64_t)b * 32, v);
    // BM: largest magnitude pattern, first one wins (Sec. 3.2).  bf16 patterns leave the low
    // 16 bits free for 31 - position, so one unsigned max finds both; fp32 takes two passes.
    uint32_t amax = 0;
    int bm = 0;
    if (sizeof(T) == 2) {
        uint32_t key = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            key = max(key, (__float_as_uint(v[i]) & 0x7FFF0000u) | (uint32_t)(31 - i));
        amax = key & 0x7FFF0000u;
        bm = 31 - (int)(key & 31u);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) amax = max(amax, __float_as_uint(v[i]) & 0x7FFFFFFFu);
        if (kPlus) {
            uint32_t mask = 0;
#pragma unroll
            for (int i = 0; i < 32; ++i)
                mask |= ((__float_as_uint(v[i]) & 0x7FFFFFFFu) == amax ? 1u : 0u) << i;
            bm = __ffs((int)mask) - 1;
        }
    }
    const uint32_t E = amax >> 23;
    const bool flush = E <= kEmax;  // floor(log2 BM) <= -127 + emax; zero and fp32 subnormals too
    const bool nonfinite = E == 255u;
    const bool dead = flush || nonfinite;
    const uint32_t sb = flush ? 0u : (nonfinite ? 255u : E - kEmax);
    const float inv = __uint_as_float((254u - sb) << 23);  // 2^-shared_exp, exact scaling
    uint32_t w[8];  // four codes each, one per byte
#pragma unroll
    for (int i = 0; i < 8; ++i)
        w[i] = dead ? 0u
                    : cvt_pair<kFmt>(v[4 * i] * inv, v[4 * i + 1] * inv) |
                          (cvt_pair<kFmt>(v[4 * i + 2] * inv, v[4 * i + 3] * inv) << 16);
    if (kPlus && !dead) {
        // Sec. 4.1: the BM's scaled value is 2^emax * 1.f; its stored mantissa is f rounded to
        // kMb bits (nearest, ties to even), clamped when it would carry into the next binade.
        // It replaces the exponent and mantissa bits of the BM's code; the sign bit the cast
        // wrote stays.
        const uint32_t frac = amax & 0x7FFFFFu;
        constexpr int sh = 23 - kMb;
        uint32_t m = frac >> sh;
        const uint32_t rem = frac & ((1u << sh) - 1u), half = 1u << (sh - 1);
        if (rem > half || (rem == half && (m & 1u))) ++m;
        m = min(m, (1u << kMb) - 1u);
        const uint32_t pos = 8u * ((uint32_t)bm & 3u);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if ((bm >> 2) == i)
                asm("bfi.b32 %0, %1, %0, %2, %3;" : "+r"(w[i]) : "r"(m), "r"(pos), "n"(kMb));
    }
    if (kFmt == 8) {
        uint4* out = reinterpret_cast<uint4*>(codes + blk * 32);
        out[0] = make_uint4(w[0], w[1], w[2], w[3]);
        out[1] = make_uint4(w[4], w[5], w[6], w[7]);
    } else {
        // four codes -> 24 bits; eight such groups -> three 64-bit words
        unsigned long long g[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            g[i] = (unsigned long long)((w[i] & 63u) | (((w[i] >> 8) & 63u) << 6) |
                                        (((w[i] >> 16) & 63u) << 12) | (((w[i] >> 24) & 63u) << 18));
        uint2* out = reinterpret_cast<uint2*>(codes + blk * 24);
        const unsigned long long w0 = g[0] | (g[1] << 24) | (g[2] << 48);
        const unsigned long long w1 = (g[2] >> 16) | (g[3] << 8) | (g[4] << 32) | (g[5] << 56);
        const unsigned long long w2 = (g[5] >> 8) | (g[6] << 16) | (g[7] << 40);
        out[0] = make_uint2((uint32_t)w0, (uint32_t)(w0 >> 32));
        out[1] = make_uint2((uint32_t)w1, (uint32_t)(w1 >> 32));
        out[2] = make_uint2((uint32_t)w2, (uint32_t)(w2 >> 32));
    }
    scales[blk] = (uint8_t)sb;
    if (bm_index != nullptr) bm_index[blk] = (uint8_t)((kPlus && !dead) ? bm : 0);
}

// bf16 sources with contiguous rows: the block stays packed two elements per register from the
// load to the cast.  Magnitudes, the maximum and the compare that finds its first position run
// on pairs (max.bf16x2, set.eq.bf16x2: 16 instead of 32 of each), the scaling is one packed
// multiply by 2^-shared_exp (exact: a result below the bf16 normal range is far below half the
// format's smallest subnormal and casts to a zero of its sign either way), and the 6-bit
// codes are packed with two selects per four codes and byte permutes.
__device__ __forceinline__ uint32_t bf16x2_mul(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_max_nan(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

template <int kFmt, bool kPlus>
__global__ void __launch_bounds__(kThreads)
quantize_wide_bf16_kernel(const uint4* __restrict__ src, int64_t total_blocks,
                          uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                          uint8_t* __restrict__ bm_index)
{
    constexpr uint32_t kEmax = kFmt == 8 ? 8u : 2u;
    constexpr int kMb = kFmt - 1;
    const int64_t blk = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (blk >= total_blocks) return;
    uint32_t x[16], t[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 v = __ldg(src + blk * 4 + i);
        x[4 * i] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) t[i] = x[i] & 0x7FFF7FFFu;
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        q[i] = bf16x2_max_nan(bf16x2_max_nan(t[4 * i], t[4 * i + 1]), bf16x2_max_nan(t[4 * i + 2], t[4 * i + 3]));
    uint32_t m2 = bf16x2_max_nan(bf16x2_max_nan(q[0], q[1]), bf16x2_max_nan(q[2], q[3]));
    m2 = bf16x2_max_nan(m2, __byte_perm(m2, m2, 0x1032));  // both halves = block maximum
    const uint32_t amax16 = m2 & 0xFFFFu;
    const uint32_t E = amax16 >> 7;
    const bool flush = E <= kEmax, nonfinite = E == 255u;
    const bool dead = flush || nonfinite;
    const uint32_t sb = flush ? 0u : (nonfinite ? 255u : E - kEmax);
    uint32_t bm = 0;
    if (kPlus) {
        // one bit per element where |x| equals the maximum; lowest set bit = first BM (Sec. 3.2)
        uint32_t r1 = 0, r2 = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t e1, e2;
            asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(e1) : "r"(t[i]), "r"(m2));
            asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(e2) : "r"(t[8 + i]), "r"(m2));
            const uint32_t sel = (1u << (2 * i)) | (1u << (16 + 2 * i));
            r1 |= e1 & sel;
            r2 |= e2 & sel;
        }
        // even elements sit in bits 0,2,..14, odd ones in bits 16,18,..30: interleave
        const uint32_t lo = (r1 & 0xFFFFu) | ((r1 >> 15) & 0xAAAAu);
        const uint32_t hi = (r2 & 0xFFFFu) | ((r2 >> 15) & 0xAAAAu);
        bm = (uint32_t)(__ffs((int)(lo | (hi << 16))) - 1) & 31u;
    }
    scales[blk] = (uint8_t)sb;
    if (bm_index != nullptr) bm_index[blk] = (uint8_t)((kPlus && !dead) ? bm : 0u);
    if (dead) {  // flushed or non-finite block: all codes zero (rare; the branch costs the others nothing)
        if (kFmt == 8) {
            uint4* out = reinterpret_cast<uint4*>(codes + blk * 32);
            out[0] = make_uint4(0, 0, 0, 0);
            out[1] = make_uint4(0, 0, 0, 0);
        } else {
            uint2* out = reinterpret_cast<uint2*>(codes + blk * 24);
            out[0] = out[1] = out[2] = make_uint2(0, 0);
        }
        return;
    }
    const uint32_t inv2 = ((254u - sb) << 7) * 0x00010001u;  // 2^-shared_exp, twice
    uint32_t w[8];  // four codes each, one per byte
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t y0 = bf16x2_mul(x[2 * i], inv2), y1 = bf16x2_mul(x[2 * i + 1], inv2);
        w[i] = cvt_pair<kFmt>(__uint_as_float(y0 << 16), __uint_as_float(y0 & 0xFFFF0000u)) |
               (cvt_pair<kFmt>(__uint_as_float(y1 << 16), __uint_as_float(y1 & 0xFFFF0000u)) << 16);
    }
    if (kPlus) {
        // Sec. 4.1: the BM's stored mantissa is its fraction rounded to kMb bits (nearest, ties
        // to even; bf16 has seven), clamped below the next binade; the cast's sign bit stays.
        // Every word is patched under a mask (no branch on the BM's position).
        const uint32_t frac = amax16 & 0x7Fu;
        constexpr int sh = 7 - kMb;
        uint32_t m = frac >> sh;
        if (sh > 0) {
            const uint32_t rem = frac & ((1u << sh) - 1u), half = 1u << (sh > 0 ? sh - 1 : 0);
            m = min(m + ((rem > half || (rem == half && (m & 1u))) ? 1u : 0u), (1u << kMb) - 1u);
        }
        const uint32_t pos = 8u * (bm & 3u);
        const uint32_t field = ((1u << kMb) - 1u) << pos, value = m << pos;
#pragma unroll
        for (int i = 0; i < 8; ++i)  // w[i] = (w[i] & ~field) | value in the BM's word, predicated
            asm("{ .reg .pred p;\n  setp.eq.u32 p, %1, %2;\n  @p lop3.b32 %0, %0, %3, %4, 0xBA; }"
                : "+r"(w[i]) : "r"(bm >> 2), "r"((uint32_t)i), "r"(field), "r"(value));
    }
    if (kFmt == 8) {
        uint4* out = reinterpret_cast<uint4*>(codes + blk * 32);
        out[0] = make_uint4(w[0], w[1], w[2], w[3]);
        out[1] = make_uint4(w[4], w[5], w[6], w[7]);
    } else {
        // bytes a b c d (six bits each) -> a | b << 6 | c << 12 | d << 18: pairs first (bits 14
        // and 15 of the intermediate hold stray bits the second select drops), then the halves
        uint32_t g[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t p = (w[i] & 0x003F003Fu) | ((w[i] >> 2) & ~0x003F003Fu);
            g[i] = (p & 0xFFFu) | ((p >> 4) & ~0xFFFu);
        }
        uint2* out = reinterpret_cast<uint2*>(codes + blk * 24);
        out[0] = make_uint2(__byte_perm(g[0], g[1], 0x4210), __byte_perm(g[1], g[2], 0x5421));
        out[1] = make_uint2(__byte_perm(g[2], g[3], 0x6542), __byte_perm(g[4], g[5], 0x4210));
        out[2] = make_uint2(__byte_perm(g[5], g[6], 0x5421), __byte_perm(g[6], g[7], 0x6542));
    }
}

// Eq. 3 at the wider formats; exact in fp32 and bf16 (at most 8 significant bits).
template <typename T, int kFmt, bool kPlus>
__global__ void __launch_bounds__(kThreads)
dequantize_wide_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                       const uint8_t* __restrict__ bm_index, int nbk, int64_t total_blocks,
                       T* __restrict__ dst, int64_t ld_dst)
{
    constexpr int kEmax = kFmt == 8 ? 8 : 2;
    constexpr int kMb = kFmt - 1;
    const int64_t blk = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (blk >= total_blocks) return;
    const int64_t row = blk / nbk;
    const int b = (int)(blk - row * nbk);
    uint32_t c[16];  // two codes each, one per byte
    if (kFmt == 8) {
        const uint4* in = reinterpret_cast<const uint4*>(codes + blk * 32);
        const uint4 a = __ldg(in), d = __ldg(in + 1);
        const uint32_t w[8] = {a.x, a.y, a.z, a.w, d.x, d.y, d.z, d.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            c[2 * i] = w[i] & 0xFFFFu;
            c[2 * i + 1] = w[i] >> 16;
        }
    } else {
        const uint2* in = reinterpret_cast<const uint2*>(codes + blk * 24);
        unsigned long long w[3];
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint2 t = __ldg(in + i);
            w[i] = (unsigned long long)t.x | ((unsigned long long)t.y << 32);
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int bit = 12 * i;  // two codes
            const int wi = bit >> 6, sh = bit & 63;
            unsigned long long x = w[wi] >> sh;
            if (sh > 52 && wi < 2) x |= w[wi + 1] << (64 - sh);
            c[i] = (uint32_t)(x & 63u) | ((uint32_t)((x >> 6) & 63u) << 8);
        }
    }
    const uint32_t sb = scales[blk];
    const int bm = kPlus ? (int)(bm_index[blk] & 31u) : -1;
    const float scale = __uint_as_float(sb << 23);  // 2^(sb - 127) for sb in 1..254
    float out[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 f = decode_pair<kFmt>(c[i]);
        out[2 * i] = f.x * scale;
        out[2 * i + 1] = f.y * scale;
    }
    if (kPlus) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (i == bm) {
                const uint32_t code = (c[i >> 1] >> ((i & 1) * 8)) & 0xFFu;
                const uint32_t m = code & ((1u << kMb) - 1u);
                // 2^emax * (1 + m / 2^kMb): mantissa bits placed at the top of the fraction
                const float mag = __uint_as_float(((127u + kEmax) << 23) | (m << (23 - kMb)));
                const float val = mag * scale;
                out[i] = ((code >> kMb) & 1u) ? -val : val;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        if (sb == 0u) out[i] = 0.0f;
        if (sb == 255u) out[i] = __uint_as_float(0x7FC00000u);
    }
    T* p = dst + row * ld_dst + (int64_t)b * 32;
    if (sizeof(T) == 4) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            reinterpret_cast<float4*>(p)[i] = make_float4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(out[8 * i + 2 * j], out[8 * i + 2 * j + 1]);
                w[j] = *reinterpret_cast<const uint32_t*>(&h);
            }
            reinterpret_cast<uint4*>(p)[i] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

template <typename T, int kFmt, bool kPlus>
cudaError_t launch_q(const void* src, int64_t rows, int64_t cols, int64_t ld_src, uint8_t* codes,
                     uint8_t* scales, uint8_t* bm_index, cudaStream_t stream)
{
    const int64_t total = rows * (cols / 32);
    if (sizeof(T) == 2 && ld_src == cols) {
        quantize_wide_bf16_kernel<kFmt, kPlus><<<(unsigned)((total + kThreads - 1) / kThreads), kThreads, 0, stream>>>(
            static_cast<const uint4*>(src), total, codes, scales, bm_index);
        return cudaGetLastError();
    }
    quantize_wide_kernel<T, kFmt, kPlus><<<(unsigned)((total + kThreads - 1) / kThreads), kThreads, 0, stream>>>(
        static_cast<const T*>(src), ld_src, (int)(cols / 32), total, codes, scales, bm_index);
    return cudaGetLastError();
}

template <typename T, int kFmt, bool kPlus>
cudaError_t launch_dq(const mxp_packed& p, void* dst, int64_t ld_dst, cudaStream_t stream)
{
    const int64_t total = p.rows * (p.cols / 32);
    dequantize_wide_kernel<T, kFmt, kPlus><<<(unsigned)((total + kThreads - 1) / kThreads), kThreads, 0, stream>>>(
        p.nibbles, p.scales, p.bm_index, (int)(p.cols / 32), total, static_cast<T*>(dst), ld_dst);
    return cudaGetLastError();
}

}  // namespace

#define MXP_WIDE_DISPATCH(FN, T, ...)                                         \
    switch (mode) {                                                           \
        case MXP_MODE_MXFP6: return FN<T, 6, false>(__VA_ARGS__);             \
        case MXP_MODE_MXFP6_PLUS: return FN<T, 6, true>(__VA_ARGS__);         \
        case MXP_MODE_MXFP8: return FN<T, 8, false>(__VA_ARGS__);             \
        case MXP_MODE_MXFP8_PLUS: return FN<T, 8, true>(__VA_ARGS__);         \
        default: return cudaErrorInvalidValue;                                \
    }

cudaError_t launch_quantize_wide(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                                 int64_t ld_src, mxp_mode mode, uint8_t* codes, uint8_t* scales,
                                 uint8_t* bm_index, cudaStream_t stream)
{
    if (dt == MXP_BF16) {
        MXP_WIDE_DISPATCH(launch_q, __nv_bfloat16, src, rows, cols, ld_src, codes, scales, bm_index, stream)
    }
    MXP_WIDE_DISPATCH(launch_q, float, src, rows, cols, ld_src, codes, scales, bm_index, stream)
}

cudaError_t launch_dequantize_wide(const mxp_packed& p, void* dst, mxp_dtype dt, int64_t ld_dst,
                                   cudaStream_t stream)
{
    const mxp_mode mode = p.mode;
    if (dt == MXP_BF16) {
        MXP_WIDE_DISPATCH(launch_dq, __nv_bfloat16, p, dst, ld_dst, stream)
    }
    MXP_WIDE_DISPATCH(launch_dq, float, p, dst, ld_dst, stream)
}
#undef MXP_WIDE_DISPATCH

}  // namespace mxp
