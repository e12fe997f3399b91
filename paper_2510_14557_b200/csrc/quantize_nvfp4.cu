// NVFP4 / NVFP4+ quantize and decode (Sec. 8, "Applicability of MX+ to NVFP4").
//
// NVFP4: E2M1 elements in blocks of 16, an E4M3 scale per block, one fp32 scale `ts` for the
// tensor.  The block scale is amax / (6 ts) rounded to E4M3, which puts the block's largest
// magnitude (the BM) next to 6, the top of the E2M1 range: its exponent field is at its
// maximum, so, as in MX+, NVFP4+ spends the BM's exponent bits on mantissa (value 4 + m/2,
// m = 0..7) and stores a 4-bit BM index per block.  Blocks whose scale byte is 2 or less keep
// the plain form (index nibble 0).
//
// What is computed is the definition in real numbers:  q = amax / (6 ts);  byte = the E4M3
// value nearest to q (ties to the even byte, saturating at 448);  d = value(byte) * ts;
// code = the E2M1 value nearest to |x| / d (ties to the even code, saturating at 6, sign of the
// input kept);  BM: m = nearest integer to (clamp(amax / d, 4, 8) - 4) * 2, ties to even, at
// most 7.  Decode: +-E * d rounded once to the output type.
// How: every quotient is first taken in binary32 through a reciprocal (error below 2^-22) and
// cast by the hardware; that is the definition's code unless a rounding boundary t of the cast
// lies within that error of the product.  Those cases are found cheaply (elements: by the
// product's bit pattern; scale byte and BM: by casting the product scaled down and up by
// 2^-20) and settled by comparing |x| with t * d (resp. amax with 6 t ts) in binary64, where
// those products (at most 33 significant bits) are exact; equality is the tie.
// Short operands (kShort: bf16 source, tensor scale with at most 12 significant bits, which
// covers every power of two): |x| has at most 8 significant bits and t * d at most 19, so a
// quotient that is not exactly on a boundary is at least 2^-20 of it away, and ties themselves
// are common (with a power-of-two d every 128th bf16 value of a binade is one).  There the
// quotient is taken with one Newton step on the reciprocal product, which returns it exactly
// whenever it is representable; the hardware cast then sees the tie as a tie, and nothing is
// left to settle per element.
//
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstring>

#include "common.cuh"

namespace mxp {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint32_t f32_to_e4m3_byte(float q)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.f), "f"(q));
    return (uint32_t)r & 0xFFu;
}
__device__ __forceinline__ float e4m3_byte_to_f32(uint32_t b)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)b));
    return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}
__device__ __forceinline__ uint32_t cvt_e2m1x8(const float* f)
{
    uint32_t r;
    asm("{ .reg .b8 b0, b1, b2, b3;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
        "  mov.b32 %0, {b0, b1, b2, b3}; }"
        : "=r"(r)
        : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "f"(f[4]), "f"(f[5]), "f"(f[6]), "f"(f[7]));
    return r;
}

constexpr float kDown = 1.f - 9.5367431640625e-07f;  // 1 - 2^-20
constexpr float kUp = 1.f + 9.5367431640625e-07f;    // 1 + 2^-20

// One block of 16: two words of codes, the scale byte and the BM index (0 when not extended).
// kKey: the values came from bf16, so their low 16 bits are zero and (magnitude bits | 15 -
// position) is a key whose unsigned maximum gives the largest magnitude and, among equal
// ones, the first position in one pass.
// The block's source words stay as loaded (bf16: two elements per word), which halves the
// registers a lane holds while it works on the other block; an element is widened where used.
template <bool kHalf>
__device__ __forceinline__ float elem(const uint32_t* raw, int i)
{
    if (!kHalf) return __uint_as_float(raw[i]);
    return __uint_as_float((i & 1) ? raw[i >> 1] & 0xFFFF0000u : raw[i >> 1] << 16);
}

template <typename T, bool kPlus, bool kShort>
__device__ __forceinline__ void nvfp4_block(const uint32_t* raw, float ts, float six_ts, uint32_t& w0, uint32_t& w1,
                                            uint32_t& scale_byte, uint32_t& index)
{
    constexpr bool kKey = sizeof(T) == 2;
#define X(i) elem<kKey>(raw, (i))
    float amax = 0.f;
    int bm = 0;
    if (kKey && kShort) {
        // bf16 pairs as loaded: the largest magnitude with a packed maximum, its first position
        // from a packed compare (one bit per element, even elements in bits 0,2,.., odd ones in
        // bits 16,18,..)
        uint32_t t[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = raw[i] & 0x7FFF7FFFu;
        uint32_t m2 = t[0];
#pragma unroll
        for (int i = 1; i < 8; ++i) asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(m2) : "r"(t[i]));
        asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(m2) : "r"(__byte_perm(m2, m2, 0x1032)));
        amax = __uint_as_float(m2 << 16);
        if (kPlus) {
            uint32_t r1 = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t eq;
                asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(eq) : "r"(t[i]), "r"(m2));
                r1 |= eq & ((1u << (2 * i)) | (1u << (16 + 2 * i)));
            }
            const uint32_t map = (r1 & 0xFFFFu) | ((r1 >> 15) & 0xAAAAu);
            bm = __ffs((int)map) - 1;
        }
    } else if (kPlus && kKey) {
        uint32_t key = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i)
            key = max(key, (__float_as_uint(X(i)) & 0x7FFFFFFFu) | (uint32_t)(15 - i));
        amax = __uint_as_float(key & 0x7FFF0000u);
        bm = 15 - (int)(key & 15u);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(X(i)));
        if (kPlus) {
#pragma unroll
            for (int i = 15; i >= 0; --i)
                if (fabsf(X(i)) == amax) bm = i;  // the first of equal maxima
        }
    }
    // scale byte: E4M3 nearest to amax / (6 ts)
    float q;
    if (kShort) {
        // the quotient by one Newton step on amax * (1 / 6 ts): exact whenever it is representable
        const float r6 = __frcp_rn(six_ts);  // (uniform over the grid: hoisted by the compiler)
        const float q0 = __fmul_rn(amax, r6);
        // (an enormous quotient needs no step: it saturates the cast; an infinite one would not)
        q = q0 < 1e30f ? __fmaf_rn(__fmaf_rn(-q0, six_ts, amax), r6, q0) : 1e30f;
    } else {
        q = fminf(__fdiv_rn(amax, six_ts), 1e30f);  // (the cast saturates finite values only)
    }
    // (short operands: 6 ts is exact, the division is correctly rounded, and a quotient that is
    // not exactly on a boundary between two bytes is at least 2^-21 of it away: one cast decides)
    uint32_t sb = f32_to_e4m3_byte(kShort ? q : __fmul_rn(q, kDown));
    const uint32_t sb_up = kShort ? sb : f32_to_e4m3_byte(__fmul_rn(q, kUp));
    if (sb != sb_up) {  // a boundary between the bytes sb and sb + 1 (never at saturation)
        const float t = 0.5f * (e4m3_byte_to_f32(sb) + e4m3_byte_to_f32(sb_up));  // exact
        const double bound = (double)t * 6.0 * (double)ts;                        // exact
        const double a = (double)amax;
        if (a > bound || (a == bound && (sb & 1u))) sb = sb_up;
    }
    const float e = e4m3_byte_to_f32(sb);
    // (short operands: the Newton step below squares the reciprocal's error, so the fast
    // approximate reciprocal serves)
    float r;
    if (kShort) asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(__fmul_rn(e, ts)));
    else r = __frcp_rn(__fmul_rn(e, ts));
    // r > 0, so x * r has the sign of x even where it underflows, and the hardware cast keeps
    // the sign of a value that rounds to zero: the codes' sign bits are the inputs'.
    // Every E2M1 rounding boundary (0.25 0.75 1.25 1.75 2.5 3.5 5) has zeros in the low 21 bits
    // of its binary32 pattern, and x * r is within 4 units in the last place of the exact
    // quotient: only a product whose pattern lies within 8 of such a pattern can be cast to
    // another code than the exact quotient.  `near` ends up below 0x8000 iff the block has one.
    float s[16];
    if (kShort) {
        // d is exact in binary32 here.  rho = x - s0 d (rounded down, so that an exact zero is
        // -0 and the sum below keeps the sign of a zero input), s = s0 + rho r.
        const float d32 = __fmul_rn(e, ts);
        if (__fmul_rn(amax, r) < 1e30f) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float x = X(i);
                const float s0 = __fmul_rn(x, r);
                s[i] = __fmaf_rn(__fmaf_rd(-s0, d32, x), r, s0);
            }
        } else {
            // a saturated scale under an enormous block: products may overflow; clamped first,
            // the step still returns the quotient (or an infinity that saturates the cast)
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float x = X(i);
                const float s0 = fminf(fmaxf(__fmul_rn(x, r), -16.f), 16.f);
                s[i] = __fmaf_rn(__fmaf_rd(-s0, d32, x), r, s0);
            }
        }
        w0 = cvt_e2m1x8(s);
        w1 = cvt_e2m1x8(s + 8);
    } else {
        uint32_t near = 0xFFFFFFFFu;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            s[i] = __fmul_rn(X(i), r);
            near = min(near, __float_as_uint(s[i]) * 2048u + 0x4000u);
        }
        w0 = cvt_e2m1x8(s);
        w1 = cvt_e2m1x8(s + 8);
        if (near < 0x8000u) {
            const double d = (double)e * (double)ts;  // exact
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const uint32_t bits = __float_as_uint(__fmul_rn(X(i), r));  // (recomputed: keeps s[] short-lived)
                if (bits * 2048u + 0x4000u < 0x8000u) {
                    const float t = __uint_as_float((bits + 8u) & 0x7FE00000u);  // the candidate boundary
                    const float t4 = fminf(t * 4.f, 31.f);
                    const uint32_t u = (uint32_t)t4;                               // 1 3 5 7 10 14 20
                    constexpr uint32_t kBoundaries = 0x1044AAu;                    // those bits set
                    if ((float)u == t4 && ((kBoundaries >> u) & 1u)) {
                        const uint32_t lower = (uint32_t)__popc(kBoundaries & ((1u << u) - 1u));  // code below it
                        const double bound = (double)t * d;                        // exact
                        const double a = fabs((double)X(i));
                        const uint32_t code = lower + ((a > bound || (a == bound && (lower & 1u))) ? 1u : 0u);
                        const uint32_t sh = (uint32_t)(i & 7) * 4u;
                        if (i < 8) w0 = (w0 & ~(7u << sh)) | (code << sh);
                        else w1 = (w1 & ~(7u << sh)) | (code << sh);
                    }
                }
            }
        }
    }
    index = 0;
    if (kPlus && sb > 2u) {
        uint32_t m, m_up;
        if (kShort) {
            // amax / d by the same Newton step as the elements: exact whenever it is representable,
            // and otherwise at least 2^-20 of a boundary 4.25 + m / 2 away from it
            const float d32 = __fmul_rn(e, ts);
            const float v0 = __fmul_rn(amax, r);
            // (an overflowed product clamps to 8 like any quotient of 8 or more)
            const float v = v0 < 1e30f ? fminf(fmaxf(__fmaf_rn(__fmaf_rn(-v0, d32, amax), r, v0), 4.f), 8.f) : 8.f;
            m = m_up = (uint32_t)__float2int_rn((v - 4.f) * 2.f);  // 0..8, ties to even
        } else {
            const float r_dn = __fmul_rn(r, kDown), r_up = __fmul_rn(r, kUp);
            const float v_dn = fminf(fmaxf(__fmul_rn(amax, r_dn), 4.f), 8.f);
            const float v_up = fminf(fmaxf(__fmul_rn(amax, r_up), 4.f), 8.f);
            m = (uint32_t)__float2int_rn((v_dn - 4.f) * 2.f);  // 0..8
            m_up = (uint32_t)__float2int_rn((v_up - 4.f) * 2.f);
        }
        if (m != m_up) {  // boundary 4.25 + m / 2 between m and m + 1
            const double bound = (double)(17u + 2u * m) * 0.25 * ((double)e * (double)ts);
            const double a = (double)amax;
            if (a > bound || (a == bound && (m & 1u))) m = m_up;
        }
        m = min(m, 7u);
        const uint32_t sh = (uint32_t)(bm & 7) * 4u;
        if (bm < 8) w0 = (w0 & ~(7u << sh)) | (m << sh);  // the sign bit stays
        else w1 = (w1 & ~(7u << sh)) | (m << sh);
        index = (uint32_t)bm;
    }
    if (sb == 0u) w0 = w1 = 0u;
    scale_byte = sb;
#undef X
}

// (bf16 rows in the short-operand form fit 32 registers: eight CTAs per SM hide the load latency
// this HBM-bound kernel is exposed to -- 40.0 -> 36.2 us on 8192 x 8192 against four CTAs)
template <typename T, bool kPlus, bool kShort>
__global__ void __launch_bounds__(kThreads, (sizeof(T) == 2 && kShort) ? 8 : 4)
nvfp4_quantize_kernel(const T* __restrict__ src, int64_t ld_src, int64_t units_per_row,
                      int64_t total_units, float ts, uint4* __restrict__ nibbles,
                      uint16_t* __restrict__ scales, uint8_t* __restrict__ bm_index)
{
    const int64_t u = (int64_t)blockIdx.x * kThreads + threadIdx.x;  // unit of 32 elements
    if (u >= total_units) return;
    const int64_t row = u / units_per_row;
    const T* p = src + row * ld_src + (u - row * units_per_row) * 32;
    constexpr int kWords = sizeof(T) == 2 ? 16 : 32;
    uint32_t raw[kWords];
#pragma unroll
    for (int i = 0; i < kWords / 4; ++i) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p) + i);
        raw[4 * i] = v.x;
        raw[4 * i + 1] = v.y;
        raw[4 * i + 2] = v.z;
        raw[4 * i + 3] = v.w;
    }
    const float six_ts = __fmul_rn(6.f, ts);
    uint32_t w[4], sb0, sb1, i0, i1;
    nvfp4_block<T, kPlus, kShort>(raw, ts, six_ts, w[0], w[1], sb0, i0);
    nvfp4_block<T, kPlus, kShort>(raw + kWords / 2, ts, six_ts, w[2], w[3], sb1, i1);
    __stcs(nibbles + u, make_uint4(w[0], w[1], w[2], w[3]));
    scales[u] = (uint16_t)(sb0 | (sb1 << 8));
    if (kPlus) bm_index[u] = (uint8_t)(i0 | (i1 << 4));
}

// One thread decodes eight elements (one word of codes, half a block).
template <typename T, bool kPlus>
__global__ void __launch_bounds__(kThreads)
nvfp4_dequantize_kernel(const uint32_t* __restrict__ nibbles, const uint8_t* __restrict__ scales,
                        const uint8_t* __restrict__ bm_index, int64_t cols, int64_t total_words,
                        float ts, T* __restrict__ dst, int64_t ld_dst)
{
    const int64_t u = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (u >= total_words) return;
    const int64_t blk = u >> 1;
    const uint32_t word = __ldg(nibbles + u);
    const uint32_t sb = scales[blk];
    const float e = e4m3_byte_to_f32(sb & 127u);
    int bm = -1;
    if (kPlus && sb > 2u) {
        bm = (int)((bm_index[blk >> 1] >> (4 * (blk & 1))) & 15u) - 8 * (int)(u & 1);  // within this word
    }
    // E * value(byte) is exact in binary32 (at most 8 significant bits), so one multiply by ts
    // rounds the exact product once.  For a bf16 destination that multiply rounds to odd
    // (truncate, then set the last bit if anything was cut off), which makes the second
    // rounding, to bf16, the single correct one.
    float out[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t c = (word >> (4 * i)) & 15u;
        const uint32_t ex = (c >> 1) & 3u, m = c & 1u;
        float mag = ex == 0u ? 0.5f * (float)m : __uint_as_float(((126u + ex) << 23) | (m << 22));
        if (kPlus && i == bm) mag = 4.f + 0.5f * (float)(c & 7u);
        const float me = __fmul_rn(mag, e);
        float v;
        if (sizeof(T) == 4) {
            v = __fmul_rn(me, ts);
        } else {
            v = __fmul_rz(me, ts);
            if (__fmaf_rn(me, ts, -v) != 0.f) v = __uint_as_float(__float_as_uint(v) | 1u);
        }
        out[i] = (c & 8u) ? -v : v;
    }
    const int64_t e0 = u * 8, row = e0 / cols;
    T* q = dst + row * ld_dst + (e0 - row * cols);
    if (sizeof(T) == 4) {
        reinterpret_cast<uint4*>(q)[0] = make_uint4(__float_as_uint(out[0]), __float_as_uint(out[1]),
                                                    __float_as_uint(out[2]), __float_as_uint(out[3]));
        reinterpret_cast<uint4*>(q)[1] = make_uint4(__float_as_uint(out[4]), __float_as_uint(out[5]),
                                                    __float_as_uint(out[6]), __float_as_uint(out[7]));
    } else {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(out[2 * i], out[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(q) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

}  // namespace

cudaError_t launch_nvfp4_quantize(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                                  int64_t ld_src, float ts, bool plus, uint8_t* nibbles,
                                  uint8_t* scales, uint8_t* bm_index, cudaStream_t stream)
{
    const int64_t units = rows * (cols / 32);
    const unsigned grid = (unsigned)((units + kThreads - 1) / kThreads);
#define MXP_NVQ(T, P, S)                                                                      \
    nvfp4_quantize_kernel<T, P, S><<<grid, kThreads, 0, stream>>>(                            \
        static_cast<const T*>(src), ld_src, cols / 32, units, ts, reinterpret_cast<uint4*>(nibbles), \
        reinterpret_cast<uint16_t*>(scales), bm_index)
    // short operands: bf16 source, at most 12 significant bits in the tensor scale, and a
    // scale large enough for value(byte) * ts to stay a normal number (bytes reach down to 2^-9)
    uint32_t ts_bits;
    memcpy(&ts_bits, &ts, 4);
    const bool shortop = dt == MXP_BF16 && (ts_bits & 0xFFFu) == 0u && ts >= 0x1p-100f && ts <= 0x1p100f;
    if (dt == MXP_BF16) {
        if (shortop) {
            if (plus) MXP_NVQ(__nv_bfloat16, true, true);
            else MXP_NVQ(__nv_bfloat16, false, true);
        } else {
            if (plus) MXP_NVQ(__nv_bfloat16, true, false);
            else MXP_NVQ(__nv_bfloat16, false, false);
        }
    } else {
        if (plus) MXP_NVQ(float, true, false);
        else MXP_NVQ(float, false, false);
    }
#undef MXP_NVQ
    return cudaGetLastError();
}

cudaError_t launch_nvfp4_dequantize(const uint8_t* nibbles, const uint8_t* scales,
                                    const uint8_t* bm_index, int64_t rows, int64_t cols, float ts,
                                    bool plus, void* dst, mxp_dtype dt, int64_t ld_dst,
                                    cudaStream_t stream)
{
    const int64_t words = rows * (cols / 8);
    const unsigned grid = (unsigned)((words + kThreads - 1) / kThreads);
#define MXP_NVD(T, P)                                                                          \
    nvfp4_dequantize_kernel<T, P><<<grid, kThreads, 0, stream>>>(                              \
        reinterpret_cast<const uint32_t*>(nibbles), scales, bm_index, cols, words, ts,         \
        static_cast<T*>(dst), ld_dst)
    if (dt == MXP_BF16) {
        if (plus) MXP_NVD(__nv_bfloat16, true);
        else MXP_NVD(__nv_bfloat16, false);
    } else {
        if (plus) MXP_NVD(float, true);
        else MXP_NVD(float, false);
    }
#undef MXP_NVD
    return cudaGetLastError();
}

}  // namespace mxp
