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
// How: every quotient is first taken in binary32 through a reciprocal, twice -- scaled down and
// up by 2^-20, which brackets the exact quotient (the binary32 steps err by < 2^-22) -- and
// both go through the hardware cast.  Where the two casts agree no rounding boundary lies in
// between and the code is the definition's.  Where they differ, exactly one boundary t lies in
// between, and the side is decided by comparing |x| with t * d (resp. amax with 6 t ts) in
// binary64, where those products (at most 33 significant bits) are exact; equality is the tie.
//
#include <cuda_bf16.h>
#include <cuda_fp16.h>

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

// Value of an E2M1 magnitude code (0..7) times four: 0 2 4 6 8 12 16 24, five bits each.
__device__ __forceinline__ uint32_t e2m1_times4(uint32_t c)
{
    return (uint32_t)((0xC418831040ull >> (5u * c)) & 31ull);
}

// One block of 16: two words of codes, the scale byte and the BM index (0 when not extended).
// `src` points at the block's 16 source elements (read again only for the rare element whose
// two bracketing casts differ).
// kKey: the values came from bf16, so their low 16 bits are zero and (magnitude bits | 15 -
// position) is a key whose unsigned maximum gives the largest magnitude and, among equal
// ones, the first position in one pass.
template <typename T, bool kPlus>
__device__ __forceinline__ void nvfp4_block(const float* x, const T* __restrict__ src, float ts,
                                            float six_ts, uint32_t& w0, uint32_t& w1,
                                            uint32_t& scale_byte, uint32_t& index)
{
    constexpr bool kKey = sizeof(T) == 2;
    float amax = 0.f;
    int bm = 0;
    if (kPlus && kKey) {
        uint32_t key = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i)
            key = max(key, (__float_as_uint(x[i]) & 0x7FFFFFFFu) | (uint32_t)(15 - i));
        amax = __uint_as_float(key & 0x7FFF0000u);
        bm = 15 - (int)(key & 15u);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(x[i]));
        if (kPlus) {
#pragma unroll
            for (int i = 15; i >= 0; --i)
                if (fabsf(x[i]) == amax) bm = i;  // the first of equal maxima
        }
    }
    // scale byte: E4M3 nearest to amax / (6 ts)
    const float q = __fdiv_rn(amax, six_ts);
    uint32_t sb = f32_to_e4m3_byte(__fmul_rn(q, kDown));
    const uint32_t sb_up = f32_to_e4m3_byte(__fmul_rn(q, kUp));
    if (sb != sb_up) {  // a boundary between the bytes sb and sb + 1 (never at saturation)
        const float t = 0.5f * (e4m3_byte_to_f32(sb) + e4m3_byte_to_f32(sb_up));  // exact
        const double bound = (double)t * 6.0 * (double)ts;                        // exact
        const double a = (double)amax;
        if (a > bound || (a == bound && (sb & 1u))) sb = sb_up;
    }
    const float e = e4m3_byte_to_f32(sb);
    const float r = __frcp_rn(__fmul_rn(e, ts));
    const float r_dn = __fmul_rn(r, kDown), r_up = __fmul_rn(r, kUp);
    // r > 0, so x * r has the sign of x even where it underflows, and the hardware cast keeps
    // the sign of a value that rounds to zero: the codes' sign bits are the inputs'
    float s[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) s[i] = __fmul_rn(x[i], r_dn);
    w0 = cvt_e2m1x8(s);
    w1 = cvt_e2m1x8(s + 8);
#pragma unroll
    for (int i = 0; i < 16; ++i) s[i] = __fmul_rn(x[i], r_up);
    const uint32_t d0 = w0 ^ cvt_e2m1x8(s), d1 = w1 ^ cvt_e2m1x8(s + 8);
    if (d0 | d1) {
        // the upper cast is the next code of the lower one; the boundary between the two is
        // the mean of their values
        const double d = (double)e * (double)ts;  // exact
        uint64_t diff = ((uint64_t)d1 << 32) | d0;
        uint64_t w = ((uint64_t)w1 << 32) | w0;
        while (diff) {
            const int i = (__ffsll((long long)diff) - 1) >> 2;
            diff &= ~(0xFull << (4 * i));
            const uint32_t c = (uint32_t)(w >> (4 * i)) & 7u;  // lower code, c < 7
            const double bound = (double)(e2m1_times4(c) + e2m1_times4(c + 1u)) * 0.125 * d;
            double a;
            if (kKey) a = (double)__bfloat162float(reinterpret_cast<const __nv_bfloat16*>(src)[i]);
            else a = (double)reinterpret_cast<const float*>(src)[i];
            a = fabs(a);
            if (a > bound || (a == bound && (c & 1u))) w += 1ull << (4 * i);
        }
        w0 = (uint32_t)w;
        w1 = (uint32_t)(w >> 32);
    }
    index = 0;
    if (kPlus && sb > 2u) {
        const float v_dn = fminf(fmaxf(__fmul_rn(amax, r_dn), 4.f), 8.f);
        const float v_up = fminf(fmaxf(__fmul_rn(amax, r_up), 4.f), 8.f);
        uint32_t m = (uint32_t)__float2int_rn((v_dn - 4.f) * 2.f);  // 0..8
        const uint32_t m_up = (uint32_t)__float2int_rn((v_up - 4.f) * 2.f);
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
}

template <typename T, bool kPlus>
__global__ void __launch_bounds__(kThreads)
nvfp4_quantize_kernel(const T* __restrict__ src, int64_t ld_src, int64_t units_per_row,
                      int64_t total_units, float ts, uint4* __restrict__ nibbles,
                      uint16_t* __restrict__ scales, uint8_t* __restrict__ bm_index)
{
    const int64_t u = (int64_t)blockIdx.x * kThreads + threadIdx.x;  // unit of 32 elements
    if (u >= total_units) return;
    const int64_t row = u / units_per_row;
    const T* p = src + row * ld_src + (u - row * units_per_row) * 32;
    float x[32];
    if (sizeof(T) == 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p) + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                x[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
                x[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p) + i);
            x[4 * i] = __uint_as_float(v.x);
            x[4 * i + 1] = __uint_as_float(v.y);
            x[4 * i + 2] = __uint_as_float(v.z);
            x[4 * i + 3] = __uint_as_float(v.w);
        }
    }
    const float six_ts = __fmul_rn(6.f, ts);
    uint32_t w[4], sb0, sb1, i0, i1;
    nvfp4_block<T, kPlus>(x, p, ts, six_ts, w[0], w[1], sb0, i0);
    nvfp4_block<T, kPlus>(x + 16, p + 16, ts, six_ts, w[2], w[3], sb1, i1);
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
#define MXP_NVQ(T, P)                                                                         \
    nvfp4_quantize_kernel<T, P><<<grid, kThreads, 0, stream>>>(                               \
        static_cast<const T*>(src), ld_src, cols / 32, units, ts, reinterpret_cast<uint4*>(nibbles), \
        reinterpret_cast<uint16_t*>(scales), bm_index)
    if (dt == MXP_BF16) {
        if (plus) MXP_NVQ(__nv_bfloat16, true);
        else MXP_NVQ(__nv_bfloat16, false);
    } else {
        if (plus) MXP_NVQ(float, true);
        else MXP_NVQ(float, false);
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
