// MXFP4 / MXFP4+ block quantization and decode kernels (HBM-bound).
//
// Quantize (Eq. 1, Sec. 4.1, Sec. 4.2).  Two kernels:
//   - bf16, contiguous rows (the hot case): one lane per 32-element block, packed bf16x2
//     arithmetic, no shuffles (quantize_bf16_lane_kernel);
//   - generic (fp32 source or strided rows): four lanes own one block, eight elements each;
//     the block maximum and its first position come out of one integer max over keys
//     (|x| bit pattern, 31 - position), reduced over the four lanes by two shuffles.
// Either way the BM falls out of the scale computation: the paper's point that it is found
// for free during conversion.
//
// Mode 2 is MX++ (Sec. 4.3): the NBMs are scaled with their own shared exponent
// shared_exp_new = CLIP(max2 - emax + 1, {shared_exp - 7, shared_exp}), max2 the largest
// exponent among the non-zero NBMs; delta = shared_exp - shared_exp_new goes into the three
// reserved bits of the index byte.  The scale byte and the BM nibble are those of MX+.
#include <cuda_bf16.h>

#include "common.cuh"
#include "e4m3_widen.cuh"

namespace mxp {
namespace {

constexpr int kThreads = 256;
constexpr int kBlocksPerWarpPass = 32;                      // 8 groups x 4 blocks
constexpr int kBlocksPerCta = kBlocksPerWarpPass * (kThreads / 32);

// Eight scaled values -> eight E2M1 codes, element 0 in the lowest nibble.
// cvt.rn.satfinite rounds to nearest-even and saturates at +-6.
__device__ __forceinline__ uint32_t cvt_e2m1x8(const float (&f)[8])
{
    uint32_t r;
    asm("{ .reg .b8 b0, b1, b2, b3;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
        "  mov.b32 %0, {b0, b1, b2, b3}; }"
        : "=r"(r)
        : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "f"(f[4]), "f"(f[5]), "f"(f[6]),
          "f"(f[7]));
    return r;
}

// bf16 path.  Key of one element: 15-bit magnitude pattern in bits 30..16 (monotone in
// |x|), 31 - position in bits 4..0, so that an unsigned max picks the largest magnitude and,
// among equal ones, the lowest position.
__device__ __forceinline__ void load_unit_bf16(const uint4 w4, int pos0, float (&v)[8],
                                               uint32_t& key)
{
    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
    uint32_t k = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        v[2 * j] = __uint_as_float(w[j] << 16);
        v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        const uint32_t a = w[j] & 0x7FFF7FFFu;
        const uint32_t klo = (a << 16) | (uint32_t)(31 - (pos0 + 2 * j));
        const uint32_t khi = (a & 0xFFFF0000u) | (uint32_t)(31 - (pos0 + 2 * j + 1));
        k = max(k, max(klo, khi));
    }
    key = k;
}

__device__ __forceinline__ uint4 ldg_stream(const void* p)
{
    return __ldcs(reinterpret_cast<const uint4*>(p));
}

// One block's worth of work for this lane (quarter q of block `blk`).
//   returns the packed nibble word; writes the block's scale / index bytes (same value in
//   all four lanes of the group).
// Biased floor(log2) of a non-zero fp32 magnitude pattern (127 = 2^0), subnormals included.
__device__ __forceinline__ int biased_floor_log2(uint32_t a)
{
    const int e = (int)(a >> 23);
    return e != 0 ? e : 9 - __clz((int)a);
}
// MX++: delta = shared_exp - shared_exp_new from the biased exponents of the BM (E) and of
// the largest NBM magnitude pattern (a2, fp32 bits; 0: every NBM is zero).
__device__ __forceinline__ uint32_t mxpp_delta(uint32_t E, uint32_t a2)
{
    const int se_b = (int)E - 2;
    int nb = se_b - 7;
    if (a2 != 0u) nb = min(max(biased_floor_log2(a2) - 1, se_b - 7), se_b);
    return (uint32_t)(se_b - nb);
}

// kMode: 0 MXFP4, 1 MXFP4+, 2 MX++.  a2_bits (MX++ only): largest NBM magnitude of the block.
template <int kMode>
__device__ __forceinline__ uint32_t encode_quarter(const float (&v)[8], uint32_t amax_bits,
                                                   uint32_t a2_bits, int bm, int q,
                                                   uint32_t& scale_byte, uint32_t& index_byte)
{
    constexpr bool kPlus = kMode >= 1;
    // amax_bits: fp32 bit pattern of the block's absolute maximum
    const uint32_t E = amax_bits >> 23;  // biased exponent (sign already cleared)
    const bool flush = E <= 2u;          // floor(log2 BM) <= -125, zero and subnormals
    const bool nonfinite = E == 255u;
    scale_byte = flush ? 0u : (nonfinite ? 255u : E - 2u);
    const uint32_t delta = (kMode == 2 && !flush && !nonfinite) ? mxpp_delta(E, a2_bits) : 0u;
    index_byte = (kPlus && !flush && !nonfinite) ? ((uint32_t)bm | (delta << 5)) : 0u;

    // 2^-shared_exp(_new) = 2^(129 - E + delta): biased exponent 256 - E + delta, in [2, 253]
    // without delta; with it the factor is applied in two exact steps
    const uint32_t kexp = 256u - E + delta;
    const float inv = __uint_as_float(min(kexp, 254u) << 23);
    const float inv_hi = __uint_as_float((127u + kexp - min(kexp, 254u)) << 23);
    float s[8];
    uint32_t sign = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        s[i] = v[i] * inv;  // exact (power of two); < 8 in magnitude
        if (kMode == 2) s[i] *= inv_hi;
        sign |= (__float_as_uint(v[i]) >> 31) << (4 * i + 3);
    }
    // codes from the hardware cast; the sign bit of each nibble is taken from the input so
    // that values rounding to zero (and -0.0) keep their sign
    uint32_t word = (cvt_e2m1x8(s) & 0x77777777u) | sign;
    if (kPlus) {
        // BM mantissa: top 3 fraction bits of amax, round to nearest even, clamp at 7
        const uint32_t mant = amax_bits & 0x7FFFFFu;
        uint32_t m = (mant + 0x7FFFFu + ((mant >> 20) & 1u)) >> 20;
        m = min(m, 7u);
        if ((bm >> 3) == q) {
            const int sh = (bm & 7) * 4;
            word = (word & ~(7u << sh)) | (m << sh);
        }
    }
    return (flush || nonfinite) ? 0u : word;
}

// Second half of a pass: the four lanes of a group hold the four quarters of blocks
// span0 .. span0+3 (v: values, key / hi_bits: the lane's maximum); blocks at or past `limit`
// are not stored.
template <typename T, int kMode>
__device__ __forceinline__ void finish_pass(const float (&v)[4][8], const uint32_t (&key)[4],
                                            const uint32_t (&hi_bits)[4], int64_t span0, int q,
                                            int64_t total_blocks, uint8_t* __restrict__ nibbles,
                                            uint8_t* __restrict__ scales,
                                            uint8_t* __restrict__ bm_index, int planes_aligned4)
{
    uint32_t words[4], sc_pack = 0, ix_pack = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t amax_bits;
        int bm;
        if (sizeof(T) == 2) {
            uint32_t k = key[j];
            k = max(k, __shfl_xor_sync(0xFFFFFFFFu, k, 1));
            k = max(k, __shfl_xor_sync(0xFFFFFFFFu, k, 2));
            amax_bits = k & 0x7FFF0000u;
            bm = 31 - (int)(k & 31u);
        } else {
            // fp32: 31 magnitude bits do not fit a 32-bit key with the position; reduce the
            // maximum first, then the first position that holds it.
            uint32_t a = hi_bits[j];
            a = max(a, __shfl_xor_sync(0xFFFFFFFFu, a, 1));
            a = max(a, __shfl_xor_sync(0xFFFFFFFFu, a, 2));
            int first = 32;
#pragma unroll
            for (int i = 7; i >= 0; --i)
                if ((__float_as_uint(v[j][i]) & 0x7FFFFFFFu) == a) first = q * 8 + i;
            first = min(first, __shfl_xor_sync(0xFFFFFFFFu, first, 1));
            first = min(first, __shfl_xor_sync(0xFFFFFFFFu, first, 2));
            amax_bits = a;
            bm = first & 31;
        }
        uint32_t a2 = 0;
        if (kMode == 2) {
            // largest magnitude among the block's other elements (fp32 bit patterns)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t a = __float_as_uint(v[j][i]) & 0x7FFFFFFFu;
                if (q * 8 + i != bm) a2 = max(a2, a);
            }
            a2 = max(a2, __shfl_xor_sync(0xFFFFFFFFu, a2, 1));
            a2 = max(a2, __shfl_xor_sync(0xFFFFFFFFu, a2, 2));
        }
        uint32_t sb, ib;
        words[j] = encode_quarter<kMode>(v[j], amax_bits, a2, bm, q, sb, ib);
        sc_pack |= sb << (8 * j);
        ix_pack |= ib << (8 * j);
    }

    // ---- stores: 4 bytes of nibbles per lane and block; one word of scales / indices per group
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int64_t blk = span0 + j;
        if (blk < total_blocks)
            __stcs(reinterpret_cast<uint32_t*>(nibbles + blk * 16 + q * 4), words[j]);
    }
    if (span0 + 3 < total_blocks && planes_aligned4) {
        if (q == 0) __stcs(reinterpret_cast<uint32_t*>(scales + span0), sc_pack);
        if (q == 1 && bm_index != nullptr)
            __stcs(reinterpret_cast<uint32_t*>(bm_index + span0), ix_pack);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (span0 + j < total_blocks) {
                if (q == 0) scales[span0 + j] = (uint8_t)(sc_pack >> (8 * j));
                if (q == 1 && bm_index != nullptr)
                    bm_index[span0 + j] = (uint8_t)(ix_pack >> (8 * j));
            }
        }
    }
}

// kContig: ld_src == cols, so the source is one flat array of blocks.
// kGather: channel reordering fused into the quantizer (Sec. 8, "Scattering outliers with
// channel reordering"): position c of the quantized row takes source channel order[c], so a
// block is 32 channels that the caller's ordering placed together; nothing else changes.
template <typename T, int kMode, bool kContig, bool kGather = false>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const T* __restrict__ src, int64_t ld_src, int64_t cols_blocks,
                int64_t total_blocks, uint8_t* __restrict__ nibbles,
                uint8_t* __restrict__ scales, uint8_t* __restrict__ bm_index, int planes_aligned4,
                const int32_t* __restrict__ order = nullptr)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int g = lane >> 2;  // lane group: blocks 4g .. 4g+3 of the warp's span
    const int q = lane & 3;   // quarter of the block owned by this lane
    const int64_t span0 =
        (int64_t)blockIdx.x * kBlocksPerCta + (int64_t)warp * kBlocksPerWarpPass + 4 * g;

    float v[4][8];
    uint32_t key[4];
    uint32_t hi_bits[4];  // fp32 path: the lane's maximum |x| bit pattern

    // ---- issue all loads of the pass first
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int64_t blk = span0 + j;
        const bool live = blk < total_blocks;
        int64_t elem;  // offset of the block's first element in src
        if (kContig) {
            elem = blk * 32;
        } else {
            const int64_t row = blk / cols_blocks;
            elem = row * ld_src + (blk - row * cols_blocks) * 32;
        }
        uint32_t ch[8];  // kGather: the lane's eight source channels, clamped into the row
        if (kGather) {
            const int64_t row = blk / cols_blocks;
            const int64_t c0 = (blk - row * cols_blocks) * 32 + q * 8;
            elem = row * ld_src;
            uint4 o0 = make_uint4(0, 0, 0, 0), o1 = o0;
            if (live) {
                o0 = __ldg(reinterpret_cast<const uint4*>(order + c0));
                o1 = __ldg(reinterpret_cast<const uint4*>(order + c0) + 1);
            }
            const uint32_t o[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
            const uint32_t last = (uint32_t)(cols_blocks * 32 - 1);
#pragma unroll
            for (int i = 0; i < 8; ++i) ch[i] = min(o[i], last);
        }
        if (sizeof(T) == 2) {
            uint4 w = make_uint4(0, 0, 0, 0);
            if (kGather) {
                if (live) {
                    const unsigned short* s16 = reinterpret_cast<const unsigned short*>(src) + elem;
                    w.x = (uint32_t)__ldg(s16 + ch[0]) | ((uint32_t)__ldg(s16 + ch[1]) << 16);
                    w.y = (uint32_t)__ldg(s16 + ch[2]) | ((uint32_t)__ldg(s16 + ch[3]) << 16);
                    w.z = (uint32_t)__ldg(s16 + ch[4]) | ((uint32_t)__ldg(s16 + ch[5]) << 16);
                    w.w = (uint32_t)__ldg(s16 + ch[6]) | ((uint32_t)__ldg(s16 + ch[7]) << 16);
                }
            } else if (live) {
                w = ldg_stream(reinterpret_cast<const char*>(src) + (elem + q * 8) * 2);
            }
            load_unit_bf16(w, q * 8, v[j], key[j]);
            hi_bits[j] = 0;
        } else {
            uint4 w0 = make_uint4(0, 0, 0, 0), w1 = w0;
            if (kGather) {
                if (live) {
                    const uint32_t* s32 = reinterpret_cast<const uint32_t*>(src) + elem;
                    w0 = make_uint4(__ldg(s32 + ch[0]), __ldg(s32 + ch[1]), __ldg(s32 + ch[2]),
                                    __ldg(s32 + ch[3]));
                    w1 = make_uint4(__ldg(s32 + ch[4]), __ldg(s32 + ch[5]), __ldg(s32 + ch[6]),
                                    __ldg(s32 + ch[7]));
                }
            } else if (live) {
                const char* p = reinterpret_cast<const char*>(src) + (elem + q * 8) * 4;
                w0 = ldg_stream(p);
                w1 = ldg_stream(p + 16);
            }
            const uint32_t w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
            uint32_t a = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[j][i] = __uint_as_float(w[i]);
                a = max(a, w[i] & 0x7FFFFFFFu);
            }
            hi_bits[j] = a;
            key[j] = 0;
            (void)w;
        }
    }

    finish_pass<T, kMode>(v, key, hi_bits, span0, q, total_blocks, nibbles, scales, bm_index,
                          planes_aligned4);
}

// Channel reordering with the row staged in shared memory: a CTA copies one source row with
// coalesced 16-byte loads, then its lanes pick their channels out of shared memory, where an
// arbitrary ordering costs bank conflicts instead of one 128-byte line per element.  Rows are
// dealt to the CTAs round robin; several CTAs per SM overlap one's copy with another's casts.
template <typename T, int kMode>
__global__ void __launch_bounds__(kThreads)
quantize_reordered_staged_kernel(const T* __restrict__ src, int64_t ld_src, int64_t rows,
                                 int cols_blocks, const int32_t* __restrict__ order,
                                 uint8_t* __restrict__ nibbles, uint8_t* __restrict__ scales,
                                 uint8_t* __restrict__ bm_index, int planes_aligned4)
{
    extern __shared__ uint4 row_smem[];
    const T* row_s = reinterpret_cast<const T*>(row_smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, q = lane & 3;
    const int cols = cols_blocks * 32;
    const int vecs = cols * (int)sizeof(T) / 16;
    const uint32_t last = (uint32_t)(cols - 1);
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4* src_row = reinterpret_cast<const uint4*>(src + row * ld_src);
        __syncthreads();  // the previous row has been read
        for (int i = threadIdx.x; i < vecs; i += kThreads) row_smem[i] = ldg_stream(src_row + i);
        __syncthreads();
        const int64_t row_blk0 = row * cols_blocks;
        // (warp-uniform trip count: finish_pass shuffles within the whole warp)
        for (int base = warp * kBlocksPerWarpPass; base < cols_blocks; base += kBlocksPerCta) {
            const int b0 = base + 4 * g;
            float v[4][8];
            uint32_t key[4], hi_bits[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool live = b0 + j < cols_blocks;
                uint4 o0 = make_uint4(0, 0, 0, 0), o1 = o0;
                if (live) {
                    const uint4* op = reinterpret_cast<const uint4*>(order + (b0 + j) * 32 + q * 8);
                    o0 = __ldg(op);
                    o1 = __ldg(op + 1);
                }
                const uint32_t o[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
                if (sizeof(T) == 2) {
                    const unsigned short* s16 = reinterpret_cast<const unsigned short*>(row_s);
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        w[i] = live ? (uint32_t)s16[min(o[2 * i], last)] |
                                          ((uint32_t)s16[min(o[2 * i + 1], last)] << 16)
                                    : 0u;
                    load_unit_bf16(make_uint4(w[0], w[1], w[2], w[3]), q * 8, v[j], key[j]);
                    hi_bits[j] = 0;
                } else {
                    const uint32_t* s32 = reinterpret_cast<const uint32_t*>(row_s);
                    uint32_t a = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t w = live ? s32[min(o[i], last)] : 0u;
                        v[j][i] = __uint_as_float(w);
                        a = max(a, w & 0x7FFFFFFFu);
                    }
                    hi_bits[j] = a;
                    key[j] = 0;
                }
            }
            // blocks past the end of this row are not stored
            finish_pass<T, kMode>(v, key, hi_bits, row_blk0 + b0, q, row_blk0 + cols_blocks, nibbles,
                                  scales, bm_index, planes_aligned4);
        }
    }
}

// ---------------------------------------------------------------- bf16 helpers (packed arithmetic)
// The power-of-two scaling is one bf16x2 multiply per pair (exact; results that underflow are
// far below the smallest code and round to a signed zero either way) and the sign bits come
// straight out of the hardware cast, which keeps the sign of values rounding to zero.
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
// Four packed bf16 pairs -> eight E2M1 codes (element 0 in the lowest nibble).
__device__ __forceinline__ uint32_t cvt_e2m1x8_bf16(uint32_t p0, uint32_t p1, uint32_t p2,
                                                    uint32_t p3)
{
    uint32_t r;
    asm("{ .reg .b8 b0, b1, b2, b3;\n"
        "  .reg .f32 l0, h0, l1, h1, l2, h2, l3, h3;\n"
        "  shl.b32 l0, %1, 16;  and.b32 h0, %1, 0xFFFF0000;\n"
        "  shl.b32 l1, %2, 16;  and.b32 h1, %2, 0xFFFF0000;\n"
        "  shl.b32 l2, %3, 16;  and.b32 h2, %3, 0xFFFF0000;\n"
        "  shl.b32 l3, %4, 16;  and.b32 h3, %4, 0xFFFF0000;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b0, h0, l0;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b1, h1, l1;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b2, h2, l2;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b3, h3, l3;\n"
        "  mov.b32 %0, {b0, b1, b2, b3}; }"
        : "=r"(r)
        : "r"(p0), "r"(p1), "r"(p2), "r"(p3));
    return r;
}

// ---------------------------------------------------------------- bf16, contiguous: one lane per block
// Every per-block scalar (exponent, scale byte, multiplier, BM mantissa) is computed once
// instead of once per cooperating lane, and no shuffles are needed: a lane reads its block's
// 64 bytes with four 128-bit loads.  Neighbouring lanes' loads fall into the same 128-byte
// lines, which L1 serves; nibbles leave as one 128-bit store per lane (fully coalesced) and
// the scale / index bytes as 32 consecutive bytes per warp.
// What the kReady variant also writes: the operand in the form the streamed tensor-core GEMM
// reads (Sec. 5: quantization fused with the preparation of the matrix-multiply operand), i.e.
// what prepack_kernel would make of the packed planes: the scale byte inside its 32-row x
// 16-byte atom and either (kReady = 1) the block's 32 codes as E2M3 codes packed into 24 bytes,
// BM included, or (kReady = 2, MXFP4+ against a plain MXFP4 partner) Eq. 4's split for the
// sparse residual instruction: the codes with BM_H in the BM's place, BM_L 2:1 compressed,
// and the metadata nibbles that say where it sits.
struct GemmReady {
    uint8_t* atoms;      // [ceil(rows/128)][nbk/4][512]
    uint4* slots;        // kReady = 1: [rows][nbk] records of 24 bytes (32 E2M3 codes)
    uint4* sp_main;      // kReady = 2: [rows][nbk] codes with BM_H
    uint2* sp_res;       //             [rows][nbk] compressed BM_L
    uint8_t* sp_meta;    //             [row group of 128][stage of 8 blocks][128 rows x 16 bytes]
    int sp_stages;       //             stages per row (nbk / 8)
    int nbk;             // blocks per row
    StatusBlock* status; // zeroed here for the GEMM that follows
};

// One block of 32 bf16 values (x: sixteen pairs, element 0 in the low half of x[0]) -> its
// codes, scale byte and index byte, stored as block number `blk`.
template <int kMode, int kReady>
__device__ __forceinline__ void quantize_block_bf16(uint32_t (&x)[16], int64_t blk,
                                                    uint4* __restrict__ nibbles,
                                                    uint8_t* __restrict__ scales,
                                                    uint8_t* __restrict__ bm_index,
                                                    const GemmReady& ready)
{
    uint32_t t[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) t[i] = x[i] & 0x7FFF7FFFu;
    uint32_t m2 = bf16x2_max_nan(t[0], t[1]);
#pragma unroll
    for (int i = 2; i < 16; ++i) m2 = bf16x2_max_nan(m2, t[i]);
    m2 = bf16x2_max_nan(m2, __byte_perm(m2, m2, 0x1032));  // both halves = block maximum
    const uint32_t amax16 = m2 & 0xFFFFu;
    const uint32_t E = amax16 >> 7;
    const bool dead = E <= 2u || E == 255u;  // flushed or non-finite: data is all zero
    const uint32_t sb = E <= 2u ? 0u : (E == 255u ? 255u : E - 2u);
    constexpr bool kPlus = kMode >= 1;
    uint32_t bm = 0, m = 0, delta = 0;
    if (kPlus) {
        // one bit per element where |x| equals the maximum; lowest set bit = first BM
        uint32_t r1 = 0, r2 = 0;
        uint32_t eq[16];
#pragma unroll
        for (int i = 0; i < 16; ++i)
            asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(eq[i]) : "r"(t[i]), "r"(m2));
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t sel = (1u << (2 * i)) | (1u << (16 + 2 * i));
            r1 |= eq[i] & sel;
            r2 |= eq[8 + i] & sel;
        }
        // even elements sit in bits 0,2,..14, odd ones in bits 16,18,..30: interleave
        const uint32_t lo = (r1 & 0xFFFFu) | ((r1 >> 15) & 0xAAAAu);
        const uint32_t hi = (r2 & 0xFFFFu) | ((r2 >> 15) & 0xAAAAu);
        const uint32_t map = lo | (hi << 16);
        bm = (uint32_t)(__ffs((int)map) - 1) & 31u;
        const uint32_t mant = amax16 & 0x7Fu;
        m = min((mant + 7u + ((mant >> 4) & 1u)) >> 4, 7u);
        if (kMode == 2) {
            // MX++: largest magnitude among the NBMs.  Clearing every element equal to the
            // maximum leaves the smaller ones; if the maximum occurs twice it is an NBM too.
            uint32_t n2 = t[0] & ~eq[0];
#pragma unroll
            for (int i = 1; i < 16; ++i) n2 = bf16x2_max_nan(n2, t[i] & ~eq[i]);
            n2 = bf16x2_max_nan(n2, __byte_perm(n2, n2, 0x1032));
            const uint32_t a2 = (__popc(map) >= 2 ? amax16 : (n2 & 0xFFFFu)) << 16;
            delta = dead ? 0u : mxpp_delta(E, a2);
        }
    }
    // 2^-shared_exp(_new) as a bf16 pair: exponent field 256 - E + delta; beyond 254 (only
    // blocks near the bottom of the bf16 range) the factor is applied in two exact steps
    const uint32_t kexp = 256u - E + delta;
    const uint32_t inv2 = (min(kexp, 254u) << 7) * 0x00010001u;
    if (kMode == 2 && kexp > 254u) {
        const uint32_t up = ((127u + kexp - 254u) << 7) * 0x00010001u;
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = bf16x2_mul(x[i], up);
    }
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        w[i] = cvt_e2m1x8_bf16(bf16x2_mul(x[4 * i], inv2), bf16x2_mul(x[4 * i + 1], inv2),
                               bf16x2_mul(x[4 * i + 2], inv2), bf16x2_mul(x[4 * i + 3], inv2));
    if (kPlus) {
        // the BM's three mantissa bits over the exponent and mantissa bits of its code, in the
        // BM's word only: w[i] = (w[i] & ~field) | value under a predicate (no branch)
        const uint32_t sh = (bm & 7u) * 4u;
        const uint32_t field = 7u << sh, value = m << sh;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            asm("{ .reg .pred p;\n  setp.eq.u32 p, %1, %2;\n  @p lop3.b32 %0, %0, %3, %4, 0xBA; }"
                : "+r"(w[i]) : "r"(bm >> 3), "r"((uint32_t)i), "r"(field), "r"(value));
    }
    const uint4 outv = dead ? make_uint4(0, 0, 0, 0) : make_uint4(w[0], w[1], w[2], w[3]);
    __stcs(nibbles + blk, outv);
    scales[blk] = (uint8_t)sb;
    if (bm_index != nullptr) bm_index[blk] = (uint8_t)(dead ? 0u : (bm | (delta << 5)));
    if (kReady == 2) {
        static_assert(kReady != 2 || kMode == 1, "split output: MXFP4+ only");
        // Eq. 4: BM = BM_H + BM_L.  The BM's code in w[] is s m2 m1 m0.
        uint32_t mw[4] = {outv.x, outv.y, outv.z, outv.w};
        unsigned long long res = 0ull;
        uint32_t meta = 0x4444u;  // pairs 0 and 1 of every group of eight: all zeros
        if (!dead) {
            const uint32_t sh = (bm & 7u) * 4u, gi = bm >> 3, pair = (bm & 7u) >> 1;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (gi == (uint32_t)i) {
                    const uint32_t sign = (mw[i] >> sh) & 8u;
                    mw[i] = (mw[i] & ~(7u << sh)) | ((6u | (m >> 2)) << sh);  // BM_H: E2M1 code 11 m2
                    if (m & 3u)  // BM_L: E2M1 code 0 m1 m0 in the kept pair's slot
                        res = (unsigned long long)(sign | (m & 3u))
                              << (4u * (4u * gi + (pair == 3u ? 2u : 0u) + (bm & 1u)));
                }
            // the BM's group keeps the BM's pair and pair 3 (pairs 0 and 3 if the BM is in pair 3)
            meta = (meta & ~(15u << (4u * gi))) | ((pair == 3u ? 0xCu : (pair | 0xCu)) << (4u * gi));
        }
        __stcs(ready.sp_main + blk, make_uint4(mw[0], mw[1], mw[2], mw[3]));
        __stcs(ready.sp_res + blk, make_uint2((uint32_t)res, (uint32_t)(res >> 32)));
        // (block numbers fit 32 bits here: the launcher checks; a 64-bit division costs ~80 instructions)
        const uint32_t row = (uint32_t)blk / (uint32_t)ready.nbk;
        const int kb = (int)((uint32_t)blk - row * (uint32_t)ready.nbk);
        const int r = (int)(row & 127);
        *reinterpret_cast<uint16_t*>(ready.sp_meta + ((size_t)(row >> 7) * ready.sp_stages + (kb >> 3)) * 2048 + r * 16 +
                                     (kb & 7) * 2) = (uint16_t)meta;
        ready.atoms[((row >> 7) * (ready.nbk >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (kb & 3)] =
            (uint8_t)sb;
    }
    if (kReady == 1) {
        static_assert(kReady != 1 || kMode <= 1, "GEMM-ready output: MXFP4 and MXFP4+ only");
        // E2M1 code s e e m -> E2M3 code s e e m 0 0 (same exponent bias): a nibble times four,
        // one code per byte first (even and odd nibbles by two masks, interleaved by byte permutes)
        const uint32_t ov[4] = {outv.x, outv.y, outv.z, outv.w};
        uint32_t c[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t ev = (ov[i] << 2) & 0x3C3C3C3Cu, od = (ov[i] >> 2) & 0x3C3C3C3Cu;
            c[2 * i] = __byte_perm(ev, od, 0x5140);
            c[2 * i + 1] = __byte_perm(ev, od, 0x7362);
        }
        if (kPlus) {
            // Eq. 3's BM branch: 4 + m/2 is the E2M3 code s 11 mmm; the sign bit the cast wrote stays
            const uint32_t pos = 8u * (bm & 3u);
            const uint32_t field = 0x1Fu << pos, value = (0x18u | m) << pos;
            const uint32_t word = dead ? 8u : bm >> 2;  // (a dead block's codes are zero already)
#pragma unroll
            for (int i = 0; i < 8; ++i)
                asm("{ .reg .pred p;\n  setp.eq.u32 p, %1, %2;\n  @p lop3.b32 %0, %0, %3, %4, 0xBA; }"
                    : "+r"(c[i]) : "r"(word), "r"((uint32_t)i), "r"(field), "r"(value));
        }
        // 32 six-bit codes = 24 bytes (the GEMM's tensor map spreads every 12 into a 16-byte slot):
        // bytes a b c d -> a | b << 6 | c << 12 | d << 18 by two bit-selects, then byte permutes
        uint32_t g[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t q = (c[i] & 0x003F003Fu) | ((c[i] >> 2) & ~0x003F003Fu);
            g[i] = (q & 0xFFFu) | ((q >> 4) & ~0xFFFu);
        }
        uint2* out6 = reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(ready.slots) + blk * 24);
        __stcs(out6, make_uint2(__byte_perm(g[0], g[1], 0x4210), __byte_perm(g[1], g[2], 0x5421)));
        __stcs(out6 + 1, make_uint2(__byte_perm(g[2], g[3], 0x6542), __byte_perm(g[4], g[5], 0x4210)));
        __stcs(out6 + 2, make_uint2(__byte_perm(g[5], g[6], 0x5421), __byte_perm(g[6], g[7], 0x6542)));
        const uint32_t row = (uint32_t)blk / (uint32_t)ready.nbk;
        const int kb = (int)((uint32_t)blk - row * (uint32_t)ready.nbk);
        const int r = (int)(row & 127);
        ready.atoms[((size_t)(row >> 7) * (ready.nbk >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (kb & 3)] =
            (uint8_t)sb;
    }
}

template <int kMode, int kReady>
__global__ void __launch_bounds__(kThreads)
quantize_bf16_lane_kernel(const uint4* __restrict__ src, int64_t total_blocks,
                          uint4* __restrict__ nibbles, uint8_t* __restrict__ scales,
                          uint8_t* __restrict__ bm_index, const GemmReady ready)
{
    const int64_t blk = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (kReady && blk == 0 && ready.status != nullptr) {
        ready.status->code = 0u;
        ready.status->where = 0u;
    }
    if (blk >= total_blocks) return;
    const uint4* p = src + blk * 4;
    uint32_t x[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 v = __ldg(p + i);
        x[4 * i] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
    }
    quantize_block_bf16<kMode, kReady>(x, blk, nibbles, scales, bm_index, ready);
}

// Channel reordering fused into the bf16 quantizer (Sec. 8, "Scattering outliers with channel
// reordering"), one lane per block as above.  A CTA keeps the ordering in shared memory for
// its whole life (clamped into the row once, and laid out so that the lanes of a warp read
// neighbouring 16-byte vectors) and copies one source row at a time with coalesced 16-byte
// loads; a lane then picks its block's 32 channels out of shared memory, where an arbitrary
// ordering costs bank conflicts instead of a 128-byte line per element.  Rows are dealt to
// the CTAs round robin; several CTAs per SM overlap one's row copy with another's casts.
// Shared memory: two rows of cols ushort + cols ushort for the ordering (cols <= 65536).
template <int kMode>
__global__ void __launch_bounds__(kThreads)
quantize_bf16_reordered_kernel(const __nv_bfloat16* __restrict__ src, int64_t ld_src, int64_t rows,
                               int cols_blocks, const int32_t* __restrict__ order,
                               uint4* __restrict__ nibbles, uint8_t* __restrict__ scales,
                               uint8_t* __restrict__ bm_index)
{
    extern __shared__ uint4 dyn_smem[];
    const int cols = cols_blocks * 32;
    // (no array of row pointers: a pointer picked from an array at run time makes the gather's
    // loads generic ones, with 64-bit address arithmetic for each)
    const uint32_t row_sa[2] = {(uint32_t)__cvta_generic_to_shared(dyn_smem),
                                (uint32_t)__cvta_generic_to_shared(dyn_smem) + 2u * (uint32_t)cols};
    unsigned short* ord_s = reinterpret_cast<unsigned short*>(dyn_smem) + 2 * cols;
    constexpr int kPerVec = 8;  // ordering entries per 16-byte vector
    constexpr int kVecs = 4;    // vectors per block
    // ordering entry e of block b sits in vector (e / kPerVec) * cols_blocks + b
    const uint32_t last = (uint32_t)(cols - 1);
    for (int c = threadIdx.x; c < cols; c += kThreads) {
        const int b = c >> 5, e = c & 31;
        ord_s[((e / kPerVec) * cols_blocks + b) * kPerVec + e % kPerVec] =
            (unsigned short)min((uint32_t)__ldg(order + c), last);
    }
    const int vecs = cols / 8;
    const GemmReady none{};
    // two row buffers filled with asynchronous 16-byte copies: the next row is on its way
    // while this one is cast
    auto fetch = [&](int64_t row, int buf) {
        if (row < rows) {
            const uint4* src_row = reinterpret_cast<const uint4*>(src + row * ld_src);
            const uint32_t dst = buf ? row_sa[1] : row_sa[0];
            for (int i = threadIdx.x; i < vecs; i += kThreads)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * (uint32_t)i),
                             "l"(src_row + i)
                             : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    fetch(blockIdx.x, 0);
    int it = 0;
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x, ++it) {
        fetch(row + gridDim.x, (it + 1) & 1);
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        __syncthreads();  // this row has landed for every thread (first pass: the ordering too)
        const unsigned short* row_s = reinterpret_cast<const unsigned short*>(dyn_smem) + ((it & 1) ? cols : 0);
        for (int b = threadIdx.x; b < cols_blocks; b += kThreads) {
            uint32_t x[16];
#pragma unroll
            for (int k = 0; k < kVecs; ++k) {
                const uint4 o = reinterpret_cast<const uint4*>(ord_s)[k * cols_blocks + b];
                const uint32_t ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    x[4 * k + i] = __byte_perm((uint32_t)row_s[ow[i] & 0xFFFFu], (uint32_t)row_s[ow[i] >> 16], 0x5410);
            }
            quantize_block_bf16<kMode, 0>(x, row * cols_blocks + b, nibbles, scales, bm_index, none);
        }
        __syncthreads();  // all reads of this buffer are done before the next pass refills it
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ------------------------------------------------------------------------- decode (Eq. 3)
// One thread decodes eight elements (one 32-bit word of nibbles).
__device__ __forceinline__ float e2m1_mag(uint32_t code)
{
    // 0, .5, 1, 1.5, 2, 3, 4, 6: subnormal step 0.5 below 1, then 1.m * 2^(e-1)
    const uint32_t e = code >> 1, m = code & 1u;
    const float normal = __uint_as_float(((126u + e) << 23) | (m << 22));
    return e == 0u ? 0.5f * (float)m : normal;
}

template <typename T, int kMode>
__global__ void __launch_bounds__(kThreads)
dequantize_kernel(const uint8_t* __restrict__ nibbles, const uint8_t* __restrict__ scales,
                  const uint8_t* __restrict__ bm_index, int64_t cols, int64_t total_units,
                  T* __restrict__ dst, int64_t ld_dst)
{
    const int64_t u = (int64_t)blockIdx.x * kThreads + threadIdx.x;  // unit of 8 elements
    if (u >= total_units) return;
    const int64_t blk = u >> 2;
    const int q = (int)(u & 3);
    const uint32_t word = __ldg(reinterpret_cast<const uint32_t*>(nibbles) + u);
    const uint32_t sb = scales[blk];
    constexpr bool kPlus = kMode >= 1;
    const uint32_t ib = kPlus ? bm_index[blk] : 0u;
    const int bm = kPlus ? (int)(ib & 31u) : -1;
    float out[8];
    // 2^(sb - 127) for sb in 1..254; sb = 0 is the reserved all-zero block; 0xFF decodes NaN
    const float scale = __uint_as_float(sb << 23);
    // MX++: the NBMs' shared exponent lies delta below (the product may be subnormal: exact)
    const float scale_nbm = kMode == 2 ? scale * __uint_as_float((127u - (ib >> 5)) << 23) : scale;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t n = (word >> (4 * i)) & 15u;
        const uint32_t code = n & 7u;
        const bool is_bm = kPlus && q * 8 + i == bm;
        const float mag = is_bm ? 4.0f + 0.5f * (float)code : e2m1_mag(code);  // "MX+ addition"
        float val = mag * (is_bm ? scale : scale_nbm);  // exact: <= 4 significant bits times 2^k
        if (sb == 0u) val = 0.0f;
        if (sb == 255u) val = __uint_as_float(0x7FC00000u);
        out[i] = (n & 8u) ? -val : val;
    }
    const int64_t e0 = u * 8;
    const int64_t row = e0 / cols;
    const int64_t off = row * ld_dst + (e0 - row * cols);
    if (sizeof(T) == 4) {
        float4* p = reinterpret_cast<float4*>(reinterpret_cast<float*>(dst) + off);
        p[0] = make_float4(out[0], out[1], out[2], out[3]);
        p[1] = make_float4(out[4], out[5], out[6], out[7]);
    } else {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(out[2 * i], out[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(dst) + off) =
            make_uint4(w[0], w[1], w[2], w[3]);
    }
}

template <typename T, int kMode>
cudaError_t launch_q(const void* src, int64_t rows, int64_t cols, int64_t ld_src,
                     uint8_t* nibbles, uint8_t* scales, uint8_t* bm_index, cudaStream_t stream)
{
    const int64_t total_blocks = rows * (cols / 32);
    const int64_t grid = (total_blocks + kBlocksPerCta - 1) / kBlocksPerCta;
    const int aligned4 = ((reinterpret_cast<uintptr_t>(scales) & 3) == 0) &&
                         ((reinterpret_cast<uintptr_t>(bm_index) & 3) == 0);
    if (ld_src == cols && sizeof(T) == 2)
        quantize_bf16_lane_kernel<kMode, 0>
            <<<(unsigned)((total_blocks + kThreads - 1) / kThreads), kThreads, 0, stream>>>(
                static_cast<const uint4*>(src), total_blocks, reinterpret_cast<uint4*>(nibbles),
                scales, bm_index, GemmReady{});
    else if (ld_src == cols)
        quantize_kernel<T, kMode, true><<<(unsigned)grid, kThreads, 0, stream>>>(
            static_cast<const T*>(src), ld_src, cols / 32, total_blocks, nibbles, scales,
            bm_index, aligned4);
    else
        quantize_kernel<T, kMode, false><<<(unsigned)grid, kThreads, 0, stream>>>(
            static_cast<const T*>(src), ld_src, cols / 32, total_blocks, nibbles, scales,
            bm_index, aligned4);
    return cudaGetLastError();
}

template <typename T, int kMode>
cudaError_t launch_q_reordered(const void* src, int64_t rows, int64_t cols, int64_t ld_src,
                               const int32_t* order, uint8_t* nibbles, uint8_t* scales,
                               uint8_t* bm_index, cudaStream_t stream)
{
    const int64_t total_blocks = rows * (cols / 32);
    const int64_t grid = (total_blocks + kBlocksPerCta - 1) / kBlocksPerCta;
    const int aligned4 = ((reinterpret_cast<uintptr_t>(scales) & 3) == 0) &&
                         ((reinterpret_cast<uintptr_t>(bm_index) & 3) == 0);
    const size_t row_bytes = (size_t)cols * sizeof(T);
    const bool vec_rows = (reinterpret_cast<uintptr_t>(src) & 15) == 0 &&
                          (ld_src * sizeof(T)) % 16 == 0;
    const int sms = sm_count();
    if (sizeof(T) == 2 && vec_rows && sms > 0 && (reinterpret_cast<uintptr_t>(nibbles) & 15) == 0) {
        // two rows and the ordering as 16-bit entries: cols <= 34112 fits, wider rows take the
        // path below
        const size_t smem = (size_t)cols * 6;
        if (smem <= 200 * 1024) {
            int per_sm = (int)((200 * 1024) / smem);
            if (per_sm > 6) per_sm = 6;
            int64_t ctas = (int64_t)sms * per_sm;
            if (ctas > rows) ctas = rows;
            auto kern = quantize_bf16_reordered_kernel<kMode>;
            static SmemAttrOnce once;
            const cudaError_t ea = ensure_dynamic_smem(kern, 200 * 1024, once);
            if (ea != cudaSuccess) return ea;
            kern<<<(unsigned)ctas, kThreads, smem, stream>>>(
                static_cast<const __nv_bfloat16*>(src), ld_src, rows, (int)(cols / 32), order,
                reinterpret_cast<uint4*>(nibbles), scales, bm_index);
            return cudaGetLastError();
        }
    }
    if (vec_rows && row_bytes <= 200 * 1024 && sms > 0) {
        auto kern = quantize_reordered_staged_kernel<T, kMode>;
        static SmemAttrOnce once;
        const cudaError_t ea = ensure_dynamic_smem(kern, 200 * 1024, once);
        if (ea != cudaSuccess) return ea;
        int per_sm = (int)((200 * 1024) / row_bytes);
        if (per_sm > 6) per_sm = 6;
        int64_t ctas = (int64_t)sms * per_sm;
        if (ctas > rows) ctas = rows;
        kern<<<(unsigned)ctas, kThreads, row_bytes, stream>>>(
            static_cast<const T*>(src), ld_src, rows, (int)(cols / 32), order, nibbles, scales,
            bm_index, aligned4 && (cols / 32) % 4 == 0);
        return cudaGetLastError();
    }
    quantize_kernel<T, kMode, false, true><<<(unsigned)grid, kThreads, 0, stream>>>(
        static_cast<const T*>(src), ld_src, cols / 32, total_blocks, nibbles, scales, bm_index,
        aligned4, order);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_quantize_reordered(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                                      int64_t ld_src, const int32_t* order, mxp_mode mode,
                                      uint8_t* nibbles, uint8_t* scales, uint8_t* bm_index,
                                      cudaStream_t stream)
{
#define MXP_QR(T, MODE) \
    launch_q_reordered<T, MODE>(src, rows, cols, ld_src, order, nibbles, scales, bm_index, stream)
    if (dt == MXP_BF16) {
        if (mode == MXP_MODE_MXFP4_PP) return MXP_QR(__nv_bfloat16, 2);
        if (mode == MXP_MODE_MXFP4_PLUS) return MXP_QR(__nv_bfloat16, 1);
        return MXP_QR(__nv_bfloat16, 0);
    }
    if (mode == MXP_MODE_MXFP4_PP) return MXP_QR(float, 2);
    if (mode == MXP_MODE_MXFP4_PLUS) return MXP_QR(float, 1);
    return MXP_QR(float, 0);
#undef MXP_QR
}

// bf16, contiguous rows, MXFP4 / MXFP4+: quantize and write the GEMM-ready form as well
// (`slots`: widened codes; or, with `split` given instead, Eq. 4's split of an MXFP4+ operand).
cudaError_t launch_quantize_ready(const void* src, int64_t rows, int64_t cols, mxp_mode mode,
                                  uint8_t* nibbles, uint8_t* scales, uint8_t* bm_index,
                                  uint8_t* atoms, uint8_t* slots, const QuantizeSplitOut* split, void* status,
                                  cudaStream_t stream)
{
    const int64_t total_blocks = rows * (cols / 32);
    if (total_blocks >= (1ll << 32)) return cudaErrorNotSupported;  // the kernel's block numbers are 32-bit
    GemmReady ready = {};
    ready.atoms = atoms;
    ready.slots = reinterpret_cast<uint4*>(slots);
    ready.nbk = (int)(cols / 32);
    ready.status = static_cast<StatusBlock*>(status);
    const unsigned grid = (unsigned)((total_blocks + kThreads - 1) / kThreads);
    if (split != nullptr) {
        if (mode != MXP_MODE_MXFP4_PLUS || cols % 256 != 0) return cudaErrorNotSupported;
        ready.sp_main = reinterpret_cast<uint4*>(split->main);
        ready.sp_res = reinterpret_cast<uint2*>(split->res);
        ready.sp_meta = split->meta;
        ready.sp_stages = (int)(cols / 256);
        // rows past the operand's end inside its last row groups: metadata only, every nibble valid
        if (split->meta_pad_bytes != 0 &&
            cudaMemsetAsync(split->meta + split->meta_pad_offset, 0x44, split->meta_pad_bytes, stream) != cudaSuccess)
            return cudaErrorUnknown;
        quantize_bf16_lane_kernel<1, 2><<<grid, kThreads, 0, stream>>>(
            static_cast<const uint4*>(src), total_blocks, reinterpret_cast<uint4*>(nibbles), scales,
            bm_index, ready);
    } else if (mode == MXP_MODE_MXFP4_PLUS)
        quantize_bf16_lane_kernel<1, 1><<<grid, kThreads, 0, stream>>>(
            static_cast<const uint4*>(src), total_blocks, reinterpret_cast<uint4*>(nibbles), scales,
            bm_index, ready);
    else
        quantize_bf16_lane_kernel<0, 1><<<grid, kThreads, 0, stream>>>(
            static_cast<const uint4*>(src), total_blocks, reinterpret_cast<uint4*>(nibbles), scales,
            bm_index, ready);
    return cudaGetLastError();
}

cudaError_t launch_quantize(const void* src, mxp_dtype dt, int64_t rows, int64_t cols,
                            int64_t ld_src, mxp_mode mode, uint8_t* nibbles, uint8_t* scales,
                            uint8_t* bm_index, cudaStream_t stream)
{
    if (dt == MXP_BF16) {
        switch (mode) {
            case MXP_MODE_MXFP4_PP:
                return launch_q<__nv_bfloat16, 2>(src, rows, cols, ld_src, nibbles, scales, bm_index, stream);
            case MXP_MODE_MXFP4_PLUS:
                return launch_q<__nv_bfloat16, 1>(src, rows, cols, ld_src, nibbles, scales, bm_index, stream);
            default:
                return launch_q<__nv_bfloat16, 0>(src, rows, cols, ld_src, nibbles, scales, bm_index, stream);
        }
    }
    switch (mode) {
        case MXP_MODE_MXFP4_PP:
            return launch_q<float, 2>(src, rows, cols, ld_src, nibbles, scales, bm_index, stream);
        case MXP_MODE_MXFP4_PLUS:
            return launch_q<float, 1>(src, rows, cols, ld_src, nibbles, scales, bm_index, stream);
        default:
            return launch_q<float, 0>(src, rows, cols, ld_src, nibbles, scales, bm_index, stream);
    }
}

template <typename T>
static cudaError_t launch_dq(const mxp_packed& p, T* dst, int64_t ld_dst, cudaStream_t stream)
{
    const int64_t units = p.rows * p.cols / 8;
    const unsigned grid = (unsigned)((units + kThreads - 1) / kThreads);
    switch (p.mode) {
        case MXP_MODE_MXFP4_PP:
            dequantize_kernel<T, 2><<<grid, kThreads, 0, stream>>>(p.nibbles, p.scales, p.bm_index,
                                                                   p.cols, units, dst, ld_dst);
            break;
        case MXP_MODE_MXFP4_PLUS:
            dequantize_kernel<T, 1><<<grid, kThreads, 0, stream>>>(p.nibbles, p.scales, p.bm_index,
                                                                   p.cols, units, dst, ld_dst);
            break;
        default:
            dequantize_kernel<T, 0><<<grid, kThreads, 0, stream>>>(p.nibbles, p.scales, p.bm_index,
                                                                   p.cols, units, dst, ld_dst);
    }
    return cudaGetLastError();
}

cudaError_t launch_dequantize(const mxp_packed& p, void* dst, mxp_dtype dt, int64_t ld_dst,
                              cudaStream_t stream)
{
    if (dt == MXP_F32) return launch_dq(p, static_cast<float*>(dst), ld_dst, stream);
    return launch_dq(p, static_cast<__nv_bfloat16*>(dst), ld_dst, stream);
}

}  // namespace mxp
