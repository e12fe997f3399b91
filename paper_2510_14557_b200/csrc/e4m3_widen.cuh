// E2M1 / MX+ / MX++ codes as E2M3 codes or E4M3 bytes: what the kernels that run
// kind::mxf8f6f4 on widened operands share.  Both types hold every E2M1 value and the BM values
// 4 + m/2 of Eq. 3 exactly; E4M3 also their power-of-two multiples used for MX++.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mxp {

// MX++ (Sec. 4.3): the tensor core gets one scale per block, the NBMs' shared exponent lies
// delta below the BM's.  The block is handed over with scale 2^(shared_exp - t),
// t = min(delta, 5, scale byte - 1): the BM becomes (4 + m/2) * 2^t (at most 240, an E4M3
// value), the NBMs E2M1 * 2^-(delta - t) (E4M3 values down to 2^-8): everything stays exact.
__device__ __forceinline__ uint32_t mxpp_shift(uint32_t scale_byte, uint32_t delta)
{
    if (scale_byte == 0u || scale_byte == 255u) return 0u;
    return min(min(delta, 5u), scale_byte - 1u);
}

// E4M3 byte of an E2M1 magnitude code (0, .5, 1, 1.5, 2, 3, 4, 6) times 2^-j, j = 0..7:
// normal while the value is at least 2^-6, a multiple of 2^-9 below.
constexpr uint32_t e4m3_of_code_shifted(int code, int j)
{
    const int e = code >> 1, m = code & 1;
    if (code == 0) return 0u;
    // value = (e ? (2 + m) << (e - 1) : m) / 2 halves -> in units of 2^-9: times 2^(8 - j)
    const int num = (e ? (2 + m) << (e - 1) : m);  // value * 2
    const int units = j <= 8 ? num << (8 - j) : 0; // value * 2^-j in units of 2^-9
    if (units < 8) return (uint32_t)units;          // subnormal
    int ex = 0, u = units;
    while (u >= 16) { u >>= 1; ++ex; }              // u in [8, 16): 1.mmm
    return (uint32_t)(((ex + 1) << 3) | (u & 7));
}
constexpr uint32_t e4m3_lut_word(int j, int hi)
{
    return e4m3_of_code_shifted(4 * hi + 0, j) | (e4m3_of_code_shifted(4 * hi + 1, j) << 8) |
           (e4m3_of_code_shifted(4 * hi + 2, j) << 16) | (e4m3_of_code_shifted(4 * hi + 3, j) << 24);
}
static_assert(e4m3_lut_word(0, 0) == 0x3C383000u && e4m3_lut_word(0, 1) == 0x4C484440u, "E4M3 table");
static __constant__ uint2 kE4m3Lut[8] = {
    {e4m3_lut_word(0, 0), e4m3_lut_word(0, 1)}, {e4m3_lut_word(1, 0), e4m3_lut_word(1, 1)},
    {e4m3_lut_word(2, 0), e4m3_lut_word(2, 1)}, {e4m3_lut_word(3, 0), e4m3_lut_word(3, 1)},
    {e4m3_lut_word(4, 0), e4m3_lut_word(4, 1)}, {e4m3_lut_word(5, 0), e4m3_lut_word(5, 1)},
    {e4m3_lut_word(6, 0), e4m3_lut_word(6, 1)}, {e4m3_lut_word(7, 0), e4m3_lut_word(7, 1)}};

// Four E2M1 codes (low 16 bits of x) -> four E4M3 bytes.  Magnitude: byte table lookup with
// the codes' low three bits as selector.  Sign: a second lookup with the raw codes as selector
// uses prmt's sign-replicate mode (selector bit 3): it returns 0xFF for a negative code and a
// table byte whose bit 0 is clear for a positive one, so bit 0 of each byte is the sign.
// `lut`: the magnitude table, kE4m3Lut[j] for codes scaled by 2^-j.
__device__ __forceinline__ uint32_t e2m1x4_to_e4m3x4(uint32_t x, uint2 lut = make_uint2(0x3C383000u, 0x4C484440u))
{
    const uint32_t mag = __byte_perm(lut.x, lut.y, x & 0x7777u);
    uint32_t neg;  // PTX prmt (not the intrinsic, which defines only three selector bits)
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(neg) : "r"(0x80808080u), "r"(x));
    return mag | ((neg << 7) & 0x80808080u);
}

// Eight E2M1 codes (nibble i of x) -> eight E2M3 codes, 6 bits each, code i at bits 6i..6i+5.
// Both formats have exponent bias 1, so the E2M3 code of an E2M1 value is its code with two
// zero mantissa bits appended: s e e m -> s e e m 0 0.  The nibbles are spread from a pitch of
// 4 bits to a pitch of 6 in three steps (by 8, 4 and 2 bits for bits 2, 1 and 0 of i).
__device__ __forceinline__ uint64_t e2m1x8_to_e2m3x8(uint32_t x)
{
    uint64_t y = x;
    y = (y & 0x000000000000FFFFull) | ((y & 0x00000000FFFF0000ull) << 8);
    y = (y & 0x00000000FF0000FFull) | ((y & 0x000000FF0000FF00ull) << 4);
    y = (y & 0x000000F00F00F00Full) | ((y & 0x00000F00F00F00F0ull) << 2);
    return y << 2;
}

// Sixteen E2M1 codes of an MXFP4 / MXFP4+ half block (w0: codes 0-7, w1: codes 8-15) as the
// 16-byte slot kind::mxf8f6f4 reads: sixteen E2M3 codes in 12 bytes, 4 bytes of padding.  bm_pos
// (0..15, or >= 16 for none): that code is the BM of an MX+ block, stored as s m2 m1 m0 and
// meaning 4 + m/2 (Eq. 3): E2M3 code s 11 mmm.
__device__ __forceinline__ uint4 e2m1x16_to_e2m3_slot(uint32_t w0, uint32_t w1, uint32_t bm_pos)
{
    unsigned long long lo = e2m1x8_to_e2m3x8(w0), hi = e2m1x8_to_e2m3x8(w1);
    if (bm_pos < 16u) {
        const uint32_t nib = (((bm_pos & 8u) ? w1 : w0) >> ((bm_pos & 7u) * 4u)) & 15u;
        const uint32_t sh = 6u * (bm_pos & 7u);
        const unsigned long long code = ((nib & 8u) << 2) | 0x18u | (nib & 7u);
        if (bm_pos & 8u)
            hi = (hi & ~(0x3Full << sh)) | (code << sh);
        else
            lo = (lo & ~(0x3Full << sh)) | (code << sh);
    }
    return make_uint4((uint32_t)lo, (uint32_t)(lo >> 32) | ((uint32_t)hi << 16), (uint32_t)(hi >> 16), 0u);
}

}  // namespace mxp
