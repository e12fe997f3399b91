// Weight-only GEMM: D[M,N] = A(bf16)[M,K] * dec(W)[N,K]^T, W in MXFP4 / MXFP4+.
//
// This is the paper's "conversion before computation" scenario (Sec. 7.1, Eq. 3): weights
// are decoded to bf16 inside the matmul kernel and multiplied on bf16 tensor cores, fp32
// accumulation.  For decode-sized M the kernel is a stream over W, so the layout follows
// the bytes: one lane loads one whole 32-element block (16 bytes) of two weight rows per
// pass, decodes it in registers and feeds it to mma.m16n8k16 with W as the 16-row operand.
//
// Decode trick: the bf16 bit pattern (code << 6) has the E2M1 exponent/mantissa bits in the
// low exponent/top mantissa positions, i.e. it *is* the E2M1 value times 2^-126, subnormals
// included.  One packed bf16x2 multiply by 2^(126 + shared_exp) then yields the decoded
// weight exactly.  The BM element of an MX+ block has the pattern 0x180 | (m << 4)
// (= (4 + m/2) * 2^-126), patched in before the multiply: this is Eq. 3's BM branch.
#include <cuda_bf16.h>

#include <cstdlib>

#include "common.cuh"

namespace mxp {
namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kRowsPerCta = 16;

__device__ __forceinline__ uint32_t hmul2_bf16(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Decode one block (four words of nibbles) into 16 bf16x2 registers.  Register 4w + i holds
// elements (8w + i, 8w + i + 4): the two nibbles sit 16 bits apart, so one shift and mask
// places both codes.
// kMode: 0 MXFP4, 1 MXFP4+, 2 MX++ (Sec. 4.3: bits 7:5 of the index byte `bm` hold delta; the
// NBMs' shared exponent lies delta below the block's, so the BM is entered 2^delta larger).
template <int kMode>
__device__ __forceinline__ void decode_block(const uint4 nib, uint32_t sb, uint32_t bm,
                                             uint32_t (&out)[16])
{
    constexpr bool kPlus = kMode >= 1;
    const uint32_t delta = kMode == 2 ? (bm >> 5) : 0u;
    const uint32_t w[4] = {nib.x, nib.y, nib.z, nib.w};
    // Left shifts are written as multiplies so that they issue on the FMA pipe (IMAD) and
    // leave the integer ALU pipe, which this kernel saturates first, to the mask / merge ops.
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t x = w[j];
        out[4 * j + 0] = ((x * 64u) & 0x01C001C0u) | ((x * 4096u) & 0x80008000u);
        out[4 * j + 1] = ((x * 4u) & 0x01C001C0u) | ((x * 256u) & 0x80008000u);
        out[4 * j + 2] = ((x >> 2) & 0x01C001C0u) | ((x * 16u) & 0x80008000u);
        out[4 * j + 3] = ((x >> 6) & 0x01C001C0u) | (x & 0x80008000u);
    }
    if (kPlus) {
        // element p lives in register 4*(p>>3) + (p&3), upper half if bit 2 of p is set
        const uint32_t p = bm & 31u;
        const uint32_t word = (p & 16u) ? ((p & 8u) ? w[3] : w[2]) : ((p & 8u) ? w[1] : w[0]);
        const uint32_t n = (word >> ((p & 7u) * 4u)) & 15u;
        const uint32_t pat =
            (0x180u + (delta << 7)) | ((n & 7u) << 4) | ((n & 8u) << 12);  // (4 + m/2) * 2^(delta - 126)
        const uint32_t reg = ((p >> 3) << 2) | (p & 3u);
        const bool upper = (p & 4u) != 0u;
        const uint32_t keep = upper ? 0x0000FFFFu : 0xFFFF0000u;
        const uint32_t ins = upper ? (pat << 16) : pat;
#pragma unroll
        for (int r = 0; r < 16; ++r)
            if (reg == (uint32_t)r) out[r] = (out[r] & keep) | ins;
    }
    // multiplier 2^(126 + shared_exp) = 2^(sb - 1): bf16 exponent field 126 + sb.  It tops
    // out at 254; the remainder goes into a second multiply (only for blocks with |x| >= 16).
    // (MX++: 126 + sb - delta; below 1 only for blocks at the very bottom of the range)
    const int total = 126 + (int)sb - (int)delta;
    const uint32_t e1 = (uint32_t)min(max(total, 1), 254);
    uint32_t m1 = (e1 << 7) * 0x00010001u;
    if (sb == 0u) m1 = 0u;                 // reserved scale: the whole block is zero
    if (sb == 255u) m1 = 0x7FC07FC0u;      // non-finite marker decodes to NaN
#pragma unroll
    for (int r = 0; r < 16; ++r) out[r] = hmul2_bf16(out[r], m1);
    if (__any_sync(0xFFFFFFFFu, total != (int)e1 && sb != 255u && sb != 0u)) {
        const uint32_t e2 = (uint32_t)(127 + total - (int)e1);
        const uint32_t m2 = (sb == 255u ? 0x3F80u : (e2 << 7)) * 0x00010001u;
#pragma unroll
        for (int r = 0; r < 16; ++r) out[r] = hmul2_bf16(out[r], m2);
    }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// kMT: number of 8-column activation tiles (M <= 8 * kMT handled per CTA pass).
template <int kMT, int kMode, typename OutT>
__global__ void __launch_bounds__(kThreads)
gemm_wo_kernel(int M, int N, int K, const __nv_bfloat16* __restrict__ A, int64_t lda,
               const uint8_t* __restrict__ nibbles, const uint8_t* __restrict__ scales,
               const uint8_t* __restrict__ bm_index, OutT* __restrict__ D, int64_t ldd)
{
    constexpr bool kPlus = kMode >= 1;
    __shared__ float red[kWarps][kRowsPerCta][8 * kMT + 1];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int n0 = blockIdx.x * kRowsPerCta;
    const int m0 = blockIdx.y * (8 * kMT);
    const int nb = K / 32;
    const int rowA = min(n0 + g, N - 1), rowB = min(n0 + g + 8, N - 1);
    const uint8_t* nibA = nibbles + (int64_t)rowA * (K / 2);
    const uint8_t* nibB = nibbles + (int64_t)rowB * (K / 2);
    const uint8_t* scA = scales + (int64_t)rowA * nb;
    const uint8_t* scB = scales + (int64_t)rowB * nb;
    const uint8_t* ixA = kPlus ? bm_index + (int64_t)rowA * nb : nullptr;
    const uint8_t* ixB = kPlus ? bm_index + (int64_t)rowB * nb : nullptr;

    float acc[kMT][4];
#pragma unroll
    for (int i = 0; i < kMT; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const int chunks = (nb + 3) / 4;
    // per-lane byte offsets of this lane's first block (4 * warp + t) in the two weight rows
    const uint8_t* pA = nibA + (int64_t)(4 * warp + t) * 16;
    const uint8_t* pB = nibB + (int64_t)(4 * warp + t) * 16;
    const __nv_bfloat16* aBase = A + (int64_t)(4 * warp + t) * 32;

    // Software pipeline: the weight bytes of the following chunk are requested before the
    // current one is decoded, so every warp keeps two chunks of W in flight.
    uint4 wa = make_uint4(0, 0, 0, 0), wb = wa;
    uint32_t sa = 0, sbb = 0, ia = 0, ib = 0;
    auto fetch = [&](int c) {
        const int b = 4 * c + t;
        wa = wb = make_uint4(0, 0, 0, 0);
        sa = sbb = ia = ib = 0;
        if (b < nb) {
            const int64_t off = (int64_t)(c - warp) * 64;  // 4 blocks x 16 bytes per chunk
            wa = __ldcs(reinterpret_cast<const uint4*>(pA + off));
            wb = __ldcs(reinterpret_cast<const uint4*>(pB + off));
            sa = scA[b];
            sbb = scB[b];
            if (kPlus) {
                ia = ixA[b];
                ib = ixB[b];
            }
        }
    };
    if (warp < chunks) fetch(warp);
    for (int c = warp; c < chunks; c += kWarps) {
        const int b = 4 * c + t;  // this lane's block within the row
        const bool live = b < nb;
        const uint4 cwa = wa, cwb = wb;
        const uint32_t csa = sa, csb = sbb, cia = ia, cib = ib;
        if (c + kWarps < chunks) fetch(c + kWarps);
        // activations of this lane's block for column m = 8*mt + g, pair-permuted to match
        uint32_t q[kMT][16];
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt) {
            const int m = m0 + 8 * mt + g;
            const bool ok = live && m < M;
            const uint4* ap =
                reinterpret_cast<const uint4*>(aBase + (int64_t)m * lda + (int64_t)(c - warp) * 128);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 x = make_uint4(0, 0, 0, 0);
                if (ok) x = __ldg(ap + j);
                q[mt][4 * j + 0] = prmt(x.x, x.z, 0x5410u);
                q[mt][4 * j + 1] = prmt(x.x, x.z, 0x7632u);
                q[mt][4 * j + 2] = prmt(x.y, x.w, 0x5410u);
                q[mt][4 * j + 3] = prmt(x.y, x.w, 0x7632u);
            }
        }
        uint32_t pa[16], pb[16];
        decode_block<kMode>(cwa, csa, cia, pa);
        decode_block<kMode>(cwb, csb, cib, pb);
#pragma unroll
        for (int s = 0; s < 8; ++s) {
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt)
                mma_bf16_16816(acc[mt], pa[2 * s], pb[2 * s], pa[2 * s + 1], pb[2 * s + 1],
                               q[mt][2 * s], q[mt][2 * s + 1]);
        }
    }

    // cross-warp reduction (fixed order -> deterministic), then store
#pragma unroll
    for (int mt = 0; mt < kMT; ++mt) {
        red[warp][g][8 * mt + 2 * t] = acc[mt][0];
        red[warp][g][8 * mt + 2 * t + 1] = acc[mt][1];
        red[warp][g + 8][8 * mt + 2 * t] = acc[mt][2];
        red[warp][g + 8][8 * mt + 2 * t + 1] = acc[mt][3];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < kRowsPerCta * 8 * kMT; e += kThreads) {
        const int r = e % kRowsPerCta, mcol = e / kRowsPerCta;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += red[w][r][mcol];
        const int n = n0 + r, m = m0 + mcol;
        if (n < N && m < M) {
            if (sizeof(OutT) == 4)
                reinterpret_cast<float*>(D)[(int64_t)m * ldd + n] = s;
            else
                reinterpret_cast<__nv_bfloat16*>(D)[(int64_t)m * ldd + n] = __float2bfloat16_rn(s);
        }
    }
}

template <int kMT, int kMode, typename OutT>
void launch(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const mxp_packed& B,
            void* D, int64_t ldd, cudaStream_t stream)
{
    dim3 grid((unsigned)((N + kRowsPerCta - 1) / kRowsPerCta),
              (unsigned)((M + 8 * kMT - 1) / (8 * kMT)));
    gemm_wo_kernel<kMT, kMode, OutT><<<grid, kThreads, 0, stream>>>(
        (int)M, (int)N, (int)K, static_cast<const __nv_bfloat16*>(A), lda, B.nibbles, B.scales,
        B.bm_index, static_cast<OutT*>(D), ldd);
}

template <int kMode, typename OutT>
void launch_mt(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const mxp_packed& B,
               void* D, int64_t ldd, cudaStream_t stream)
{
    if (M <= 8)
        launch<1, kMode, OutT>(M, N, K, A, lda, B, D, ldd, stream);
    else
        launch<2, kMode, OutT>(M, N, K, A, lda, B, D, ldd, stream);
}

}  // namespace

size_t skinny_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }  // a status block is optional

cudaError_t launch_gemm_weight_only(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                    const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                                    void* workspace, size_t workspace_bytes, cudaStream_t stream)
{
    if (M > (1 << 20) || N > (1ll << 30) || K > (1ll << 30)) return cudaErrorNotSupported;
    // Decode shapes go to the streamed kernel (mxp_debug_override can force the general one).
    // A workspace, if given, receives the status of its bounded waits.
    const bool want_old = override_get(MXP_KNOB_WEIGHT_ONLY_KERNEL) == 1;
    if (!want_old && M <= 64 && wo_stream_supported(M, N, K, A, lda, B)) {
        void* status = nullptr;
        if (workspace != nullptr && workspace_bytes >= sizeof(StatusBlock)) {
            status = workspace;
            if (cudaMemsetAsync(status, 0, sizeof(StatusBlock), stream) != cudaSuccess)
                return cudaErrorUnknown;
        }
        return launch_gemm_wo_stream(M, N, K, A, lda, B, D, d_dt, ldd, status, stream);
    }
    if ((M + 15) / 16 > 65535) return cudaErrorNotSupported;
    if (d_dt == MXP_F32) {
        if (B.mode == MXP_MODE_MXFP4_PP) launch_mt<2, float>(M, N, K, A, lda, B, D, ldd, stream);
        else if (B.mode == MXP_MODE_MXFP4_PLUS) launch_mt<1, float>(M, N, K, A, lda, B, D, ldd, stream);
        else launch_mt<0, float>(M, N, K, A, lda, B, D, ldd, stream);
    } else {
        if (B.mode == MXP_MODE_MXFP4_PP) launch_mt<2, __nv_bfloat16>(M, N, K, A, lda, B, D, ldd, stream);
        else if (B.mode == MXP_MODE_MXFP4_PLUS) launch_mt<1, __nv_bfloat16>(M, N, K, A, lda, B, D, ldd, stream);
        else launch_mt<0, __nv_bfloat16>(M, N, K, A, lda, B, D, ldd, stream);
    }
    return cudaGetLastError();
}

}  // namespace mxp
