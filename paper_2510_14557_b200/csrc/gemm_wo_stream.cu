// Weight-only GEMM for decode shapes, streamed: D[M,N] = A(bf16)[M,K] * dec(W)[N,K]^T.
//
// Same operation as gemm_weight_only.cu (Sec. 7.1 "conversion before computation", Eq. 3),
// organised as a stream over W: persistent CTAs, one per SM.  Roles per CTA:
//   * a producer warp moves 16 weight rows x 2048 elements per stage into shared memory with
//     bulk copies (mbarrier ring), plus the 16 rows' scale and BM-index bytes per row group;
//   * sixteen consumer warps each take one 128-element chunk of every stage;
//   * two reducer warps add the partial sums in a fixed order and store D, so the consumers
//     go straight on to the next row group;
//   * MX+ modes: two correction warps handle the BM (below).
// Per 32-element block the four lanes of a quad hold the block's four words for two rows and
//   * turn the E2M1 codes into f16 pairs with the hardware cast (cvt.rn.f16x2.e2m1x2),
//   * run two m16n8k16 f16 MMAs against the activations of the block (fresh accumulator),
//   * add that partial sum times 2^(shared_exp) of the weight block into the running fp32 sum.
// The BM (Eq. 3's BM branch: 4 + m/2 instead of the E2M1 value of the same bits) never enters
// that loop: a quad would spend as many instructions on locating and patching one element as
// on the other 31 together, in all four lanes.  The consumers multiply the BM's code as E2M1
// and one thread per weight row and eighth of the blocks adds
// (4 + m/2 - E2M1(m)) * 2^shared_exp * a[k_BM] per block: a dozen scalar instructions.
// Activations are bf16; so that they fit f16 each 256-element chunk of an activation row is
// normalised by the power of two that puts its largest magnitude in [2^14, 2^15): every
// element within 2^28 of that maximum stays exact (f16 keeps 11 significant bits), smaller
// ones are rounded at 2^-39 of the maximum, far inside the GEMM's error bound, which is
// relative to the row's norm.  The power of two goes back in once per chunk.  No scale
// multiply touches the weights, so the weight side costs one cast per element pair.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdlib>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mxp {
namespace {

constexpr int kCW = 16;                      // consumer warps
constexpr int kRW = 2;                       // reducer warps
constexpr int kXW = 4;                       // BM correction warps (MX+ modes)
constexpr int kXSub = 32 * kXW / 16;         // correction threads per weight row: 8
constexpr int kProducerWarp = kCW;
constexpr int kThreadsBase = 32 * (kCW + 1 + kRW);
constexpr int kThreadsCorr = kThreadsBase + 32 * kXW;  // with the correction warps
constexpr int kLutBytes = 32 * 4 * 16;       // [BM position][lane of the quad] -> 4 keep masks
constexpr int kRows = 16;                    // weight rows per step
constexpr int kSlab = 4096;                  // elements of K per stage
constexpr int kChunkBlocks = kSlab / 32 / kCW;  // 8 blocks of 32 per warp and stage
constexpr int kMaxStages = 6;
constexpr int kMaxMetaBufs = 4;              // row groups whose scale / index bytes may be in flight
constexpr int kRowStride = kSlab / 2 + 16;   // bytes; the pad spreads the rows over the banks
constexpr int kStageBytes = kRows * kRowStride;
constexpr long long kWaitLimit = 4000000000ll;
constexpr size_t kSmemMax = 227 * 1024;

struct WoParams {
    int M, N, K;
    const __nv_bfloat16* A;
    int64_t lda;
    const uint8_t* nibbles;
    const uint8_t* scales;
    const uint8_t* bm_index;
    void* D;
    int64_t ldd;
    StatusBlock* status;  // may be nullptr
    int stages;           // ring depth
    int red_buffers;      // 1 or 2 partial-sum buffers
    int meta_bufs;        // 2 or 4 buffers of scale / index bytes
};

__device__ __forceinline__ void report(StatusBlock* st, volatile uint32_t* abort, uint32_t where)
{
    *abort = 1u;
    if (st != nullptr) {
        atomicCAS(&st->code, 0u, (uint32_t)MXP_ERR_TIMEOUT);
        st->where = where;
    }
}

__host__ __device__ constexpr size_t align16(size_t x) { return (x + 15) / 16 * 16; }

// Shared-memory layout (bytes from the 128-byte aligned base).
struct WoLayout {
    size_t lut, act, fa, meta, red, ring, fixed;
    int meta_stride;  // bytes of one metadata buffer (scales + index of 16 rows)
    int red_stride;   // bytes of one partial-sum buffer
};
__host__ __device__ inline WoLayout wo_layout(int K, int mp, bool plus, bool corr, int red_buffers,
                                              int meta_bufs)
{
    WoLayout l;
    const size_t nb = (size_t)K / 32;
    size_t off = 256;  // barriers
    l.lut = off;
    off += kLutBytes;
    l.act = off;
    off += nb * mp * 64;
    l.fa = off;
    off += (nb / 8 + 1) * (size_t)mp * 4;  // factor per 256-element chunk and column
    l.meta = off;
    l.meta_stride = (int)(kRows * nb * (plus ? 2 : 1));
    off += (size_t)meta_bufs * l.meta_stride;
    l.red = off = align16(off);
    l.red_stride = (kCW + (corr ? 1 : 0)) * kRows * (mp + 1) * 4;
    off += (size_t)red_buffers * l.red_stride;
    l.ring = off = align16(off);
    l.fixed = off + 128;  // + slack for aligning the base; the ring follows
    return l;
}

__device__ __forceinline__ void bulk_copy(uint32_t smem_dst, const void* gmem_src, uint32_t bytes,
                                          uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(smem_dst),
        "l"(gmem_src), "r"(bytes), "r"(ptx::smem_u32(bar))
        : "memory");
}

// Shared-memory loads by 32-bit shared address (keeps them out of the generic path).
__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds8(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(a));
    return v;
}

// Eight E2M1 codes (one word) -> four f16x2 registers, element 2i in the low half.
__device__ __forceinline__ void cvt_e2m1x8(uint32_t w, uint32_t (&h)[4])
{
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "mov.b32 {b0, b1, b2, b3}, %4;\n\t"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n\t"
        "cvt.rn.f16x2.e2m1x2 %1, b1;\n\t"
        "cvt.rn.f16x2.e2m1x2 %2, b2;\n\t"
        "cvt.rn.f16x2.e2m1x2 %3, b3;\n\t}"
        : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3])
        : "r"(w));
}

// Eq. 3, BM branch: the element at position p of the block is 4 + m/2 with the stored sign.
// `lut_t` points at this lane's column of the mask table: entry p holds, for each of the
// lane's four f16x2 registers, which bits to keep (all of them unless the lane's word holds
// element p).  The f16 pattern of the BM is built from the lane's own word; where the lane
// does not hold the BM the pattern is garbage and fully masked.
// `ib` is the block's index byte: position in bits 4:0; in MX++ mode (kPP) bits 7:5 hold
// delta, and the BM, which keeps the block's own shared exponent, is entered 2^delta larger
// than the NBMs it sits among (at most 7.5 * 128, an f16 value).
template <bool kPP>
__device__ __forceinline__ void patch_bm(uint32_t w, uint32_t ib, uint32_t lut_t, uint32_t (&h)[4])
{
    const uint32_t p = ib & 31u;
    const uint4 keep = lds128(lut_t + p * 64u);
    const uint32_t x = w >> ((p & 7u) * 4u);
    uint32_t pat = ((x << 7) & 0x0380u) | 0x4400u;  // 4 + m/2
    if (kPP) pat += (ib >> 5) << 10;                 // times 2^delta
    pat |= (x << 12) & 0x8000u;                      // sign
    pat *= 0x00010001u;                              // both halves; the mask picks one
    h[0] = (h[0] & keep.x) | (pat & ~keep.x);
    h[1] = (h[1] & keep.y) | (pat & ~keep.y);
    h[2] = (h[2] & keep.z) | (pat & ~keep.z);
    h[3] = (h[3] & keep.w) | (pat & ~keep.w);
}

// c = a * b (no accumulator input: the zero operands cost no register moves)
__device__ __forceinline__ void mma_f16_16816_first(float (&c)[4], uint32_t a0, uint32_t a1,
                                                    uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1)
{
    // not volatile: the compiler may interleave the MMAs of independent blocks
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Largest bf16 magnitude (bit pattern) in one block of 32.
__device__ __forceinline__ uint32_t block_max(const uint4 (&x)[4])
{
    const uint32_t* xi = reinterpret_cast<const uint32_t*>(x);
    uint32_t mx = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint32_t v = xi[i] & 0x7FFF7FFFu;
        mx = max(mx, max(v & 0xFFFFu, v >> 16));
    }
    return mx;
}
// Multiplier field and factor for a row whose largest magnitude has bit pattern mx: the row
// times 2^(mulfield - 127) has its maximum in [2^14, 2^15); factor = 2^(127 - mulfield).
__device__ __forceinline__ int row_mulfield(uint32_t mx) { return min(253, 268 - (int)(mx >> 7)); }
// One block of 32 bf16 activations times 2^(mulfield - 127) -> 32 f16.
__device__ __forceinline__ void normalise_block(const uint4 (&x)[4], int mulfield, uint4 (&y)[4])
{
    const uint32_t* xi = reinterpret_cast<const uint32_t*>(x);
    const uint32_t mul2 = ((uint32_t)mulfield << 7) * 0x00010001u;
    uint32_t* yo = reinterpret_cast<uint32_t*>(y);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        uint32_t s;
        asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(s) : "r"(xi[i]), "r"(mul2));
        const float lo = __uint_as_float(s << 16), hi = __uint_as_float(s & 0xFFFF0000u);
        const __half2 h2 = __floats2half2_rn(lo, hi);
        yo[i] = *reinterpret_cast<const uint32_t*>(&h2);
    }
}

// Optional timeline (build with -DMXP_WO_TIMELINE, pass a workspace of >= 64 KB): the first
// CTAs record globaltimer stamps of a few events behind the status block.
#ifdef MXP_WO_TIMELINE
#define WO_TL(slot)                                                                        \
    do {                                                                                   \
        if (prm.status != nullptr && blockIdx.x < 8 && (slot) < 64) {                      \
            long long t_;                                                                  \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                         \
            reinterpret_cast<long long*>(reinterpret_cast<char*>(prm.status) + 256)[blockIdx.x * 64 + (slot)] = t_; \
        }                                                                                  \
    } while (0)
#else
#define WO_TL(slot) \
    do {            \
    } while (0)
#endif

// kCorr (MX+ modes, one or two activation rows): the BM is handled by the correction warps; otherwise
// the consumers patch it into their f16 fragments, which costs the same for any number of
// activation columns, while the correction threads' work grows with each column.
template <int kMT, int kMode, bool kCorr, typename OutT>
__global__ void __launch_bounds__(kCorr ? kThreadsCorr : kThreadsBase, 1)
gemm_wo_stream_kernel(const WoParams prm)
{
    constexpr bool kPlus = kMode >= 1;  // 1: MXFP4+, 2: MX++ (Sec. 4.3)
    constexpr bool kPP = kMode == 2;
    constexpr bool kPatch = kPlus && !kCorr;
    static_assert(!kCorr || kPlus, "correction warps are for the MX+ modes");
    constexpr int kMp = 8 * kMT;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) &
                                               ~(uintptr_t)127);
    const WoLayout L = wo_layout(prm.K, kMp, kPlus, kCorr, prm.red_buffers, prm.meta_bufs);
    const uint32_t kMetaBufs = (uint32_t)prm.meta_bufs;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    uint64_t* empty = full + kMaxStages;
    uint64_t* meta_full = empty + kMaxStages;
    uint64_t* meta_empty = meta_full + kMaxMetaBufs;
    uint64_t* red_full = meta_empty + kMaxMetaBufs;
    uint64_t* red_free = red_full + 2;
    uint64_t* setup_bar = red_free + 2;
    volatile uint32_t* abort = reinterpret_cast<volatile uint32_t*>(setup_bar + 1);
    const uint32_t sbase = ptx::smem_u32(smem);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = prm.stages;
    const int nb = prm.K / 32;
    const int slabs = (prm.K + kSlab - 1) / kSlab;
    const int rgs = prm.N / kRows;
    const int m0 = blockIdx.y * kMp;
    const bool two_red = prm.red_buffers == 2;

    // Chained launches (Sec. 7.1's decode loop runs one such GEMM after another): let the next
    // grid on the stream be scheduled as soon as SMs free up.  What this grid must not touch
    // before the previous one has finished is fenced below (activations in, D out); the weight
    // planes are read at once.
    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        WO_TL(0);
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], kCW + (kCorr ? kXW : 0));
        }
        for (int b = 0; b < kMaxMetaBufs; ++b) {
            ptx::mbar_init(&meta_full[b], 1);
            ptx::mbar_init(&meta_empty[b], kCW + (kCorr ? kXW : 0));
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&red_full[b], kCW + (kCorr ? kXW : 0));
            ptx::mbar_init(&red_free[b], kRW);
        }
        ptx::mbar_init(setup_bar, kCW);
        *abort = 0u;
        ptx::fence_mbar_init();
    }
    __syncthreads();

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer warp
        uint32_t it = 0;
        int s = 0;
        uint32_t round = 0;
        bool ok = true;
        for (int rg = blockIdx.x; rg < rgs && ok; rg += gridDim.x, ++it) {
            const int64_t n0 = (int64_t)rg * kRows;
            const uint32_t mb = it % kMetaBufs, muse = it / kMetaBufs;
            if (muse > 0 && !ptx::mbar_wait(&meta_empty[mb], (muse - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x3000);
                break;
            }
            if (lane == 0) {
                const uint32_t dst = sbase + (uint32_t)L.meta + mb * (uint32_t)L.meta_stride;
                ptx::mbar_arrive_expect_tx(&meta_full[mb], (uint32_t)L.meta_stride);
                bulk_copy(dst, prm.scales + n0 * nb, (uint32_t)(kRows * nb), &meta_full[mb]);
                if (kPlus)
                    bulk_copy(dst + kRows * nb, prm.bm_index + n0 * nb, (uint32_t)(kRows * nb),
                              &meta_full[mb]);
            }
            for (int sl = 0; sl < slabs; ++sl) {
                if (round > 0 && !ptx::mbar_wait(&empty[s], (round - 1) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x3100 + s);
                    ok = false;
                    break;
                }
                const uint32_t bytes = (uint32_t)(min(kSlab, prm.K - sl * kSlab) / 2);
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(&full[s], bytes * kRows);
                    WO_TL(16 + (int)it * slabs + sl);
                }
                __syncwarp();
                if (lane < kRows)
                    bulk_copy(sbase + (uint32_t)L.ring + (uint32_t)(s * kStageBytes + lane * kRowStride),
                              prm.nibbles + (n0 + lane) * (int64_t)(prm.K / 2) + (int64_t)sl * (kSlab / 2),
                              bytes, &full[s]);
                if (++s == S) {
                    s = 0;
                    ++round;
                }
            }
        }
    } else if (warp < kCW) {
        // ------------------------------------------------------------------ consumer warps
        const int g = lane >> 2, t = lane & 3;
        constexpr int kCT = 32 * kCW;  // consumer threads
        // BM mask table: entry [p][t] keeps everything unless word t holds element p
        if (kPatch && threadIdx.x < 128) {
            const uint32_t p = threadIdx.x >> 2, tt = threadIdx.x & 3;
            uint32_t k[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
            if ((p >> 3) == tt) k[(p & 7u) >> 1] = (p & 1u) ? 0x0000FFFFu : 0xFFFF0000u;
            reinterpret_cast<uint4*>(smem + L.lut)[threadIdx.x] = make_uint4(k[0], k[1], k[2], k[3]);
        }
        // Activations -> f16 [block][column][32].  Every warp prepares exactly the chunks it
        // will consume (no cross-warp step): each 256-element chunk of a column is normalised
        // by its own power of two, kept in fa[chunk][column].
        float* fa = reinterpret_cast<float*>(smem + L.fa);
        constexpr int kItems = kChunkBlocks * kMp / 32;  // blocks per lane and chunk
        ptx::grid_dependency_wait();  // A may be the previous grid's output
        for (int sl = 0; sl < slabs; ++sl) {
            const int chunk = sl * kCW + warp;
            const int kb0 = chunk * kChunkBlocks;
            if (kb0 >= nb) break;
            const int mc = lane % kMp;
            uint4 x[kItems][4];
            uint32_t mx = 0;
#pragma unroll
            for (int u = 0; u < kItems; ++u) {
                const int kb = kb0 + lane / kMp + u * (32 / kMp);
#pragma unroll
                for (int q = 0; q < 4; ++q) x[u][q] = make_uint4(0, 0, 0, 0);
                if (m0 + mc < prm.M) {
                    const uint4* src = reinterpret_cast<const uint4*>(
                        prm.A + (int64_t)(m0 + mc) * prm.lda + kb * 32);
#pragma unroll
                    for (int q = 0; q < 4; ++q) x[u][q] = __ldg(src + q);
                }
                mx = max(mx, block_max(x[u]));
            }
#pragma unroll
            for (int o = kMp; o < 32; o <<= 1) mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            const int mulfield = row_mulfield(mx);
#pragma unroll
            for (int u = 0; u < kItems; ++u) {
                const int kb = kb0 + lane / kMp + u * (32 / kMp);
                uint4 y[4];
                normalise_block(x[u], mulfield, y);
                uint4* dst = reinterpret_cast<uint4*>(smem + L.act + ((size_t)kb * kMp + mc) * 64);
#pragma unroll
                for (int q = 0; q < 4; ++q) dst[q] = y[q];
            }
            if (lane < kMp) fa[chunk * kMp + mc] = __uint_as_float((uint32_t)(254 - mulfield) << 23);
        }
        // every warp's share of the activations (and the mask table) is in place before use
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(setup_bar);
        bool ok = ptx::mbar_wait(setup_bar, 0, abort, kWaitLimit);
        if (!ok && lane == 0) report(prm.status, abort, 0x3500);
        if (threadIdx.x == 0) WO_TL(1);

        const uint32_t lut_t = sbase + (uint32_t)L.lut + (uint32_t)t * 16u;
        const uint32_t act_gt = sbase + (uint32_t)L.act + (uint32_t)(g * 32 + 8 * t) * 2u;
        const uint32_t w_gt = sbase + (uint32_t)L.ring + (uint32_t)(g * kRowStride + warp * (kChunkBlocks * 16) + t * 4);
        float* red = reinterpret_cast<float*>(smem + L.red);

        uint32_t it = 0, round = 0;
        int s = 0;
        for (int rg = blockIdx.x; rg < rgs && ok; rg += gridDim.x, ++it) {
            const uint32_t mb = it % kMetaBufs;
            if (!ptx::mbar_wait(&meta_full[mb], (it / kMetaBufs) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x3200);
                break;
            }
            const uint32_t sc = sbase + (uint32_t)L.meta + mb * (uint32_t)L.meta_stride + (uint32_t)(g * nb);
            const uint32_t ix = sc + (uint32_t)(kRows * nb);
            float acc[kMT][4];
#pragma unroll
            for (int i = 0; i < kMT; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

            for (int sl = 0; sl < slabs && ok; ++sl) {
                if (!ptx::mbar_wait(&full[s], round & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x3400 + s);
                    ok = false;
                    break;
                }
                if (threadIdx.x == 0) WO_TL(32 + (int)it * slabs + sl);
                const int kb0 = sl * (kSlab / 32) + warp * kChunkBlocks;
                if (kb0 < nb) {
                    float cacc[kMT][4];
#pragma unroll
                    for (int i = 0; i < kMT; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) cacc[i][j] = 0.f;
                    const uint2 scA = lds64(sc + kb0), scB = lds64(sc + 8 * nb + kb0);
                    uint2 ixA = make_uint2(0, 0), ixB = ixA;
                    if (kPP || kPatch) {  // MX++: delta; patching: the BM's position
                        ixA = lds64(ix + kb0);
                        ixB = lds64(ix + 8 * nb + kb0);
                    }
                    const uint32_t wp = w_gt + (uint32_t)(s * kStageBytes);
                    const uint32_t ap = act_gt + (uint32_t)(kb0 * kMp) * 64u;
#pragma unroll
                    for (int j = 0; j < kChunkBlocks; ++j) {
                        const uint32_t wA = lds32(wp + j * 16);
                        const uint32_t wB = lds32(wp + 8 * kRowStride + j * 16);
                        uint32_t hA[4], hB[4];
                        cvt_e2m1x8(wA, hA);
                        cvt_e2m1x8(wB, hB);
                        const int sh = 8 * (j & 3);
                        const uint32_t ibA = ((j < 4 ? ixA.x : ixA.y) >> sh) & 255u;
                        const uint32_t ibB = ((j < 4 ? ixB.x : ixB.y) >> sh) & 255u;
                        if (kPatch) {
                            patch_bm<kPP>(wA, ibA, lut_t, hA);
                            patch_bm<kPP>(wB, ibB, lut_t, hB);
                        }
                        // 2^(scale byte - 127) as a float: a zero byte (flushed block) gives 0;
                        // MX++: the NBMs' exponent lies delta below (exact, subnormals included)
                        float sA = __uint_as_float((((j < 4 ? scA.x : scA.y) >> sh) & 255u) << 23);
                        float sB = __uint_as_float((((j < 4 ? scB.x : scB.y) >> sh) & 255u) << 23);
                        if (kPP) {
                            sA *= __uint_as_float((127u - (ibA >> 5)) << 23);
                            sB *= __uint_as_float((127u - (ibB >> 5)) << 23);
                        }
#pragma unroll
                        for (int mt = 0; mt < kMT; ++mt) {
                            const uint4 b = lds128(ap + (uint32_t)((j * kMp + 8 * mt) * 64));
                            float c[4];
                            mma_f16_16816_first(c, hA[0], hB[0], hA[1], hB[1], b.x, b.y);
                            mma_f16_16816(c, hA[2], hB[2], hA[3], hB[3], b.z, b.w);
                            cacc[mt][0] = fmaf(c[0], sA, cacc[mt][0]);
                            cacc[mt][1] = fmaf(c[1], sA, cacc[mt][1]);
                            cacc[mt][2] = fmaf(c[2], sB, cacc[mt][2]);
                            cacc[mt][3] = fmaf(c[3], sB, cacc[mt][3]);
                        }
                    }
                    // the power of two taken out of this chunk of the activation columns
#pragma unroll
                    for (int mt = 0; mt < kMT; ++mt) {
                        const float2 f2 = *reinterpret_cast<const float2*>(
                            fa + (kb0 / kChunkBlocks) * kMp + 8 * mt + 2 * t);
                        acc[mt][0] = fmaf(cacc[mt][0], f2.x, acc[mt][0]);
                        acc[mt][1] = fmaf(cacc[mt][1], f2.y, acc[mt][1]);
                        acc[mt][2] = fmaf(cacc[mt][2], f2.x, acc[mt][2]);
                        acc[mt][3] = fmaf(cacc[mt][3], f2.y, acc[mt][3]);
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&empty[s]);
                if (++s == S) {
                    s = 0;
                    ++round;
                }
            }
            if (!ok) break;
            if (threadIdx.x == 0) WO_TL(2 + (int)it);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&meta_empty[mb]);

            // hand the partial sums to the reducer warps
            const uint32_t rbuf = two_red ? (it & 1u) : 0u;
            const uint32_t ruse = two_red ? (it >> 1) : it;
            if (ruse > 0 && !ptx::mbar_wait(&red_free[rbuf], (ruse - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x3300);
                break;
            }
            float* rb = red + (size_t)rbuf * (L.red_stride / 4);
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) {
                float* r0 = rb + ((size_t)warp * kRows + g) * (kMp + 1) + 8 * mt + 2 * t;
                r0[0] = acc[mt][0];
                r0[1] = acc[mt][1];
                r0[8 * (kMp + 1)] = acc[mt][2];
                r0[8 * (kMp + 1) + 1] = acc[mt][3];
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&red_full[rbuf]);
        }
    } else if (kCorr && warp >= kCW + 1 + kRW) {
        // ------------------------------------------------------------------ BM correction warps
        // The consumers multiply every code as E2M1, the BM's `s m2 m1 m0` included (as the
        // value of its low three bits, at the NBMs' scale).  Eq. 3's BM branch says 4 + m/2 at
        // the block's own scale; per block and weight row these warps add the difference times
        // the activation at the BM's position.  One thread per weight row and eighth of the
        // blocks; a row's eight threads add up their sums, which go to the reducers as one
        // more partial sum per row.
        {
            const int tid = threadIdx.x - 32 * (kCW + 1 + kRW);
            const int row = tid / kXSub, sub = tid % kXSub;  // a row's threads are neighbouring lanes
            const int mcols = min(kMp, prm.M - m0);
            // per code `s m2 m1 m0` (entry = lane & 15): Eq. 3's BM value 4 + m/2 and the E2M1
            // value of the same bits, both signed
            const uint32_t lm = (uint32_t)lane & 7u;
            const float sgn = (lane & 8) ? -1.f : 1.f;
            const float bm_true = sgn * (4.f + 0.5f * (float)lm);
            const float bm_e2m1 =
                sgn * (lm < 2u ? 0.5f * (float)lm : __uint_as_float(((126u + (lm >> 1)) << 23) | ((lm & 1u) << 22)));
            const float* fa = reinterpret_cast<const float*>(smem + L.fa);
            float* red = reinterpret_cast<float*>(smem + L.red);
            bool ok = ptx::mbar_wait(setup_bar, 0, abort, kWaitLimit);  // activations are in place
            if (!ok && lane == 0) report(prm.status, abort, 0x3700);
            uint32_t it = 0, round = 0;
            int s = 0;
            for (int rg = blockIdx.x; rg < rgs && ok; rg += gridDim.x, ++it) {
                const uint32_t mb = it % kMetaBufs;
                if (!ptx::mbar_wait(&meta_full[mb], (it / kMetaBufs) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x3800);
                    break;
                }
                const uint32_t sc = sbase + (uint32_t)L.meta + mb * (uint32_t)L.meta_stride + (uint32_t)(row * nb);
                const uint32_t ix = sc + (uint32_t)(kRows * nb);
                float acc[kMp];
#pragma unroll
                for (int c = 0; c < kMp; ++c) acc[c] = 0.f;
                for (int sl = 0; sl < slabs && ok; ++sl) {
                    if (!ptx::mbar_wait(&full[s], round & 1, abort, kWaitLimit)) {
                        if (lane == 0) report(prm.status, abort, 0x3900 + s);
                        ok = false;
                        break;
                    }
                    const int nblk = min(kSlab, prm.K - sl * kSlab) / 32;
                    const uint32_t wrow = sbase + (uint32_t)L.ring + (uint32_t)(s * kStageBytes + row * kRowStride);
                    // eight blocks at a time (one 8-byte word of index and of scale bytes), the
                    // groups dealt round robin to the row's eight threads; the loads of a group
                    // are issued together so that their latencies overlap
                    // (warp-uniform trip count: the table lookups are full-warp shuffles; a
                    // thread past the last group works on group 0 and adds nothing)
                    for (int g0 = 0; g0 < nblk / 8; g0 += kXSub) {
                        const bool on = g0 + sub < nblk / 8;
                        const int g8 = on ? g0 + sub : 0;
                        const int kb0 = sl * (kSlab / 32) + 8 * g8;
                        const uint2 ib8 = lds64(ix + kb0), sc8 = lds64(sc + kb0);
                        uint32_t pos[8], byte[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            pos[u] = __byte_perm(u < 4 ? ib8.x : ib8.y, 0u, 0x4440u + (u & 3));
                            byte[u] = lds8(wrow + (8 * g8 + u) * 16 + ((pos[u] & 31u) >> 1));
                        }
                        float cf[8];
                        uint32_t ap[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const uint32_t p = pos[u] & 31u;
                            // (bit 4 may hold the neighbouring code's low bit: the tables repeat
                            // every 16 lanes and a shuffle takes its source lane modulo 32)
                            const uint32_t nib = byte[u] >> ((p << 2) & 4u);
                            // 2^(scale byte - 127); a zero byte (flushed block) gives 0
                            const float scale =
                                __uint_as_float(__byte_perm(u < 4 ? sc8.x : sc8.y, 0u, 0x4440u + (u & 3)) << 23);
                            // the tables sit one entry per lane: a shuffle is the lookup
                            if (kPP) {  // the consumers entered E2M1(m) at the NBMs' scale, delta binades down
                                const float tv = __shfl_sync(0xFFFFFFFFu, bm_true, (int)nib);
                                const float ev = __shfl_sync(0xFFFFFFFFu, bm_e2m1, (int)nib);
                                cf[u] = fmaf(-ev, __uint_as_float((127u - (pos[u] >> 5)) << 23), tv) * scale;
                            } else {
                                cf[u] = __shfl_sync(0xFFFFFFFFu, bm_true - bm_e2m1, (int)nib) * scale;
                            }
                            ap[u] = sbase + (uint32_t)L.act + (uint32_t)((kb0 + u) * kMp) * 64u + p * 2u;
                        }
                        const float* fk = fa + (kb0 / kChunkBlocks) * kMp;  // one chunk = these 8 blocks
#pragma unroll
                        for (int c = 0; c < kMp; ++c) {
                            if (c < mcols) {
                                float part = 0.f;
#pragma unroll
                                for (int u = 0; u < 8; ++u)
                                    part = fmaf(cf[u], __half2float(__ushort_as_half(
                                                           (unsigned short)lds16(ap[u] + c * 64))), part);
                                acc[c] = fmaf(part, on ? fk[c] : 0.f, acc[c]);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&empty[s]);
                    if (++s == S) {
                        s = 0;
                        ++round;
                    }
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&meta_empty[mb]);
                const uint32_t rbuf = two_red ? (it & 1u) : 0u;
                const uint32_t ruse = two_red ? (it >> 1) : it;
                if (ruse > 0 && !ptx::mbar_wait(&red_free[rbuf], (ruse - 1) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x3A00);
                    break;
                }
                float* r0 = red + (size_t)rbuf * (L.red_stride / 4) + ((size_t)kCW * kRows + row) * (kMp + 1);
#pragma unroll
                for (int c = 0; c < kMp; ++c) {
                    float v = acc[c];
#pragma unroll
                    for (int o = 1; o < kXSub; o <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                    if (sub == 0) r0[c] = v;
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&red_full[rbuf]);
            }
        }
    } else {
        // ------------------------------------------------------------------ reducer warps
        const int tid = threadIdx.x - 32 * (kCW + 1);
        const float* red = reinterpret_cast<const float*>(smem + L.red);
        uint32_t it = 0;
        ptx::grid_dependency_wait();  // D may still be read by the previous grid
        for (int rg = blockIdx.x; rg < rgs; rg += gridDim.x, ++it) {
            const int64_t n0 = (int64_t)rg * kRows;
            const uint32_t rbuf = two_red ? (it & 1u) : 0u;
            const uint32_t ruse = two_red ? (it >> 1) : it;
            if (!ptx::mbar_wait(&red_full[rbuf], ruse & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x3600);
                break;
            }
            const float* rb = red + (size_t)rbuf * (L.red_stride / 4);
            for (int e = tid; e < kRows * kMp; e += 32 * kRW) {
                const int r = e % kRows, mcol = e / kRows;
                float sum = 0.f;
#pragma unroll
                for (int w = 0; w < kCW + (kCorr ? 1 : 0); ++w)
                    sum += rb[((size_t)w * kRows + r) * (kMp + 1) + mcol];
                const int m = m0 + mcol;
                if (m < prm.M) {
                    if (sizeof(OutT) == 4)
                        static_cast<float*>(prm.D)[(int64_t)m * prm.ldd + n0 + r] = sum;
                    else
                        static_cast<__nv_bfloat16*>(prm.D)[(int64_t)m * prm.ldd + n0 + r] =
                            __float2bfloat16_rn(sum);
                }
            }
            __syncwarp();
            if (tid == 0) WO_TL(48 + (int)it);
            if (lane == 0) ptx::mbar_arrive(&red_free[rbuf]);
        }
    }
    // Leave together: no CTA exits while bulk copies into its shared memory may be in flight
    // (after a timeout the producer stops issuing; what it issued lands within the wait below).
    if (*abort != 0u && threadIdx.x == 0) {
        const long long t0 = clock64();
        for (int s = 0; s < S; ++s)
            while (!ptx::mbar_try_wait(&full[s], 0) && !ptx::mbar_try_wait(&full[s], 1) &&
                   clock64() - t0 < kWaitLimit) {
            }
    }
    __syncthreads();
}

// Ring depth and numbers of partial-sum and metadata buffers that fit; the roomier choices
// are tried first.  False if not even two stages fit.
inline bool wo_plan(int K, int mp, bool plus, bool corr, int* stages, int* red_buffers, int* meta_bufs)
{
    const int rbs[3] = {2, 1, 1}, mbs[3] = {4, 4, 2};
    for (int c = 0; c < 3; ++c) {
        const size_t fixed = wo_layout(K, mp, plus, corr, rbs[c], mbs[c]).fixed;
        if (fixed >= kSmemMax) continue;
        const int st = (int)((kSmemMax - fixed) / kStageBytes);
        if (st >= 3 || (c == 2 && st >= 2)) {
            *stages = st > kMaxStages ? kMaxStages : st;
            *red_buffers = rbs[c];
            *meta_bufs = mbs[c];
            return true;
        }
    }
    return false;
}

template <int kMT, int kMode, bool kCorr, typename OutT>
cudaError_t launch(WoParams prm, int num_sms, bool chained, cudaStream_t stream)
{
    constexpr bool kPlus = kMode >= 1;
    constexpr int kThreads = kCorr ? kThreadsCorr : kThreadsBase;
    if (!wo_plan(prm.K, 8 * kMT, kPlus, kCorr, &prm.stages, &prm.red_buffers, &prm.meta_bufs))
        return cudaErrorNotSupported;
    const size_t smem = wo_layout(prm.K, 8 * kMT, kPlus, kCorr, prm.red_buffers, prm.meta_bufs).fixed +
                        (size_t)prm.stages * kStageBytes;
    auto kern = gemm_wo_stream_kernel<kMT, kMode, kCorr, OutT>;
    static SmemAttrOnce once;
    const cudaError_t ea = ensure_dynamic_smem(kern, (int)kSmemMax, once);
    if (ea != cudaSuccess) return ea;
    const int rgs = prm.N / kRows;
    const int mtiles = (prm.M + 8 * kMT - 1) / (8 * kMT);
    int gx = num_sms / mtiles;
    if (gx < 1) gx = 1;
    if (gx > rgs) gx = rgs;
    if (!chained) {
        kern<<<dim3((unsigned)gx, (unsigned)mtiles), kThreads, smem, stream>>>(prm);
        return cudaGetLastError();
    }
    // programmatic dependent launch: this grid may start while the previous one on the stream
    // is draining; only its weight stream runs ahead of the in-kernel dependency wait
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)gx, (unsigned)mtiles);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, prm);
}


// Largest M for which the correction warps beat patching (measured on config 3, CUDA graph:
// 14.1 vs 15.2 us at M = 1, 14.8 vs 15.5 at M = 2, 15.7 vs 15.6 at M = 3, 21.3 vs 17.4 at
// M = 8).
constexpr int kCorrMaxM = 2;

}  // namespace

bool wo_stream_supported(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                         const mxp_packed& B)
{
    if (M < 1 || N < kRows || N % kRows != 0 || K % 256 != 0) return false;
    if (M > 4096 || N > (1ll << 30) || K > (1 << 20)) return false;
    if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B.nibbles) |
         reinterpret_cast<uintptr_t>(B.scales)) & 15)
        return false;
    if (lda % 8 != 0) return false;
    const bool plus = B.mode != MXP_MODE_MXFP4;
    if (plus && (reinterpret_cast<uintptr_t>(B.bm_index) & 15)) return false;
    int st, rb, mb;
    return wo_plan((int)K, M <= 8 ? 8 : 16, plus, plus && M <= kCorrMaxM, &st, &rb, &mb);
}

cudaError_t launch_gemm_wo_stream(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                  const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                                  void* status, cudaStream_t stream, bool chained)
{
    WoParams prm;
    prm.status = static_cast<StatusBlock*>(status);
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.A = static_cast<const __nv_bfloat16*>(A);
    prm.lda = lda;
    prm.nibbles = B.nibbles;
    prm.scales = B.scales;
    prm.bm_index = B.bm_index;
    prm.D = D;
    prm.ldd = ldd;
    prm.stages = prm.red_buffers = prm.meta_bufs = 0;
    const int sms = sm_count();
    if (sms <= 0) return cudaErrorUnknown;
    const bool f32 = d_dt == MXP_F32;
    const int mode = (int)B.mode;
#define MXP_WO_LAUNCH(MT, CORR)                                                            \
    switch (mode) {                                                                        \
        case 2:                                                                            \
            return f32 ? launch<MT, 2, CORR, float>(prm, sms, chained, stream)             \
                       : launch<MT, 2, CORR, __nv_bfloat16>(prm, sms, chained, stream);    \
        case 1:                                                                            \
            return f32 ? launch<MT, 1, CORR, float>(prm, sms, chained, stream)             \
                       : launch<MT, 1, CORR, __nv_bfloat16>(prm, sms, chained, stream);    \
        default:                                                                           \
            return f32 ? launch<MT, 0, false, float>(prm, sms, chained, stream)            \
                       : launch<MT, 0, false, __nv_bfloat16>(prm, sms, chained, stream);   \
    }
    // one or two activation rows: the BM goes to the correction warps (see the kernel)
    if (M <= kCorrMaxM) {
        MXP_WO_LAUNCH(1, true)
    }
    if (M <= 8) {
        MXP_WO_LAUNCH(1, false)
    }
    MXP_WO_LAUNCH(2, false)
#undef MXP_WO_LAUNCH
}

}  // namespace mxp
