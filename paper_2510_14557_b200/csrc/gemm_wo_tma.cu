// Weight-only GEMM for decode shapes, weights untouched by any thread:
//
//   D[M,N] = A(bf16)[M,K] * dec(W)[N,K]^T          (Sec. 7.1 setting; decode per Eq. 3)
//
// The 4-bit codes go from HBM to the tensor core without passing through registers:
//   * TMA loads the nibble plane with the 16U4_ALIGN16B tensor-map type, which writes every
//     8 bytes of codes to a 16-byte slot of shared memory: the layout in which tcgen05.mma
//     kind::mxf8f6f4 reads E2M1 operands.  Every CTA (one per SM) owns a contiguous range of at
//     most 128 weight rows and walks the whole K with them: no split along K, no cross-CTA
//     reduction; the rows of the 128-row MMA tile it does not own are padding.
//   * The activations are the MMA's narrow operand: each bf16 activation is split into two E4M3
//     terms (hi + lo, each with its own E8M0 block scale), exact whenever the element lies within
//     2^16 of its block's maximum and within 2^-20 of that maximum otherwise; the two terms are
//     separate operand rows whose accumulator columns the epilogue adds.
//   * MX+ weights: the tensor core reads the BM's code s m2 m1 m0 as the E2M1 value of its low
//     three bits instead of 4 + m/2 (Eq. 3).  One thread per weight row adds the difference,
//     (4 + m/2 - e2m1(m)) * 2^shared_exp * a[k_BM], on the CUDA cores: one multiply-add per block
//     and activation row, with the BM code read from the tile TMA wrote.
//   * The same four warps turn the row-major scale bytes (TMA, 16 blocks per row at a time) into
//     the 32-row x 16-byte atoms tcgen05.cp wants, and drain the accumulator at the end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdlib>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mxp {
namespace {

// warp 0: TMA producer; 1-4: MMA issuers; 5-8: row warps (scale atoms, epilogue); 9-16: BM
// correction (MX+ weights; otherwise they only help with the set-up)
constexpr int kIssueWarp0 = 1, kIssuers = 4;
constexpr int kRowWarp0 = 5;
constexpr int kCorrWarp0 = 9, kCorrWarps = 8;
constexpr int kWarps = kCorrWarp0 + kCorrWarps;
constexpr int kThreads = 32 * kWarps;
constexpr int kStageK = 128;         // elements of K per stage
constexpr int kTok = 8;              // activation rows per CTA (grid.y walks M)
constexpr int kNrows = 2 * kTok;     // MMA N: hi rows, lo rows
constexpr int kAcc = 2 * kIssuers;   // accumulators: two per issuer, used in turn
constexpr uint32_t kTmemCols = 256;  // kAcc * kNrows accumulator columns + 8 per issuer for scales
constexpr int kAtom = 512;
constexpr int kMaxStages = 16;
constexpr int kMaxGroups = 16;       // groups of four stages per tile: K <= 8192
constexpr int kMetaBufs = 4;         // groups of four stages of scale / index bytes in flight
constexpr long long kWaitLimit = 4000000000ll;
constexpr size_t kSmemMax = 227 * 1024;
constexpr uint32_t kFmtE4M3 = 0, kFmtE2M1 = 5;

struct TmaParams {
    int M, N, K;
    const __nv_bfloat16* A;
    int64_t lda;
    void* D;
    int64_t ldd;
    StatusBlock* status;  // may be nullptr
    int rows_per_tile;    // <= 128
    int tiles_per_cta;
    int stages;
};

// Shared-memory layout (bytes from the 1024-byte aligned base).  The ring comes first: the MMA
// reads 128 rows from a slot that holds fewer, i.e. into what follows, which must exist.
struct TmaLayout {
    size_t ring, ring_stride, sfa, meta, meta_stride, act, sfb, abf, corr, bars, total;
};
__host__ __device__ inline TmaLayout tma_layout(int K, int M, int rows_per_tile, int stages, bool plus)
{
    TmaLayout l;
    const size_t nst = (size_t)K / kStageK;
    const size_t rows8 = ((size_t)rows_per_tile + 7) / 8 * 8;
    size_t off = 0;
    l.ring = off;
    l.ring_stride = rows8 * 128;
    off += (size_t)stages * l.ring_stride;
    l.sfa = off;  // one atom per stage of the tile: written once per tile, no reuse inside it
    off += nst * kAtom;
    l.meta = off;
    l.meta_stride = rows8 * 16 * 2;  // scale tile, then index tile
    off += kMetaBufs * l.meta_stride;
    off = (off + 1023) / 1024 * 1024;
    l.act = off;
    off += nst * kNrows * 128;
    l.sfb = off;
    off += nst * kAtom;
    l.abf = off;
    if (plus) off += (size_t)(M < kTok ? M : kTok) * (size_t)K * 2;
    off = (off + 15) / 16 * 16;
    l.corr = off;  // partial corrections [2 halves][kTok][128 rows], fp32
    if (plus) off += 2 * kTok * 128 * 4;
    l.bars = off;
    off += 640;
    // the last slot's 128-row read must stay inside the allocation
    const size_t ring_read_end = l.ring + (size_t)(stages - 1) * l.ring_stride + 128 * 128;
    if (off < ring_read_end) off = ring_read_end;
    l.total = off + 1024;  // slack for aligning the base
    return l;
}

__device__ __forceinline__ void report(StatusBlock* st, volatile uint32_t* abort, uint32_t where)
{
    *abort = 1u;
    if (st != nullptr && atomicCAS(&st->code, 0u, (uint32_t)MXP_ERR_TIMEOUT) == 0u)
        st->where = where;  // the first wait that gave up
}

// Offset of 16-byte chunk c (0..7) of row r inside a 128B-swizzled tile.
__device__ __forceinline__ uint32_t swz_chunk(uint32_t r, uint32_t c)
{
    return r * 128u + ((c ^ (r & 7u)) << 4);
}

// Four floats -> four E4M3 bytes (round to nearest even, saturating), a in the low byte.
__device__ __forceinline__ uint32_t cvt_e4m3x4(float a, float b, float c, float d)
{
    uint32_t r;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(r)
        : "f"(a), "f"(b), "f"(c), "f"(d));
    return r;
}
// Four E4M3 bytes -> four floats.
__device__ __forceinline__ void e4m3x4_to_float(uint32_t v, float (&f)[4])
{
    uint32_t h0, h1;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "mov.b32 {lo, hi}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, lo;\n\t"
        "cvt.rn.f16x2.e4m3x2 %1, hi;\n\t}"
        : "=r"(h0), "=r"(h1)
        : "r"(v));
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&h0));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&h1));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}

#ifdef MXP_WOTMA_TIMELINE
#define TL(slot)                                                                               \
    do {                                                                                       \
        if (prm.status != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && (slot) < 96)        \
            reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(prm.status) + 256)[slot] = \
                ptx::globaltimer_ns();                                                         \
    } while (0)
#else
#define TL(slot) \
    do {         \
    } while (0)
#endif

// kPlus: the weights are MXFP4+ (the BM correction runs).
template <bool kPlus, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_wo_tma_kernel(const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_sc,
                   const __grid_constant__ CUtensorMap tmap_ix, const TmaParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~(uintptr_t)1023);
    const int S = prm.stages;
    const TmaLayout L = tma_layout(prm.K, prm.M, prm.rows_per_tile, S, kPlus);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);  // TMA: weight tile landed
    uint64_t* empty = full + kMaxStages;       // MMAs (and BM reads) of the slot are done
    uint64_t* sfa_ready = empty + kMaxStages;  // [kMaxGroups] row warps wrote the group's scale atoms
    uint64_t* meta_full = sfa_ready + kMaxGroups;
    uint64_t* meta_empty = meta_full + kMetaBufs;
    uint64_t* acc_full = meta_empty + kMetaBufs;
    uint64_t* acc_empty = acc_full + 1;
    uint64_t* corr_full = acc_empty + 1;       // correction warps wrote their partial sums
    uint64_t* corr_empty = corr_full + 1;      // row warps have read them
    uint64_t* setup_bar = corr_empty + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(setup_bar + 1);
    volatile uint32_t* abort = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nb = prm.K / 32;
    const int nst = prm.K / kStageK;
    const int m0 = blockIdx.y * kTok;
    const int mrows = min(kTok, prm.M - m0);
    const int rows8 = (prm.rows_per_tile + 7) / 8 * 8;

    auto ring = [&](int s) { return smem + L.ring + (size_t)s * L.ring_stride; };
    auto sfa = [&](int st) { return smem + L.sfa + (size_t)st * kAtom; };
    auto meta_sc = [&](int g) { return smem + L.meta + (size_t)g * L.meta_stride; };
    auto meta_ix = [&](int g) { return smem + L.meta + (size_t)g * L.meta_stride + (size_t)rows8 * 16; };
    auto tile_n0 = [&](int t) {
        return ((int64_t)blockIdx.x * prm.tiles_per_cta + t) * prm.rows_per_tile;
    };

    if (threadIdx.x == 0) {
        TL(0);
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], kPlus ? 1 + kCorrWarps : 1);
        }
        for (int g = 0; g < kMaxGroups; ++g) ptx::mbar_init(&sfa_ready[g], 4);
        for (int g = 0; g < kMetaBufs; ++g) {
            ptx::mbar_init(&meta_full[g], 1);
            ptx::mbar_init(&meta_empty[g], kPlus ? 4 + kCorrWarps : 4);
        }
        ptx::mbar_init(acc_full, kIssuers);
        ptx::mbar_init(acc_empty, 4);
        ptx::mbar_init(corr_full, kCorrWarps);
        ptx::mbar_init(corr_empty, 4);
        ptx::mbar_init(setup_bar, kWarps - 1);
        *abort = 0u;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_w);
        ptx::prefetch_tmap(&tmap_sc);
        if (kPlus) ptx::prefetch_tmap(&tmap_ix);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) TL(1);
    // An MMA that adds to an accumulator waits for the one before it on the same accumulator,
    // and these MMAs are tiny (128 x 16 x 32): every issuer alternates between two accumulators
    // of its own; the epilogue adds all of them up.
    const uint32_t tmem_acc = tmem_base;                   // kAcc x kNrows columns
    const uint32_t tmem_sf = tmem_base + kAcc * kNrows;    // per issuer: 4 columns for W, 4 for A

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // Starts at once: the weights do not depend on the activation set-up below.
        if (lane == 0) {
            uint32_t c = 0, gc = 0;
            bool ok = true;
            const uint32_t meta_bytes = (uint32_t)prm.rows_per_tile * 16u * (kPlus ? 2u : 1u);
            for (int t = 0; t < prm.tiles_per_cta && ok; ++t) {
                const int64_t n0 = tile_n0(t);
                if (n0 >= prm.N) break;
                for (int st = 0; st < nst; ++st, ++c) {
                    if ((st & 3) == 0) {
                        const int g = gc % kMetaBufs;
                        const uint32_t ug = gc / kMetaBufs;
                        if (ug > 0 && !ptx::mbar_wait(&meta_empty[g], (ug - 1) & 1, abort, kWaitLimit)) {
                            report(prm.status, abort, 0x5000 + g);
                            ok = false;
                            break;
                        }
                        ptx::mbar_arrive_expect_tx(&meta_full[g], meta_bytes);
                        ptx::tma_load_2d(meta_sc(g), &tmap_sc, &meta_full[g], (st >> 2) * 16, (int)n0);
                        if (kPlus)
                            ptx::tma_load_2d(meta_ix(g), &tmap_ix, &meta_full[g], (st >> 2) * 16, (int)n0);
                        ++gc;
                    }
                    const int s = c % S;
                    const uint32_t u = c / S;
                    if (u > 0 && !ptx::mbar_wait(&empty[s], (u - 1) & 1, abort, kWaitLimit)) {
                        report(prm.status, abort, 0x5100 + s);
                        ok = false;
                        break;
                    }
                    // the unpacking load counts the packed bytes it reads (64 per row), not the
                    // 128 it writes
                    ptx::mbar_arrive_expect_tx(&full[s], (uint32_t)prm.rows_per_tile * 64u);
                    ptx::tma_load_2d(ring(s), &tmap_w, &full[s], st * kStageK, (int)n0);
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- activations
        // bf16 -> two E4M3 terms per element, each with its own E8M0 block scale; written as
        // the MMA's K-major, 128B-swizzled narrow operand (hi rows, then lo rows) plus the
        // scale atoms; MX+ also keeps the bf16 values for the BM correction.
        const int tid = threadIdx.x - 32;
        if (mrows < kTok) {
            // rows of absent activations: zero codes (their scale bytes may be anything finite)
            for (int i = tid; i < nst * 128; i += kThreads - 32)
                reinterpret_cast<uint4*>(smem + L.act)[i] = make_uint4(0u, 0u, 0u, 0u);
            for (int i = tid; i < nst * 32; i += kThreads - 32)
                reinterpret_cast<uint4*>(smem + L.sfb)[i] = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
            // the writes below land in the same buffers: order them behind the fill
            asm volatile("bar.sync 1, %0;" ::"r"(kThreads - 32) : "memory");
        }
        for (int i = tid; i < nb * mrows; i += kThreads - 32) {
            const int kb = i / mrows, mc = i - kb * mrows;
            uint32_t x[16] = {};
            {
                const uint4* src = reinterpret_cast<const uint4*>(
                    prm.A + (int64_t)(m0 + mc) * prm.lda + kb * 32);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 v = __ldg(src + q);
                    x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
                    if (kPlus)
                        reinterpret_cast<uint4*>(smem + L.abf + ((size_t)mc * prm.K + kb * 32) * 2)[q] = v;
                }
            }
            uint32_t mx = 0;
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const uint32_t v = x[q] & 0x7FFF7FFFu;
                mx = max(mx, max(v & 0xFFFFu, v >> 16));
            }
            const uint32_t ef = mx >> 7;
            const bool nonfinite = ef == 255u;
            // hi: the block maximum lands in [128, 256); lo: what is left, 16 times finer
            const uint32_t sb_hi = nonfinite ? 255u : max(ef, 8u) - 7u;
            const uint32_t sb_lo = nonfinite ? 255u : max(sb_hi, 5u) - 4u;
            const float inv_hi = __uint_as_float((254u - min(sb_hi, 253u)) << 23);
            const float up_lo = __uint_as_float((127u + sb_hi - sb_lo) << 23);
            uint8_t* tile = smem + L.act + (size_t)(kb >> 2) * (kNrows * 128);
            const uint32_t c0 = (uint32_t)(kb & 3) * 2u;
#pragma unroll
            for (int half = 0; half < 2; ++half) {  // 16 elements = one 16-byte chunk per term
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t x0 = x[8 * half + 2 * q], x1 = x[8 * half + 2 * q + 1];
                    float f[4], back[4];
                    f[0] = __uint_as_float(x0 << 16) * inv_hi;
                    f[1] = __uint_as_float(x0 & 0xFFFF0000u) * inv_hi;
                    f[2] = __uint_as_float(x1 << 16) * inv_hi;
                    f[3] = __uint_as_float(x1 & 0xFFFF0000u) * inv_hi;
                    hi[q] = cvt_e4m3x4(f[0], f[1], f[2], f[3]);
                    e4m3x4_to_float(hi[q], back);
                    lo[q] = cvt_e4m3x4((f[0] - back[0]) * up_lo, (f[1] - back[1]) * up_lo,
                                       (f[2] - back[2]) * up_lo, (f[3] - back[3]) * up_lo);
                    if (nonfinite) hi[q] = lo[q] = 0u;
                }
                *reinterpret_cast<uint4*>(tile + swz_chunk(mc, c0 + half)) =
                    make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(tile + swz_chunk(kTok + mc, c0 + half)) =
                    make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
            uint8_t* atom = smem + L.sfb + (size_t)(kb >> 2) * kAtom + (kb & 3);
            atom[mc * 16] = (uint8_t)sb_hi;
            atom[(kTok + mc) * 16] = (uint8_t)sb_lo;
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (threadIdx.x == 32) TL(2);
        if (lane == 0) ptx::mbar_arrive(setup_bar);
    }

    if (warp >= kIssueWarp0 && warp < kIssueWarp0 + kIssuers) {
        // ------------------------------------------------------------------ MMA issuers
        // Issuer i takes the stages st = i (mod kIssuers), with two accumulators and one set of
        // scale-factor columns of its own: issuing a tcgen05 instruction costs its thread tens
        // of nanoseconds, and these MMAs are too small to hide that behind one thread.
        const int iss = warp - kIssueWarp0;
        const uint32_t tmem_sfa = tmem_sf + 8u * (uint32_t)iss, tmem_sfb = tmem_sfa + 4u;
        bool ok = ptx::mbar_wait(setup_bar, 0, abort, kWaitLimit);
        if (!ok && lane == 0) report(prm.status, abort, 0x5200);
        if (lane == 0 && iss == 0) TL(3);
        ptx::tc_fence_after_sync();
        uint32_t c = 0, ti = 0;
        for (int t = 0; t < prm.tiles_per_cta && ok; ++t, ++ti) {
            if (tile_n0(t) >= prm.N) break;
            if (ti > 0 && !ptx::mbar_wait(acc_empty, (ti - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x5300);
                break;
            }
            ptx::tc_fence_after_sync();
            // Stages are dealt out by their running number and the number of slots is a multiple
            // of kIssuers: slot and issuer stay paired, an issuer sees every fill of its slots in
            // turn, and the parity of the fill it waits for is never ambiguous.
            const int first = (iss - (int)(c % kIssuers) + kIssuers) % kIssuers;
            for (int st = first; st < nst; st += kIssuers) {
                const uint32_t cc = c + (uint32_t)st;
                const int s = cc % S;
                const uint32_t ph = (cc / S) & 1;
                if (!ptx::mbar_wait(&full[s], ph, abort, kWaitLimit) ||
                    !ptx::mbar_wait(&sfa_ready[st >> 2], ti & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x5400 + s);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                if (lane == 0) TL(8 + st);
                const uint64_t da = ptx::smem_desc_sw128(ptx::smem_u32(ring(s)));
                const uint64_t db = ptx::smem_desc_sw128(
                    ptx::smem_u32(smem + L.act + (size_t)st * (kNrows * 128)));
                const uint64_t d_sfa = ptx::smem_desc_sf(ptx::smem_u32(sfa(st)));
                const uint64_t d_sfb = ptx::smem_desc_sf(ptx::smem_u32(smem + L.sfb + (size_t)st * kAtom));
                if (ptx::elect_one()) {
                    ptx::tc_cp_sf(tmem_sfa, d_sfa);
                    ptx::tc_cp_sf(tmem_sfb, d_sfb);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)  // first use of an accumulator: overwrite
                        ptx::mma_mxf8f6f4(tmem_acc + (uint32_t)((2 * iss + (kk & 1)) * kNrows),
                                          da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk),
                                          ptx::idesc_block_scaled(kFmtE2M1, kFmtE4M3, 128, kNrows, kk, kk),
                                          tmem_sfa, tmem_sfb, (st == first && kk < 2) ? 0u : 1u);
                    ptx::tc_commit(&empty[s]);
                }
                __syncwarp();
            }
            c += (uint32_t)nst;
            if (!ok) break;
            if (ptx::elect_one()) ptx::tc_commit(acc_full);
            __syncwarp();
        }
    } else if (warp >= kRowWarp0 && warp < kRowWarp0 + 4) {
        // ------------------------------------------------------------------ row warps
        // Thread = weight row of the tile = TMEM lane: scale atoms while the tile streams, the
        // accumulators at its end.
        const int q = warp & 3;  // the TMEM lane quarter this warp may read
        const int row = 32 * q + lane;
        const uint32_t sfa_off = (uint32_t)(row & 31) * 16u + (uint32_t)(row >> 5) * 4u;
        const float* corr_s = reinterpret_cast<const float*>(smem + L.corr);
        uint32_t gc = 0, ti = 0;
        bool ok = true;
        for (int t = 0; t < prm.tiles_per_cta && ok; ++t, ++ti) {
            const int64_t n0 = tile_n0(t);
            if (n0 >= prm.N) break;
            const int rows_here = (int)min((int64_t)prm.rows_per_tile, (int64_t)prm.N - n0);
            const bool live = row < rows_here;
            // (the MMAs of the tile before have completed: this warp drained its accumulators)
            for (int st0 = 0; st0 < nst && ok; st0 += 4, ++gc) {
                const int g = gc % kMetaBufs;
                if (!ptx::mbar_wait(&meta_full[g], (gc / kMetaBufs) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x5600 + g);
                    ok = false;
                    break;
                }
                uint4 sc4 = make_uint4(0, 0, 0, 0);
                if (live) sc4 = *reinterpret_cast<const uint4*>(meta_sc(g) + row * 16);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&meta_empty[g]);
                if (live) {
                    *reinterpret_cast<uint32_t*>(sfa(st0) + sfa_off) = sc4.x;
                    *reinterpret_cast<uint32_t*>(sfa(st0 + 1) + sfa_off) = sc4.y;
                    *reinterpret_cast<uint32_t*>(sfa(st0 + 2) + sfa_off) = sc4.z;
                    *reinterpret_cast<uint32_t*>(sfa(st0 + 3) + sfa_off) = sc4.w;
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&sfa_ready[st0 >> 2]);
            }
            if (!ok) break;
            // epilogue: every accumulator's hi and lo columns, plus the BM correction
            if (!ptx::mbar_wait(acc_full, ti & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x5900);
                break;
            }
            ptx::tc_fence_after_sync();
            if (threadIdx.x == 32 * kRowWarp0) TL(4);
            float acc[kNrows];
#pragma unroll
            for (int j = 0; j < kNrows; ++j) acc[j] = 0.f;
            for (int a = 0; a < kAcc; ++a) {
                // issuer a / 2 wrote its accumulators only if it had a stage of this tile
                if (((a >> 1) - (int)((ti * (uint32_t)nst) % kIssuers) + kIssuers) % kIssuers >= nst) continue;
                uint32_t r2[kNrows];
                ptx::tmem_ld_32x16(tmem_acc + ((uint32_t)(32 * q) << 16) + (uint32_t)(a * kNrows), r2);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < kNrows; ++j) acc[j] += __uint_as_float(r2[j]);
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty);
            float corr[kTok];
#pragma unroll
            for (int m = 0; m < kTok; ++m) corr[m] = 0.f;
            if (kPlus) {
                if (!ptx::mbar_wait(corr_full, ti & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x5A00);
                    break;
                }
#pragma unroll
                for (int m = 0; m < kTok; ++m)
                    if (m < mrows) corr[m] = corr_s[m * 128 + row] + corr_s[(kTok + m) * 128 + row];
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(corr_empty);
            }
            if (live) {
#pragma unroll
                for (int m = 0; m < kTok; ++m) {
                    if (m < mrows) {
                        const float v = acc[m] + acc[kTok + m] + corr[m];
                        const int64_t off = (int64_t)(m0 + m) * prm.ldd + n0 + row;
                        if (sizeof(OutT) == 4)
                            static_cast<float*>(prm.D)[off] = v;
                        else
                            static_cast<__nv_bfloat16*>(prm.D)[off] = __float2bfloat16_rn(v);
                    }
                }
            }
        }
    } else if (kPlus && warp >= kCorrWarp0) {
        // ------------------------------------------------------------------ correction warps
        // Two threads per weight row, two blocks of the stage each: Eq. 3's BM value minus the
        // E2M1 value the tensor core read in its place, times the block's scale and the
        // activation at the BM's position.
        const int tc = threadIdx.x - 32 * kCorrWarp0;
        const int row = tc >> 1, half = tc & 1;
        const __nv_bfloat16* abf = reinterpret_cast<const __nv_bfloat16*>(smem + L.abf);
        float* corr_s = reinterpret_cast<float*>(smem + L.corr);
        uint32_t c = 0, gc = 0, ti = 0;
        bool ok = ptx::mbar_wait(setup_bar, 0, abort, kWaitLimit);  // the bf16 activations
        if (!ok && lane == 0) report(prm.status, abort, 0x5500);
        for (int t = 0; t < prm.tiles_per_cta && ok; ++t, ++ti) {
            const int64_t n0 = tile_n0(t);
            if (n0 >= prm.N) break;
            const int rows_here = (int)min((int64_t)prm.rows_per_tile, (int64_t)prm.N - n0);
            const bool live = row < rows_here;
            float corr[kTok];
#pragma unroll
            for (int m = 0; m < kTok; ++m) corr[m] = 0.f;
            for (int st0 = 0; st0 < nst && ok; st0 += 4, ++gc) {
                const int g = gc % kMetaBufs;
                if (!ptx::mbar_wait(&meta_full[g], (gc / kMetaBufs) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x5B00 + g);
                    ok = false;
                    break;
                }
                uint4 sc4 = make_uint4(0, 0, 0, 0), ix4 = make_uint4(0, 0, 0, 0);
                if (live) {
                    sc4 = *reinterpret_cast<const uint4*>(meta_sc(g) + row * 16);
                    ix4 = *reinterpret_cast<const uint4*>(meta_ix(g) + row * 16);
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&meta_empty[g]);
#pragma unroll
                for (int i = 0; i < 4; ++i, ++c) {
                    const int st = st0 + i;
                    const int s = c % S;
                    if (!ptx::mbar_wait(&full[s], (c / S) & 1, abort, kWaitLimit)) {
                        if (lane == 0) report(prm.status, abort, 0x5800 + s);
                        ok = false;
                        break;
                    }
                    const uint32_t sw = i == 0 ? sc4.x : i == 1 ? sc4.y : i == 2 ? sc4.z : sc4.w;
                    const uint32_t iw = i == 0 ? ix4.x : i == 1 ? ix4.y : i == 2 ? ix4.z : ix4.w;
                    if (live) {
                        const uint8_t* tile = ring(s);
#pragma unroll
                        for (int bb = 0; bb < 2; ++bb) {
                            const uint32_t b = 2u * (uint32_t)half + (uint32_t)bb;
                            const uint32_t sc = (sw >> (8 * b)) & 255u;
                            const uint32_t e = 32u * b + ((iw >> (8 * b)) & 31u);  // element of the stage
                            const uint32_t byte = tile[swz_chunk((uint32_t)row, e >> 4) + ((e & 15u) >> 1)];
                            const uint32_t nib = (e & 1u) ? byte >> 4 : byte & 15u;
                            // 2 * (4 + m/2 - e2m1(m)) for m = 0..7: 8 8 8 8 8 7 6 3
                            const uint32_t d2 = (0x36788888u >> (4u * (nib & 7u))) & 15u;
                            float v = (float)d2 * 0.5f * __uint_as_float(sc << 23);
                            if (nib & 8u) v = -v;
                            if (sc == 0u || sc == 255u) v = 0.f;  // flushed block / non-finite scale
                            const __nv_bfloat16* ap = abf + (size_t)st * kStageK + e;
#pragma unroll
                            for (int m = 0; m < kTok; ++m)
                                if (m < mrows) corr[m] = fmaf(v, __bfloat162float(ap[(size_t)m * prm.K]), corr[m]);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&empty[s]);
                }
            }
            if (!ok) break;
            if (ti > 0 && !ptx::mbar_wait(corr_empty, (ti - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x5C00);
                break;
            }
#pragma unroll
            for (int m = 0; m < kTok; ++m) corr_s[(half * kTok + m) * 128 + row] = corr[m];
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(corr_full);
        }
    }

    // ---------------------------------------------------------------------- teardown
    // After a timeout, copies may still be in flight into this CTA's shared memory: give them
    // (bounded) time to land before the CTA leaves.
    __syncthreads();
    if (*abort != 0u && threadIdx.x == 0) {
        const long long t0 = clock64();
        for (int s = 0; s < S; ++s)
            while (!ptx::mbar_try_wait(&full[s], 0) && !ptx::mbar_try_wait(&full[s], 1) &&
                   clock64() - t0 < kWaitLimit) {
            }
        for (int g = 0; g < kMetaBufs; ++g)
            while (!ptx::mbar_try_wait(&meta_full[g], 0) && !ptx::mbar_try_wait(&meta_full[g], 1) &&
                   clock64() - t0 < kWaitLimit) {
            }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) TL(5);
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Nibble plane [N][K/2 bytes] as a tensor of 4-bit elements; every 16 codes (8 bytes) land in a
// 16-byte slot of shared memory.  Boxes of 128 codes x `box_rows` rows, 128B swizzle.
bool make_tmap_codes(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t K, int box_rows)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
    const cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 2, const_cast<uint8_t*>(base), dims, strides,
              box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Scale or index plane [N][K/32 bytes]; boxes of 16 bytes (four stages) x `box_rows` rows.
bool make_tmap_meta(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t nb, int box_rows)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)nb, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)nb};
    const cuuint32_t box[2] = {16u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TmaPlan {
    int gx, mtiles, rows_per_tile, tiles_per_cta, stages;
    size_t smem;
};
// Rows per CTA so that every SM gets work, at most 128 per tile; as many ring slots as fit.
bool tma_plan(int64_t M, int64_t N, int64_t K, bool plus, int num_sms, TmaPlan* p)
{
    p->mtiles = (int)((M + kTok - 1) / kTok);
    p->gx = num_sms / p->mtiles;
    if (p->gx < 1) p->gx = 1;
    const int64_t rows_per_cta = (N + p->gx - 1) / p->gx;
    p->tiles_per_cta = (int)((rows_per_cta + 127) / 128);
    p->rows_per_tile = (int)((N + (int64_t)p->gx * p->tiles_per_cta - 1) / ((int64_t)p->gx * p->tiles_per_cta));
    const size_t fixed = tma_layout((int)K, (int)M, p->rows_per_tile, 0, plus).total;
    const size_t per_stage = (size_t)((p->rows_per_tile + 7) / 8 * 8) * 128;
    if (fixed + 4 * per_stage + 128 * 128 > kSmemMax) return false;
    int stages = (int)((kSmemMax - fixed - 128 * 128) / per_stage);
    stages = stages > kMaxStages ? kMaxStages : stages;
    p->stages = stages / kIssuers * kIssuers;  // every slot belongs to one issuer
    p->smem = tma_layout((int)K, (int)M, p->rows_per_tile, p->stages, plus).total;
    return p->smem <= kSmemMax;
}

template <bool kPlus, typename OutT>
cudaError_t launch(const CUtensorMap& tw, const CUtensorMap& ts, const CUtensorMap& ti, TmaParams prm,
                   const TmaPlan& plan, cudaStream_t stream)
{
    auto kern = gemm_wo_tma_kernel<kPlus, OutT>;
    static SmemAttrOnce once;
    cudaError_t e = ensure_dynamic_smem(kern, (int)kSmemMax, once);
    if (e != cudaSuccess) return e;
    kern<<<dim3((unsigned)plan.gx, (unsigned)plan.mtiles), kThreads, plan.smem, stream>>>(tw, ts, ti, prm);
    return cudaGetLastError();
}

}  // namespace

bool wo_tma_supported(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const mxp_packed& B)
{
    if (B.mode != MXP_MODE_MXFP4 && B.mode != MXP_MODE_MXFP4_PLUS) return false;
    if (M < 1 || M > 64 || N < 1 || N > (1ll << 30) || K < 512 || K % 512 != 0 || K > 8192) return false;
    if ((reinterpret_cast<uintptr_t>(A) & 15) || (reinterpret_cast<uintptr_t>(B.nibbles) & 31) ||
        (reinterpret_cast<uintptr_t>(B.scales) & 15))
        return false;
    if (B.mode != MXP_MODE_MXFP4 && (reinterpret_cast<uintptr_t>(B.bm_index) & 15)) return false;
    if (lda % 8 != 0) return false;
    const int sms = sm_count();
    TmaPlan plan;
    return sms > 0 && tma_plan(M, N, K, B.mode != MXP_MODE_MXFP4, sms, &plan);
}

cudaError_t launch_gemm_wo_tma(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                               const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                               void* status, cudaStream_t stream)
{
    const bool plus = B.mode != MXP_MODE_MXFP4;
    const int sms = sm_count();
    TmaPlan plan;
    if (sms <= 0 || !tma_plan(M, N, K, plus, sms, &plan)) return cudaErrorNotSupported;
    CUtensorMap tw, ts, ti;
    if (!make_tmap_codes(&tw, B.nibbles, N, K, plan.rows_per_tile) ||
        !make_tmap_meta(&ts, B.scales, N, K / 32, plan.rows_per_tile) ||
        !make_tmap_meta(&ti, plus ? B.bm_index : B.scales, N, K / 32, plan.rows_per_tile))
        return cudaErrorInvalidValue;
    TmaParams prm;
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.A = static_cast<const __nv_bfloat16*>(A);
    prm.lda = lda;
    prm.D = D;
    prm.ldd = ldd;
    prm.status = static_cast<StatusBlock*>(status);
    prm.rows_per_tile = plan.rows_per_tile;
    prm.tiles_per_cta = plan.tiles_per_cta;
    prm.stages = plan.stages;
    const bool f32 = d_dt == MXP_F32;
    if (plus)
        return f32 ? launch<true, float>(tw, ts, ti, prm, plan, stream)
                   : launch<true, __nv_bfloat16>(tw, ts, ti, prm, plan, stream);
    return f32 ? launch<false, float>(tw, ts, ti, prm, plan, stream)
               : launch<false, __nv_bfloat16>(tw, ts, ti, prm, plan, stream);
}

}  // namespace mxp
